// Decode attention, reference-quality CUDA-core path (any dtype, head_dim 64 or
// 128, any GQA group size) and the split-KV combine kernel shared by all paths.
//
// Partials of one (layer, b, kv head, chunk, head-in-group), log2 domain:
//   M = max_j t_j,  l = sum_j 2^(t_j - M),  o[d] = sum_j 2^(t_j - M) v_j[d]
// with t_j = scale * log2(e) * (q . k_j).
#include <cuda_bf16.h>

#include "lt_internal.h"

namespace lt {

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) {
  return x;
}
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) {
  return __bfloat162float(x);
}

// grid (chunk, b*Hkv + h, layer_rel); block = 128 threads = 4 warps; warp w
// takes heads w, w+4, ... of the group and walks the chunk key by key.
template <typename T, int D>
__global__ void decode_generic_kernel(DecodeArgs a, LayerTable kf, LayerTable vf, LayerTable ks, LayerTable vs) {
  constexpr int EPL = D / 32;  // elements per lane
  const lt_shape& s = a.s;
  const int l = a.layer_begin + blockIdx.z;
  const int bh = blockIdx.y;
  const int b = bh / s.n_kv_heads, h = bh % s.n_kv_heads;
  const int G = s.n_q_heads / s.n_kv_heads;
  const bool lazy = a.mask[l] != 0;
  const T* K = (const T*)(lazy ? ks.p[l] : kf.p[l]);
  const T* V = (const T*)(lazy ? vs.p[l] : vf.p[l]);
  const int rows = lazy ? s.n_sink + s.n_recent : s.full_capacity;
  int n = a.seq_lens[b];
  if (!K || !V) {
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(a.dev_err, LT_DEVERR_NULL_LAYER);
    return;
  }
  if (n > rows) {
    if (!lazy && threadIdx.x == 0 && blockIdx.x == 0) atomicOr(a.dev_err, LT_DEVERR_LEN_CLAMPED);
    n = rows;
  }
  if (n > a.n_chunks_launch * a.chunk_keys) {
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(a.dev_err, LT_DEVERR_LEN_CLAMPED);
    n = a.n_chunks_launch * a.chunk_keys;
  }
  const int j0 = blockIdx.x * a.chunk_keys;
  const int j1 = min(n, j0 + a.chunk_keys);
  if (j0 >= j1) return;
  const float cs = a.cs;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const T* Kb = K + ((long long)bh * rows) * D;
  const T* Vb = V + ((long long)bh * rows) * D;
  for (int g = warp; g < G; g += 4) {
    const int hq = h * G + g;
    const T* qp = (const T*)a.q + (((long long)l * s.batch + b) * s.n_q_heads + hq) * D;
    float qr[EPL], acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      qr[e] = to_f32<T>(qp[lane * EPL + e]);
      acc[e] = 0.f;
    }
    float M = -INFINITY, lsum = 0.f;
    for (int j = j0; j < j1; ++j) {
      float part = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) part += qr[e] * to_f32<T>(Kb[(long long)j * D + lane * EPL + e]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      const float t = part * cs;
      const float Mn = fmaxf(M, t);
      const float corr = exp2f(M - Mn);  // exp2f(-inf) = 0 on the first key
      const float p = exp2f(t - Mn);
      lsum = lsum * corr + p;
#pragma unroll
      for (int e = 0; e < EPL; ++e)
        acc[e] = acc[e] * corr + p * to_f32<T>(Vb[(long long)j * D + lane * EPL + e]);
      M = Mn;
    }
    const long long unit = (((long long)l * s.batch + b) * s.n_kv_heads + h) * a.n_chunks_max + blockIdx.x;
    float* po = a.part_o + (unit * G + g) * D;
#pragma unroll
    for (int e = 0; e < EPL; ++e) po[lane * EPL + e] = acc[e];
    if (lane == 0) {
      float* pml = a.part_ml + (unit * G + g) * 2;
      pml[0] = M;
      pml[1] = lsum;
    }
  }
}

cudaError_t launch_decode_generic(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                                  const LayerTable& ks, const LayerTable& vs, cudaStream_t st) {
  dim3 grid(a.n_chunks_launch, a.s.batch * a.s.n_kv_heads, a.layer_count);
  const bool bf = a.s.dtype == LT_BF16;
  if (a.s.head_dim == 128) {
    if (bf) decode_generic_kernel<__nv_bfloat16, 128><<<grid, 128, 0, st>>>(a, kf, vf, ks, vs);
    else decode_generic_kernel<float, 128><<<grid, 128, 0, st>>>(a, kf, vf, ks, vs);
  } else {
    if (bf) decode_generic_kernel<__nv_bfloat16, 64><<<grid, 128, 0, st>>>(a, kf, vf, ks, vs);
    else decode_generic_kernel<float, 64><<<grid, 128, 0, st>>>(a, kf, vf, ks, vs);
  }
  return cudaGetLastError();
}

// grid (Hq, B, layer_rel); block = D threads; thread d merges the chunks of its
// (layer, b, hq) in chunk order (fixed order => run-to-run identical bits).
__global__ void decode_combine_kernel(DecodeArgs a) {
  const lt_shape& s = a.s;
  const int l = a.layer_begin + blockIdx.z;
  const int b = blockIdx.y, hq = blockIdx.x;
  const int D = s.head_dim;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int h = hq / G, g = hq % G;
  const int d = threadIdx.x;
  const bool lazy = a.mask[l] != 0;
  const int rows = lazy ? s.n_sink + s.n_recent : s.full_capacity;
  int n = min(a.seq_lens[b], rows);
  n = min(n, a.n_chunks_launch * a.chunk_keys);
  const int nc = (n + a.chunk_keys - 1) / a.chunk_keys;
  const long long unit0 = (((long long)l * s.batch + b) * s.n_kv_heads + h) * a.n_chunks_max;
  float M = -INFINITY;
  for (int c = 0; c < nc; ++c) M = fmaxf(M, a.part_ml[((unit0 + c) * G + g) * 2]);
  float num = 0.f, den = 0.f;
  for (int c = 0; c < nc; ++c) {
    const float* pml = a.part_ml + ((unit0 + c) * G + g) * 2;
    const float w = exp2f(pml[0] - M);
    den += w * pml[1];
    num += w * a.part_o[((unit0 + c) * G + g) * D + d];
  }
  const float r = nc > 0 ? num / den : 0.f;
  const long long oi = (((long long)l * s.batch + b) * s.n_q_heads + hq) * D + d;
  if (a.out_dtype == LT_F32) ((float*)a.out)[oi] = r;
  else ((__nv_bfloat16*)a.out)[oi] = __float2bfloat16_rn(r);
}

cudaError_t launch_decode_combine(const DecodeArgs& a, cudaStream_t st) {
  dim3 grid(a.s.n_q_heads, a.s.batch, a.layer_count);
  decode_combine_kernel<<<grid, a.s.head_dim, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace lt
