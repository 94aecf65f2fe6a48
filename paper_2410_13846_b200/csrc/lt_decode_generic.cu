// Decode step, reference-quality CUDA-core path (any dtype, head_dim 64 or 128,
// any GQA group size).  Same persistent work-list structure, fused append and
// in-kernel merge as the tensor-core path.
//
// Partials of one (layer, b, kv head, chunk, head-in-group), log2 domain:
//   M = max_j t_j,  l = sum_j 2^(t_j - M),  o[d] = sum_j 2^(t_j - M) v_j[d]
// with t_j = scale * log2(e) * (q . k_j).
#include <cuda_bf16.h>

#include "lt_decode_common.cuh"
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

// Persistent launch; block = 128 threads = 4 warps; per item warp w takes heads
// w, w+4, ... of the group and walks the chunk key by key.
template <typename T, int D>
__global__ void __launch_bounds__(128) decode_generic_kernel(DecodeArgs a, LayerTable kf, LayerTable vf,
                                                             LayerTable ks, LayerTable vs) {
  constexpr int EPL = D / 32;  // elements per lane
  extern __shared__ __align__(16) uint8_t smem[];
  __shared__ int s_flag;
  __shared__ float2 s_ml[kCombineStagePairs];
  const lt_shape& s = a.s;
  const int G = s.n_q_heads / s.n_kv_heads;
  pdl_wait_prior_grid();
  pdl_allow_next_grid();
  WorkList wl;
  wl.carve(smem, a.layer_count, s.batch);
  wl.build(a, kf, vf, ks, vs);
  const int n_items = wl.total(a);
  const float cs = a.cs;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const WorkItem w = wl.item(a, item);
    const int l = w.l, b = w.b, h = w.h;
    const long long bh = (long long)b * s.n_kv_heads + h;
    const T* Kl = (const T*)(w.lazy ? ks.p[l] : kf.p[l]);
    const T* Vl = (const T*)(w.lazy ? vs.p[l] : vf.p[l]);
    // element offset of cache row j of this (b, kv head): stream caches are contiguous, full caches may be paged
    auto row_off = [&](int j) { return (w.lazy ? bh * w.rows + j : full_cache_row(s, b, h, j)) * D; };
    const T* k_new_row = nullptr;
    const T* v_new_row = nullptr;
    if (w.new_row >= 0) {
      const long long src = (((long long)l * s.batch + b) * s.n_kv_heads + h) * D;
      k_new_row = (const T*)a.k_new + src;
      v_new_row = (const T*)a.v_new + src;
      T* kd = const_cast<T*>(Kl) + row_off(w.new_row);
      T* vd = const_cast<T*>(Vl) + row_off(w.new_row);
      for (int d = threadIdx.x; d < D; d += blockDim.x) {
        kd[d] = k_new_row[d];
        vd[d] = v_new_row[d];
      }
    }
    const long long unit = partial_unit(a, w);
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
      for (int j = w.j0; j < w.j1; ++j) {
        const long long ro = row_off(j);
        const T* kr = (j == w.new_row) ? k_new_row : Kl + ro;
        const T* vr = (j == w.new_row) ? v_new_row : Vl + ro;
        float part = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) part += qr[e] * to_f32<T>(kr[lane * EPL + e]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        const float t = part * cs;
        const float Mn = fmaxf(M, t);
        const float corr = exp2f(M - Mn);  // exp2f(-inf) = 0 on the first key
        const float p = exp2f(t - Mn);
        lsum = lsum * corr + p;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = acc[e] * corr + p * to_f32<T>(vr[lane * EPL + e]);
        M = Mn;
      }
      float* po = a.part_o + (unit * G + g) * D;
#pragma unroll
      for (int e = 0; e < EPL; ++e) po[lane * EPL + e] = acc[e];
      if (lane == 0) {
        float* pml = a.part_ml + (unit * G + g) * 2;
        pml[0] = M;
        pml[1] = lsum;
      }
    }
    if (count_item_in(a, w, &s_flag)) combine_unit(a, w, s_ml);
    __syncthreads();
  }
  finish_launch(a);
}

template <typename T, int D>
static cudaError_t launch_generic_variant(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                                          const LayerTable& ks, const LayerTable& vs, cudaStream_t st) {
  const int smem = worklist_smem_bytes(a.layer_count * a.s.batch, a.s.batch);
  auto kern = decode_generic_kernel<T, D>;
  int per_sm = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 128, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  return launch_decode_kernel(kern, persistent_grid(a, per_sm), 128, smem, st, a, kf, vf, ks, vs);
}

cudaError_t launch_decode_generic(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                                  const LayerTable& ks, const LayerTable& vs, cudaStream_t st) {
  const bool bf = a.s.dtype == LT_BF16;
  if (a.s.head_dim == 128) {
    return bf ? launch_generic_variant<__nv_bfloat16, 128>(a, kf, vf, ks, vs, st)
              : launch_generic_variant<float, 128>(a, kf, vf, ks, vs, st);
  }
  return bf ? launch_generic_variant<__nv_bfloat16, 64>(a, kf, vf, ks, vs, st)
            : launch_generic_variant<float, 64>(a, kf, vf, ks, vs, st);
}

}  // namespace lt
