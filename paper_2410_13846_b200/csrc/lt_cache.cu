// KV-cache movement: per-step append (full layers and lazy layers) and the
// prefill -> decode compaction of the lazy layers.  Pure data movement with
// integer addressing; every row is copied bit for bit in 16-byte vectors.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "lt_internal.h"

namespace lt {

__device__ __forceinline__ int ring_slot_dev(int p, int S, int R) { return p < S ? p : S + (p - S) % R; }

// One thread per 16-byte vector of one (layer, b, kv head) row of k_new / v_new.
__global__ void append_kernel(lt_shape s, const uint8_t* __restrict__ mask, const uint4* __restrict__ k_new,
                              const uint4* __restrict__ v_new, const int32_t* __restrict__ seq_lens,
                              LayerTable kf, LayerTable vf, LayerTable ks, LayerTable vs, int layer_begin,
                              int layer_count, int vec_per_row, uint32_t* dev_err) {
  const int B = s.batch, Hkv = s.n_kv_heads, S = s.n_sink, R = s.n_recent;
  const long long total = (long long)layer_count * B * Hkv * vec_per_row;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int v = (int)(idx % vec_per_row);
  long long row = idx / vec_per_row;  // ((lrel*B)+b)*Hkv+h
  const int h = (int)(row % Hkv);
  const int b = (int)((row / Hkv) % B);
  const int l = layer_begin + (int)(row / ((long long)Hkv * B));
  const int pos = seq_lens[b];
  const bool lazy = mask[mask_index(s, l, b)] != 0;
  uint4* kdst = (uint4*)(lazy ? ks.p[l] : kf.p[l]);
  uint4* vdst = (uint4*)(lazy ? vs.p[l] : vf.p[l]);
  if (!kdst || !vdst) {
    if (dev_err && v == 0) atomicOr(dev_err, LT_DEVERR_NULL_LAYER);
    return;
  }
  const int slot = lazy ? ring_slot_dev(pos, S, R) : pos;
  const int rows = lazy ? S + R : s.full_capacity;
  if (pos < 0 || slot >= rows) {
    if (dev_err && v == 0) atomicOr(dev_err, LT_DEVERR_POS_OUT_OF_RANGE);
    return;
  }
  const long long src = ((long long)(l * B + b) * Hkv + h) * vec_per_row + v;
  const long long drow = lazy ? ((long long)b * Hkv + h) * rows + slot : full_cache_row(s, b, h, slot);
  if (s.kv_fp8) {
    // 8 bf16 values -> 8 E4M3 bytes: float32 division by the layer's scale, round to nearest even, saturate
    auto quantize8 = [](uint4 x, float scale) {
      const uint32_t w[4] = {x.x, x.y, x.z, x.w};
      uint2 out = make_uint2(0u, 0u);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const uint32_t pair = w[e >> 1];
        const float f = __uint_as_float((e & 1) ? (pair & 0xffff0000u) : (pair << 16));
        const uint32_t code = (uint32_t)__nv_cvt_float_to_fp8(__fdiv_rn(f, scale), __NV_SATFINITE, __NV_E4M3);
        if (e < 4) out.x |= code << (8 * e);
        else out.y |= code << (8 * (e - 4));
      }
      return out;
    };
    const long long dst8 = drow * vec_per_row + v;  // 8-byte units: a cached row has vec_per_row of them
    reinterpret_cast<uint2*>(kdst)[dst8] = quantize8(k_new[src], s.kv_scales[2 * l]);
    reinterpret_cast<uint2*>(vdst)[dst8] = quantize8(v_new[src], s.kv_scales[2 * l + 1]);
    return;
  }
  const long long dst = drow * vec_per_row + v;
  kdst[dst] = k_new[src];
  vdst[dst] = v_new[src];
}

__global__ void advance_seq_lens_kernel(int32_t* seq_lens, int B) {
  for (int b = threadIdx.x; b < B; b += blockDim.x) seq_lens[b] += 1;
}

cudaError_t launch_append(const lt_shape& s, const uint8_t* mask, const void* k_new, const void* v_new,
                          int32_t* seq_lens, const LayerTable& kf, const LayerTable& vf, const LayerTable& ks,
                          const LayerTable& vs, int layer_begin, int layer_count, int advance, uint32_t* dev_err,
                          cudaStream_t st) {
  const int vec_per_row = (int)(s.head_dim * elem_bytes(s.dtype) / 16);
  const long long total = (long long)layer_count * s.batch * s.n_kv_heads * vec_per_row;
  const int threads = 256;
  const long long blocks = (total + threads - 1) / threads;
  append_kernel<<<(unsigned)blocks, threads, 0, st>>>(s, mask, (const uint4*)k_new, (const uint4*)v_new, seq_lens, kf,
                                                      vf, ks, vs, layer_begin, layer_count, vec_per_row, dev_err);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (advance) {
    advance_seq_lens_kernel<<<1, 256, 0, st>>>(seq_lens, s.batch);
    e = cudaGetLastError();
  }
  return e;
}

// Gather by destination slot: slot s of the stream cache receives the prompt
// row of the last position that maps to it, so no two threads write one row.
__global__ void stream_init_kernel(lt_shape s, const uint8_t* __restrict__ mask, LayerTable kf, LayerTable vf,
                                   const int32_t* __restrict__ seq_lens, LayerTable ks, LayerTable vs,
                                   int vec_per_row, const int32_t* __restrict__ only_layer, uint32_t* dev_err) {
  const int Hkv = s.n_kv_heads, S = s.n_sink, R = s.n_recent, cap = s.full_capacity;
  const int l = blockIdx.z;
  const int bh = blockIdx.y;
  const int b = bh / Hkv, h = bh - b * Hkv;
  if (only_layer && *only_layer != l) return;  // compaction of the one layer named on the device
  if (mask[mask_index(s, l, b)] == 0) return;
  const int C = S + R;
  const uint4* ksrc = (const uint4*)kf.p[l];
  const uint4* vsrc = (const uint4*)vf.p[l];
  uint4* kdst = (uint4*)ks.p[l];
  uint4* vdst = (uint4*)vs.p[l];
  if (!ksrc || !vsrc || !kdst || !vdst) {
    if (dev_err && threadIdx.x == 0 && blockIdx.x == 0) atomicOr(dev_err, LT_DEVERR_NULL_LAYER);
    return;
  }
  int n = seq_lens[b];
  if (n > cap) {
    if (dev_err && threadIdx.x == 0 && blockIdx.x == 0) atomicOr(dev_err, LT_DEVERR_LEN_CLAMPED);
    n = cap;
  }
  const long long total = (long long)C * vec_per_row;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int slot = (int)(idx / vec_per_row);
    const int v = (int)(idx % vec_per_row);
    int p = -1;
    if (slot < S) {
      if (slot < n) p = slot;
    } else {
      const int ri = slot - S;
      const int last = n - S - 1;  // ring index space: position p maps to (p - S)
      if (last >= ri) p = S + last - ((last - ri) % R);
    }
    if (p < 0) continue;
    const long long src = full_cache_row(s, b, h, p) * vec_per_row + v;
    const long long dst = ((long long)bh * C + slot) * vec_per_row + v;
    kdst[dst] = ksrc[src];
    vdst[dst] = vsrc[src];
  }
}

cudaError_t launch_stream_init(const lt_shape& s, const uint8_t* mask, const LayerTable& kf, const LayerTable& vf,
                               const int32_t* seq_lens, const LayerTable& ks, const LayerTable& vs,
                               const int32_t* only_layer, uint32_t* dev_err, cudaStream_t st) {
  const int vec_per_row = (int)(cache_row_bytes(s) / 16);
  const int C = s.n_sink + s.n_recent;
  const long long total = (long long)C * vec_per_row;
  const int threads = 256;
  int bx = (int)((total + threads - 1) / threads);
  if (bx > 64) bx = 64;
  dim3 grid(bx, s.batch * s.n_kv_heads, s.n_layers);
  stream_init_kernel<<<grid, threads, 0, st>>>(s, mask, kf, vf, seq_lens, ks, vs, vec_per_row, only_layer, dev_err);
  return cudaGetLastError();
}

}  // namespace lt
