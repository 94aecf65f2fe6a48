// Lazy ratio (Eq. 1), reference-quality CUDA-core path (any dtype, head_dim 64
// or 128), the merge kernel shared by all scoring paths, and the selection.
//
// Partial statistics of one tail row (layer, b, hq, t) over one key split, log2
// domain with t_j = scale * log2(e) * (q . k_j):
//   M = max_j t_j,  A = sum_j 2^(t_j - M),  W = sum_{j in window} 2^(t_j - M)
// over the visible keys j <= n_ctx - w_last + t of the split; the window is
// {j < n_sink} U {j >= n_ctx - n_recent}.
#include <cuda_bf16.h>

#include "lt_internal.h"

namespace lt {

template <typename T>
__device__ __forceinline__ float ld_f32(const T* p);
template <>
__device__ __forceinline__ float ld_f32<float>(const float* p) {
  return *p;
}
template <>
__device__ __forceinline__ float ld_f32<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(*p);
}

// grid (w_last * n_splits, B * Hq, L); block 128.
template <typename T, int D>
__global__ void scores_generic_kernel(ScoreArgs a, LayerTable kf) {
  const lt_shape& s = a.s;
  const int t = blockIdx.x / a.n_splits, sp = blockIdx.x % a.n_splits;
  const int b = blockIdx.y / s.n_q_heads, hq = blockIdx.y % s.n_q_heads;
  const int l = a.layer_begin + blockIdx.z;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int h = hq / G;
  __shared__ float qs[D];
  __shared__ float red[3][128];
  const T* qp = (const T*)a.q_tail + ((((long long)l * s.batch + b) * s.n_q_heads + hq) * a.w_last + t) * D;
  for (int d = threadIdx.x; d < D; d += blockDim.x) qs[d] = ld_f32<T>(qp + d);
  __syncthreads();
  const int i = a.n_ctx - a.w_last + t;  // position of this query; sees keys 0..i
  int j0, j1;
  score_split_range(a, sp, &j0, &j1);
  j1 = min(i + 1, j1);
  const T* Kl = (const T*)kf.p[l];
  const int win_lo = s.recent_per_row ? i - s.n_recent + 1 : a.n_ctx - s.n_recent;  // first recent key of this row
  float M = -INFINITY, A = 0.f, W = 0.f;
  for (int j = j0 + threadIdx.x; j < j1; j += blockDim.x) {
    const T* kr = Kl + full_cache_row(s, b, h, j) * D;
    float dot = 0.f;
#pragma unroll 8
    for (int d = 0; d < D; ++d) dot += qs[d] * ld_f32<T>(kr + d);
    const float tj = dot * a.cs;
    const float Mn = fmaxf(M, tj);
    const float corr = exp2f(M - Mn), p = exp2f(tj - Mn);
    A = A * corr + p;
    W = W * corr + ((j < s.n_sink || j >= win_lo) ? p : 0.f);
    M = Mn;
  }
  red[0][threadIdx.x] = M;
  red[1][threadIdx.x] = A;
  red[2][threadIdx.x] = W;
  __syncthreads();
  if (threadIdx.x == 0) {
    float Mx = -INFINITY;
    for (int k = 0; k < 128; ++k) Mx = fmaxf(Mx, red[0][k]);
    float As = 0.f, Ws = 0.f;
    if (Mx > -INFINITY) {
      for (int k = 0; k < 128; ++k) {
        const float w = exp2f(red[0][k] - Mx);
        As += w * red[1][k];
        Ws += w * red[2][k];
      }
    }
    float* st = a.stats +
                ((((((long long)blockIdx.z * s.batch + b) * s.n_q_heads + hq) * a.w_last + t) * a.n_splits) + sp) * 3;
    st[0] = Mx;
    st[1] = As;
    st[2] = Ws;
  }
}

cudaError_t launch_scores_generic(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st) {
  dim3 grid(a.w_last * a.n_splits, a.s.batch * a.s.n_q_heads, a.layer_count);
  const bool bf = a.s.dtype == LT_BF16;
  if (a.s.head_dim == 128) {
    if (bf) scores_generic_kernel<__nv_bfloat16, 128><<<grid, 128, 0, st>>>(a, kf);
    else scores_generic_kernel<float, 128><<<grid, 128, 0, st>>>(a, kf);
  } else {
    if (bf) scores_generic_kernel<__nv_bfloat16, 64><<<grid, 128, 0, st>>>(a, kf);
    else scores_generic_kernel<float, 64><<<grid, 128, 0, st>>>(a, kf);
  }
  return cudaGetLastError();
}

// One warp per (layer, b, hq): lane t, t + 32, ... merges the statistics slots of its tail rows and takes the
// row's mass W/A; the lanes' sums are added in a fixed tree and divided by w_last.  The statistics are indexed by
// the layer's position in the scored range.
__global__ void scores_finish_kernel(ScoreArgs a) {
  const lt_shape& s = a.s;
  const long long per_layer = (long long)s.batch * s.n_q_heads;
  const int lane = threadIdx.x & 31;
  const long long rel = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (rel >= a.layer_count * per_layer) return;  // whole warps leave together
  const long long idx = a.layer_begin * per_layer + rel;
  const int T = a.w_last;
  int n_slots = a.n_splits;
  long long unit_row0 = 0;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int hq = (int)(rel % s.n_q_heads);
  if (a.streamk) unit_row0 = ((rel / s.n_q_heads) * s.n_kv_heads + hq / G) * a.row_blocks;  // first unit of this kv head
  float sum = 0.f;
  for (int t = lane; t < T; t += 32) {
    const float* st = a.stats + ((rel * T + t) * a.n_splits) * 3;
    if (a.streamk) {
      // the persistent kernel wrote two slots per piece of this row's unit: the CTAs from the owner of the
      // unit's first tile to the owner of its last one (two slots each: halves of a tile's keys)
      const int r = (hq % G) * T + t;  // row among the kv head's G * T query rows
      const long long g0 = (unit_row0 + r / kScoreBlockM) * a.tiles_per_unit;
      n_slots = 2 * (score_tile_owner(a.total_tiles, a.grid, g0 + a.tiles_per_unit - 1) -
                     score_tile_owner(a.total_tiles, a.grid, g0) + 1);
    }
    float Mx = -INFINITY;
    for (int sp = 0; sp < n_slots; ++sp) Mx = fmaxf(Mx, st[sp * 3]);
    if (a.window_only) {
      // denominator given: mass = sum over splits of W * 2^(M - lse * log2(e))
      const float lse2 = a.lse[idx * T + t] * 1.4426950408889634f;
      float W = 0.f;
      for (int sp = 0; sp < n_slots; ++sp) W += st[sp * 3 + 2] * exp2f(st[sp * 3] - lse2);
      sum += W;
    } else {
      float A = 0.f, W = 0.f;
      for (int sp = 0; sp < n_slots; ++sp) {
        const float w = exp2f(st[sp * 3] - Mx);
        A += w * st[sp * 3 + 1];
        W += w * st[sp * 3 + 2];
      }
      sum += W / A;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
  if (lane == 0) a.scores[idx] = sum / (float)T;
}

cudaError_t launch_scores_finish(const ScoreArgs& a, cudaStream_t st) {
  const long long warps = (long long)a.layer_count * a.s.batch * a.s.n_q_heads;
  scores_finish_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(a);
  return cudaGetLastError();
}

// Selection: one CTA.  Thread l sums its layer's scores in double in index
// order, then ranks itself by counting the layers that beat it under the total
// order (ratio descending, index ascending).
__global__ void select_kernel(const float* __restrict__ scores, int L, int per_layer, int n_lazy,
                              uint8_t* __restrict__ mask, float* __restrict__ ratio) {
  __shared__ double r[LT_MAX_LAYERS];
  const int l = threadIdx.x;
  if (l < L) {
    double acc = 0.0;
    const float* p = scores + (long long)l * per_layer;
    for (int k = 0; k < per_layer; ++k) acc += (double)p[k];
    r[l] = acc / (double)per_layer;
  }
  __syncthreads();
  if (l < L) {
    int rank = 0;
    for (int m = 0; m < L; ++m) rank += (r[m] > r[l]) || (r[m] == r[l] && m < l);
    mask[l] = rank < n_lazy ? 1 : 0;
    if (ratio) ratio[l] = (float)r[l];
  }
}

// Per-prompt selection: block b ranks the layers by the mean over the query
// heads of scores[l][b][:] (same total order as select_kernel).
__global__ void select_per_seq_kernel(const float* __restrict__ scores, int L, int B, int Hq, int n_lazy,
                                      uint8_t* __restrict__ mask, float* __restrict__ ratio) {
  __shared__ double r[LT_MAX_LAYERS];
  const int l = threadIdx.x, b = blockIdx.x;
  if (l < L) {
    double acc = 0.0;
    const float* p = scores + ((long long)l * B + b) * Hq;
    for (int k = 0; k < Hq; ++k) acc += (double)p[k];
    r[l] = acc / (double)Hq;
  }
  __syncthreads();
  if (l < L) {
    int rank = 0;
    for (int m = 0; m < L; ++m) rank += (r[m] > r[l]) || (r[m] == r[l] && m < l);
    mask[(long long)b * L + l] = rank < n_lazy ? 1 : 0;
    if (ratio) ratio[(long long)b * L + l] = (float)r[l];
  }
}

cudaError_t launch_select_per_seq(const float* scores, int L, int B, int Hq, int n_lazy, uint8_t* mask, float* ratio,
                                  cudaStream_t st) {
  select_per_seq_kernel<<<B, LT_MAX_LAYERS, 0, st>>>(scores, L, B, Hq, n_lazy, mask, ratio);
  return cudaGetLastError();
}

// One arrival at the priority queue of Figure 3.  The queue is "the layers
// 0..layer whose mask is still 0"; state[l] holds their ratios (double).  When
// more than n_full layers are queued, the one with the highest ratio (lower
// index on ties) leaves: mask = 1, *popped = its index.
__global__ void select_push_kernel(const float* __restrict__ scores_l, int layer, int L, int per_layer, int n_full,
                                   double* __restrict__ state, uint8_t* __restrict__ mask,
                                   int32_t* __restrict__ popped) {
  __shared__ double r[LT_MAX_LAYERS];
  __shared__ uint8_t queued[LT_MAX_LAYERS];
  const int t = threadIdx.x;
  if (layer == 0 && t < L) mask[t] = 0;  // a new prompt: empty queue, nothing lazy yet
  if (t == 0) {
    double acc = 0.0;
    for (int k = 0; k < per_layer; ++k) acc += (double)scores_l[k];
    state[layer] = acc / (double)per_layer;
  }
  __syncthreads();
  const bool in_queue = t <= layer && mask[t] == 0;
  queued[t] = in_queue ? 1 : 0;
  r[t] = (t <= layer) ? state[t] : 0.0;
  const int count = __syncthreads_count(in_queue);
  if (count <= n_full) {
    if (t == 0 && popped) *popped = -1;
    return;
  }
  if (in_queue) {
    int beaten_by = 0;
    for (int m = 0; m <= layer; ++m)
      if (queued[m]) beaten_by += (r[m] > r[t]) || (r[m] == r[t] && m < t);
    if (beaten_by == 0) {
      mask[t] = 1;
      if (popped) *popped = t;
    }
  }
}

cudaError_t launch_select_push(const float* scores_l, int layer, int L, int per_layer, int n_full, double* state,
                               uint8_t* mask, int32_t* popped, cudaStream_t st) {
  select_push_kernel<<<1, LT_MAX_LAYERS, 0, st>>>(scores_l, layer, L, per_layer, n_full, state, mask, popped);
  return cudaGetLastError();
}

// Frequency-count choice: thread l counts the samples that labelled layer l lazy
// (integer, exact), then ranks itself (count descending, index ascending).
__global__ void select_frequency_kernel(const uint8_t* __restrict__ masks, int N, int L, int n_lazy,
                                        uint8_t* __restrict__ mask, int32_t* __restrict__ counts) {
  __shared__ int c[LT_MAX_LAYERS];
  const int l = threadIdx.x;
  if (l < L) {
    int acc = 0;
    for (int i = 0; i < N; ++i) acc += masks[(long long)i * L + l] != 0;
    c[l] = acc;
  }
  __syncthreads();
  if (l < L) {
    int rank = 0;
    for (int m = 0; m < L; ++m) rank += (c[m] > c[l]) || (c[m] == c[l] && m < l);
    mask[l] = rank < n_lazy ? 1 : 0;
    if (counts) counts[l] = c[l];
  }
}

cudaError_t launch_select_frequency(const uint8_t* masks, int N, int L, int n_lazy, uint8_t* mask, int32_t* counts,
                                    cudaStream_t st) {
  select_frequency_kernel<<<1, LT_MAX_LAYERS, 0, st>>>(masks, N, L, n_lazy, mask, counts);
  return cudaGetLastError();
}

cudaError_t launch_select(const float* scores, int L, int B, int Hq, int n_lazy, uint8_t* mask, float* ratio,
                          cudaStream_t st) {
  select_kernel<<<1, LT_MAX_LAYERS, 0, st>>>(scores, L, B * Hq, n_lazy, mask, ratio);
  return cudaGetLastError();
}

}  // namespace lt
