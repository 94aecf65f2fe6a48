// Lazy ratio (Eq. 1), CUDA-core path (fp32 stacks; head_dim 64 or 128), the merge
// kernel shared by all scoring paths, and the selection.
//
// Partial statistics of one tail row (layer, b, hq, t) over one key split, log2
// domain with t_j = scale * log2(e) * (q . k_j):
//   M = max_j t_j,  A = sum_j 2^(t_j - M),  W = sum_{j in window} 2^(t_j - M)
// over the visible keys j <= n_ctx - w_last + t of the split; the window is
// {j < n_sink} U {j >= n_ctx - n_recent}.
//
// One CTA of 128 threads per (layer, batch row, kv head, key split).  It serves the G * w_last query rows of
// the kv head in blocks of 32 rows; for each block it walks the split in tiles of 16 KB of K rows (two tiles in
// shared memory, the next one copied under the arithmetic of this one):
//   scores      a thread owns one key of the tile and a share of the block's rows.  It walks its K row starting
//               at element `key` and wrapping around (the 32 rows of a warp, a multiple of 128 bytes apart,
//               fall into 32 banks); one K element feeds every row of the thread, q (times scale * log2 e)
//               comes from shared memory at the same rotated index.
//   statistics  a warp per query row: tile maximum, new running maximum, the tile's sums of 2^(t - M) over all
//               visible keys and over the window keys, folded into the row's running (M, A, W).
// A K row is read from memory once per block of rows (from L2 after the first block) instead of once per row.
#include <cuda_bf16.h>

#include "lt_internal.h"

namespace lt {

namespace {

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

__device__ __forceinline__ void copy16_async(void* smem_dst, const void* src, int src_bytes) {
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void copy_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void copy_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

constexpr int kSgThreads = 128;
constexpr int kSgRows = 32;           // query rows per pass over the split
constexpr int kSgTileBytes = 16384;   // K rows of one tile

}  // namespace

// grid (n_splits, B * Hkv, layers of the call); block 128.
template <typename T, int D>
__global__ void __launch_bounds__(kSgThreads) scores_generic_kernel(ScoreArgs a, LayerTable kf) {
  constexpr int RB = kSgRows;
  constexpr int TK = kSgTileBytes / (D * (int)sizeof(T));  // keys per tile: 32, 64 or 128
  constexpr int ROW = D * (int)sizeof(T), VEC = ROW / 16;
  constexpr int NRG = kSgThreads / TK;                      // row shares in the score phase
  constexpr int RPT = RB / NRG;                             // rows per thread
  static_assert(TK >= 32 && TK <= kSgThreads && kSgThreads % TK == 0 && RB % NRG == 0, "geometry");
  extern __shared__ __align__(16) uint8_t sg_smem[];
  uint8_t* tiles = sg_smem;                                             // [2][TK rows of K]
  float* q_s = reinterpret_cast<float*>(sg_smem + 2 * kSgTileBytes);    // [RB][D] the block's query rows, times scale * log2 e
  float* sc = q_s + RB * D;                                             // [RB][TK] scores of the tile
  float* st_M = sc + RB * TK;                                           // [RB] running (M, A, W) of the block's rows
  float* st_A = st_M + RB;
  float* st_W = st_A + RB;
  const lt_shape& s = a.s;
  const int sp = blockIdx.x;
  const int b = blockIdx.y / s.n_kv_heads, h = blockIdx.y % s.n_kv_heads;
  const int l = a.layer_begin + blockIdx.z;
  const int G = s.n_q_heads / s.n_kv_heads, T_ = a.w_last;
  const int n_rows = G * T_;  // rows of this kv head: row = g * w_last + t, contiguous in q_tail
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int j0, j1;
  score_split_range(a, sp, &j0, &j1);  // keys [j0, j1) of this split (j1 <= n_ctx)
  const int n_tiles = j1 > j0 ? (j1 - j0 + TK - 1) / TK : 0;
  const T* Kl = (const T*)kf.p[l];
  const T* qbase = (const T*)a.q_tail + (((long long)l * s.batch + b) * s.n_q_heads + (long long)h * G) * T_ * D;
  auto fetch_tile = [&](int it) {
    uint8_t* kt = tiles + (it & 1) * kSgTileBytes;
    for (int i = tid; i < TK * VEC; i += kSgThreads) {
      const int r = i / VEC, p = i - r * VEC;
      const int j = j0 + it * TK + r;
      const bool valid = j < j1;
      const uint8_t* src = reinterpret_cast<const uint8_t*>(Kl + full_cache_row(s, b, h, valid ? j : j0) * D);
      copy16_async(kt + r * ROW + p * 16, src + p * 16, valid ? 16 : 0);
    }
  };
  for (int r0 = 0; r0 < n_rows; r0 += RB) {
    const int RBn = min(RB, n_rows - r0);
    for (int i = tid; i < RB * D; i += kSgThreads) q_s[i] = i < RBn * D ? ld_f32<T>(qbase + (long long)r0 * D + i) * a.cs : 0.f;
    if (tid < RB) {
      st_M[tid] = -INFINITY;
      st_A[tid] = 0.f;
      st_W[tid] = 0.f;
    }
    if (n_tiles > 0) fetch_tile(0);
    copy_commit();
    for (int it = 0; it < n_tiles; ++it) {
      if (it + 1 < n_tiles) fetch_tile(it + 1);
      copy_commit();
      copy_wait<1>();
      __syncthreads();  // tile `it` has landed; the block's q rows and state are visible
      const int tile_j0 = j0 + it * TK;
      // ---- scores -------------------------------------------------------------------
      {
        const int key = tid % TK, rg = tid / TK;
        if (rg * RPT < RBn) {
          const T* krow = reinterpret_cast<const T*>(tiles + (it & 1) * kSgTileBytes) + key * D;
          const float* qr = q_s + rg * RPT * D;
          float t[RPT];
#pragma unroll
          for (int i = 0; i < RPT; ++i) t[i] = 0.f;
#pragma unroll 4
          for (int dd = 0; dd < D; ++dd) {
            const int d = (dd + key) & (D - 1);
            const float kv = ld_f32<T>(krow + d);
#pragma unroll
            for (int i = 0; i < RPT; ++i) t[i] = fmaf(kv, qr[i * D + d], t[i]);
          }
          const int j = tile_j0 + key;
#pragma unroll
          for (int i = 0; i < RPT; ++i) {
            const int row = r0 + rg * RPT + i;
            const int pos = a.n_ctx - T_ + row % T_;  // position of this query: it sees keys 0 .. pos
            sc[(rg * RPT + i) * TK + key] = (j < j1 && j <= pos) ? t[i] : -INFINITY;
          }
        }
      }
      __syncthreads();
      // ---- statistics: a warp per row ---------------------------------------------------
      for (int r = warp; r < RBn; r += kSgThreads / 32) {
        const int pos = a.n_ctx - T_ + (r0 + r) % T_;
        const int win_lo = s.recent_per_row ? pos - s.n_recent + 1 : a.n_ctx - s.n_recent;  // first recent key of this row
        float v[TK / 32];
        float m = -INFINITY;
#pragma unroll
        for (int c = 0; c < TK / 32; ++c) {
          v[c] = sc[r * TK + lane + 32 * c];
          m = fmaxf(m, v[c]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (m > -INFINITY) {  // the row sees at least one key of this tile (uniform over the warp)
          const float Mo = st_M[r];
          const float Mn = fmaxf(Mo, m);
          float sa = 0.f, sw = 0.f;
#pragma unroll
          for (int c = 0; c < TK / 32; ++c) {
            const int j = tile_j0 + lane + 32 * c;
            const float p = exp2f(v[c] - Mn);
            sa += p;
            sw += (j < s.n_sink || j >= win_lo) ? p : 0.f;
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            sa += __shfl_xor_sync(0xffffffffu, sa, o);
            sw += __shfl_xor_sync(0xffffffffu, sw, o);
          }
          if (lane == 0) {
            const float corr = exp2f(Mo - Mn);  // 0 while the row has seen nothing yet
            st_M[r] = Mn;
            st_A[r] = st_A[r] * corr + sa;
            st_W[r] = st_W[r] * corr + sw;
          }
        }
      }
      __syncthreads();  // the stage and the scores are free for the tile after next
    }
    copy_wait<0>();
    if (tid < RBn) {
      const int row = r0 + tid;
      const int hq = h * G + row / T_, t = row % T_;
      float* st = a.stats +
                  ((((((long long)blockIdx.z * s.batch + b) * s.n_q_heads + hq) * T_ + t) * a.n_splits) + sp) * 3;
      st[0] = st_M[tid];
      st[1] = st_A[tid];
      st[2] = st_W[tid];
    }
    __syncthreads();  // q and the state are rewritten by the next block of rows
  }
}

template <typename T, int D>
static cudaError_t launch_scores_generic_variant(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st) {
  constexpr int TK = kSgTileBytes / (D * (int)sizeof(T));
  constexpr int smem = 2 * kSgTileBytes + (kSgRows * D + kSgRows * TK + 3 * kSgRows) * 4;
  auto kern = scores_generic_kernel<T, D>;
  // the same value on every call, so concurrent first calls from several host threads agree
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  dim3 grid(a.n_splits, a.s.batch * a.s.n_kv_heads, a.layer_count);
  kern<<<grid, kSgThreads, smem, st>>>(a, kf);
  return cudaGetLastError();
}

cudaError_t launch_scores_generic(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st) {
  const bool bf = a.s.dtype == LT_BF16;
  if (a.s.head_dim == 128) {
    return bf ? launch_scores_generic_variant<__nv_bfloat16, 128>(a, kf, st)
              : launch_scores_generic_variant<float, 128>(a, kf, st);
  }
  return bf ? launch_scores_generic_variant<__nv_bfloat16, 64>(a, kf, st)
            : launch_scores_generic_variant<float, 64>(a, kf, st);
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
      // the row's log-sum-exp over its visible keys, as a prefill's attention kernel would hand it over
      if (a.lse_out) a.lse_out[idx * T + t] = (Mx + log2f(A)) * 0.6931471805599453f;
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
