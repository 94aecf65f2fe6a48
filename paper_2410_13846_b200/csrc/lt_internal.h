// Internal declarations shared by the translation units of liblt.
// Host-side plumbing only; each kernel family lives in its own .cu file.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "lt.h"

namespace lt {

// Host tables of device pointers travel to the kernels by value.
struct LayerTable {
  const void* p[LT_MAX_LAYERS];
};

// Workspace layout: [header 256 B: error word][counters of the decode step]
// [region used by the running call: split-KV partials or scoring statistics].
constexpr size_t kWsHeaderBytes = 256;
constexpr size_t kWsAlign = 256;
// Bytes of header + counters ([L][B][Hkv] unit counters, then two launch
// counters per layer: a launch uses the pair of its first layer); everything
// here must be zero between calls (lt_workspace_init).
size_t ws_prefix_bytes(const lt_shape& s);

// Split-KV plan of the decode step; a function of the shape alone so that the
// workspace query and every later call agree.
struct DecodePlan {
  int min_chunk, max_chunk;  // the kernels pick the chunk length of a launch in this range (multiples of 64)
  int mid_chunk;             // upper end of the range for launches with few keys (see make_decode_plan)
  int target_items;          // items a launch aims for when its keys allow (a few per CTA)
  int items_cap;             // most items (= partial slots) any launch over this shape can have
  int layer_items_cap;       // most items per layer of any launch (a launch over k layers has at most k times this):
                             // what a step issued as concurrent per-layer launches reserves for every layer
  size_t ml_floats;          // [items_cap][G][2]
  size_t o_floats;           // [items_cap][G][D]
};
DecodePlan make_decode_plan(const lt_shape& s);

// Split plan of the scoring pass.  With the denominator given (window_only)
// only the kept keys are visited: split 0 is the sink range when n_sink > 0,
// the other splits are equal parts of the recent range.
struct ScorePlan {
  int n_splits;        // statistics slots per tail row: key-range splits of its (layer, batch row, kv head), or
                       // the pieces that the persistent tensor-core kernel may cut its unit into
  int split_len;       // keys per split (of the whole prompt, or of the recent range)
  size_t stat_floats;  // [L][B][Hq][T][n_splits][3] partial (reference exponent, sum_all, sum_window)
};
// layer_count: layers scored by one call; 0 = the bound that holds for any layer range (workspace query).
ScorePlan make_score_plan(const lt_shape& s, int n_ctx, int w_last, bool window_only, int layer_count = 0);

// Geometry of the tensor-core scoring kernel.
constexpr int kScoreBlockM = 256;   // query rows per unit
constexpr int kScoreBlockN = 256;   // keys per tile
constexpr int kScoreMaxCtas = 192;  // the persistent launch never has more CTAs than this (one per SM)
// The persistent launch cuts the sequence of all tiles, [0, total), into `grid` contiguous ranges:
// tile g belongs to CTA g * grid / total.
__host__ __device__ inline int score_tile_owner(long long total, int grid, long long g) {
  return (int)((g * grid) / total);
}
__host__ __device__ inline void score_cta_tiles(long long total, int grid, int cta, long long* g0, long long* g1) {
  *g0 = ((long long)cta * total + grid - 1) / grid;
  *g1 = ((long long)(cta + 1) * total + grid - 1) / grid;
}

// Index of (layer l, batch row b) in layer_mask.
__host__ __device__ inline int mask_index(const lt_shape& s, int l, int b) {
  return s.per_sequence_mask ? b * s.n_layers + l : l;
}
// Row (in units of head_dim elements) of token j of (batch row b, kv head h) in a layer's full cache.
// The block table is dereferenced on the device only.
__device__ __forceinline__ long long full_cache_row(const lt_shape& s, int b, int h, int j) {
  if (s.page_size <= 0) return ((long long)b * s.n_kv_heads + h) * s.full_capacity + j;
  const int page = s.block_table[(long long)b * s.pages_per_seq + j / s.page_size];
  return ((long long)page * s.n_kv_heads + h) * s.page_size + j % s.page_size;
}
inline float resolved_scale(const lt_shape& s) {
  return s.softmax_scale > 0.f ? s.softmax_scale : 1.0f / sqrtf((float)s.head_dim);
}
inline size_t elem_bytes(int dtype) { return dtype == LT_BF16 ? 2 : 4; }
// Bytes of one cached K or V row.
inline size_t cache_row_bytes(const lt_shape& s) { return s.kv_fp8 ? (size_t)s.head_dim : s.head_dim * elem_bytes(s.dtype); }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

lt_status validate_shape(const lt_shape* s);

// ---- launchers (each returns cudaGetLastError() of its launches) ----------
cudaError_t launch_append(const lt_shape& s, const uint8_t* mask, const void* k_new, const void* v_new,
                          int32_t* seq_lens, const LayerTable& kf, const LayerTable& vf,
                          const LayerTable& ks, const LayerTable& vs, int layer_begin, int layer_count,
                          int advance, uint32_t* dev_err, cudaStream_t st);

cudaError_t launch_stream_init(const lt_shape& s, const uint8_t* mask, const LayerTable& kf,
                               const LayerTable& vf, const int32_t* seq_lens, const LayerTable& ks,
                               const LayerTable& vs, const int32_t* only_layer, uint32_t* dev_err, cudaStream_t st);

// One decode step (or the attention half of it).  `fused` = the step appends
// k_new / v_new itself: the visible length is seq_lens[b] + 1 and the item that
// owns the new token's row stores it into the cache.
struct DecodeArgs {
  lt_shape s;
  const void* q;
  const void* k_new;  // fused only
  const void* v_new;  // fused only
  const uint8_t* mask;
  const int32_t* seq_lens;
  int32_t* seq_lens_rw;  // fused + advance: incremented by the last CTA of the launch
  void* out;
  int out_dtype;
  int layer_begin, layer_count;
  int min_chunk, mid_chunk, max_chunk, target_items, items_cap;
  int fused, advance;
  int pdl;   // launch with the programmatic-serialization attribute (the step comes as several launches)
  int overlap;    // the caller vouches that this launch shares nothing with the launches before it on the stream
                  // (another layer range of the same step): it does not wait for them before it starts
  int slot_base;  // first partial slot of this launch (0, or the launch's own region when launches may overlap)
  float cs;  // softmax scale * log2(e)
  float* part_ml;
  float* part_o;
  int* unit_counters;  // [L][B][Hkv], zero between launches
  int* launch_counters;  // [L][2], zero between launches; the two below are the pair of layer_begin
  int* done_counter;     // zero between launches
  int* work_counter;     // zero between launches: dynamic item hand-out
  uint32_t* dev_err;
};
// Most (layer, batch row) pairs one launch can take (its work list lives in
// shared memory); larger stacks are split by layers on the host.
constexpr int kMaxWorkEntries = 2048;
// CTAs of a persistent decode launch: per_sm * SM count, but no more than the
// most items the launch can have.
int persistent_grid(const DecodeArgs& a, int ctas_per_sm);
// SM count of the current device (looked up once per device, behind a lock).
int sm_count_of_current_device();
// Launch of a decode kernel, with the programmatic-serialization attribute when a.pdl is set.
template <typename Kern>
inline cudaError_t launch_decode_kernel(Kern kern, int grid, int threads, int smem, cudaStream_t st, const DecodeArgs& a,
                                        const LayerTable& kf, const LayerTable& vf, const LayerTable& ks,
                                        const LayerTable& vs) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, a, kf, vf, ks, vs);
}
cudaError_t launch_decode_generic(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                                  const LayerTable& ks, const LayerTable& vs, cudaStream_t st);
// bf16, head_dim 128 or 64, group size <= 32: tensor-core path.
bool decode_mma_supported(const lt_shape& s);
cudaError_t launch_decode_mma(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                              const LayerTable& ks, const LayerTable& vs, cudaStream_t st);

// A validated decode call, ready to launch: the two halves of lt_hybrid_decode_attn / lt_decode_step,
// split so that a caller can put its own stream work between the host-side checks and the launches.
struct DecodeCall {
  DecodeArgs a;
  LayerTable kf, vf, ks, vs;
};
// Every check the host can make; enqueues nothing.  `ws` only has its address and size looked at.
lt_status decode_prepare(DecodeCall* c, const lt_shape* shape, const void* q, const void* k_new, const void* v_new,
                         const void* const* k_full, const void* const* v_full, const void* const* k_stream,
                         const void* const* v_stream, const uint8_t* layer_mask, int32_t* seq_lens, void* out,
                         int32_t out_dtype, int32_t layer_begin, int32_t layer_count, int fused, int advance,
                         void* ws, size_t ws_bytes, int layered = 0, int independent = 0);
// Bytes of the split-KV region when every layer has partial slots of its own (lt_decode_step_layers).
size_t layered_decode_bytes(const lt_shape& s);
lt_status decode_launch(const DecodeCall& c, void* stream);

struct ScoreArgs {
  lt_shape s;
  const void* q_tail;
  const float* lse;  // window_only: natural-log denominators [L][B][Hq][T]
  float* lse_out;    // full pass only, may be NULL: receives the denominators it computed, same layout
  int n_ctx, w_last;
  int layer_begin, layer_count;  // layers scored by this call; q_tail, stats and scores keep their whole-stack indexing
  int window_only;
  int n_splits, split_len;
  // tensor-core path only: the persistent launch
  int streamk;             // 1: CTAs own contiguous tile ranges and n_splits = 2 x the pieces of a unit; 0: n_splits = 2 x
                           // the host splits (a row's statistics of a piece or split come in two slots, one per half
                           // of a tile's keys)
  int grid;                // CTAs
  int row_blocks;          // blocks of kScoreBlockM query rows per (layer, b, kv head)
  int n_units;             // layer_count * B * Hkv * row_blocks
  int tiles_per_unit;      // streamk: ceil(n_ctx / kScoreBlockN)
  long long total_tiles;   // streamk: n_units * tiles_per_unit
  float cs;      // softmax scale * log2(e)
  float* stats;  // workspace
  float* scores;
  uint32_t* dev_err;
  // 8-bit keys (tensor-core path): q_tail as two E4M3 terms per element, q = q8_scale[row] * (hi + lo), made by
  // the call itself in the workspace: q8 holds the hi rows [q8_rows][head_dim], then the lo rows
  uint8_t* q8;
  float* q8_scale;     // [q8_rows]
  long long q8_rows;   // n_layers * batch * n_q_heads * w_last
};
// Workspace bytes of the two-term query copy for w_last tail queries (0 unless the caches are 8-bit).
size_t score_q8_bytes(const lt_shape& s, int w_last);
// Key range [*k0, *k1) of split sp (see ScorePlan).
__host__ __device__ inline void score_split_range(const ScoreArgs& a, int sp, int* k0, int* k1) {
  if (!a.window_only) {
    *k0 = sp * a.split_len;
    *k1 = (*k0 + a.split_len < a.n_ctx) ? *k0 + a.split_len : a.n_ctx;
    if (*k0 > a.n_ctx) *k0 = a.n_ctx;
    return;
  }
  const int S = a.s.n_sink < a.n_ctx ? a.s.n_sink : a.n_ctx;
  if (a.s.n_sink > 0) {
    if (sp == 0) {
      *k0 = 0;
      *k1 = S;
      return;
    }
    sp -= 1;
  }
  int w0 = a.n_ctx - a.s.n_recent - (a.s.recent_per_row ? a.w_last - 1 : 0);  // first key any tail row keeps
  if (w0 < S) w0 = S;
  *k0 = w0 + sp * a.split_len;
  if (*k0 > a.n_ctx) *k0 = a.n_ctx;
  *k1 = (*k0 + a.split_len < a.n_ctx) ? *k0 + a.split_len : a.n_ctx;
}
cudaError_t launch_scores_generic(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st);
// bf16 queries, head_dim 128 or 64 (8-bit keys: 128): tcgen05 / TMEM path.
bool scores_umma_supported(const lt_shape& s, int w_last);
cudaError_t launch_scores_umma(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st);
cudaError_t launch_scores_finish(const ScoreArgs& a, cudaStream_t st);

cudaError_t launch_select(const float* scores, int L, int B, int Hq, int n_lazy, uint8_t* mask,
                          float* ratio, cudaStream_t st);

cudaError_t launch_select_per_seq(const float* scores, int L, int B, int Hq, int n_lazy, uint8_t* mask, float* ratio,
                                  cudaStream_t st);
cudaError_t launch_select_frequency(const uint8_t* masks, int N, int L, int n_lazy, uint8_t* mask, int32_t* counts,
                                    cudaStream_t st);
cudaError_t launch_select_push(const float* scores_l, int layer, int L, int per_layer, int n_full, double* state,
                               uint8_t* mask, int32_t* popped, cudaStream_t st);

}  // namespace lt
