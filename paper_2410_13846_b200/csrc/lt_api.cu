// C-ABI entry points of liblt: argument validation, workspace carving and
// stream-ordered launches.  No device memory is allocated here.  The only state
// that survives a call is what the library looks up once per device (SM count,
// kernel attributes, the driver's tensor-map encoder), each behind a lock, so
// calls from several host threads are safe.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "lt_internal.h"

namespace lt {

lt_status validate_shape(const lt_shape* s) {
  if (!s) return LT_ERR_INVALID_ARG;
  if (s->n_layers < 1 || s->batch < 1 || s->n_kv_heads < 1 || s->n_q_heads < 1) return LT_ERR_INVALID_ARG;
  if (s->n_q_heads % s->n_kv_heads != 0) return LT_ERR_INVALID_ARG;
  if (s->n_sink < 0 || s->n_recent < 1 || s->full_capacity < 1) return LT_ERR_INVALID_ARG;
  if ((int64_t)s->n_sink + s->n_recent > (1 << 30)) return LT_ERR_INVALID_ARG;
  if (s->n_layers > LT_MAX_LAYERS) return LT_ERR_UNSUPPORTED;
  if (s->head_dim != 64 && s->head_dim != 128) return LT_ERR_UNSUPPORTED;
  if (s->dtype != LT_F32 && s->dtype != LT_BF16) return LT_ERR_UNSUPPORTED;
  if (!(s->softmax_scale == s->softmax_scale)) return LT_ERR_INVALID_ARG;  // NaN
  if ((s->per_sequence_mask | s->recent_per_row) & ~1) return LT_ERR_INVALID_ARG;
  if (s->page_size < 0 || s->reserved_ != 0 || s->reserved2_ != 0) return LT_ERR_INVALID_ARG;
  if (s->kv_fp8 & ~1) return LT_ERR_INVALID_ARG;
  if (s->kv_fp8) {
    if (!s->kv_scales) return LT_ERR_INVALID_ARG;
    if (s->dtype != LT_BF16 || s->head_dim != 128 || s->n_q_heads / s->n_kv_heads > 32) return LT_ERR_UNSUPPORTED;
  }
  if (s->page_size > 0) {
    if (s->page_size % 128 != 0) return LT_ERR_UNSUPPORTED;
    if (s->pages_per_seq < 1 || s->n_pages < 1 || !s->block_table) return LT_ERR_INVALID_ARG;
    if ((int64_t)s->pages_per_seq * s->page_size != s->full_capacity) return LT_ERR_INVALID_ARG;
    if ((int64_t)s->n_pages * s->n_kv_heads * s->page_size >= (1ll << 31)) return LT_ERR_UNSUPPORTED;
  }
  return LT_OK;
}

DecodePlan make_decode_plan(const lt_shape& s) {
  DecodePlan p;
  const int64_t n_max = (int64_t)((s.full_capacity > s.n_sink + s.n_recent) ? s.full_capacity
                                                                            : s.n_sink + s.n_recent);
  const int64_t units = (int64_t)s.n_layers * s.batch * s.n_kv_heads;
  // Measured on B200 (32K context, whole stack and one layer per call): long chunks win, per-item
  // hand-off costs more than an uneven last round; shorter chunks only pay when a launch has very few keys.
  p.min_chunk = 512;
  // 8-bit caches: 8192-key chunks measured 9 % faster than 2048-key ones (the hand-off between items, four CTA
  // barriers, weighs more the less time an item's bytes take).
  // The 16-bit path: 4096-key chunks when the launch still has a few of them per CTA (at least 2 * target_items *
  // 4096 keys, a whole stack at long context: fewer hand-offs, and contexts up to 4096 need no split at all),
  // 2048 otherwise (one layer per call, where long chunks leave the last round of the grid half empty).
  p.max_chunk = s.kv_fp8 ? 8192 : 4096;
  p.mid_chunk = s.kv_fp8 ? 8192 : 2048;
  p.target_items = 592;
  // chunk = clamp(ceil(keys / target), min, max or mid) gives at most target + units items when it is not clamped
  // from above, units * ceil(n_max / max) when it is clamped at max, fewer than 2 * target * max / mid + units when
  // it is clamped at mid (such a launch has fewer than 2 * target * max keys), and never more than with every
  // chunk at its shortest
  int64_t cap = units * ((n_max + p.max_chunk - 1) / p.max_chunk);
  const int64_t few = 2 * (int64_t)p.target_items * p.max_chunk / p.mid_chunk;
  if (cap < few) cap = few;
  cap += p.target_items + units;
  const int64_t shortest = units * ((n_max + p.min_chunk - 1) / p.min_chunk);
  if (cap > shortest) cap = shortest;
  if (cap > (int64_t)0x7fffffff) cap = 0x7fffffff;
  p.items_cap = (int)cap;
  // One layer's share of any launch: chunk >= ceil(keys / target) gives at most target + units items, a chunk
  // clamped from above is at least mid_chunk long; a launch over k layers has at most k times this.
  const int64_t units_l = (int64_t)s.batch * s.n_kv_heads;
  int64_t lcap = units_l * ((n_max + p.mid_chunk - 1) / p.mid_chunk);
  if (lcap < p.target_items + units_l) lcap = p.target_items + units_l;
  if (lcap * s.n_layers > (int64_t)0x7fffffff) lcap = 0x7fffffff / s.n_layers;
  p.layer_items_cap = (int)lcap;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int gp = G;  // heads per partial slot
  p.ml_floats = (size_t)cap * gp * 2;
  p.o_floats = (size_t)cap * gp * s.head_dim;
  return p;
}

// Host-side key splits of one (layer, batch row, kv head) when `layers` layers are scored by one call.
static int host_score_splits(const lt_shape& s, int n_ctx, int w_last, bool window_only, int layers, int* split_len) {
  const int64_t units = (int64_t)layers * s.batch * s.n_kv_heads;
  int64_t want = (148 * 4 + units - 1) / units;  // a few CTAs per SM even for small stacks
  int span = n_ctx;                              // keys that are divided among the splits
  if (window_only) {
    const int S = s.n_sink < n_ctx ? s.n_sink : n_ctx;
    int w0 = n_ctx - s.n_recent - (s.recent_per_row ? w_last - 1 : 0);
    if (w0 < S) w0 = S;
    span = n_ctx - w0;
  }
  // shortest split: 1024 keys on the tensor-core path; the CUDA-core kernel walks a split tile by tile in one CTA,
  // so small problems are cut finer there to fill the GPU
  const int shortest = scores_umma_supported(s, w_last) ? 1024 : 128;
  int64_t most = (span + shortest - 1) / shortest;
  if (want > most) want = most;
  if (want < 1) want = 1;
  int len = (int)((span + want - 1) / want);
  len = (len + 63) / 64 * 64;
  if (len < 64) len = 64;
  *split_len = len;
  int n = (int)((span + len - 1) / len);
  if (n < 1) n = 1;
  if (window_only && s.n_sink > 0) n += 1;
  return n;
}

ScorePlan make_score_plan(const lt_shape& s, int n_ctx, int w_last, bool window_only, int layer_count) {
  ScorePlan p;
  const size_t rows_per_layer = (size_t)s.batch * s.n_q_heads * w_last;
  if (layer_count > 0) {
    p.n_splits = host_score_splits(s, n_ctx, w_last, window_only, layer_count, &p.split_len);
    p.stat_floats = (size_t)layer_count * rows_per_layer * p.n_splits * 3;
    return p;
  }
  // Workspace query: room for a call over any layer range with any prompt length up to n_ctx and any
  // tail length up to w_last, through either kernel.  The persistent tensor-core kernel cuts a unit into at
  // most (CTAs / units) + 2 pieces, never more than it has tiles.
  // The tensor-core kernel writes two slots per piece or split (one per half of a tile's keys).
  const bool umma = scores_umma_supported(s, w_last);
  const int64_t tiles = (n_ctx + kScoreBlockN - 1) / kScoreBlockN;
  size_t most_slots = 0;  // max over c of c * slots(c)
  p.n_splits = 1;
  p.split_len = 64;
  for (int c = 1; c <= s.n_layers; ++c) {
    int len = 0;
    int64_t slots = host_score_splits(s, n_ctx, w_last, window_only, c, &len) + 1;  // + 1: rounding of shorter prompts
    if (umma) {
      slots *= 2;
      if (!window_only) {
        int64_t pieces = kScoreMaxCtas / ((int64_t)c * s.batch * s.n_kv_heads) + 2;
        if (pieces > tiles) pieces = tiles;
        if (2 * pieces > slots) slots = 2 * pieces;
      }
    }
    if ((size_t)(c * slots) > most_slots) most_slots = (size_t)(c * slots);
    if (slots > p.n_splits) p.n_splits = (int)slots;
  }
  p.stat_floats = rows_per_layer * most_slots * 3;
  return p;
}

size_t score_q8_bytes(const lt_shape& s, int w_last) {
  if (!s.kv_fp8 || w_last < 1) return 0;
  const size_t rows = (size_t)s.n_layers * s.batch * s.n_q_heads * w_last;
  return round_up(2 * rows * s.head_dim, kWsAlign) + round_up(rows * sizeof(float), kWsAlign);
}

size_t ws_prefix_bytes(const lt_shape& s) {
  const size_t counters = ((size_t)s.n_layers * s.batch * s.n_kv_heads + 2 * (size_t)s.n_layers) * sizeof(int);
  return kWsHeaderBytes + round_up(counters, kWsAlign);
}

size_t layered_decode_bytes(const lt_shape& s) {
  const DecodePlan dp = make_decode_plan(s);
  const size_t slots = (size_t)dp.layer_items_cap * s.n_layers;
  const size_t G = s.n_q_heads / s.n_kv_heads;
  return round_up(slots * G * 2 * 4, kWsAlign) + round_up(slots * G * s.head_dim * 4, kWsAlign);
}

int sm_count_of_current_device() {
  static std::mutex mu;
  static int sm_count[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  std::lock_guard<std::mutex> lock(mu);
  if (sm_count[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    sm_count[dev] = n;
  }
  return sm_count[dev];
}

int persistent_grid(const DecodeArgs& a, int ctas_per_sm) {
  const long long most = a.items_cap;
  long long grid = (long long)sm_count_of_current_device() * ctas_per_sm;
  if (grid > most) grid = most;
  return (int)(grid < 1 ? 1 : grid);
}

static lt_status fill_table(LayerTable* t, const void* const* host, int L, bool require_all) {
  memset(t, 0, sizeof(*t));
  if (!host) return require_all ? LT_ERR_INVALID_ARG : LT_OK;
  for (int l = 0; l < L; ++l) {
    t->p[l] = host[l];
    if (require_all && !host[l]) return LT_ERR_INVALID_ARG;
    if (((uintptr_t)host[l] & 15u) != 0) return LT_ERR_INVALID_ARG;
  }
  return LT_OK;
}

// Entries of [begin, begin + count) must be present; the rest of the table is not looked at.
static lt_status fill_table_range(LayerTable* t, const void* const* host, int begin, int count) {
  memset(t, 0, sizeof(*t));
  if (!host) return LT_ERR_INVALID_ARG;
  for (int l = begin; l < begin + count; ++l) {
    if (!host[l] || ((uintptr_t)host[l] & 15u) != 0) return LT_ERR_INVALID_ARG;
    t->p[l] = host[l];
  }
  return LT_OK;
}

static lt_status check_layer_range(const lt_shape* s, int begin, int count) {
  if (begin < 0 || count < 1 || begin + count > s->n_layers) return LT_ERR_INVALID_ARG;
  return LT_OK;
}

static inline uint32_t* err_word(void* ws) { return reinterpret_cast<uint32_t*>(ws); }

}  // namespace lt

using namespace lt;

extern "C" {

const char* lt_status_string(lt_status s) {
  switch (s) {
    case LT_OK: return "ok";
    case LT_ERR_INVALID_ARG: return "invalid argument";
    case LT_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case LT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case LT_ERR_CUDA: return "CUDA runtime error";
    case LT_ERR_TIMEOUT: return "device wait timed out";
    case LT_ERR_DEVICE_RANGE: return "device error word set (position or length out of range)";
    default: return "unknown status";
  }
}

int32_t lt_version(void) { return 200; }

int32_t lt_ring_slot(int32_t pos, int32_t n_sink, int32_t n_recent) {
  if (pos < 0 || n_sink < 0 || n_recent < 1) return -1;
  if (pos < n_sink) return pos;
  return n_sink + (pos - n_sink) % n_recent;
}

lt_status lt_workspace_bytes(const lt_shape* shape, int32_t n_ctx_max, int32_t w_last_max, size_t* bytes_out) {
  lt_status st = validate_shape(shape);
  if (st != LT_OK) return st;
  if (!bytes_out || n_ctx_max < 0 || w_last_max < 0) return LT_ERR_INVALID_ARG;
  DecodePlan dp = make_decode_plan(*shape);
  size_t decode_bytes = round_up(dp.ml_floats * 4, kWsAlign) + round_up(dp.o_floats * 4, kWsAlign);
  size_t score_bytes = 0;
  if (n_ctx_max > 0 && w_last_max > 0) {
    const ScorePlan sp = make_score_plan(*shape, n_ctx_max, w_last_max, false);
    const ScorePlan sw = make_score_plan(*shape, n_ctx_max, w_last_max, true);
    score_bytes = round_up((sp.stat_floats > sw.stat_floats ? sp.stat_floats : sw.stat_floats) * 4, kWsAlign);
    score_bytes += score_q8_bytes(*shape, w_last_max);  // 8-bit keys: the call's two-term copy of q_tail
  }
  *bytes_out = ws_prefix_bytes(*shape) + (decode_bytes > score_bytes ? decode_bytes : score_bytes);
  return LT_OK;
}

lt_status lt_workspace_bytes_layers(const lt_shape* shape, int32_t n_ctx_max, int32_t w_last_max, size_t* bytes_out) {
  lt_status st = lt_workspace_bytes(shape, n_ctx_max, w_last_max, bytes_out);
  if (st != LT_OK) return st;
  const size_t layered = ws_prefix_bytes(*shape) + layered_decode_bytes(*shape);
  if (layered > *bytes_out) *bytes_out = layered;
  return LT_OK;
}

lt_status lt_workspace_init(void* ws, size_t ws_bytes, void* stream) {
  if (!ws || ws_bytes < kWsHeaderBytes || ((uintptr_t)ws % kWsAlign) != 0) return LT_ERR_WORKSPACE;
  // error word and the decode step's counters start at zero; the rest is scratch
  cudaError_t e = cudaMemsetAsync(ws, 0, ws_bytes, (cudaStream_t)stream);
  return e == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

lt_status lt_check(void* ws, uint32_t* flags_out, void* stream) {
  if (!ws) return LT_ERR_WORKSPACE;
  uint32_t flags = 0;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(&flags, ws, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess) return LT_ERR_CUDA;
  if (cudaMemsetAsync(ws, 0, sizeof(flags), st) != cudaSuccess) return LT_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LT_ERR_CUDA;
  if (flags_out) *flags_out = flags;
  if (flags & LT_DEVERR_TIMEOUT) return LT_ERR_TIMEOUT;  // the scores of that call are invalid
  return flags ? LT_ERR_DEVICE_RANGE : LT_OK;
}

// Shared body of lt_lazy_scores (lse == NULL) and lt_lazy_scores_lse.
static lt_status scores_impl(const lt_shape* shape, const void* q_tail, const void* const* k_full, const float* lse,
                             int window_only, int32_t n_ctx, int32_t w_last, int32_t layer_begin,
                             int32_t layer_count, float* scores, void* ws, size_t ws_bytes, void* stream,
                             float* lse_out = nullptr) {
  lt_status st = validate_shape(shape);
  if (st != LT_OK) return st;
  if (!q_tail || !k_full || !scores) return LT_ERR_INVALID_ARG;
  if (window_only && !lse) return LT_ERR_INVALID_ARG;
  // 8-bit keys are scored by the tensor-core kernel only (E4M3 MMAs on the stored bytes)
  if (shape->kv_fp8 && !scores_umma_supported(*shape, w_last)) return LT_ERR_UNSUPPORTED;
  if (w_last < 1 || w_last > n_ctx || n_ctx > shape->full_capacity) return LT_ERR_INVALID_ARG;
  if (((uintptr_t)q_tail & 15u) != 0 || ((uintptr_t)lse & 3u) != 0 || ((uintptr_t)lse_out & 3u) != 0)
    return LT_ERR_INVALID_ARG;
  if ((st = check_layer_range(shape, layer_begin, layer_count)) != LT_OK) return st;
  LayerTable kf;
  if ((st = fill_table_range(&kf, k_full, layer_begin, layer_count)) != LT_OK) return st;
  const bool umma = scores_umma_supported(*shape, w_last);
  ScorePlan sp = make_score_plan(*shape, n_ctx, w_last, window_only != 0, layer_count);
  ScoreArgs a;
  memset(&a, 0, sizeof(a));
  if (umma) {
    // the persistent launch: one CTA per SM; with the whole prompt scored the CTAs own contiguous tile ranges
    a.row_blocks = ((shape->n_q_heads / shape->n_kv_heads) * w_last + kScoreBlockM - 1) / kScoreBlockM;
    a.n_units = layer_count * shape->batch * shape->n_kv_heads * a.row_blocks;
    a.streamk = window_only ? 0 : 1;
    a.tiles_per_unit = (n_ctx + kScoreBlockN - 1) / kScoreBlockN;
    a.total_tiles = (long long)a.n_units * a.tiles_per_unit;
    const long long work = a.streamk ? a.total_tiles : (long long)a.n_units * sp.n_splits;  // tiles, or host splits
    int grid = sm_count_of_current_device();
    if (grid > kScoreMaxCtas) grid = kScoreMaxCtas;
    if (grid > work) grid = (int)work;
    a.grid = grid < 1 ? 1 : grid;
    if (a.streamk) {
      // most pieces any unit is cut into under this grid: owner(last tile) - owner(first tile) + 1
      long long pieces = ((long long)(a.tiles_per_unit - 1) * a.grid) / a.total_tiles + 2;
      if (pieces > a.tiles_per_unit) pieces = a.tiles_per_unit;
      sp.n_splits = (int)pieces;
    }
    sp.n_splits *= 2;  // two statistics slots per piece or split: one per half of a tile's keys
    sp.stat_floats = (size_t)layer_count * shape->batch * shape->n_q_heads * w_last * sp.n_splits * 3;
  }
  if (!ws || ((uintptr_t)ws % kWsAlign) != 0) return LT_ERR_WORKSPACE;
  const size_t prefix = ws_prefix_bytes(*shape);
  const size_t stat_bytes = round_up(sp.stat_floats * 4, kWsAlign);
  if (ws_bytes < prefix + stat_bytes + score_q8_bytes(*shape, w_last)) return LT_ERR_WORKSPACE;
  a.s = *shape;
  a.q_tail = q_tail;
  a.lse = lse;
  a.lse_out = lse_out;
  a.n_ctx = n_ctx;
  a.w_last = w_last;
  a.layer_begin = layer_begin;
  a.layer_count = layer_count;
  a.window_only = window_only;
  a.n_splits = sp.n_splits;
  a.split_len = sp.split_len;
  a.stats = reinterpret_cast<float*>((char*)ws + prefix);
  a.scores = scores;
  a.cs = resolved_scale(*shape) * 1.4426950408889634f;
  a.dev_err = err_word(ws);
  if (shape->kv_fp8) {
    a.q8_rows = (long long)shape->n_layers * shape->batch * shape->n_q_heads * w_last;
    a.q8 = reinterpret_cast<uint8_t*>((char*)ws + prefix + stat_bytes);
    a.q8_scale = reinterpret_cast<float*>(a.q8 + round_up(2 * (size_t)a.q8_rows * shape->head_dim, kWsAlign));
  }
  cudaStream_t cs = (cudaStream_t)stream;
  cudaError_t e = umma ? launch_scores_umma(a, kf, cs) : launch_scores_generic(a, kf, cs);
  if (e != cudaSuccess) return LT_ERR_CUDA;
  e = launch_scores_finish(a, cs);
  return e == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

lt_status lt_lazy_scores(const lt_shape* shape, const void* q_tail, const void* const* k_full, int32_t n_ctx,
                         int32_t w_last, int32_t layer_begin, int32_t layer_count, float* scores, void* ws,
                         size_t ws_bytes, void* stream) {
  return scores_impl(shape, q_tail, k_full, nullptr, 0, n_ctx, w_last, layer_begin, layer_count, scores, ws, ws_bytes,
                     stream);
}

lt_status lt_lazy_scores_with_lse(const lt_shape* shape, const void* q_tail, const void* const* k_full, int32_t n_ctx,
                                  int32_t w_last, int32_t layer_begin, int32_t layer_count, float* scores,
                                  float* lse_out, void* ws, size_t ws_bytes, void* stream) {
  if (!lse_out) return LT_ERR_INVALID_ARG;
  return scores_impl(shape, q_tail, k_full, nullptr, 0, n_ctx, w_last, layer_begin, layer_count, scores, ws, ws_bytes,
                     stream, lse_out);
}

lt_status lt_lazy_scores_lse(const lt_shape* shape, const void* q_tail, const void* const* k_full, const float* lse,
                             int32_t n_ctx, int32_t w_last, int32_t layer_begin, int32_t layer_count, float* scores,
                             void* ws, size_t ws_bytes, void* stream) {
  return scores_impl(shape, q_tail, k_full, lse, 1, n_ctx, w_last, layer_begin, layer_count, scores, ws, ws_bytes,
                     stream);
}

lt_status lt_select_lazy(const float* scores, int32_t n_layers, int32_t batch, int32_t n_q_heads, int32_t n_lazy,
                         uint8_t* layer_mask, float* layer_ratio, void* stream) {
  if (!scores || !layer_mask) return LT_ERR_INVALID_ARG;
  if (n_layers < 1 || batch < 1 || n_q_heads < 1) return LT_ERR_INVALID_ARG;
  if (n_layers > LT_MAX_LAYERS) return LT_ERR_UNSUPPORTED;
  if (n_lazy < 0 || n_lazy > n_layers) return LT_ERR_INVALID_ARG;
  cudaError_t e = launch_select(scores, n_layers, batch, n_q_heads, n_lazy, layer_mask, layer_ratio,
                                (cudaStream_t)stream);
  return e == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

lt_status lt_select_lazy_per_seq(const float* scores, int32_t n_layers, int32_t batch, int32_t n_q_heads,
                                 int32_t n_lazy, uint8_t* layer_mask, float* layer_ratio, void* stream) {
  if (!scores || !layer_mask) return LT_ERR_INVALID_ARG;
  if (n_layers < 1 || batch < 1 || n_q_heads < 1) return LT_ERR_INVALID_ARG;
  if (n_layers > LT_MAX_LAYERS) return LT_ERR_UNSUPPORTED;
  if (n_lazy < 0 || n_lazy > n_layers) return LT_ERR_INVALID_ARG;
  cudaError_t e = launch_select_per_seq(scores, n_layers, batch, n_q_heads, n_lazy, layer_mask, layer_ratio,
                                        (cudaStream_t)stream);
  return e == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

lt_status lt_select_lazy_frequency(const uint8_t* sample_masks, int32_t n_samples, int32_t n_layers, int32_t n_lazy,
                                   uint8_t* layer_mask, int32_t* layer_counts, void* stream) {
  if (!sample_masks || !layer_mask) return LT_ERR_INVALID_ARG;
  if (n_samples < 1 || n_layers < 1) return LT_ERR_INVALID_ARG;
  if (n_layers > LT_MAX_LAYERS) return LT_ERR_UNSUPPORTED;
  if (n_lazy < 0 || n_lazy > n_layers) return LT_ERR_INVALID_ARG;
  cudaError_t e = launch_select_frequency(sample_masks, n_samples, n_layers, n_lazy, layer_mask, layer_counts,
                                          (cudaStream_t)stream);
  return e == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

lt_status lt_select_lazy_push(const float* layer_scores, int32_t layer, int32_t n_layers, int32_t batch,
                              int32_t n_q_heads, int32_t n_full, void* queue_state, uint8_t* layer_mask,
                              int32_t* popped_layer, void* stream) {
  if (!layer_scores || !queue_state || !layer_mask) return LT_ERR_INVALID_ARG;
  if (n_layers < 1 || batch < 1 || n_q_heads < 1) return LT_ERR_INVALID_ARG;
  if (n_layers > LT_MAX_LAYERS) return LT_ERR_UNSUPPORTED;
  if (layer < 0 || layer >= n_layers || n_full < 0 || n_full > n_layers) return LT_ERR_INVALID_ARG;
  if (((uintptr_t)queue_state & 7u) != 0) return LT_ERR_INVALID_ARG;
  cudaError_t e = launch_select_push(layer_scores, layer, n_layers, batch * n_q_heads, n_full,
                                     reinterpret_cast<double*>(queue_state), layer_mask, popped_layer,
                                     (cudaStream_t)stream);
  return e == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

static lt_status stream_init_impl(const lt_shape* shape, const uint8_t* layer_mask, const void* const* k_full,
                                  const void* const* v_full, const int32_t* seq_lens, void* const* k_stream,
                                  void* const* v_stream, const int32_t* only_layer, void* ws, void* stream) {
  lt_status st = validate_shape(shape);
  if (st != LT_OK) return st;
  if (!layer_mask || !k_full || !v_full || !seq_lens || !k_stream || !v_stream) return LT_ERR_INVALID_ARG;
  if (ws && ((uintptr_t)ws % kWsAlign) != 0) return LT_ERR_WORKSPACE;
  LayerTable kf, vf, ks, vs;
  const int L = shape->n_layers;
  if ((st = fill_table(&kf, k_full, L, false)) != LT_OK) return st;
  if ((st = fill_table(&vf, v_full, L, false)) != LT_OK) return st;
  if ((st = fill_table(&ks, (const void* const*)k_stream, L, false)) != LT_OK) return st;
  if ((st = fill_table(&vs, (const void* const*)v_stream, L, false)) != LT_OK) return st;
  cudaError_t e = launch_stream_init(*shape, layer_mask, kf, vf, seq_lens, ks, vs, only_layer,
                                     ws ? err_word(ws) : nullptr, (cudaStream_t)stream);
  return e == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

lt_status lt_stream_init(const lt_shape* shape, const uint8_t* layer_mask, const void* const* k_full,
                         const void* const* v_full, const int32_t* seq_lens, void* const* k_stream,
                         void* const* v_stream, void* ws, void* stream) {
  return stream_init_impl(shape, layer_mask, k_full, v_full, seq_lens, k_stream, v_stream, nullptr, ws, stream);
}

lt_status lt_stream_init_layer(const lt_shape* shape, const uint8_t* layer_mask, const int32_t* layer,
                               const void* const* k_full, const void* const* v_full, const int32_t* seq_lens,
                               void* const* k_stream, void* const* v_stream, void* ws, void* stream) {
  if (!layer) return LT_ERR_INVALID_ARG;
  return stream_init_impl(shape, layer_mask, k_full, v_full, seq_lens, k_stream, v_stream, layer, ws, stream);
}

lt_status lt_kv_append(const lt_shape* shape, const uint8_t* layer_mask, const void* k_new, const void* v_new,
                       int32_t* seq_lens, void* const* k_full, void* const* v_full, void* const* k_stream,
                       void* const* v_stream, int32_t layer_begin, int32_t layer_count, int32_t advance_seq_lens,
                       void* ws, void* stream) {
  lt_status st = validate_shape(shape);
  if (st != LT_OK) return st;
  if (!layer_mask || !k_new || !v_new || !seq_lens) return LT_ERR_INVALID_ARG;
  if (!k_full && !k_stream) return LT_ERR_INVALID_ARG;
  if ((k_full == nullptr) != (v_full == nullptr) || (k_stream == nullptr) != (v_stream == nullptr))
    return LT_ERR_INVALID_ARG;
  if ((((uintptr_t)k_new | (uintptr_t)v_new) & 15u) != 0) return LT_ERR_INVALID_ARG;
  if ((st = check_layer_range(shape, layer_begin, layer_count)) != LT_OK) return st;
  if (ws && ((uintptr_t)ws % kWsAlign) != 0) return LT_ERR_WORKSPACE;
  LayerTable kf, vf, ks, vs;
  const int L = shape->n_layers;
  if ((st = fill_table(&kf, (const void* const*)k_full, L, false)) != LT_OK) return st;
  if ((st = fill_table(&vf, (const void* const*)v_full, L, false)) != LT_OK) return st;
  if ((st = fill_table(&ks, (const void* const*)k_stream, L, false)) != LT_OK) return st;
  if ((st = fill_table(&vs, (const void* const*)v_stream, L, false)) != LT_OK) return st;
  cudaError_t e = launch_append(*shape, layer_mask, k_new, v_new, seq_lens, kf, vf, ks, vs, layer_begin, layer_count,
                                advance_seq_lens, ws ? err_word(ws) : nullptr, (cudaStream_t)stream);
  return e == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

}  // extern "C"

// Shared body of lt_hybrid_decode_attn (k_new == NULL) and lt_decode_step, in two halves: every check that
// the host can make (nothing is enqueued), then the launches.
lt_status lt::decode_prepare(DecodeCall* c, const lt_shape* shape, const void* q, const void* k_new, const void* v_new,
                             const void* const* k_full, const void* const* v_full, const void* const* k_stream,
                             const void* const* v_stream, const uint8_t* layer_mask, int32_t* seq_lens, void* out,
                             int32_t out_dtype, int32_t layer_begin, int32_t layer_count, int fused, int advance,
                             void* ws, size_t ws_bytes, int layered, int independent) {
  lt_status st = validate_shape(shape);
  if (st != LT_OK) return st;
  if (!q || !layer_mask || !seq_lens || !out) return LT_ERR_INVALID_ARG;
  if (fused && (!k_new || !v_new)) return LT_ERR_INVALID_ARG;
  if (!k_full && !k_stream) return LT_ERR_INVALID_ARG;
  if ((k_full == nullptr) != (v_full == nullptr) || (k_stream == nullptr) != (v_stream == nullptr))
    return LT_ERR_INVALID_ARG;
  if (out_dtype != LT_F32 && out_dtype != LT_BF16) return LT_ERR_UNSUPPORTED;
  if ((((uintptr_t)q | (uintptr_t)out | (uintptr_t)k_new | (uintptr_t)v_new) & 15u) != 0) return LT_ERR_INVALID_ARG;
  if ((st = check_layer_range(shape, layer_begin, layer_count)) != LT_OK) return st;
  if (shape->batch > kMaxWorkEntries) return LT_ERR_UNSUPPORTED;
  const int L = shape->n_layers;
  if ((st = fill_table(&c->kf, k_full, L, false)) != LT_OK) return st;
  if ((st = fill_table(&c->vf, v_full, L, false)) != LT_OK) return st;
  if ((st = fill_table(&c->ks, k_stream, L, false)) != LT_OK) return st;
  if ((st = fill_table(&c->vs, v_stream, L, false)) != LT_OK) return st;

  DecodePlan dp = make_decode_plan(*shape);
  const size_t prefix = ws_prefix_bytes(*shape);
  // layered: every layer owns layer_items_cap partial slots, so that launches over different layers can be in
  // flight together; otherwise every launch starts at slot 0
  const size_t slots = layered ? (size_t)dp.layer_items_cap * shape->n_layers : (size_t)dp.items_cap;
  const size_t G = shape->n_q_heads / shape->n_kv_heads;
  const size_t ml_bytes = round_up(slots * G * 2 * 4, kWsAlign);
  const size_t o_bytes = round_up(slots * G * shape->head_dim * 4, kWsAlign);
  if (!ws || ((uintptr_t)ws % kWsAlign) != 0) return LT_ERR_WORKSPACE;
  if (ws_bytes < prefix + ml_bytes + o_bytes) return LT_ERR_WORKSPACE;

  DecodeArgs& a = c->a;
  a.s = *shape;
  a.q = q;
  a.k_new = k_new;
  a.v_new = v_new;
  a.mask = layer_mask;
  a.seq_lens = seq_lens;
  a.seq_lens_rw = seq_lens;
  a.out = out;
  a.out_dtype = out_dtype;
  a.min_chunk = dp.min_chunk;
  a.max_chunk = dp.max_chunk;
  a.mid_chunk = dp.mid_chunk;
  a.target_items = dp.target_items;
  a.items_cap = layered ? dp.layer_items_cap : dp.items_cap;  // layered: per layer, scaled by decode_launch
  a.overlap = (layered && independent) ? 1 : 0;
  a.slot_base = layered ? 1 : 0;  // layered: turned into layer_begin * layer_items_cap by decode_launch
  a.fused = fused;
  a.advance = advance;
  // A call over part of the stack is one of several launches of a step (a model calls layer by layer):
  // let each of them become resident under the tail of the one before.
  a.pdl = layer_count < shape->n_layers ? 1 : 0;
  a.layer_begin = layer_begin;
  a.layer_count = layer_count;
  a.unit_counters = reinterpret_cast<int*>((char*)ws + kWsHeaderBytes);
  a.launch_counters = a.unit_counters + (size_t)shape->n_layers * shape->batch * shape->n_kv_heads;
  a.done_counter = a.launch_counters + 2 * (size_t)layer_begin;
  a.work_counter = a.done_counter + 1;
  a.part_ml = reinterpret_cast<float*>((char*)ws + prefix);
  a.part_o = reinterpret_cast<float*>((char*)ws + prefix + ml_bytes);
  a.dev_err = err_word(ws);
  a.cs = resolved_scale(*shape) * 1.4426950408889634f;
  return LT_OK;
}

lt_status lt::decode_launch(const DecodeCall& c, void* stream) {
  // One launch takes at most kMaxWorkEntries (layer, batch row) pairs; a larger
  // stack goes in consecutive launches by layers (only the last one advances).
  DecodeArgs a = c.a;
  cudaStream_t cs = (cudaStream_t)stream;
  const int layer_begin = c.a.layer_begin, layer_count = c.a.layer_count;
  const int layers_per_launch = kMaxWorkEntries / a.s.batch;
  const bool mma = decode_mma_supported(a.s);
  const bool layered = c.a.slot_base != 0;
  for (int done = 0; done < layer_count; done += layers_per_launch) {
    a.layer_begin = layer_begin + done;
    a.layer_count = layer_count - done < layers_per_launch ? layer_count - done : layers_per_launch;
    a.advance = (c.a.advance && done + a.layer_count == layer_count) ? 1 : 0;
    if (layer_count > layers_per_launch) a.pdl = 1;  // a stack that is split here is several launches too
    a.done_counter = a.launch_counters + 2 * (size_t)a.layer_begin;
    a.work_counter = a.done_counter + 1;
    if (layered) {
      a.slot_base = a.layer_begin * c.a.items_cap;
      a.items_cap = a.layer_count * c.a.items_cap;
      // the later launches of a split call share nothing with the ones before them either; only the tensor-core
      // kernel starts without waiting
      a.overlap = (mma && (c.a.overlap || done > 0)) ? 1 : 0;
      a.pdl = 1;
    }
    cudaError_t e = mma ? launch_decode_mma(a, c.kf, c.vf, c.ks, c.vs, cs) : launch_decode_generic(a, c.kf, c.vf, c.ks, c.vs, cs);
    if (e != cudaSuccess) return LT_ERR_CUDA;
  }
  return LT_OK;
}

static lt_status decode_impl(const lt_shape* shape, const void* q, const void* k_new, const void* v_new,
                             const void* const* k_full, const void* const* v_full, const void* const* k_stream,
                             const void* const* v_stream, const uint8_t* layer_mask, int32_t* seq_lens, void* out,
                             int32_t out_dtype, int32_t layer_begin, int32_t layer_count, int fused, int advance,
                             void* ws, size_t ws_bytes, void* stream) {
  DecodeCall c;
  const lt_status st = decode_prepare(&c, shape, q, k_new, v_new, k_full, v_full, k_stream, v_stream, layer_mask,
                                      seq_lens, out, out_dtype, layer_begin, layer_count, fused, advance, ws, ws_bytes);
  if (st != LT_OK) return st;
  return decode_launch(c, stream);
}

extern "C" {

lt_status lt_hybrid_decode_attn(const lt_shape* shape, const void* q, const void* const* k_full,
                                const void* const* v_full, const void* const* k_stream, const void* const* v_stream,
                                const uint8_t* layer_mask, const int32_t* seq_lens, void* out, int32_t out_dtype,
                                int32_t max_seq_len_hint, int32_t layer_begin, int32_t layer_count, void* ws,
                                size_t ws_bytes, void* stream) {
  (void)max_seq_len_hint;  // the persistent launch sizes itself from the device-side lengths
  return decode_impl(shape, q, nullptr, nullptr, k_full, v_full, k_stream, v_stream, layer_mask,
                     const_cast<int32_t*>(seq_lens), out, out_dtype, layer_begin, layer_count, 0, 0, ws, ws_bytes,
                     stream);
}

lt_status lt_decode_step(const lt_shape* shape, const void* q, const void* k_new, const void* v_new,
                         void* const* k_full, void* const* v_full, void* const* k_stream, void* const* v_stream,
                         const uint8_t* layer_mask, int32_t* seq_lens, void* out, int32_t out_dtype,
                         int32_t layer_begin, int32_t layer_count, int32_t advance_seq_lens, void* ws,
                         size_t ws_bytes, void* stream) {
  return decode_impl(shape, q, k_new, v_new, (const void* const*)k_full, (const void* const*)v_full,
                     (const void* const*)k_stream, (const void* const*)v_stream, layer_mask, seq_lens, out, out_dtype,
                     layer_begin, layer_count, 1, advance_seq_lens ? 1 : 0, ws, ws_bytes, stream);
}

lt_status lt_decode_step_layers(const lt_shape* shape, const void* q, const void* k_new, const void* v_new,
                                void* const* k_full, void* const* v_full, void* const* k_stream,
                                void* const* v_stream, const uint8_t* layer_mask, int32_t* seq_lens, void* out,
                                int32_t out_dtype, int32_t layer_begin, int32_t layer_count,
                                int32_t advance_seq_lens, int32_t independent_of_previous, void* ws, size_t ws_bytes,
                                void* stream) {
  DecodeCall c;
  const lt_status st = decode_prepare(&c, shape, q, k_new, v_new, (const void* const*)k_full,
                                      (const void* const*)v_full, (const void* const*)k_stream,
                                      (const void* const*)v_stream, layer_mask, seq_lens, out, out_dtype, layer_begin,
                                      layer_count, 1, advance_seq_lens ? 1 : 0, ws, ws_bytes, 1,
                                      independent_of_previous ? 1 : 0);
  if (st != LT_OK) return st;
  return decode_launch(c, stream);
}

lt_status lt_decode_step_host(const lt_shape* shape, const void* q_host, const void* k_new_host,
                              const void* v_new_host, void* out_host, void* q_dev, void* k_new_dev, void* v_new_dev,
                              void* out_dev, void* const* k_full, void* const* v_full, void* const* k_stream,
                              void* const* v_stream, const uint8_t* layer_mask, int32_t* seq_lens, int32_t out_dtype,
                              void* ws, size_t ws_bytes, void* stream) {
  lt_status st = validate_shape(shape);
  if (st != LT_OK) return st;
  if (!q_host || !k_new_host || !v_new_host || !out_host || !q_dev || !k_new_dev || !v_new_dev || !out_dev)
    return LT_ERR_INVALID_ARG;
  if (out_dtype != LT_F32 && out_dtype != LT_BF16) return LT_ERR_UNSUPPORTED;
  const size_t e = elem_bytes(shape->dtype);
  const size_t rows = (size_t)shape->n_layers * shape->batch;
  const size_t q_bytes = rows * shape->n_q_heads * shape->head_dim * e;
  const size_t kv_bytes = rows * shape->n_kv_heads * shape->head_dim * e;
  const size_t out_bytes = rows * shape->n_q_heads * shape->head_dim * (out_dtype == LT_F32 ? 4 : 2);
  cudaStream_t cs = (cudaStream_t)stream;
  if (cudaMemcpyAsync(q_dev, q_host, q_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return LT_ERR_CUDA;
  if (cudaMemcpyAsync(k_new_dev, k_new_host, kv_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return LT_ERR_CUDA;
  if (cudaMemcpyAsync(v_new_dev, v_new_host, kv_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return LT_ERR_CUDA;
  st = lt_decode_step(shape, q_dev, k_new_dev, v_new_dev, k_full, v_full, k_stream, v_stream, layer_mask, seq_lens,
                      out_dev, out_dtype, 0, shape->n_layers, 1, ws, ws_bytes, stream);
  if (st != LT_OK) return st;
  if (cudaMemcpyAsync(out_host, out_dev, out_bytes, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return LT_ERR_CUDA;
  return LT_OK;
}

}  // extern "C"
