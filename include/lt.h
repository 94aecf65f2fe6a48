/*
 * lt.h - C ABI of liblt: the hybrid decode-attention path of LightTransfer on
 * one NVIDIA B200 (sm_100a).
 *
 * The method (LightTransfer-Test, Section 5.1 of the paper): after the prompt
 * has been prefilled, every layer gets a "lazy ratio" (Eq. 1) - the share of
 * attention that its last w_last prompt queries put on the first n_sink keys
 * and on the last n_recent keys.  The layers with the highest ratios become
 * "lazy": they keep only those keys/values (a constant-size cache) and decode
 * with streaming attention; every other layer keeps its whole cache and
 * decodes with full attention.
 *
 * Conventions
 *   - Every function returns an lt_status; nothing aborts, throws or traps.
 *   - The caller owns all memory.  The library allocates nothing on the
 *     device and never synchronises the device unless a function says so.  All
 *     device work is enqueued on `stream` (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream).
 *   - State between calls: none that belongs to a caller.  The library caches,
 *     per device and behind locks, what it looks up on first use (SM count,
 *     kernel attributes and occupancy, the driver's tensor-map encoder), so any
 *     number of host threads may call it, first calls included.  Two calls that
 *     share a workspace must still be ordered by the caller.
 *   - "dev" marks a device pointer, "host" a host pointer.
 *   - Layer tables (k_full, v_full, k_stream, v_stream) are HOST arrays of
 *     n_layers DEVICE pointers, read during the call only.  An entry may be
 *     NULL when that layer never takes that role (a layer's role is known
 *     only after lt_select_lazy, so a caller may allocate both kinds for all
 *     layers, or re-allocate after selection).  A NULL entry that the device
 *     mask selects is skipped and reported through the error word.
 *   - Layouts are dense row-major, last index fastest:
 *       full cache of one layer    [batch][n_kv_heads][full_capacity][head_dim]
 *                                  (or a page pool, see lt_shape.page_size)
 *       stream cache of one layer  [batch][n_kv_heads][n_sink+n_recent][head_dim]
 *     Every cache pointer must be 16-byte aligned.
 *   - layer_mask is uint8[n_layers] on the device, 1 = lazy (streaming); with
 *     shape.per_sequence_mask it is uint8[batch][n_layers], one row per prompt.
 *   - seq_lens is int32[batch] on the device: tokens already in the cache of
 *     that batch row = position of the next token.
 *   - A decode step is "append, then attend": the new token attends to itself
 *     (causal mask with i >= j, Appendix E).
 *   - GQA: query head hq reads kv head hq / (n_q_heads / n_kv_heads).
 *   - Every shape the calls accept is computed on the GPU by this library's own
 *     kernels.  The bandwidth-bound tensor-core kernels serve bf16 stacks with
 *     head_dim 64 or 128 (decode: query groups of up to 32 heads; scoring: any
 *     group); fp32 stacks and larger groups run on
 *     tiled CUDA-core kernels, several times slower per byte.
 */
#ifndef LT_H_
#define LT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t lt_status;
enum {
  LT_OK = 0,
  LT_ERR_INVALID_ARG = 1, /* null pointer, bad size, n_lazy outside [0, L], ... */
  LT_ERR_UNSUPPORTED = 2, /* head_dim not in {64,128}, unknown dtype, too many layers */
  LT_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
  LT_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch error) */
  LT_ERR_TIMEOUT = 5,     /* reported by lt_check: a bounded wait inside the scoring kernel (on its copy engine
                             or tensor-core barriers) ran out; that call's scores are invalid */
  LT_ERR_DEVICE_RANGE = 6 /* reported by lt_check: a position left its cache, or a selected layer's table entry was NULL */
};

enum { LT_F32 = 0, LT_BF16 = 1 };

#define LT_MAX_LAYERS 128

/* Bits of the device error word (see lt_check). */
#define LT_DEVERR_POS_OUT_OF_RANGE 1u /* append: seq_len >= full_capacity; store skipped */
#define LT_DEVERR_NULL_LAYER 2u       /* mask selected a layer whose table entry is NULL */
#define LT_DEVERR_LEN_CLAMPED 4u      /* attend: seq_len > full_capacity; clamped */
#define LT_DEVERR_TIMEOUT 8u          /* scoring: a bounded wait inside a kernel expired; scores invalid */

/* Zero-initialise the struct and set what you need: every field after softmax_scale has a zero default. */
typedef struct lt_shape {
  int32_t n_layers;      /* L, 1..LT_MAX_LAYERS */
  int32_t batch;         /* B >= 1 */
  int32_t n_q_heads;     /* Hq, multiple of n_kv_heads */
  int32_t n_kv_heads;    /* Hkv >= 1 */
  int32_t head_dim;      /* D, 64 or 128 */
  int32_t n_sink;        /* w_sink >= 0 (0 = pure sliding window) */
  int32_t n_recent;      /* w_recent >= 1 */
  int32_t full_capacity; /* rows per (batch, kv head) of a full cache */
  int32_t dtype;         /* LT_F32 or LT_BF16: q, k, v and both caches */
  float softmax_scale;   /* <= 0 means 1/sqrt(head_dim) */
  int32_t per_sequence_mask; /* 0: layer_mask is uint8[n_layers], one hybrid for the batch;
                                1: uint8[batch][n_layers], every prompt has its own lazy layers
                                   (Section 4: the lazy layers vary with the prompt) */
  int32_t recent_per_row;    /* scoring only.  0: X_recent is the fixed block of the last n_recent prompt
                                positions (Table 1, the set a lazy layer retains); 1: the recent set of the
                                tail query at position i is i - n_recent + 1 .. i (Appendix E, M_lazy row by row) */
  /* Paged full caches (block tables, as serving engines keep them).  page_size = 0: contiguous caches as
     described above.  page_size > 0 (a multiple of 128): the full cache of a layer is a pool
     [n_pages][n_kv_heads][page_size][head_dim]; token j of batch row b lives in page
     block_table[b][j / page_size] at row j % page_size, and full_capacity must equal
     pages_per_seq * page_size.  One table serves every layer (each layer has its own pool of the same
     geometry).  Stream caches are constant-size and stay contiguous. */
  int32_t page_size;
  int32_t pages_per_seq;       /* columns of block_table */
  int32_t n_pages;             /* pages in every layer's pool */
  int32_t reserved_;           /* keep the pointer 8-byte aligned; must be 0 */
  const int32_t* block_table;  /* dev int32 [batch][pages_per_seq], entries in [0, n_pages); read during device work */
  /* 8-bit caches (not in the paper, which keeps BF16 everywhere, Appendix A; a deployment option).
     kv_fp8 = 1: full and stream caches hold FP8 E4M3 bytes (rows of head_dim bytes) while q, k_new,
     v_new and out stay in `dtype`.  A stored byte c of layer l means E4M3(c) * kv_scales[l][0] for K and
     * kv_scales[l][1] for V; lt_kv_append / lt_decode_step store code(x) = E4M3 nearest to
     float32(x) / scale (float32 division, round to nearest even, saturating at +-448).  Needs
     dtype = LT_BF16, head_dim = 128 and a query group of at most 32.  The kernels turn the stored bytes into
     f16 in registers (exact) and multiply on the tensor cores with fp32 accumulation, q as f16 at one
     power-of-two scale per head (exact for bf16 inputs), the probabilities as one f16 term.  lt_lazy_scores and
     lt_lazy_scores_lse read 8-bit keys too (k_full holds the E4M3 bytes; q_tail stays bf16): the stored bytes go
     through E4M3 tensor-core MMAs against q as two E4M3 terms per element at one power-of-two scale per query
     row (exact for bf16 inputs down to 2^-10 of the row's largest value), which the call writes into the
     workspace; size the workspace with this shape (lt_workspace_bytes adds the room for it). */
  int32_t kv_fp8;
  int32_t reserved2_;      /* must be 0 */
  const float* kv_scales;  /* dev float [n_layers][2] (K scale, V scale), positive; read during device work */
} lt_shape;

/* Text for a status code (static storage, never NULL). */
const char* lt_status_string(lt_status s);

/* Library version, major*10000 + minor*100 + patch. */
int32_t lt_version(void);

/*
 * Slot of token position `pos` in a lazy layer's cache (Section 5.1: a lazy
 * layer retains only the KV of {X_initial, X_recent}): pos itself while
 * pos < n_sink, else n_sink + (pos - n_sink) mod n_recent.  Pure host function;
 * returns -1 on pos < 0, n_sink < 0 or n_recent < 1.
 */
int32_t lt_ring_slot(int32_t pos, int32_t n_sink, int32_t n_recent);

/*
 * Bytes of workspace that lt_lazy_scores / lt_lazy_scores_lse (prompt length up
 * to n_ctx_max, up to w_last_max tail queries, any layer range) and
 * lt_hybrid_decode_attn / lt_decode_step (any seq_len up to
 * max(full_capacity, n_sink + n_recent), any layer range) need for this shape.
 * Host only; pass 0, 0 when the workspace will not be used for scoring.
 * The workspace is device memory, 256-byte aligned, owned by the caller; it
 * starts with the device error word and the counters of the decode step, which
 * must be zeroed once with lt_workspace_init (every call leaves them zero).
 * Two calls that overlap on the device must not share it.
 */
lt_status lt_workspace_bytes(const lt_shape* shape, int32_t n_ctx_max, int32_t w_last_max,
                             size_t* bytes_out /* host */);

/*
 * lt_workspace_bytes for a workspace that lt_decode_step_layers can use as well
 * (Appendix A's per-layer call): never less than lt_workspace_bytes, and room
 * for every layer's own partial slots.  Host only.
 */
lt_status lt_workspace_bytes_layers(const lt_shape* shape, int32_t n_ctx_max, int32_t w_last_max,
                                    size_t* bytes_out /* host */);

/* Zero the workspace (async on `stream`); once, before its first use. */
lt_status lt_workspace_init(void* ws /* dev */, size_t ws_bytes, void* stream);

/*
 * Copy the device error word to *flags_out and clear it.  SYNCHRONISES the
 * stream.  Returns LT_ERR_TIMEOUT when LT_DEVERR_TIMEOUT is set (whatever else
 * is), LT_ERR_DEVICE_RANGE when any other bit is set, LT_OK when the word is 0.
 */
lt_status lt_check(void* ws /* dev */, uint32_t* flags_out /* host, may be NULL */, void* stream);

/*
 * Lazy ratio (Eq. 1; Table 1 for the log-sum-exp identity it equals).
 *   q_tail  dev [L][B][Hq][w_last][D]: queries of prompt positions
 *           n_ctx - w_last .. n_ctx - 1
 *   k_full  host table of dev pointers; rows 0 .. n_ctx-1 of every (b, kv head)
 *           hold the prompt keys.  Entries of the scored layers must be
 *           non-NULL; the others are not looked at.
 *   layers [layer_begin, layer_begin + layer_count) are scored (0 and n_layers
 *           for the whole stack).  Scoring one layer at a time, right after its
 *           prefill, is what Figure 3's queue needs: the keys of a layer that
 *           was popped and compacted are never read again, so its full cache
 *           can be freed and its table entry set to NULL.
 *   scores  dev float [L][B][Hq]: for each query head the mean over the w_last
 *           tail queries of the causal-softmax mass on keys j < n_sink or
 *           j >= n_ctx - n_recent (a set union; 1.0 when the window covers all).
 *           Only the scored layers' slices are written.
 * The mean over heads and batch rows that completes Eq. 1 is taken by
 * lt_select_lazy.  Requires 1 <= w_last <= n_ctx <= full_capacity.
 */
lt_status lt_lazy_scores(const lt_shape* shape, const void* q_tail /* dev */,
                         const void* const* k_full /* host table */, int32_t n_ctx, int32_t w_last,
                         int32_t layer_begin, int32_t layer_count, float* scores /* dev */, void* ws /* dev */,
                         size_t ws_bytes, void* stream);

/*
 * lt_lazy_scores that also hands out the denominators it computed (Table 1:
 * the `lse` that the prefill's attention returns next to its output):
 *   lse_out  dev float [L][B][Hq][w_last]: natural logarithm of
 *            sum_{j <= i} exp(scale * q_i . k_j) for the tail rows
 *            i = n_ctx - w_last .. n_ctx - 1; only the scored layers' slices are
 *            written.  It is the input lt_lazy_scores_lse expects, for callers
 *            whose prefill does not export it.
 * Everything else as lt_lazy_scores (same pass over the keys, same scores).
 */
lt_status lt_lazy_scores_with_lse(const lt_shape* shape, const void* q_tail /* dev */,
                                  const void* const* k_full /* host table */, int32_t n_ctx, int32_t w_last,
                                  int32_t layer_begin, int32_t layer_count, float* scores /* dev */,
                                  float* lse_out /* dev */, void* ws /* dev */, size_t ws_bytes, void* stream);

/*
 * Lazy ratio with the denominator given (Section 5.1: FlashAttention's prefill
 * already produced the log-sum-exp of every attention row, so only the product of
 * the tail queries with the kept keys is left to compute, a constant-size one; Table 1).
 * Same result as lt_lazy_scores, but only the kept keys are read:
 *   lse     dev float [L][B][Hq][w_last]: natural logarithm of
 *           sum_{j <= i} exp(scale * q_i . k_j) for the tail rows
 *           i = n_ctx - w_last .. n_ctx - 1 (what the prefill attention returns)
 *   k_full  rows j < n_sink and j >= n_ctx - n_recent of every (b, kv head) are
 *           read; the rest of the prompt keys is not touched.
 *   scores[l][b][hq] = mean over the tail rows of
 *           sum_{j kept, j <= i} exp(scale * q_i . k_j - lse_i).
 * Cost is independent of n_ctx.  Same workspace and layer range as lt_lazy_scores.
 */
lt_status lt_lazy_scores_lse(const lt_shape* shape, const void* q_tail /* dev */,
                             const void* const* k_full /* host table */, const float* lse /* dev */,
                             int32_t n_ctx, int32_t w_last, int32_t layer_begin, int32_t layer_count,
                             float* scores /* dev */, void* ws /* dev */, size_t ws_bytes, void* stream);

/*
 * Selection (Section 5.1, the max-priority queue of size P = L - n_lazy; Fig. 3):
 * r_l = mean over [B][Hq] of scores[l] (accumulated in double, fixed order);
 * layer_mask[l] = 1 for the n_lazy layers with the largest r_l, ties to the
 * lower layer index - the same set the streaming priority queue leaves lazy.
 *   layer_ratio  dev float [L] or NULL: r_l rounded to float.
 * Runs on the device; no host round trip.
 */
lt_status lt_select_lazy(const float* scores /* dev [L][B][Hq] */, int32_t n_layers, int32_t batch,
                         int32_t n_q_heads, int32_t n_lazy, uint8_t* layer_mask /* dev [L] */,
                         float* layer_ratio /* dev [L] or NULL */, void* stream);

/*
 * Per-prompt selection (Section 4: which layers are lazy differs from prompt to
 * prompt): for every batch row b, r = mean over [Hq] of
 * scores[l][b] and the n_lazy layers with the largest r become lazy for that
 * prompt.  layer_mask dev uint8 [B][L], layer_ratio dev float [B][L] or NULL.
 * Use the result with shape.per_sequence_mask = 1.
 */
lt_status lt_select_lazy_per_seq(const float* scores /* dev [L][B][Hq] */, int32_t n_layers, int32_t batch,
                                 int32_t n_q_heads, int32_t n_lazy, uint8_t* layer_mask /* dev [B][L] */,
                                 float* layer_ratio /* dev [B][L] or NULL */, void* stream);

/*
 * Frequency-count choice of the lazy layers over many samples (Section 5.2,
 * LightTransfer-Train: every training sample reveals its own lazy layers; the
 * layers that are lazy in the most samples are chosen).
 *   sample_masks  dev uint8 [n_samples][L]: per-sample masks, e.g. the rows that
 *                 lt_select_lazy_per_seq wrote for successive batches
 *   layer_mask    dev uint8 [L]: 1 for the n_lazy layers with the highest counts,
 *                 ties to the lower layer index
 *   layer_counts  dev int32 [L] or NULL
 */
lt_status lt_select_lazy_frequency(const uint8_t* sample_masks /* dev */, int32_t n_samples, int32_t n_layers,
                                   int32_t n_lazy, uint8_t* layer_mask /* dev [L] */,
                                   int32_t* layer_counts /* dev [L] or NULL */, void* stream);

/*
 * Streaming selection, one layer at a time (Section 5.1 and Figure 3: the
 * ratios enter a priority queue of capacity P = n_full during prefilling; when
 * the queue overflows, the layer with the highest ratio is popped, labelled
 * lazy and its KV reduced at once, so at most P full caches ever exist).
 * Call in layer order, right after layer `layer`'s scores are known:
 *   layer_scores  dev float [B][Hq]: this layer's slice of the lt_lazy_scores output
 *   queue_state   dev, 8 * n_layers bytes, 8-byte aligned, owned by the caller;
 *                 layer 0 starts a new prompt (state and mask are reset)
 *   layer_mask    dev uint8 [L]: updated in place (the popped layer becomes 1)
 *   popped_layer  dev int32 or NULL: the layer that left the queue, or -1
 * After the last layer the mask equals lt_select_lazy(n_lazy = L - n_full) on
 * the same scores.  lt_stream_init_layer compacts the popped layer without a
 * host round trip.
 */
lt_status lt_select_lazy_push(const float* layer_scores /* dev */, int32_t layer, int32_t n_layers, int32_t batch,
                              int32_t n_q_heads, int32_t n_full, void* queue_state /* dev */,
                              uint8_t* layer_mask /* dev [L] */, int32_t* popped_layer /* dev or NULL */,
                              void* stream);

/*
 * Prefill -> decode compaction of the lazy layers (Section 5.1: a lazy
 * layer keeps the KV of its initial and its most recent tokens and drops the rest;
 * Fig. 3).  For every layer with mask 1 and every (b, kv head), prompt rows
 * p in {0 .. min(n_sink,n)-1} U {max(n_sink, n - n_recent) .. n-1}, n = seq_lens[b],
 * are copied bit for bit from the full cache to row lt_ring_slot(p) of the
 * stream cache, so later appends continue the ring.  Layers with mask 0 are
 * untouched.
 */
lt_status lt_stream_init(const lt_shape* shape, const uint8_t* layer_mask /* dev */,
                         const void* const* k_full, const void* const* v_full /* host tables */,
                         const int32_t* seq_lens /* dev [B] */, void* const* k_stream,
                         void* const* v_stream /* host tables */, void* ws /* dev, for the error word; may be NULL */,
                         void* stream);

/*
 * lt_stream_init for the one layer whose index is stored at *layer on the
 * device (nothing happens when it is -1 or the mask of that layer is 0): the
 * compaction step of the streaming selection above.
 */
lt_status lt_stream_init_layer(const lt_shape* shape, const uint8_t* layer_mask /* dev */,
                               const int32_t* layer /* dev */, const void* const* k_full,
                               const void* const* v_full /* host tables */, const int32_t* seq_lens /* dev [B] */,
                               void* const* k_stream, void* const* v_stream /* host tables */,
                               void* ws /* dev, for the error word; may be NULL */, void* stream);

/*
 * Per-step KV append (Section 3: decoding stores the KV of every generated token; Section 5.1
 * for the lazy layers).  With p = seq_lens[b]:
 *   mask 0: k_new[l][b][h][:] -> full cache row p        (skipped and flagged
 *           LT_DEVERR_POS_OUT_OF_RANGE when p >= full_capacity)
 *   mask 1: -> stream cache row lt_ring_slot(p): sinks are never overwritten,
 *           later tokens overwrite the oldest ring row.
 * Then seq_lens[b] += 1 for every b (once per call, not per layer).
 *   k_new, v_new  dev [L][B][Hkv][D]
 *   layers [layer_begin, layer_begin + layer_count) are written; pass 0 and
 *   n_layers for the whole stack.  seq_lens is advanced only when
 *   advance_seq_lens != 0 (a per-layer caller advances on its last layer).
 */
lt_status lt_kv_append(const lt_shape* shape, const uint8_t* layer_mask /* dev */,
                       const void* k_new /* dev */, const void* v_new /* dev */,
                       int32_t* seq_lens /* dev [B] */, void* const* k_full, void* const* v_full,
                       void* const* k_stream, void* const* v_stream /* host tables */,
                       int32_t layer_begin, int32_t layer_count, int32_t advance_seq_lens,
                       void* ws /* dev, for the error word; may be NULL */, void* stream);

/*
 * One decode step of attention for the whole stack (Appendix E: MHA with the
 * causal mask in layers outside I, with M_lazy in layers inside I; Section 3).
 * With n = seq_lens[b] (the new token already appended):
 *   mask 0: out[l][b][hq] = softmax(scale * q . K[0..n-1]^T) V[0..n-1]  over the
 *           full cache;
 *   mask 1: the same over the min(n, n_sink + n_recent) valid rows of the stream
 *           cache (order of rows is irrelevant to softmax, so the ring is read
 *           linearly).
 *   q    dev [L][B][Hq][D], dtype of the shape
 *   out  dev [L][B][Hq][D], LT_F32 or LT_BF16 (out_dtype); zeros where n = 0
 *   max_seq_len_hint  ignored (kept for source compatibility): the launch
 *           sizes itself from the device-side lengths.
 *   layers [layer_begin, layer_begin + layer_count).
 * Split-KV: partial (max, sum, weighted values) per KV chunk go to the
 * workspace; the last chunk of each (layer, b, kv head) to finish merges them
 * in chunk order inside the same launch.  batch <= 2048.
 * A call over part of the stack (layer_count < n_layers: a model that calls
 * layer by layer, as the cache-updating attention call of Appendix A is used)
 * is launched with CUDA's programmatic-serialization attribute: its CTAs may
 * become resident while the previous kernel of the stream finishes and wait
 * there until that kernel has completed, so back-to-back per-layer calls do not
 * pay a launch gap each.  Results and ordering are those of plain stream order.
 */
lt_status lt_hybrid_decode_attn(const lt_shape* shape, const void* q /* dev */,
                                const void* const* k_full, const void* const* v_full,
                                const void* const* k_stream, const void* const* v_stream /* host tables */,
                                const uint8_t* layer_mask /* dev */, const int32_t* seq_lens /* dev */,
                                void* out /* dev */, int32_t out_dtype, int32_t max_seq_len_hint,
                                int32_t layer_begin, int32_t layer_count, void* ws /* dev */,
                                size_t ws_bytes, void* stream);

/*
 * One whole decode step in a single launch: lt_kv_append followed by
 * lt_hybrid_decode_attn (Section 3: each decoding step saves the new token's KV
 * and attends over the cache; the experimental setup of Appendix A runs that as
 * one cache-updating attention call).  With p = seq_lens[b]:
 *   - k_new / v_new [L][B][Hkv][D] are stored at row p of the full cache
 *     (mask 0) or row lt_ring_slot(p) of the stream cache (mask 1), exactly as
 *     lt_kv_append does; p >= full_capacity in a full layer skips the store
 *     and raises LT_DEVERR_POS_OUT_OF_RANGE;
 *   - out [L][B][Hq][D] is the attention of q over the p + 1 tokens (full
 *     layers) or the min(p + 1, n_sink + n_recent) retained tokens (lazy
 *     layers), exactly as lt_hybrid_decode_attn would return after the append;
 *   - seq_lens[b] += 1 at the end of the launch when advance_seq_lens != 0
 *     (a per-layer caller passes 0 except for its last layer).
 * The workspace must have been zeroed once by lt_workspace_init.  Results are
 * bit-identical to the two separate calls.
 */
lt_status lt_decode_step(const lt_shape* shape, const void* q /* dev */, const void* k_new /* dev */,
                         const void* v_new /* dev */, void* const* k_full, void* const* v_full,
                         void* const* k_stream, void* const* v_stream /* host tables */,
                         const uint8_t* layer_mask /* dev */, int32_t* seq_lens /* dev [B] */, void* out /* dev */,
                         int32_t out_dtype, int32_t layer_begin, int32_t layer_count, int32_t advance_seq_lens,
                         void* ws /* dev */, size_t ws_bytes, void* stream);

/*
 * lt_decode_step for a caller that issues one step as several launches over
 * disjoint layer ranges (Appendix A runs the cache-updating attention call once
 * per layer) and can tell the library which of them do not depend on the launch
 * before them.  Same operation, arguments and results as lt_decode_step, plus:
 *   independent_of_previous  0: plain stream order, as lt_decode_step.
 *       1: the caller vouches that the work enqueued on `stream` since the last
 *       call of this function with independent_of_previous = 0 consists only of
 *       calls of this function for the same step (same shape, tables, mask,
 *       seq_lens and workspace) over layer ranges disjoint from this one, none
 *       of them with advance_seq_lens != 0, and that nothing this call reads (q,
 *       k_new, v_new of its layers) is written by them.  The launch then starts
 *       on its items as soon as SMs come free under the tail of the launches
 *       before it instead of waiting for them to complete; its own completion
 *       still implies theirs, so whatever follows on the stream sees plain
 *       stream order.  The first call of every step passes 0 (it reads the
 *       seq_lens that the previous step's last call advanced).
 * A model whose other layers produce q for layer l + 1 from the output of layer
 * l has a true dependency and passes 0 throughout; the flag is for callers that
 * hold the inputs of several layers at once (speculative or batched layer
 * execution, benchmarks of the attention stack).
 * Every layer owns its partial slots and launch counters in the workspace, which
 * therefore must have lt_workspace_bytes_layers bytes (zeroed once with
 * lt_workspace_init); LT_ERR_WORKSPACE otherwise.  Results are bit-identical to
 * the same sequence of calls with independent_of_previous = 0.
 */
lt_status lt_decode_step_layers(const lt_shape* shape, const void* q /* dev */, const void* k_new /* dev */,
                                const void* v_new /* dev */, void* const* k_full, void* const* v_full,
                                void* const* k_stream, void* const* v_stream /* host tables */,
                                const uint8_t* layer_mask /* dev */, int32_t* seq_lens /* dev [B] */,
                                void* out /* dev */, int32_t out_dtype, int32_t layer_begin, int32_t layer_count,
                                int32_t advance_seq_lens, int32_t independent_of_previous, void* ws /* dev */,
                                size_t ws_bytes, void* stream);

/*
 * lt_decode_step for a caller whose step inputs and outputs live in HOST
 * memory (the same operation, Section 3; the sampler of a serving loop reads
 * the step's result on the host).  Enqueues on `stream`: q_host, k_new_host,
 * v_new_host -> the device staging buffers, the whole-stack lt_decode_step
 * (all layers, seq_lens advanced), out staging -> out_host.  Does not
 * synchronise: out_host is valid once the stream has reached this point.
 *   q_host, k_new_host, v_new_host, out_host  host, layouts and dtypes as in
 *       lt_decode_step; page-locked memory keeps the copies asynchronous
 *   q_dev, k_new_dev, v_new_dev, out_dev      dev staging buffers of the same
 *       sizes, owned by the caller
 */
lt_status lt_decode_step_host(const lt_shape* shape, const void* q_host, const void* k_new_host,
                              const void* v_new_host, void* out_host, void* q_dev, void* k_new_dev,
                              void* v_new_dev, void* out_dev, void* const* k_full, void* const* v_full,
                              void* const* k_stream, void* const* v_stream /* host tables */,
                              const uint8_t* layer_mask /* dev */, int32_t* seq_lens /* dev [B] */,
                              int32_t out_dtype, void* ws /* dev */, size_t ws_bytes, void* stream);

/*
 * The decode-attention step for callers that cannot allocate device memory.
 * (No counterpart in the paper: this is a deployment convenience of the library.)
 *
 * Some hosts are handed pointers but no allocator - a serving engine that has
 * already given all free HBM to its KV-cache pool, a plug-in inside another
 * program's memory plan, a loop in which cudaMalloc would stall the device.
 * This call is lt_hybrid_decode_attn without the workspace arguments: the
 * split-KV partials live in a fixed array of LT_STATIC_SCRATCH_BYTES inside the
 * library image, resident on every GPU that loads the library until the process
 * exits.  The call allocates and frees nothing.
 *
 *   - Same arguments, layouts and result as lt_hybrid_decode_attn.
 *   - dev_error (dev, 4-byte aligned, may be NULL): receives this call's error
 *     word (the LT_DEVERR_* bits), stream-ordered; there is no workspace to
 *     lt_check.  It is written only by a call that returns LT_OK: a call refused
 *     on the host enqueues nothing and leaves both *dev_error and the shared
 *     array as they were.
 *   - A shape whose lt_workspace_bytes(shape, 0, 0, ..) exceeds
 *     LT_STATIC_SCRATCH_BYTES returns LT_ERR_WORKSPACE before any device work.
 *   - The first call on each device looks up the array's device address; make
 *     that call before beginning any stream capture.  The address is kept for
 *     the life of the process, which assumes that the device's primary context
 *     is not reset in between.
 *   - All calls on a device share the array, which still holds the previous
 *     call's partials.  The error word is cleared at the start of every call and
 *     partials are written before they are read, so calls in stream order are
 *     independent; calls that overlap on the GPU race and must be serialised.
 */
#define LT_STATIC_SCRATCH_BYTES (16u << 20)
lt_status lt_hybrid_decode_attn_static(const lt_shape* shape, const void* q /* dev */,
                                       const void* const* k_full, const void* const* v_full,
                                       const void* const* k_stream, const void* const* v_stream /* host tables */,
                                       const uint8_t* layer_mask /* dev */, const int32_t* seq_lens /* dev */,
                                       void* out /* dev */, int32_t out_dtype, int32_t max_seq_len_hint,
                                       int32_t layer_begin, int32_t layer_count,
                                       uint32_t* dev_error /* dev, may be NULL */, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LT_H_ */
