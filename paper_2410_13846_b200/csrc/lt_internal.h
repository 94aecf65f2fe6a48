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

// Workspace layout: [header 256 B][region used by the running call].
constexpr size_t kWsHeaderBytes = 256;
constexpr size_t kWsAlign = 256;

// Split-KV plan of the decode step; a function of the shape alone so that the
// workspace query and every later call agree.
struct DecodePlan {
  int chunk_keys;    // keys per KV chunk (multiple of 64)
  int n_chunks_max;  // chunks that cover max(full_capacity, n_sink + n_recent)
  size_t ml_floats;  // [L][B][Hkv][n_chunks_max][G][2]
  size_t o_floats;   // [L][B][Hkv][n_chunks_max][G][D]
};
DecodePlan make_decode_plan(const lt_shape& s);

// Split plan of the scoring pass.
struct ScorePlan {
  int n_splits;        // key-range splits per (layer, batch row, kv head)
  size_t stat_floats;  // [L][B][Hq][T][n_splits][3] partial (max, sum_all, sum_window)
};
ScorePlan make_score_plan(const lt_shape& s, int n_ctx, int w_last);

inline float resolved_scale(const lt_shape& s) {
  return s.softmax_scale > 0.f ? s.softmax_scale : 1.0f / sqrtf((float)s.head_dim);
}
inline size_t elem_bytes(int dtype) { return dtype == LT_BF16 ? 2 : 4; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

lt_status validate_shape(const lt_shape* s);

// ---- launchers (each returns cudaGetLastError() of its launches) ----------
cudaError_t launch_append(const lt_shape& s, const uint8_t* mask, const void* k_new, const void* v_new,
                          int32_t* seq_lens, const LayerTable& kf, const LayerTable& vf,
                          const LayerTable& ks, const LayerTable& vs, int layer_begin, int layer_count,
                          int advance, uint32_t* dev_err, cudaStream_t st);

cudaError_t launch_stream_init(const lt_shape& s, const uint8_t* mask, const LayerTable& kf,
                               const LayerTable& vf, const int32_t* seq_lens, const LayerTable& ks,
                               const LayerTable& vs, uint32_t* dev_err, cudaStream_t st);

struct DecodeArgs {
  lt_shape s;
  const void* q;
  const uint8_t* mask;
  const int32_t* seq_lens;
  void* out;
  int out_dtype;
  int layer_begin, layer_count;
  int chunk_keys, n_chunks_max, n_chunks_launch;
  float cs;  // softmax scale * log2(e)
  float* part_ml;
  float* part_o;
  uint32_t* dev_err;
};
cudaError_t launch_decode_generic(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                                  const LayerTable& ks, const LayerTable& vs, cudaStream_t st);
// bf16, head_dim 128, group size <= 8: tensor-core path.
bool decode_mma_supported(const lt_shape& s);
cudaError_t launch_decode_mma(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                              const LayerTable& ks, const LayerTable& vs, cudaStream_t st);
cudaError_t launch_decode_combine(const DecodeArgs& a, cudaStream_t st);

struct ScoreArgs {
  lt_shape s;
  const void* q_tail;
  int n_ctx, w_last;
  int n_splits;
  float cs;      // softmax scale * log2(e)
  float* stats;  // workspace
  float* scores;
  uint32_t* dev_err;
};
cudaError_t launch_scores_generic(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st);
bool scores_mma_supported(const lt_shape& s, int w_last);
cudaError_t launch_scores_mma(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st);
// bf16, head_dim 128: tcgen05 / TMEM path.
bool scores_umma_supported(const lt_shape& s, int w_last);
cudaError_t launch_scores_umma(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st);
cudaError_t launch_scores_finish(const ScoreArgs& a, cudaStream_t st);

cudaError_t launch_select(const float* scores, int L, int B, int Hq, int n_lazy, uint8_t* mask,
                          float* ratio, cudaStream_t st);

}  // namespace lt
