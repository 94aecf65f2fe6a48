// lt_hybrid_decode_attn_static: the decode-attention step for callers that
// cannot allocate device memory.
//
// Some hosts of this library are handed pointers but no allocator: a serving
// engine that has already given every free byte of HBM to its KV-cache pool, a
// plug-in that runs inside someone else's memory plan, a loop that must not
// call cudaMalloc because an allocation would stall or fragment the device.
// The ordinary entry point wants a caller-provided workspace for the split-KV
// partial results; this one keeps that scratch in a fixed array that is part of
// the library image, so the caller passes inputs and outputs only.
//
// Cost and limits: the array (LT_STATIC_SCRATCH_BYTES) is resident on every GPU
// that loads the library, for the life of the process.  Shapes whose partials
// do not fit are rejected with LT_ERR_WORKSPACE.  Every call on a device shares
// the one array and finds the previous call's partials in it: the error word is
// cleared at the start of each call, partials are always written before they
// are read within a call, and two calls that overlap on the GPU (different
// streams, no dependency) race on it - serialise them.
//
// The first call on each device resolves the array's device address
// (cudaGetSymbolAddress, with that device current); make that first call before
// starting any stream capture.
#include <mutex>

#include "lt_internal.h"

namespace lt {
namespace {

// In host code this name is only a handle for the runtime; the address a kernel
// may dereference comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[LT_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device (resolved once).
cudaError_t scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace lt

using namespace lt;

extern "C" lt_status lt_hybrid_decode_attn_static(const lt_shape* shape, const void* q, const void* const* k_full,
                                                  const void* const* v_full, const void* const* k_stream,
                                                  const void* const* v_stream, const uint8_t* layer_mask,
                                                  const int32_t* seq_lens, void* out, int32_t out_dtype,
                                                  int32_t max_seq_len_hint, int32_t layer_begin, int32_t layer_count,
                                                  uint32_t* dev_error, void* stream) {
  // Size check first: it needs no CUDA call, so an oversized shape is refused
  // even where no device is present.
  size_t need = 0;
  lt_status st = lt_workspace_bytes(shape, 0, 0, &need);
  if (st != LT_OK) return st;
  if (need > (size_t)LT_STATIC_SCRATCH_BYTES) return LT_ERR_WORKSPACE;

  // Every check the host can make comes before any CUDA call and before anything is enqueued: a refused
  // call touches neither the shared array nor *dev_error.  (The checks only look at the workspace's address
  // and size, so they can run against a stand-in address before the array's own is known.)
  (void)max_seq_len_hint;  // ignored, as in lt_hybrid_decode_attn
  DecodeCall call;
  st = decode_prepare(&call, shape, q, nullptr, nullptr, k_full, v_full, k_stream, v_stream, layer_mask,
                      const_cast<int32_t*>(seq_lens), out, out_dtype, layer_begin, layer_count, 0, 0,
                      reinterpret_cast<void*>(kWsAlign), (size_t)LT_STATIC_SCRATCH_BYTES);
  if (st != LT_OK) return st;
  if (dev_error && ((uintptr_t)dev_error & 3u) != 0) return LT_ERR_INVALID_ARG;

  void* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) return LT_ERR_CUDA;
  st = decode_prepare(&call, shape, q, nullptr, nullptr, k_full, v_full, k_stream, v_stream, layer_mask,
                      const_cast<int32_t*>(seq_lens), out, out_dtype, layer_begin, layer_count, 0, 0, scratch,
                      (size_t)LT_STATIC_SCRATCH_BYTES);
  if (st != LT_OK) return st;
  cudaStream_t cs = (cudaStream_t)stream;
  // The header holds the error word and the merge counters; start every call from zero.
  if (cudaMemsetAsync(scratch, 0, ws_prefix_bytes(*shape), cs) != cudaSuccess) return LT_ERR_CUDA;
  st = decode_launch(call, stream);
  if (st != LT_OK) return st;
  if (dev_error) {
    // hand the step's error word to the caller's own device word (stream-ordered, 4 bytes)
    if (cudaMemcpyAsync(dev_error, scratch, sizeof(uint32_t), cudaMemcpyDeviceToDevice, cs) != cudaSuccess)
      return LT_ERR_CUDA;
  }
  return LT_OK;
}
