// Pieces shared by the decode-step kernels (tensor-core and CUDA-core paths):
// the flattened work list of a persistent launch, the fused KV append, and the
// in-kernel merge of the split-KV partials by the last CTA of each unit.
//
// A decode step over a hybrid stack is very uneven: a full layer at 32K context
// has sixteen 2048-key chunks per (batch row, kv head), a lazy layer has one.
// Which layers are lazy is known on the device only (layer_mask), so instead of
// a rectangular grid with mostly empty CTAs for the lazy layers, the kernels
// launch a fixed number of CTAs (a multiple of the SM count) and every CTA walks
// the same work list:
//   entry e = (layer, batch row)      n_e = visible keys, nc_e = chunks
//   items of e = n_kv_heads * nc_e    item -> (kv head, chunk)
// The prefix sum over entries lives in shared memory; an item index is turned
// into (entry, kv head, chunk) by binary search.  The chunk length is chosen on
// the device from the total number of keys of the launch, so that a whole stack
// (2048-key chunks) and a single layer (shorter chunks) both give every CTA
// several items; the partials of item i live in slot i of the workspace.
#pragma once

#include <cuda_bf16.h>

#include "lt_internal.h"

namespace lt {

// Programmatic dependent launch, for callers that issue a step as several launches (one per layer):
// a launch made with the programmatic-serialization attribute may become resident while the previous
// kernel of the stream is still running its last items.  Its CTAs then sit in pdl_wait_prior_grid()
// until that kernel has completed and its writes are visible, so the launch latency and the CTA
// ramp-up are paid under the previous kernel's tail.  Everything a launch shares with its predecessor -
// seq_lens (advanced by a step's last launch), the launch counters and the partial slots of the
// workspace - is touched only after the wait, which is the first statement of the kernels.  Without the
// attribute both calls are no-ops.
//
// A launch with DecodeArgs::overlap set does not wait at its start: the caller has vouched that it shares
// nothing with the launches before it (another layer range of the same step, none of which advances
// seq_lens), its counters and partial slots are those of its own layers, and so its CTAs start on their
// items as soon as SMs come free under the previous launch's tail.  Two rules keep stream order intact.
// A launch lets its successor in only after every one of its CTAs has read seq_lens (the trigger follows
// the work-list build), so a successor that advances seq_lens at its end cannot be read too early by
// anyone: by induction every earlier launch has all its CTAs past that read.  And the last CTA of an
// overlapped launch waits for the prior grid before it retires, so the completion of a launch still
// implies the completion of everything before it.
__device__ __forceinline__ void pdl_wait_prior_grid() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_allow_next_grid() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

struct WorkItem {
  int l, b, h, c;  // layer, batch row, kv head, chunk
  int nc;          // chunks of this (layer, batch row)
  int n;           // visible keys of this (layer, batch row), clamped to the cache
  int j0, j1;      // key rows [j0, j1) of this chunk
  int rows;        // rows per (b, kv head) of the cache that is read
  int new_row;     // fused append: row taken from k_new / v_new (and stored) by this item, else -1
  int slot0;       // partial slot of chunk 0 of this (layer, b, kv head); chunk c uses slot0 + c
  bool lazy;
};

__device__ __forceinline__ int ring_slot_of(int p, int S, int R) { return p < S ? p : S + (p - S) % R; }

// Shared-memory footprint of the work list (bytes) for `entries` (layer, b) pairs.
__host__ __device__ constexpr inline int worklist_smem_bytes(int entries, int batch) {
  return ((entries + 1 + batch) * 4 + entries + 15) / 16 * 16;
}

struct WorkList {
  int* prefix;    // [entries + 1]
  int* seq;       // [batch]   seq_lens as read at kernel start
  uint8_t* kind;  // [entries]  bit 0 lazy, bit 1 table entry missing
  int entries;
  int chunk;      // keys per chunk of this launch (before balancing)

  __device__ __forceinline__ void carve(uint8_t* mem, int layer_count, int batch) {
    entries = layer_count * batch;
    prefix = reinterpret_cast<int*>(mem);
    seq = prefix + entries + 1;
    kind = reinterpret_cast<uint8_t*>(seq + batch);
  }

  // visible keys of (layer kind, batch row) after clamping; raises the error bits
  __device__ __forceinline__ int visible(const DecodeArgs& a, int e, int b, bool report) const {
    const lt_shape& s = a.s;
    const bool lazy = kind[e] & 1;
    const int rows = lazy ? s.n_sink + s.n_recent : s.full_capacity;
    int n = seq[b] + (a.fused ? 1 : 0);
    if (n < 0) n = 0;
    if (n > rows) {
      if (!lazy && report) atomicOr(a.dev_err, a.fused ? LT_DEVERR_POS_OUT_OF_RANGE : LT_DEVERR_LEN_CLAMPED);
      n = rows;
    }
    return n;
  }

  // Called by every thread of the CTA.  Ends with a barrier.
  __device__ void build(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf, const LayerTable& ks,
                        const LayerTable& vs) {
    const lt_shape& s = a.s;
    const int B = s.batch;
    for (int b = threadIdx.x; b < B; b += blockDim.x) seq[b] = a.seq_lens[b];
    for (int e = threadIdx.x; e < entries; e += blockDim.x) {
      const int lr = e / B, b = e - lr * B;
      const int l = a.layer_begin + lr;
      const bool lazy = a.mask[mask_index(s, l, b)] != 0;
      const bool missing = lazy ? (!ks.p[l] || !vs.p[l]) : (!kf.p[l] || !vf.p[l]);
      kind[e] = (lazy ? 1 : 0) | (missing ? 2 : 0);
      if (missing && blockIdx.x == 0) atomicOr(a.dev_err, LT_DEVERR_NULL_LAYER);
    }
    __syncthreads();
    // thread t owns a contiguous run of entries
    const int per = (entries + blockDim.x - 1) / blockDim.x;
    const int e0 = min(entries, (int)threadIdx.x * per), e1 = min(entries, e0 + per);
    // chunk length: total keys of the launch spread over a few items per CTA
    __shared__ unsigned long long total_keys;
    if (threadIdx.x == 0) total_keys = 0ull;
    __syncthreads();
    {
      unsigned long long mine = 0ull;
      for (int e = e0; e < e1; ++e)
        if (!(kind[e] & 2)) mine += (unsigned long long)visible(a, e, e % B, blockIdx.x == 0) * s.n_kv_heads;
      if (mine) atomicAdd(&total_keys, mine);
    }
    __syncthreads();
    {
      const long long target = min((long long)gridDim.x * 8, (long long)a.target_items);
      long long c = (long long)((total_keys + target - 1) / target);
      c = (c + 63) / 64 * 64;
      // the longest chunks only for launches that keep a few of them per CTA
      const long long hi =
          total_keys >= 2ull * (unsigned long long)a.target_items * (unsigned long long)a.max_chunk ? a.max_chunk : a.mid_chunk;
      chunk = (int)max((long long)a.min_chunk, min(hi, c));
    }
    // items per entry, then an exclusive scan
    int run = 0;
    for (int e = e0; e < e1; ++e) {
      const int b = e % B;
      int items = 0;
      if (!(kind[e] & 2)) {
        const int n = visible(a, e, b, false);
        const int nc = max(1, (n + chunk - 1) / chunk);
        items = s.n_kv_heads * nc;
      }
      prefix[e + 1] = items;  // turned into the prefix below
      run += items;
    }
    // block-wide exclusive scan of the per-thread sums: shuffles inside a warp, then the warp totals
    __shared__ int warp_total[8];  // blockDim.x <= 256
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int incl = run;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += t;
    }
    if (lane == 31) warp_total[wid] = incl;
    if (threadIdx.x == 0) prefix[0] = 0;
    __syncthreads();
    int before = 0;
    for (int w = 0; w < wid; ++w) before += warp_total[w];
    int acc = before + incl - run;
    for (int e = e0; e < e1; ++e) {
      acc += prefix[e + 1];
      prefix[e + 1] = acc;
    }
    __syncthreads();
  }

  // Items of the launch; never more than the partial slots the workspace holds
  // (the plan's bound covers every chunk length this build can choose).
  __device__ __forceinline__ int total(const DecodeArgs& a) const {
    const int t = prefix[entries];
    if (t > a.items_cap) {
      if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(a.dev_err, LT_DEVERR_LEN_CLAMPED);
      return a.items_cap;
    }
    return t;
  }

  __device__ __forceinline__ WorkItem item(const DecodeArgs& a, int idx) const {
    const lt_shape& s = a.s;
    int lo = 0, hi = entries;  // largest e with prefix[e] <= idx
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (prefix[mid] <= idx) lo = mid;
      else hi = mid;
    }
    WorkItem w;
    const int lr = lo / s.batch;
    w.b = lo - lr * s.batch;
    w.l = a.layer_begin + lr;
    w.lazy = kind[lo] & 1;
    w.rows = w.lazy ? s.n_sink + s.n_recent : s.full_capacity;
    w.n = visible(a, lo, w.b, false);
    w.nc = max(1, (w.n + chunk - 1) / chunk);
    const int rem = idx - prefix[lo];
    w.h = rem / w.nc;
    w.c = rem - w.h * w.nc;
    w.slot0 = idx - w.c;
    int len = (w.n + w.nc - 1) / w.nc;  // balanced chunks: no tiny last chunk
    if (s.page_size > 0) len = (len + 31) & ~31;  // paged caches: a 16- or 32-key tile never straddles two pages
    w.j0 = min(w.n, w.c * len);
    w.j1 = min(w.n, w.j0 + len);
    w.new_row = -1;
    if (a.fused) {
      const int pos = seq[w.b];
      const int slot = w.lazy ? ring_slot_of(pos, s.n_sink, s.n_recent) : pos;
      if (pos >= 0 && slot < w.rows && slot >= w.j0 && slot < w.j1) w.new_row = slot;
    }
    return w;
  }
};

// Slot of the partials of (layer, b, kv head, chunk): the item's own index.
__device__ __forceinline__ long long partial_unit(const DecodeArgs& a, const WorkItem& w) {
  return (long long)a.slot_base + w.slot0 + w.c;
}

// Staging buffer (shared memory) for the (max, sum) pairs of a unit's chunks
// while they are merged; units with more pairs read them from global memory.
constexpr int kCombineStagePairs = 512;

// After a CTA has written the partials of its item (one thread's fence after a
// CTA barrier publishes them all): count the item in; true for every thread of
// the CTA that finished the last chunk of its (layer, b, kv head).  Two CTA
// barriers.  A unit with a single chunk needs no count.
__device__ __forceinline__ bool count_item_in(const DecodeArgs& a, const WorkItem& w, int* s_flag) {
  if (w.nc <= 1) {
    __syncthreads();
    return true;
  }
  const long long unit = ((long long)w.l * a.s.batch + w.b) * a.s.n_kv_heads + w.h;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();  // cumulative: the partials written before the barrier are visible device-wide
    const int prev = atomicAdd(a.unit_counters + unit, 1);
    const int last = prev == w.nc - 1;
    if (last) {
      a.unit_counters[unit] = 0;  // ready for the next launch
      __threadfence();            // acquire side: the other chunks' partials are visible to this CTA
    }
    *s_flag = last;
  }
  __syncthreads();
  return *s_flag != 0;
}

// Merge the chunk partials of w's (layer, b, kv head) in chunk order (fixed
// order => run-to-run identical bits) and write the outputs of the group's
// query heads.  Called by every thread of the CTA; one thread owns four
// consecutive d of one head and keeps eight chunk loads in flight.
__device__ __forceinline__ void combine_unit(const DecodeArgs& a, const WorkItem& w, float2* s_ml) {
  const lt_shape& s = a.s;
  const int G = s.n_q_heads / s.n_kv_heads, D = s.head_dim;
  const int GP = G;             // heads per partial slot
  const int Gn = G;
  const long long unit0 = (long long)a.slot_base + w.slot0;
  const long long cs_ml = GP;   // float2s between the slots of consecutive chunks
  const int pairs = w.nc * Gn;
  const bool staged = pairs <= kCombineStagePairs;
  const float2* ml_g = reinterpret_cast<const float2*>(a.part_ml) + unit0 * GP;  // chunk c, head g at c * cs_ml + g
  if (staged) {
    for (int i = threadIdx.x; i < pairs; i += blockDim.x) {
      const int c = i / Gn, g = i - c * Gn;
      s_ml[i] = __ldcg(ml_g + c * cs_ml + g);
    }
  }
  __syncthreads();
  const int dq = D / 4;
  for (int idx = threadIdx.x; idx < Gn * dq; idx += blockDim.x) {
    const int g = idx / dq, d = (idx - g * dq) * 4;
    float M = -INFINITY;
    for (int c = 0; c < w.nc; ++c) M = fmaxf(M, staged ? s_ml[c * Gn + g].x : __ldcg(ml_g + c * cs_ml + g).x);
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    if (M > -INFINITY) {
      const float4* po = reinterpret_cast<const float4*>(a.part_o + (unit0 * GP + g) * D + d);
      const long long cstride = cs_ml * D / 4;  // float4s between chunks
      for (int c0 = 0; c0 < w.nc; c0 += 8) {
        float4 ov[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (c0 + i < w.nc) ov[i] = __ldcg(po + (c0 + i) * cstride);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (c0 + i < w.nc) {
            const float2 ml = staged ? s_ml[(c0 + i) * Gn + g] : __ldcg(ml_g + (c0 + i) * cs_ml + g);
            const float wgt = exp2f(ml.x - M);
            den += wgt * ml.y;
            num.x += wgt * ov[i].x;
            num.y += wgt * ov[i].y;
            num.z += wgt * ov[i].z;
            num.w += wgt * ov[i].w;
          }
        }
      }
    }
    // 8-bit caches: V's scale comes in here
    const float vsc = s.kv_fp8 ? s.kv_scales[2 * w.l + 1] : 1.f;
    const float r0 = den > 0.f ? (num.x / den) * vsc : 0.f, r1 = den > 0.f ? (num.y / den) * vsc : 0.f;
    const float r2 = den > 0.f ? (num.z / den) * vsc : 0.f, r3 = den > 0.f ? (num.w / den) * vsc : 0.f;
    const long long oi = (((long long)w.l * s.batch + w.b) * s.n_q_heads + w.h * G + g) * D + d;
    if (a.out_dtype == LT_F32) {
      *reinterpret_cast<float4*>((float*)a.out + oi) = make_float4(r0, r1, r2, r3);
    } else {
      __nv_bfloat162 lo = __floats2bfloat162_rn(r0, r1), hi = __floats2bfloat162_rn(r2, r3);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>((__nv_bfloat16*)a.out + oi) = pk;
    }
  }
}

// End of a persistent launch: the last CTA to finish re-arms the launch's
// counters and, for a fused step that advances, increments seq_lens (every CTA
// has read them by then).  Called by every thread.
__device__ __forceinline__ void finish_launch(const DecodeArgs& a) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const int prev = atomicAdd(a.done_counter, 1);
    if (prev == (int)gridDim.x - 1) {
      if (a.overlap) pdl_wait_prior_grid();  // this launch is complete only when the ones before it are
      *a.done_counter = 0;
      *a.work_counter = 0;
      if (a.fused && a.advance)
        for (int b = 0; b < a.s.batch; ++b) a.seq_lens_rw[b] += 1;
    }
  }
}

}  // namespace lt
