// Lazy ratio (Eq. 1), Blackwell tensor-core path: bf16, head_dim 128.
//
// S = Q K^T is a real dense contraction here (G * w_last query rows against
// every prompt key), so it runs on the 5th-generation tensor cores:
// tcgen05.mma (M = 128, N = 128, K = 16 per instruction, bf16 in, fp32 out)
// issued by one thread, operands in shared memory in the 128-byte-swizzled
// K-major layout, accumulators in tensor memory (TMEM).
//
// One CTA per (layer, batch row, kv head, key split, block of 256 query rows),
// three warpgroups with fixed roles:
//   warp 0      producer: one lane streams 128-key K tiles into a 4-stage ring
//               with TMA (cp.async.bulk.tensor, two 64-column boxes per tile, the
//               128-byte swizzle applied by the copy engine), completion counted
//               in bytes on full[s];
//   warp 1      allocates TMEM; lane 0 issues the MMAs of a tile (2 row blocks x
//               8 k-steps) into one of two accumulator buffers and commits to
//               empty[s] (stage may be refilled) and sfull[t] (scores ready);
//   warps 2-3   fill up the first warpgroup (register hand-over is per warpgroup);
//   warps 4-11  statistics: thread = one query row (TMEM lane), reads its row of
//               the 128 x 128 score block with tcgen05.ld and keeps only the
//               running max, sum exp and windowed sum exp - no shuffles, no
//               shared memory, nothing written until the end.  The exponentials
//               (one MUFU instruction each) are the floor of this kernel, so
//               these warps take the registers the first warpgroup gives up and
//               hold a whole 128-column row in flight.
// Every wait on an mbarrier is bounded in time; on expiry the kernel raises
// LT_DEVERR_TIMEOUT in the workspace header, all roles leave their loops, TMEM
// is freed and the kernel returns.
#include <cuda.h>  // CUtensorMap and its enums; the encoder is looked up at run time, nothing links to libcuda
#include <cuda_bf16.h>

#include "lt_internal.h"

namespace lt {

namespace {

constexpr int kD = 128;  // head_dim
constexpr int kRowBytes = 256;
constexpr int kBlockM = 256;   // query rows per CTA (2 UMMA row blocks)
constexpr int kBlockN = 128;   // keys per tile
constexpr int kStages = 4;
constexpr int kQHalfBytes = kBlockM * 128;        // one d-half of Q: [256 rows][128 B]
constexpr int kQBytes = 2 * kQHalfBytes;          // 64 KB
constexpr int kKHalfBytes = kBlockN * 128;        // one d-half of a K tile
constexpr int kStageBytes = 2 * kKHalfBytes;      // 32 KB
constexpr int kBarBytes = 256;
constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kBarBytes + 1024;  // + alignment slack
constexpr int kThreads = 384;
constexpr int kRegsLight = 56;   // producer / MMA warpgroup after setmaxnreg.dec
constexpr int kRegsStats = 224;  // statistics warpgroups after setmaxnreg.inc
constexpr int kTmemCols = 512;
constexpr long long kWaitCycles = 4000000000ll;  // ~2 s at 1.9 GHz

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
// One box of a 2-D tensor map into shared memory; completes `bar` by the box's bytes.
// x * element size must be a multiple of 16 bytes (here x is 0 or 64 bf16 elements).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// Bounded wait.  Returns false when the wait expired or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitCycles) {
      *abort_flag = 1;
      return false;
    }
  }
}

// Bounded wait that ignores the abort flag: used to let copies in flight land before the CTA exits.
__device__ __forceinline__ void mbar_wait_quiet(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity) && clock64() - t0 < kWaitCycles) {
  }
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of
// 128 bytes, 8-row groups 1024 bytes apart (dense), descriptor version 1.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address, 16-byte units
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused with swizzle): 1
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                          // version
  d |= (uint64_t)2 << 61;                          // SWIZZLE_128B
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, N = 128, M = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlockN >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
// 32 consecutive columns of this thread's TMEM lane into v[OFF .. OFF+31] (asynchronous until tmem_ld_wait)
template <int OFF, int N>
__device__ __forceinline__ void tmem_ld32_at(uint32_t taddr, uint32_t (&v)[N]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(v[OFF + 0]), "=r"(v[OFF + 1]), "=r"(v[OFF + 2]), "=r"(v[OFF + 3]), "=r"(v[OFF + 4]), "=r"(v[OFF + 5]),
        "=r"(v[OFF + 6]), "=r"(v[OFF + 7]), "=r"(v[OFF + 8]), "=r"(v[OFF + 9]), "=r"(v[OFF + 10]), "=r"(v[OFF + 11]),
        "=r"(v[OFF + 12]), "=r"(v[OFF + 13]), "=r"(v[OFF + 14]), "=r"(v[OFF + 15]), "=r"(v[OFF + 16]),
        "=r"(v[OFF + 17]), "=r"(v[OFF + 18]), "=r"(v[OFF + 19]), "=r"(v[OFF + 20]), "=r"(v[OFF + 21]),
        "=r"(v[OFF + 22]), "=r"(v[OFF + 23]), "=r"(v[OFF + 24]), "=r"(v[OFF + 25]), "=r"(v[OFF + 26]),
        "=r"(v[OFF + 27]), "=r"(v[OFF + 28]), "=r"(v[OFF + 29]), "=r"(v[OFF + 30]), "=r"(v[OFF + 31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
// One MUFU instruction: 2^x, relative error 2^-22, results below 2^-126 flush to zero.
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
// max of 64 values: four interleaved chains, then a small tree (short dependency depth)
__device__ __forceinline__ float max64(const uint32_t (&v)[64]) {
  float m0 = __uint_as_float(v[0]), m1 = __uint_as_float(v[1]), m2 = __uint_as_float(v[2]),
        m3 = __uint_as_float(v[3]);
#pragma unroll
  for (int i = 4; i < 64; i += 4) {
    m0 = fmaxf(m0, __uint_as_float(v[i]));
    m1 = fmaxf(m1, __uint_as_float(v[i + 1]));
    m2 = fmaxf(m2, __uint_as_float(v[i + 2]));
    m3 = fmaxf(m3, __uint_as_float(v[i + 3]));
  }
  return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}
// sum_i 2^(v_i * cs + off): four accumulators
__device__ __forceinline__ float sum_ex2_64(const uint32_t (&v)[64], float cs, float off) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int i = 0; i < 64; i += 4) {
    s0 += ex2(fmaf(__uint_as_float(v[i]), cs, off));
    s1 += ex2(fmaf(__uint_as_float(v[i + 1]), cs, off));
    s2 += ex2(fmaf(__uint_as_float(v[i + 2]), cs, off));
    s3 += ex2(fmaf(__uint_as_float(v[i + 3]), cs, off));
  }
  return (s0 + s1) + (s2 + s3);
}

}  // namespace

// grid (n_splits * row_blocks, B * Hkv, L); block 384.
struct KeyMaps {
  CUtensorMap m[LT_MAX_LAYERS];  // layer l's K cache as a [B * Hkv * capacity][128] bf16 matrix, box 64 x 128
};

__global__ void __launch_bounds__(kThreads, 1)
    scores_umma_kernel(ScoreArgs a, const __grid_constant__ KeyMaps maps) {
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: the swizzle pattern of the MMA is a function of address bits 4..9
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sK = sQ + kQBytes;
  uint8_t* bar_mem = smem + kQBytes + kStages * kStageBytes;
  const uint32_t bar0 = smem_u32(bar_mem);
  const uint32_t bar_full = bar0;                      // [kStages]
  const uint32_t bar_empty = bar0 + 8 * kStages;       // [kStages]
  const uint32_t bar_sfull = bar0 + 16 * kStages;      // [2]
  const uint32_t bar_sempty = bar_sfull + 16;          // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + 16 * kStages + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 16 * kStages + 40);

  const lt_shape& s = a.s;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int T = a.w_last;
  const int M = G * T;
  const int sp = blockIdx.x % a.n_splits, rb = blockIdx.x / a.n_splits;
  const int b = blockIdx.y / s.n_kv_heads, h = blockIdx.y % s.n_kv_heads;
  const int l = a.layer_begin + blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_ctx = a.n_ctx;
  int k0, k1;
  score_split_range(a, sp, &k0, &k1);
  // Paged caches: tiles start on multiples of 128 keys so that none straddles two pages (the page size
  // is a multiple of 128); the keys before k0 in the first tile are masked by the statistics warps.
  const int ts0 = s.page_size > 0 ? (k0 & ~(kBlockN - 1)) : k0;
  const int n_tiles = k1 > k0 ? (k1 - ts0 + kBlockN - 1) / kBlockN : 0;
  const int rows_here = min(kBlockM, M - rb * kBlockM);  // valid query rows of this CTA
  const int n_mb = (rows_here + 127) / 128;              // UMMA row blocks in use

  // ---- set-up: barriers, TMEM, Q tile ------------------------------------------
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_sfull + 8 * i, 1);
      mbar_init(bar_sempty + 8 * i, 256);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  {
    const uint8_t* qb = (const uint8_t*)a.q_tail +
                        ((((long long)l * s.batch + b) * s.n_q_heads + (long long)h * G) * T + (long long)rb * kBlockM) *
                            kRowBytes;
    for (int idx = threadIdx.x; idx < kBlockM * 16; idx += kThreads) {
      const int r = idx >> 4, p = idx & 15;
      const bool valid = r < rows_here;
      cp_async16(sQ + (p >> 3) * kQHalfBytes + r * 128 + (((p & 7) ^ (r & 7)) << 4),
                 qb + (long long)(valid ? r : 0) * kRowBytes + p * 16, valid ? 16 : 0);
    }
    cp_async_commit();
    cp_async_wait<0>();
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // tensor-map row of key j of this (b, kv head); j is a tile start
  auto map_row = [&](int j) {
    if (s.page_size <= 0) return (b * s.n_kv_heads + h) * s.full_capacity + j;
    const int page = s.block_table[(long long)b * s.pages_per_seq + j / s.page_size];
    return (page * s.n_kv_heads + h) * s.page_size + j % s.page_size;
  };

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegsLight));
  if (warp == 0) {
    // ===== producer =====
    // Rows past the split end are real cache rows (or zero past the end of the
    // cache): the statistics warps never look at those columns.
    if (lane == 0) {
      const CUtensorMap* map = &maps.m[l];
      bool ok = true;
      int issued = 0;
      for (int it = 0; it < n_tiles && ok; ++it) {
        const int st = it % kStages;
        if (it >= kStages) ok = mbar_wait(bar_empty + 8 * st, ((it / kStages) & 1) ^ 1, abort_flag);
        if (!ok) break;
        const uint32_t dst = sK + st * kStageBytes;
        const uint32_t bar = bar_full + 8 * st;
        mbar_expect_tx(bar, kStageBytes);
        const int y = map_row(ts0 + it * kBlockN);
        tma_load_2d(dst, map, 0, y, bar);
        tma_load_2d(dst + kKHalfBytes, map, 64, y, bar);
        issued = it + 1;
      }
      if (!ok) {
        // gave up: let the copies already issued land before the shared memory goes away
        for (int j = max(0, issued - kStages); j < issued; ++j)
          mbar_wait_quiet(bar_full + 8 * (j % kStages), (j / kStages) & 1);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ===== MMA issuer =====
    if (lane == 0) {
      bool ok = true;
      for (int it = 0; it < n_tiles && ok; ++it) {
        const int st = it % kStages, t = it & 1;
        if (it >= 2) ok = mbar_wait(bar_sempty + 8 * t, ((it >> 1) & 1) ^ 1, abort_flag);
        if (ok) ok = mbar_wait(bar_full + 8 * st, (it / kStages) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        fence_proxy_async();
        for (int mb = 0; mb < n_mb; ++mb) {
          const uint32_t d_tmem = tmem_base + t * 256 + mb * 128;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t a_addr = sQ + (ks >> 2) * kQHalfBytes + mb * (128 * 128) + (ks & 3) * 32;
            const uint32_t b_addr = sK + st * kStageBytes + (ks >> 2) * kKHalfBytes + (ks & 3) * 32;
            umma_bf16(d_tmem, umma_desc(a_addr), umma_desc(b_addr), ks > 0 ? 1u : 0u);
          }
        }
        umma_commit(bar_empty + 8 * st);
        umma_commit(bar_sfull + 8 * t);
      }
    }
    __syncwarp();
  }
  } else {
    // ===== statistics =====
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegsStats));
    // A tile's 128 columns are taken in two halves of 64 registers.  The load of
    // one half is in flight while the exponentials of the other half run, and
    // the accumulator buffer is handed back to the MMA warp as soon as both
    // halves sit in registers.
    const int sw = warp - 4;
    const int mb = sw >> 2;          // row block of this warp
    const int quad = warp & 3;       // TMEM lane quadrant this warp may read
    const int r_local = mb * 128 + quad * 32 + lane;
    const int r = rb * kBlockM + r_local;
    const bool row_valid = r_local < rows_here;
    const int vis = n_ctx - T + (r % T);  // last visible key of this row
    const float cs = a.cs;
    const int S = s.n_sink;
    const int win_lo = s.recent_per_row ? vis - s.n_recent + 1 : n_ctx - s.n_recent;  // first recent key of this row
    const int lim = min(vis, k1 - 1);     // last key of this split that the row may see
    float m = -INFINITY, sA = 0.f, sWn = 0.f;
    const bool active = mb < n_mb;
    const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16) + mb * 128;

    // statistics of one half (64 keys from jb) already in registers
    auto half_stats = [&](uint32_t (&v)[64], int jb) {
      const int jend = jb + 64;
      const bool all_win = (jend <= S) || (jb >= win_lo);
      const bool no_win = (jb >= S) && (jend <= win_lo);
      if ((jb >= k0) && (jend - 1 <= lim) && (all_win || no_win)) {
        const float mn = fmaxf(m, max64(v));
        const float corr = ex2((m - mn) * cs);
        const float ps = sum_ex2_64(v, cs, -mn * cs);
        sA = fmaf(sA, corr, ps);
        sWn = fmaf(sWn, corr, all_win ? ps : 0.f);
        m = mn;
      } else if (max(jb, k0) <= min(jend - 1, lim)) {
        // boundary half (split start, causal tail, split end or window edge): mask in place.
        // 2^(-inf) = 0, and at least one key is visible, so the maximum is finite.
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (jb + i > lim || jb + i < k0) v[i] = 0xff800000u;
        const float mn = fmaxf(m, max64(v));
        const float corr = ex2((m - mn) * cs);
        const float off = -mn * cs;
        const float ps = sum_ex2_64(v, cs, off);
#pragma unroll
        for (int i = 0; i < 64; ++i) {
          const int j = jb + i;
          if (!(j < S || j >= win_lo)) v[i] = 0xff800000u;
        }
        const float pw = sum_ex2_64(v, cs, off);
        sA = fmaf(sA, corr, ps);
        sWn = fmaf(sWn, corr, pw);
        m = mn;
      }
    };

    bool ok = true;
    uint32_t va[64], vb[64];
    if (n_tiles > 0) {
      ok = mbar_wait(bar_sfull, 0, abort_flag);
      tc_fence_after();
      if (ok && active) {
        tmem_ld32_at<0>(lane_base, va);
        tmem_ld32_at<32>(lane_base + 32, va);
      }
    }
    for (int it = 0; it < n_tiles && ok; ++it) {
      const int t = it & 1;
      const int kb = ts0 + it * kBlockN;
      const uint32_t taddr = lane_base + t * 256;
      // first half is (being) loaded; start the second half, then work on the first
      tmem_ld_wait();
      if (active) {
        tmem_ld32_at<0>(taddr + 64, vb);
        tmem_ld32_at<32>(taddr + 96, vb);
        half_stats(va, kb);
      }
      tmem_ld_wait();
      // both halves are in registers: the accumulator buffer may be overwritten
      tc_fence_before();
      mbar_arrive(bar_sempty + 8 * t);
      if (it + 1 < n_tiles) {
        const int tn = (it + 1) & 1;
        ok = mbar_wait(bar_sfull + 8 * tn, ((it + 1) >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        if (active) {
          tmem_ld32_at<0>(lane_base + tn * 256, va);
          tmem_ld32_at<32>(lane_base + tn * 256 + 32, va);
        }
      }
      if (active) half_stats(vb, kb + 64);
    }
    tmem_ld_wait();
    if (ok && row_valid) {
      const int g = r / T, tq = r - g * T;
      const long long rowid = (((long long)l * s.batch + b) * s.n_q_heads + h * G + g) * T + tq;
      float* stp = a.stats + (rowid * a.n_splits + sp) * 3;
      stp[0] = m * cs;
      stp[1] = sA;
      stp[2] = sWn;
    }
  }

  // ---- teardown ------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(a.dev_err, LT_DEVERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                 : "memory");
  }
}

bool scores_umma_supported(const lt_shape& s, int /*w_last*/) {
  return s.dtype == LT_BF16 && s.head_dim == 128 &&
         (long long)s.batch * s.n_kv_heads * s.full_capacity < (1ll << 31);  // tensor-map rows fit an int32 coordinate
}

namespace {
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// The driver's tensor-map encoder, looked up through the runtime (no link-time dependency on libcuda).
EncodeTiledFn lookup_encode_tiled() {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess)
    return nullptr;
  return reinterpret_cast<EncodeTiledFn>(p);
}
EncodeTiledFn encode_tiled_fn() {
  static const EncodeTiledFn fn = lookup_encode_tiled();  // initialised once, thread-safe
  return fn;
}
}  // namespace

cudaError_t launch_scores_umma(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st) {
  const int G = a.s.n_q_heads / a.s.n_kv_heads;
  const int M = G * a.w_last;
  const int row_blocks = (M + kBlockM - 1) / kBlockM;
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return cudaErrorNotSupported;
  const cuuint64_t rows_total = a.s.page_size > 0 ? (cuuint64_t)a.s.n_pages * a.s.n_kv_heads * a.s.page_size
                                                  : (cuuint64_t)a.s.batch * a.s.n_kv_heads * a.s.full_capacity;
  const cuuint64_t gdim[2] = {(cuuint64_t)kD, rows_total};
  const cuuint64_t gstride[1] = {(cuuint64_t)kRowBytes};
  const cuuint32_t box[2] = {64u, (cuuint32_t)kBlockN};
  const cuuint32_t estride[2] = {1u, 1u};
  KeyMaps local;
  const int l_end = a.layer_begin + a.layer_count;
  for (int l = a.layer_begin; l < l_end; ++l) {
    const CUresult r = encode(&local.m[l], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(kf.p[l]), gdim,
                              gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  for (int l = 0; l < LT_MAX_LAYERS; ++l)
    if (l < a.layer_begin || l >= l_end) local.m[l] = local.m[a.layer_begin];
  cudaError_t e = cudaFuncSetAttribute(scores_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  dim3 grid(a.n_splits * row_blocks, a.s.batch * a.s.n_kv_heads, a.layer_count);
  scores_umma_kernel<<<grid, kThreads, kSmemBytes, st>>>(a, local);
  return cudaGetLastError();
}

}  // namespace lt
