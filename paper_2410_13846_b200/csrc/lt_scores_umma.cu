// Lazy ratio (Eq. 1), Blackwell tensor-core path: bf16, head_dim 128.
//
// S = Q K^T is a real dense contraction here (G * w_last query rows against
// every prompt key), so it runs on the 5th-generation tensor cores:
// tcgen05.mma (M = 128, N = 128, K = 16 per instruction, bf16 in, fp32 out)
// issued by one thread, operands in shared memory in the 128-byte-swizzled
// K-major layout, accumulators in tensor memory (TMEM).
//
// One CTA per (layer, batch row, kv head, key split, block of 256 query rows),
// 10 warps with fixed roles:
//   warp 0      producer: streams 128-key K tiles into a 4-stage ring with
//               16-byte cp.async (rows past the split end are zero-filled),
//               makes them visible to the async proxy and arrives on full[s];
//   warp 1      allocates TMEM; lane 0 issues the MMAs of a tile (2 row blocks x
//               8 k-steps) into one of two accumulator buffers and commits to
//               empty[s] (stage may be refilled) and sfull[t] (scores ready);
//   warps 2-9   statistics: thread = one query row (TMEM lane), reads its row of
//               the 128 x 128 score block with tcgen05.ld and keeps only the
//               running max, sum exp and windowed sum exp - no shuffles, no
//               shared memory, nothing written until the end.
// Every wait on an mbarrier is bounded in time; on expiry the kernel raises
// LT_DEVERR_TIMEOUT in the workspace header, all roles leave their loops, TMEM
// is freed and the kernel returns.
#include <cuda_bf16.h>

#include "lt_internal.h"

namespace lt {

namespace {

constexpr int kD = 128;
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
constexpr int kThreads = 320;
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
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }

__host__ __device__ inline int split_len_umma(int n_ctx, int n_splits) {
  int len = (n_ctx + n_splits - 1) / n_splits;
  return (len + 63) / 64 * 64;
}

}  // namespace

// grid (n_splits * row_blocks, B * Hkv, L); block 320.
__global__ void __launch_bounds__(kThreads, 1) scores_umma_kernel(ScoreArgs a, LayerTable kf) {
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
  const int l = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_ctx = a.n_ctx;
  const int len = split_len_umma(n_ctx, a.n_splits);
  const int k0 = sp * len;
  const int k1 = min(n_ctx, k0 + len);
  const int n_tiles = k1 > k0 ? (k1 - k0 + kBlockN - 1) / kBlockN : 0;
  const int rows_here = min(kBlockM, M - rb * kBlockM);  // valid query rows of this CTA
  const int n_mb = (rows_here + 127) / 128;              // UMMA row blocks in use

  // ---- set-up: barriers, TMEM, Q tile ------------------------------------------
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bar_full + 8 * i, 32);
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

  const uint8_t* Kb = (const uint8_t*)kf.p[l] + ((long long)(b * s.n_kv_heads + h) * s.full_capacity) * kRowBytes;

  if (warp == 0) {
    // ===== producer =====
    constexpr int LAG = 2;  // tiles whose copies may still be in flight
    bool ok = true;
    for (int it = 0; it < n_tiles + LAG && ok; ++it) {
      if (it < n_tiles) {
        const int st = it % kStages;
        if (it >= kStages) ok = mbar_wait(bar_empty + 8 * st, ((it / kStages) & 1) ^ 1, abort_flag);
        if (ok) {
          const int kb = k0 + it * kBlockN;
          const uint32_t dst = sK + st * kStageBytes;
#pragma unroll 8
          for (int i = 0; i < (kBlockN * 16) / 32; ++i) {
            const int idx = i * 32 + lane;
            const int r = idx >> 4, p = idx & 15;
            const int row = kb + r;
            const bool valid = row < k1;
            cp_async16(dst + (p >> 3) * kKHalfBytes + r * 128 + (((p & 7) ^ (r & 7)) << 4),
                       Kb + (long long)(valid ? row : (k1 - 1)) * kRowBytes + p * 16, valid ? 16 : 0);
          }
        }
      }
      cp_async_commit();
      if (it >= LAG && ok) {
        cp_async_wait<LAG>();
        fence_proxy_async();
        mbar_arrive(bar_full + 8 * ((it - LAG) % kStages));
      }
    }
    cp_async_wait<0>();
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
  } else {
    // ===== statistics =====
    const int sw = warp - 2;
    const int mb = sw >> 2;          // row block of this warp
    const int quad = warp & 3;       // TMEM lane quadrant this warp may read
    const int r_local = mb * 128 + quad * 32 + lane;
    const int r = rb * kBlockM + r_local;
    const bool row_valid = r_local < rows_here;
    const int vis = n_ctx - T + (r % T);  // last visible key of this row
    const float cs = a.cs;
    const int S = s.n_sink, win_lo = n_ctx - s.n_recent;
    float m = -INFINITY, sA = 0.f, sWn = 0.f;
    bool ok = true;
    for (int it = 0; it < n_tiles && ok; ++it) {
      const int t = it & 1;
      ok = mbar_wait(bar_sfull + 8 * t, (it >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      if (mb < n_mb) {
        const int kb = k0 + it * kBlockN;
        const int kend = kb + kBlockN;
        const bool all_win = (kend <= S) || (kb >= win_lo);
        const bool no_win = (kb >= S) && (kend <= win_lo);
        const bool plain = (kend <= k1) && (kend - 1 <= n_ctx - T) && (all_win || no_win);
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + t * 256 + mb * 128;
#pragma unroll 1
        for (int ch = 0; ch < kBlockN / 32; ++ch) {
          uint32_t v[32];
          tmem_ld32(taddr + ch * 32, v);
          tmem_ld_wait();
          if (plain) {
            float cm = __uint_as_float(v[0]);
#pragma unroll
            for (int i = 1; i < 32; ++i) cm = fmaxf(cm, __uint_as_float(v[i]));
            const float mn = fmaxf(m, cm);
            const float corr = exp2f((m - mn) * cs);
            const float off = -mn * cs;
            float ps = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) ps += exp2f(fmaf(__uint_as_float(v[i]), cs, off));
            sA = sA * corr + ps;
            sWn = sWn * corr + (all_win ? ps : 0.f);
            m = mn;
          } else {
            const int lim = min(vis, k1 - 1);
            const int jb = kb + ch * 32;
            float cm = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (jb + i <= lim) cm = fmaxf(cm, __uint_as_float(v[i]));
            const float mn = fmaxf(m, cm);
            if (mn > -INFINITY) {
              const float corr = exp2f((m - mn) * cs);
              const float off = -mn * cs;
              float ps = 0.f, pw = 0.f;
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const int j = jb + i;
                if (j <= lim) {
                  const float p = exp2f(fmaf(__uint_as_float(v[i]), cs, off));
                  ps += p;
                  if (j < S || j >= win_lo) pw += p;
                }
              }
              sA = sA * corr + ps;
              sWn = sWn * corr + pw;
              m = mn;
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar_sempty + 8 * t);
    }
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

bool scores_umma_supported(const lt_shape& s, int /*w_last*/) { return s.dtype == LT_BF16 && s.head_dim == 128; }

cudaError_t launch_scores_umma(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st) {
  const int G = a.s.n_q_heads / a.s.n_kv_heads;
  const int M = G * a.w_last;
  const int row_blocks = (M + kBlockM - 1) / kBlockM;
  cudaError_t e = cudaFuncSetAttribute(scores_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  dim3 grid(a.n_splits * row_blocks, a.s.batch * a.s.n_kv_heads, a.s.n_layers);
  scores_umma_kernel<<<grid, kThreads, kSmemBytes, st>>>(a, kf);
  return cudaGetLastError();
}

}  // namespace lt
