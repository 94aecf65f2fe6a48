// Lazy ratio (Eq. 1), Blackwell tensor-core path: bf16 queries, head_dim 128 or 64; keys in bf16, or (head_dim 128,
// template branch K8) as the E4M3 bytes of an 8-bit cache, which go through tcgen05.mma kind::f8f6f4 against the
// queries as two E4M3 terms (see Geo and q_split_kernel).
//
// S = Q K^T is a real dense contraction here (G * w_last query rows against
// every prompt key), so it runs on the 5th-generation tensor cores:
// tcgen05.mma (M = 128, N = 256, K = 16 per instruction, bf16 in, fp32 out)
// issued by one thread, operands in shared memory in the 128-byte-swizzled
// K-major layout, accumulators in tensor memory (TMEM).  N = 256 on purpose: the
// issuing thread pays a fixed cost per instruction group (barrier wait, commit)
// during which it issues nothing, and only instructions of 128 clocks each keep
// the tensor pipe fed across those gaps (measured: groups of eight N = 128
// instructions run at 92 clocks per instruction instead of 64, N = 256 at 128).
//
// The launch is persistent: one CTA per SM.  With the whole prompt scored
// (lt_lazy_scores) the 256-key tiles of all (layer, batch row, kv head, block of
// 256 query rows) units form one sequence that is cut into equal contiguous
// ranges, one per CTA, so every SM gets the same number of tiles whatever the
// unit count; a unit that straddles a cut gets its own statistics slots per piece.
// With the denominator given (lt_lazy_scores_lse) the work items are the host's
// key splits of the kept ranges, a contiguous run of them per CTA.
//
// Roles (18 warps):
//   warp 0      producer: one lane streams the unit's query block (64 KB, at a change
//               of unit) and the 256-key K tiles (64 KB each, two stages) into shared
//               memory with TMA (cp.async.bulk.tensor, 64-column x 128/256-row boxes),
//               completion counted in bytes;
//   warp 1      allocates TMEM; lane 0 issues the MMAs of a tile (8 k-steps per row
//               block of 128 query rows) into that row block's accumulator (256
//               columns) and commits to its slot_full and, after the tile's last row
//               block, to empty[s];
//   warps 2-17  statistics, four per scheduler: thread = one query row (one TMEM lane)
//               x one half of the tile's 256 keys.  It reads its 128 scores in chunks of
//               32 registers with tcgen05.ld (the other warps of its scheduler run under
//               the load) and keeps only a reference exponent, sum exp and windowed sum
//               exp - no shuffles, no shared memory, nothing written until the end of the
//               piece.  The accumulator goes back to the MMA warp as soon as the row's last
//               chunk is in registers.
// Warps 2-9 read accumulator 0 and warps 10-17 accumulator 1.  A unit with more than 128
// query rows fills both with every tile (one row block each).  A unit with at most 128
// rows (multi-head attention, short tails) alternates instead: tile i goes to
// accumulator i & 1, so the MMAs of a tile run under the statistics of the tile before
// it, and the second group hands its sums to the first through shared memory at the
// end of the piece (two mbarriers, waits bounded like all others).
//
// Exponentials.  One ex2 per score on the special-function unit (16 per clock per
// SM) makes that unit the busiest of the SM (~80 %), so a fixed share of the columns
// takes 2^x on the FMA pipe
// instead: the reference of a row is an INTEGER M >= max (log2 domain), so x = t - M
// splits exactly into round(x) and a remainder f in [-1/2, 1/2]; 2^f is a cubic
// (relative error 7.5e-5, far inside the 1e-3 absolute tolerance of a ratio of sums)
// and round(x) goes into the exponent field with one integer add.  The FMA-pipe work
// uses the packed two-lane fp32 instructions (fma / add .f32x2).  The share is small
// (an eighth): measured, an ex2 costs the scheduler about five issue slots and the
// polynomial about twelve, so a larger share only trades one bound for another.
//
// On B200 the pass as a whole runs at the board's power limit (about 1 kW with the
// key stream, the MMAs and the statistics all active): its time follows its energy,
// and changes to the instruction stream mostly change the clock the governor leaves.
//
// Every wait on an mbarrier is bounded in time; on expiry the kernel raises
// LT_DEVERR_TIMEOUT in the workspace header, all roles leave their loops, TMEM
// is freed and the kernel returns.
#include <cuda.h>  // CUtensorMap and its enums; the encoder is looked up at run time, nothing links to libcuda
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "lt_internal.h"

#ifndef LT_SCORES_POLY_OF8
#define LT_SCORES_POLY_OF8 1  // of every 8 column pairs, this many take 2^x on the FMA pipe
#endif

namespace lt {

namespace {

constexpr int kBlockM = kScoreBlockM;  // query rows per unit (2 UMMA row blocks)
constexpr int kBlockN = kScoreBlockN;  // keys per tile (one UMMA instruction wide)
constexpr int kQHalfBytes = kBlockM * 128;        // 64 d (one 128-byte half of a row) of the query block: [256 rows][128 B]
constexpr int kKHalfBytes = kBlockN * 128;        // 64 d of a K tile: [256 rows][128 B]
constexpr int kBarBytes = 256;
constexpr int kMergeBytes = 2 * 128 * 3 * 4;      // (reference, sum, windowed sum) of 128 rows x two key halves
// Geometry that depends on the head dimension DH (128 or 64): a row has DH / 64 halves of 128 bytes; the K ring
// holds 128 KB either way (2 stages of 64 KB, or 4 of 32 KB).
// K8 (8-bit keys, head_dim 128): a K row is one 128-byte span of E4M3 bytes and a tile 32 KB (four stages); the
// query block comes as two E4M3 terms (q = scale * (hi + lo), see q_split_kernel) of 32 KB each, which take the
// places of the two 64-d halves of a 16-bit query block, and the contraction runs as four 32-wide k-steps per term.
template <int DH, bool K8 = false>
struct Geo {
  static_assert(!K8 || DH == 128, "8-bit keys: head_dim 128");
  static constexpr int kHalves = DH / 64;                               // 128-byte spans of a 16-bit row; K8: terms of q
  static constexpr int kKHalves = K8 ? 1 : kHalves;                     // 128-byte spans of a K row
  static constexpr int kQBytes = kHalves * kQHalfBytes;                 // 64 KB or 32 KB
  static constexpr int kStageBytes = kKHalves * kKHalfBytes;            // 64 KB or 32 KB
  static constexpr int kStages = 4 / kKHalves;
  static constexpr int kKSteps = DH / 16;                               // MMAs per row block and tile (K8: 2 terms x 4)
  static constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kBarBytes + kMergeBytes + 1024;  // + alignment slack
};
constexpr int kStatWarps = 16;
constexpr int kThreads = 64 + kStatWarps * 32;    // 576 (registers are granted as for 640: 96 per thread)
constexpr int kTmemCols = 512;   // two accumulators of 256 columns, one per row block
constexpr int kChunk = 32;       // columns per tcgen05.ld
constexpr int kPolyOf8 = LT_SCORES_POLY_OF8;
constexpr long long kWaitCycles = 4000000000ll;  // ~2 s at 1.9 GHz
constexpr uint32_t kSuspendHintNs = 1000000u;    // a waiting thread may stay suspended this long before try_wait returns

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
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
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
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
  for (uint32_t polls = 1;; ++polls) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((polls & 15u) == 0u) {  // the flag and the clock are looked at every 16th poll: a poll stays four instructions
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        return false;
      }
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
// Instruction descriptor: D fp32, A and B bf16, both K-major, N = 256, M = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlockN >> 3) << 17) | ((128u >> 4) << 24);

// The same with A and B in E4M3 (format code 0 in both fields), for tcgen05.mma.kind::f8f6f4: K = 32 per instruction.
constexpr uint32_t kIdesc8 = (1u << 4) | ((uint32_t)(kBlockN >> 3) << 17) | ((128u >> 4) << 24);

// D[tmem] (+)= A[smem] . B[smem]^T over 32 E4M3 values per row: A a 128-row slice of one term of the query block,
// B a 256-key slice of the K tile.
__device__ __forceinline__ void umma_e4m3_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}\n" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(kIdesc8), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[smem] . B[smem]^T: A a 128-row x 16-d slice of the query block, B a 256-key x 16-d slice of the K tile.
__device__ __forceinline__ void umma_bf16_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
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
// 32 consecutive columns of this thread's TMEM lane into v[0 .. 31] (asynchronous until tmem_ld_wait)
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
// One MUFU instruction: 2^x, relative error 2^-22, results below 2^-126 flush to zero.
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
// Three-input maximum (one instruction on sm_100).
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;\n" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Packed two-lane fp32 arithmetic (one instruction per pair).
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ f32x2 pack2u(uint32_t lo, uint32_t hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;\n" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// max of 32 values: four interleaved chains of three-input maxima, then a small tree
__device__ __forceinline__ float max32(const uint32_t (&v)[32]) {
  float m0 = max3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
  float m1 = max3(__uint_as_float(v[3]), __uint_as_float(v[4]), __uint_as_float(v[5]));
  float m2 = max3(__uint_as_float(v[6]), __uint_as_float(v[7]), __uint_as_float(v[8]));
  float m3 = max3(__uint_as_float(v[9]), __uint_as_float(v[10]), __uint_as_float(v[11]));
#pragma unroll
  for (int i = 12; i < 28; i += 8) {
    m0 = max3(m0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
    m1 = max3(m1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
    m2 = max3(m2, __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
    m3 = max3(m3, __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
  }
  m0 = max3(m0, __uint_as_float(v[28]), __uint_as_float(v[29]));
  m1 = max3(m1, __uint_as_float(v[30]), __uint_as_float(v[31]));
  return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// 2^f on [-1/2, 1/2] as a cubic: least maximum relative error (7.5e-5), from a weighted least-squares
// (Lawson) fit of p(f) / 2^f to 1 on 4001 Chebyshev nodes, coefficients rounded to float.
constexpr float kP0 = 0.9999280571937561f, kP1 = 0.6932609677314758f, kP2 = 0.2426111251115799f,
                kP3 = 0.0551716685295105f;
constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it leaves round-to-nearest(x) in the low mantissa bits
constexpr float kMinX = -125.0f;       // 2^x below this is treated as 2^-125 (keeps the exponent field positive)

// sum_i 2^(v_i * cs - M) over the 32 values, M an integer (as a float): MUFU for most column pairs, the
// FMA-pipe polynomial for kPolyOf8 of every 8 pairs.
__device__ __forceinline__ float sum_ex2_32_mixed(const uint32_t (&v)[32], float cs, float M) {
  const f32x2 cs2 = pack2(cs, cs), nM2 = pack2(-M, -M);
  const f32x2 magic2 = pack2(kMagic, kMagic), mone2 = pack2(-1.f, -1.f);
  const f32x2 p3 = pack2(kP3, kP3), p2 = pack2(kP2, kP2), p1 = pack2(kP1, kP1), p0 = pack2(kP0, kP0);
  f32x2 acc0 = pack2(0.f, 0.f), acc1 = acc0, acc2 = acc0, acc3 = acc0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {  // pair i = columns 2i, 2i + 1
    const f32x2 x2 = fma2(pack2u(v[2 * i], v[2 * i + 1]), cs2, nM2);
    float xl, xh;
    unpack2(x2, xl, xh);
    f32x2 e2;
    // the polynomial pairs are spread over the group of 8 so that both pipes stay fed
    const bool poly = ((i & 7) * kPolyOf8) / 8 != (((i & 7) + 1) * kPolyOf8) / 8;
    if (poly) {
      const f32x2 xc = pack2(fmaxf(xl, kMinX), fmaxf(xh, kMinX));
      const f32x2 t2 = add2(xc, magic2);                     // magic + round(x)
      const f32x2 f2 = add2(xc, fma2(t2, mone2, magic2));    // x - round(x), exact
      f32x2 p = fma2(p3, f2, p2);
      p = fma2(p, f2, p1);
      p = fma2(p, f2, p0);
      float pl, ph, tl, th;
      unpack2(p, pl, ph);
      unpack2(t2, tl, th);
      // 2^round(x): the integer sits in the low bits of t; shifted into the exponent field it adds to p's exponent
      const float rl = __int_as_float(__float_as_int(pl) + (__float_as_int(tl) << 23));
      const float rh = __int_as_float(__float_as_int(ph) + (__float_as_int(th) << 23));
      e2 = pack2(rl, rh);
    } else {
      e2 = pack2(ex2(xl), ex2(xh));
    }
    if ((i & 3) == 0) acc0 = add2(acc0, e2);
    else if ((i & 3) == 1) acc1 = add2(acc1, e2);
    else if ((i & 3) == 2) acc2 = add2(acc2, e2);
    else acc3 = add2(acc3, e2);
  }
  float a, b;
  unpack2(add2(add2(acc0, acc1), add2(acc2, acc3)), a, b);
  return a + b;
}
// The same sum with every exponential on the MUFU; -inf entries (masked columns) contribute 0.
__device__ __forceinline__ float sum_ex2_32(const uint32_t (&v)[32], float cs, float off) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    s0 += ex2(fmaf(__uint_as_float(v[i]), cs, off));
    s1 += ex2(fmaf(__uint_as_float(v[i + 1]), cs, off));
    s2 += ex2(fmaf(__uint_as_float(v[i + 2]), cs, off));
    s3 += ex2(fmaf(__uint_as_float(v[i + 3]), cs, off));
  }
  return (s0 + s1) + (s2 + s3);
}

}  // namespace

struct KeyMaps {
  CUtensorMap q;                 // q_tail as a [L * B * Hq * w_last][128] bf16 matrix, box 64 x 256
  CUtensorMap m[LT_MAX_LAYERS];  // layer l's K cache as a [B * Hkv * capacity][128] bf16 matrix, box 64 x 128
};

// One contiguous run of tiles of one unit, handled by one CTA.
struct Piece {
  int l, b, h, rb;  // the unit: layer, batch row, kv head, block of 256 query rows
  int unit;         // its index (changes <=> the query block in shared memory must be replaced)
  int k0, k1;       // keys of the piece: statistics cover [k0, k1)
  int ts0;          // first key of the piece's first tile
  int n_tiles;
  int slot;         // statistics slot pair of the piece within its rows (one slot per column half)
};

// The pieces of this CTA, in order.  `cursor` starts at 0 (every role walks the same list on its own).
__device__ __forceinline__ bool next_piece(const ScoreArgs& a, long long& cursor, Piece& p) {
  const lt_shape& s = a.s;
  int unit, k0, k1, ts0, n_tiles, slot;
  if (a.streamk) {
    long long g_begin, g_end;
    score_cta_tiles(a.total_tiles, gridDim.x, blockIdx.x, &g_begin, &g_end);
    const long long g = g_begin + cursor;
    if (g >= g_end) return false;
    const int TU = a.tiles_per_unit;
    unit = (int)(g / TU);
    const int ta = (int)(g - (long long)unit * TU);
    const int tb = (int)min((long long)TU, ta + (g_end - g));
    k0 = ta * kBlockN;
    k1 = min(tb * kBlockN, a.n_ctx);
    ts0 = k0;
    n_tiles = tb - ta;
    slot = (int)blockIdx.x - score_tile_owner(a.total_tiles, gridDim.x, (long long)unit * TU);
    cursor += n_tiles;
  } else {
    // host splits of the kept key ranges: every CTA takes a contiguous run of (unit, split) items, so that the
    // query block in shared memory is replaced only when the run moves on to the next unit
    const int host_splits = a.n_splits / 2;
    const long long n_items = (long long)a.n_units * host_splits;
    long long i_begin, i_end;
    score_cta_tiles(n_items, gridDim.x, blockIdx.x, &i_begin, &i_end);
    const long long item = i_begin + cursor;
    if (item >= i_end) return false;
    unit = (int)(item / host_splits);
    slot = (int)(item - (long long)unit * host_splits);
    score_split_range(a, slot, &k0, &k1);
    // Paged caches: tiles start on multiples of 128 keys so that no 128-key box straddles two pages (the page
    // size is a multiple of 128); the keys before k0 in the first tile are masked by the statistics warps.
    ts0 = s.page_size > 0 ? (k0 & ~127) : k0;
    n_tiles = k1 > k0 ? (k1 - ts0 + kBlockN - 1) / kBlockN : 0;
    cursor += 1;
  }
  p.unit = unit;
  p.rb = unit % a.row_blocks;
  int x = unit / a.row_blocks;
  p.h = x % s.n_kv_heads;
  x /= s.n_kv_heads;
  p.b = x % s.batch;
  p.l = a.layer_begin + x / s.batch;
  p.k0 = k0;
  p.k1 = k1;
  p.ts0 = ts0;
  p.n_tiles = n_tiles;
  p.slot = slot;
  return true;
}

template <int DH, bool K8>
__global__ void __launch_bounds__(kThreads, 1)
    scores_umma_kernel(ScoreArgs a, const __grid_constant__ KeyMaps maps) {
  using G_ = Geo<DH, K8>;
  constexpr int kHalves = G_::kHalves, kKHalves = G_::kKHalves, kQBytes = G_::kQBytes, kStageBytes = G_::kStageBytes;
  constexpr int kStages = G_::kStages, kKSteps = G_::kKSteps;
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: the swizzle pattern of the MMA is a function of address bits 4..9
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sK = sQ + kQBytes;
  uint8_t* bar_mem = smem + kQBytes + kStages * kStageBytes;
  const uint32_t bar0 = smem_u32(bar_mem);
  const uint32_t bar_full = bar0;                      // [kStages]  K tile landed
  const uint32_t bar_empty = bar0 + 8 * kStages;       // [kStages]  K tile consumed by the MMAs
  const uint32_t bar_sfull = bar0 + 16 * kStages;      // [2]        row block's accumulator holds a score block
  const uint32_t bar_sempty = bar_sfull + 16;          // [2]        score block is in registers
  const uint32_t bar_qfull = bar_sempty + 16;          //            query block landed
  const uint32_t bar_qfree = bar_qfull + 8;            //            every MMA that reads the query block has completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + 16 * kStages + 56);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 16 * kStages + 64);
  const uint32_t bar_mgfull = bar0 + 16 * kStages + 72;  // second statistics group has published its partial sums
  const uint32_t bar_mgfree = bar_mgfull + 8;            // first group has read them
  float* merge_buf = reinterpret_cast<float*>(bar_mem + kBarBytes);
  static_assert(16 * kStages + 88 <= kBarBytes, "barrier area too small");

  const lt_shape& s = a.s;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int T = a.w_last;
  const int M = G * T;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_ctx = a.n_ctx;

  // ---- set-up: barriers, TMEM ----------------------------------------------------
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_sfull + 8 * i, 1);
      mbar_init(bar_sempty + 8 * i, kStatWarps * 32 / 2);  // every statistics thread of the row block
    }
    mbar_init(bar_qfull, 1);
    mbar_init(bar_qfree, 1);
    mbar_init(bar_mgfull, kStatWarps * 32 / 2);
    mbar_init(bar_mgfree, kStatWarps * 32 / 2);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // rows of query block rb that exist, and the UMMA row blocks they fill
  auto rows_of = [&](int rb) { return min(kBlockM, M - rb * kBlockM); };
  auto mbs_of = [&](int rb) { return (rows_of(rb) + 127) / 128; };

  if (warp < 2) {
    if (warp == 0) {
      // ===== producer =====
      // Rows past the piece's last key are real cache rows (or zero past the end of the
      // cache): the statistics warps never look at those columns.  Query rows past the unit's last
      // row are the next head's rows (or zero past the end of q_tail): their scores are never read.
      if (lane == 0) {
        bool ok = true;
        long long cursor = 0;
        int kt = 0;        // tiles issued by this CTA so far: stage kt % kStages, use kt / kStages of that stage
        int q_loads = 0;   // query blocks loaded so far
        int prev_unit = -1;
        Piece p;
        while (ok && next_piece(a, cursor, p)) {
          if (p.n_tiles == 0) continue;
          if (p.unit != prev_unit) {
            // the MMAs of the previous unit must be done with the query block before it is replaced
            if (q_loads > 0) ok = mbar_wait(bar_qfree, (q_loads - 1) & 1, abort_flag);
            if (!ok) break;
            mbar_expect_tx(bar_qfull, kQBytes);
            const int yq = ((p.l * s.batch + p.b) * s.n_q_heads + p.h * G) * T + p.rb * kBlockM;
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) {
              // 16-bit queries: the two 64-d halves of the rows; 8-bit keys: the rows of the two E4M3 terms of q
              if constexpr (K8) tma_load_2d(sQ + hf * kQHalfBytes, &maps.q, 0, hf * a.q8_rows + yq, bar_qfull);
              else tma_load_2d(sQ + hf * kQHalfBytes, &maps.q, 64 * hf, yq, bar_qfull);
            }
            ++q_loads;
            prev_unit = p.unit;
          }
          const CUtensorMap* map = &maps.m[p.l];
          for (int it = 0; it < p.n_tiles; ++it, ++kt) {
            const int st = kt % kStages;
            if (kt >= kStages) ok = mbar_wait(bar_empty + 8 * st, ((kt / kStages) & 1) ^ 1, abort_flag);
            if (!ok) break;
            const uint32_t dst = sK + st * kStageBytes;
            const uint32_t bar = bar_full + 8 * st;
            mbar_expect_tx(bar, kStageBytes);
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {  // two boxes of 128 keys (a box never straddles a page)
              const int j = p.ts0 + it * kBlockN + rh * 128;
              int y;
              if (s.page_size <= 0) {
                y = (p.b * s.n_kv_heads + p.h) * s.full_capacity + j;
              } else {
                // keys past the end of the cache take the last page: never read by the statistics
                const int pg = min(j / s.page_size, s.pages_per_seq - 1);
                const int page = s.block_table[(long long)p.b * s.pages_per_seq + pg];
                y = (page * s.n_kv_heads + p.h) * s.page_size + j % s.page_size;
              }
#pragma unroll
              for (int hf = 0; hf < kKHalves; ++hf)
                tma_load_2d(dst + hf * kKHalfBytes + rh * (128 * 128), map, 64 * hf, y, bar);
            }
          }
        }
        if (!ok) {
          // gave up: let the copies already issued land before the shared memory goes away
          for (int j = max(0, kt - kStages); j < kt; ++j)
            mbar_wait_quiet(bar_full + 8 * (j % kStages), (j / kStages) & 1);
          if (q_loads > 0) mbar_wait_quiet(bar_qfull, (q_loads - 1) & 1);
        }
      }
      __syncwarp();
    } else if (warp == 1) {
      // ===== MMA issuer =====
      if (lane == 0) {
        bool ok = true;
        long long cursor = 0;
        int kt = 0;            // tiles consumed so far
        int uses0 = 0, uses1 = 0;  // score blocks issued so far into each row block's accumulator
        int q_loads = 0;
        int prev_unit = -1;
        Piece p;
        while (ok && next_piece(a, cursor, p)) {
          if (p.n_tiles == 0) continue;
          const int n_mb = mbs_of(p.rb);
          if (p.unit != prev_unit) {
            if (q_loads > 0) umma_commit(bar_qfree);  // arrives once every MMA issued so far has completed
            ok = mbar_wait(bar_qfull, q_loads & 1, abort_flag);
            if (!ok) break;
            ++q_loads;
            prev_unit = p.unit;
          }
          for (int it = 0; it < p.n_tiles && ok; ++it, ++kt) {
            const int st = kt % kStages;
            ok = mbar_wait(bar_full + 8 * st, (kt / kStages) & 1, abort_flag);
            if (!ok) break;
            // A unit with two row blocks fills both accumulators with every tile.  A unit with one (at most 128
            // query rows) alternates: tile `it` goes to accumulator it & 1, so that the MMAs of one tile run
            // while the statistics of the tile before it are taken, by the other group of statistics warps.
            for (int j = 0; j < n_mb; ++j) {
              const int acc = n_mb == 1 ? (it & 1) : j;  // accumulator (and statistics group)
              int& uses = acc ? uses1 : uses0;
              if (uses > 0) {
                ok = mbar_wait(bar_sempty + 8 * acc, (uses - 1) & 1, abort_flag);
                if (!ok) break;
              }
              ++uses;
              tc_fence_after();
              const uint32_t d_tmem = tmem_base + acc * 256;
#pragma unroll
              for (int ks = 0; ks < kKSteps; ++ks) {
                const uint32_t a_addr = sQ + (ks >> 2) * kQHalfBytes + j * (128 * 128) + (ks & 3) * 32;
                if constexpr (K8) {
                  // term ks >> 2 of q against the tile's 32 bytes ks & 3: both terms add into the same scores
                  const uint32_t b_addr = sK + st * kStageBytes + (ks & 3) * 32;
                  umma_e4m3_ss(d_tmem, umma_desc(a_addr), umma_desc(b_addr), ks > 0 ? 1u : 0u);
                } else {
                  const uint32_t b_addr = sK + st * kStageBytes + (ks >> 2) * kKHalfBytes + (ks & 3) * 32;
                  umma_bf16_ss(d_tmem, umma_desc(a_addr), umma_desc(b_addr), ks > 0 ? 1u : 0u);
                }
              }
              umma_commit(bar_sfull + 8 * acc);
            }
            if (!ok) break;
            umma_commit(bar_empty + 8 * st);
          }
        }
      }
      __syncwarp();
    }
  } else {
    // ===== statistics =====
    // Four consecutive warps cover the four TMEM lane quadrants (a warp may access lanes 32 * (warp % 4) ...).
    const int sw = warp - 2;
    const int quad = warp & 3;       // TMEM lane quadrant this warp may access
    const int mb = (sw >> 2) & 1;    // statistics group = accumulator of this warp
    const int ch = sw >> 3;          // half of the tile's 256 keys that this warp reads
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + mb * 256 + ch * 128;
    const int S = s.n_sink;

    bool ok = true;
    long long cursor = 0;
    int uses = 0;    // score blocks of this accumulator consumed so far
    int merges = 0;  // pieces whose partial sums went from the second group to the first
    Piece p;
    uint32_t va[kChunk];
    while (ok && next_piece(a, cursor, p)) {
      const int rows_here = rows_of(p.rb);
      const int n_mb = (rows_here + 127) / 128;
      // one row block: both groups serve it, tile `it` belongs to group it & 1, and the second group hands
      // its sums to the first at the end of the piece
      const bool alt = n_mb == 1;
      const bool active = alt || mb < n_mb;
      const int rblk = alt ? 0 : mb;  // row block of the unit that this warp's rows are in
      const int r_local = rblk * 128 + quad * 32 + lane;
      const int r = p.rb * kBlockM + r_local;   // row of the kv head's G * T query rows
      const bool row_valid = r_local < rows_here;
      const int g = r / T, tq = r - g * T;
      const long long rowid =
          (((long long)(p.l - a.layer_begin) * s.batch + p.b) * s.n_q_heads + p.h * G + g) * T + tq;
      float* stp = a.stats + (rowid * a.n_splits + 2 * p.slot + ch) * 3;
      float cs = a.cs;
      if constexpr (K8) {
        // scores come out in units of (row's q scale) x (layer's K scale)
        const long long qrow = (((long long)p.l * s.batch + p.b) * s.n_q_heads + p.h * G + g) * T + tq;
        cs = a.cs * s.kv_scales[2 * p.l] * (row_valid ? a.q8_scale[qrow] : 1.f);
      }
      if (!active || p.n_tiles == 0) {
        // nothing to read: an idle row block, or an empty key range (its slots still get neutral statistics)
        if (active && row_valid && (!alt || mb == 0)) {
          stp[0] = -INFINITY;
          stp[1] = 0.f;
          stp[2] = 0.f;
        }
        continue;
      }
      const int k0 = p.k0, k1 = p.k1;
      const int vis = n_ctx - T + tq;  // last visible key of this row
      const int win_lo = s.recent_per_row ? vis - s.n_recent + 1 : n_ctx - s.n_recent;  // first recent key of this row
      const int lim = min(vis, k1 - 1);     // last key of this piece that the row may see
      float Mr = -INFINITY, sA = 0.f, sWn = 0.f;  // reference exponent (an integer), sum, windowed sum

      // statistics of one chunk whose 32 keys all count, inside the window (in_win) or all outside it
      auto plain_stats = [&](uint32_t (&v)[kChunk], bool in_win) {
        const float Mn = fmaxf(Mr, ceilf(max32(v) * cs));
        const float corr = ex2(Mr - Mn);
        const float ps = sum_ex2_32_mixed(v, cs, Mn);
        sA = fmaf(sA, corr, ps);
        sWn = fmaf(sWn, corr, in_win ? ps : 0.f);
        Mr = Mn;
      };
      // statistics of one chunk (32 keys from jb) already in registers
      auto chunk_stats = [&](uint32_t (&v)[kChunk], int jb) {
        const int jend = jb + kChunk;
        const bool all_win = (jend <= S) || (jb >= win_lo);
        const bool no_win = (jb >= S) && (jend <= win_lo);
        if ((jb >= k0) && (jend - 1 <= lim) && (all_win || no_win)) {
          plain_stats(v, all_win);
        } else if (max(jb, k0) <= min(jend - 1, lim)) {
          // boundary chunk (piece start, causal tail, piece end or window edge): mask in place.
          // 2^(-inf) = 0, and at least one key is visible, so the maximum is finite.
#pragma unroll
          for (int i = 0; i < kChunk; ++i)
            if (jb + i > lim || jb + i < k0) v[i] = 0xff800000u;
          const float Mn = fmaxf(Mr, ceilf(max32(v) * cs));
          const float corr = ex2(Mr - Mn);
          const float ps = sum_ex2_32(v, cs, -Mn);
#pragma unroll
          for (int i = 0; i < kChunk; ++i) {
            const int j = jb + i;
            if (!(j < S || j >= win_lo)) v[i] = 0xff800000u;
          }
          const float pw = sum_ex2_32(v, cs, -Mn);
          sA = fmaf(sA, corr, ps);
          sWn = fmaf(sWn, corr, pw);
          Mr = Mn;
        }
      };

      for (int it = 0; it < p.n_tiles; ++it) {
        if (alt && (it & 1) != mb) continue;  // the other group's tile
        const int kb = p.ts0 + it * kBlockN + ch * 128;  // first key of this thread's 128 columns
        ok = mbar_wait(bar_sfull + 8 * mb, uses & 1, abort_flag);
        if (!ok) break;
        ++uses;
        tc_fence_after();
        if (rblk * 128 + quad * 32 >= rows_here) {
          // none of this warp's 32 rows exists (a ragged query block): nothing to read, hand the accumulator back
          tc_fence_before();
          mbar_arrive(bar_sempty + 8 * mb);
          continue;
        }
        // Four chunks of 32 columns through one register buffer: the load of a chunk is not overlapped
        // by this warp's own arithmetic but by the three other statistics warps of its scheduler (two
        // buffers would not fit the 96 registers a thread gets).
        // Most tiles lie inside the piece, before every row's last visible key and on one side of the window's
        // edges for all 32 rows of the warp: their chunks need no per-chunk tests.
        const int kend = kb + 128;
        const bool span_in = (kend <= S) || (kb >= win_lo);
        const bool span_out = (kb >= S) && (kend <= win_lo);
        const bool plain = __all_sync(0xffffffffu, (kb >= k0) && (kend - 1 <= lim) && (span_in || span_out));
        if (plain) {
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            tmem_ld32(lane_addr + c * kChunk, va);
            tmem_ld_wait();
            if (c == 3) {
              tc_fence_before();
              mbar_arrive(bar_sempty + 8 * mb);
            }
            plain_stats(va, span_in);
          }
        } else {
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            tmem_ld32(lane_addr + c * kChunk, va);
            tmem_ld_wait();
            if (c == 3) {
              // the row's last chunk is in registers: the accumulator may be overwritten
              tc_fence_before();
              mbar_arrive(bar_sempty + 8 * mb);
            }
            chunk_stats(va, kb + c * kChunk);
          }
        }
      }
      if (!ok) break;
      if (alt) {
        // every thread of both groups takes part (also those whose rows do not exist): the barriers count threads
        float* mg = merge_buf + ((ch * 128 + quad * 32 + lane) * 3);
        if (mb == 1) {
          if (merges > 0) ok = mbar_wait(bar_mgfree, (merges - 1) & 1, abort_flag);  // the last piece's values were read
          if (!ok) break;
          mg[0] = Mr;
          mg[1] = sA;
          mg[2] = sWn;
          mbar_arrive(bar_mgfull);
          ++merges;
          continue;  // the first group writes the piece's statistics
        }
        ok = mbar_wait(bar_mgfull, merges & 1, abort_flag);
        if (!ok) break;
        const float M1 = mg[0], sA1 = mg[1], sW1 = mg[2];
        mbar_arrive(bar_mgfree);
        ++merges;
        const float Mn = fmaxf(Mr, M1);
        if (Mn > -INFINITY) {
          const float c0 = ex2(Mr - Mn), c1 = ex2(M1 - Mn);  // 2^(-inf) = 0 for a side that saw no key
          sA = sA * c0 + sA1 * c1;
          sWn = sWn * c0 + sW1 * c1;
          Mr = Mn;
        }
      }
      if (row_valid) {
        stp[0] = Mr;
        stp[1] = sA;
        stp[2] = sWn;
      }
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
  return s.dtype == LT_BF16 && (s.head_dim == 128 || s.head_dim == 64) &&
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

// 8-bit keys: the tail queries as two E4M3 terms.  A warp per query row of 128 values: the row's scale is the power
// of two that puts its largest magnitude into [128, 256) (inside E4M3's range of 448), hi = E4M3 nearest to
// q / scale, lo = E4M3 nearest to q / scale - hi.  A bf16 value has eight significant bits and each term four, so
// hi + lo is exact unless the value is more than 2^10 below the row's largest, where what is dropped is below
// 2^-17 of that largest value.
__global__ void q_split_kernel(const __nv_bfloat16* __restrict__ q_tail, long long row_begin, long long row_end,
                               long long rows_total, uint8_t* __restrict__ q8, float* __restrict__ q8_scale) {
  const long long row = row_begin + (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= row_end) return;  // whole warps leave together
  const int lane = threadIdx.x & 31;
  const uint2 raw = *reinterpret_cast<const uint2*>(q_tail + row * 128 + lane * 4);
  float x[4] = {__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u), __uint_as_float(raw.y << 16),
                __uint_as_float(raw.y & 0xffff0000u)};
  float amax = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  const int e2 = (amax > 0.f && amax < INFINITY) ? ilogbf(amax) - 7 : 0;
  const float scale = exp2f((float)e2), inv = exp2f((float)-e2);
  uint32_t hi = 0, lo = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float y = x[i] * inv;  // exact: a power of two
    const __nv_fp8_storage_t h = __nv_cvt_float_to_fp8(y, __NV_SATFINITE, __NV_E4M3);
    const float hf = __half2float(__half(__nv_cvt_fp8_to_halfraw(h, __NV_E4M3)));
    const __nv_fp8_storage_t l = __nv_cvt_float_to_fp8(y - hf, __NV_SATFINITE, __NV_E4M3);
    hi |= (uint32_t)h << (8 * i);
    lo |= (uint32_t)l << (8 * i);
  }
  *reinterpret_cast<uint32_t*>(q8 + row * 128 + lane * 4) = hi;
  *reinterpret_cast<uint32_t*>(q8 + (rows_total + row) * 128 + lane * 4) = lo;
  if (lane == 0) q8_scale[row] = scale;
}

// grid = a.grid CTAs (fixed with the plan, so that the merge kernel finds the pieces of a unit); block 576.
template <int DH, bool K8>
static cudaError_t launch_scores_umma_dh(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st) {
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return cudaErrorNotSupported;
  constexpr int kElem = K8 ? 1 : 2;  // bytes of a cached key element
  const CUtensorMapDataType dt = K8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  const cuuint64_t rows_total = a.s.page_size > 0 ? (cuuint64_t)a.s.n_pages * a.s.n_kv_heads * a.s.page_size
                                                  : (cuuint64_t)a.s.batch * a.s.n_kv_heads * a.s.full_capacity;
  const cuuint64_t gdim[2] = {(cuuint64_t)DH, rows_total};
  const cuuint64_t gstride[1] = {(cuuint64_t)(kElem * DH)};
  const cuuint32_t box[2] = {K8 ? 128u : 64u, 128u};  // 128 bytes x 128 keys either way
  const cuuint32_t estride[2] = {1u, 1u};
  KeyMaps local;
  const cuuint64_t q_rows = (cuuint64_t)a.s.n_layers * a.s.batch * a.s.n_q_heads * (cuuint64_t)a.w_last;
  if (K8) {
    // this call's layers of q_tail as two E4M3 terms, then one matrix of 2 x q_rows rows of 128 bytes over them
    const long long per_layer = (long long)a.s.batch * a.s.n_q_heads * a.w_last;
    const long long r0 = a.layer_begin * per_layer, r1 = r0 + a.layer_count * per_layer;
    q_split_kernel<<<(unsigned)((r1 - r0 + 7) / 8), 256, 0, st>>>((const __nv_bfloat16*)a.q_tail, r0, r1,
                                                                    (long long)q_rows, a.q8, a.q8_scale);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const cuuint64_t qdim[2] = {128u, 2 * q_rows};
    const cuuint32_t qbox[2] = {128u, (cuuint32_t)kBlockM};
    const CUresult r = encode(&local.q, dt, 2, a.q8, qdim, gstride, qbox, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  } else {
    // the tail queries of the whole stack as one matrix of head_dim-element rows; a box is 64 d of a unit's 256 rows
    const cuuint64_t qdim[2] = {(cuuint64_t)DH, q_rows};
    const cuuint32_t qbox[2] = {64u, (cuuint32_t)kBlockM};
    const CUresult r = encode(&local.q, dt, 2, const_cast<void*>(a.q_tail), qdim, gstride, qbox, estride,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  const int l_end = a.layer_begin + a.layer_count;
  for (int l = a.layer_begin; l < l_end; ++l) {
    const CUresult r = encode(&local.m[l], dt, 2, const_cast<void*>(kf.p[l]), gdim, gstride, box, estride,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  for (int l = 0; l < LT_MAX_LAYERS; ++l)
    if (l < a.layer_begin || l >= l_end) local.m[l] = local.m[a.layer_begin];
  constexpr int smem = Geo<DH, K8>::kSmemBytes;
  cudaError_t e = cudaFuncSetAttribute(scores_umma_kernel<DH, K8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  scores_umma_kernel<DH, K8><<<a.grid, kThreads, smem, st>>>(a, local);
  return cudaGetLastError();
}

cudaError_t launch_scores_umma(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st) {
  if (a.s.kv_fp8) return launch_scores_umma_dh<128, true>(a, kf, st);
  return a.s.head_dim == 64 ? launch_scores_umma_dh<64, false>(a, kf, st) : launch_scores_umma_dh<128, false>(a, kf, st);
}

}  // namespace lt
