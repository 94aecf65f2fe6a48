// Decode step, bandwidth path: bf16 activations, head_dim 128 or 64, GQA group <= 32 (groups above 8 by
// warps that share a tile ring and serve eight heads each: template parameter ROLES);
// caches in bf16 or (template branch FP8, head_dim 128) in E4M3 bytes.
//
// A persistent launch (two CTAs per SM) walks the flattened work list of
// (layer, batch row, kv head, KV chunk) items; items are handed out through a
// device counter so that faster SMs take more of them.  One item serves every
// query head of the group, so each cached K and V byte is read from HBM exactly
// once per step.
//
// Each warp streams its own 16-key tiles of the chunk through a private
// multi-stage cp.async ring in shared memory (16-byte vectors, fully coalesced
// rows, XOR swizzle of the 16-byte column so that ldmatrix is conflict-free).
// The ring never drains between items: while a warp finishes the tiles of one
// item its look-ahead already fetches the first tiles of the CTA's next item,
// so the merge of the four warps, the hand-off of the partials and the merge of
// a finished (layer, b, kv head) all happen with loads in flight.
//
// Fused append: the item that owns the new token's row takes that row from
// k_new / v_new and stores it into the cache.  The last item of a (layer, batch
// row, kv head) to finish merges the chunk partials and writes the output, so a
// whole decode step is one launch.
//
// Tensor-core mapping (mma.sync m16n8k16, bf16 in, fp32 accumulate):
//   S^T[key][head]  = K[key][d] . Q^T[d][head]      keys are M (16), heads are N (8)
//   O^T[d][head]   += V^T[d][key] . P[key][head]    d is M (8 tiles), keys are K
// K is the A operand through ldmatrix, V^T through ldmatrix.trans, Q sits in
// registers for the whole chunk, and P moves from the accumulator layout to the
// B layout with one movmatrix per 8x8 block.  P is split into a bf16 head and a
// bf16 residual (two MMAs) so that the probabilities keep ~16 bits.
#include <cuda_bf16.h>

#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <mutex>

#include "lt_decode_common.cuh"
#include "lt_internal.h"

namespace lt {

namespace {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Two 16 x 16 byte matrices, transposed: lane i gives the address of the 16 bytes of matrix row i (rows 0-15:
// first matrix, 16-31: second).  Thread (g = lane / 4, c = lane % 4) receives, four bytes per register,
// r0 = rows 4c .. 4c+3 of byte column g, r1 = the same rows of column g + 8, r2 / r3 = rows 16 + 4c .. of
// columns g / g + 8.  With rows = keys and columns = d, a register is V^T[d][four keys]: its two halves
// convert to the f16 pairs of an m16n8k16 A fragment (r0, r1: first 16 keys; r2, r3: second 16).
__device__ __forceinline__ void ldmatrix_b8_x2_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m16n16.x2.trans.shared.b8 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// The two low / two high E4M3 bytes of a word -> two f16 (exact: every E4M3 value is an f16 value).
__device__ __forceinline__ uint32_t e4m3_lo2_to_f16x2(uint32_t w) {
  uint32_t d;
  asm("{\n.reg .b16 lo, hi;\nmov.b32 {lo, hi}, %1;\ncvt.rn.f16x2.e4m3x2 %0, lo;\n}\n" : "=r"(d) : "r"(w));
  return d;
}
__device__ __forceinline__ uint32_t e4m3_hi2_to_f16x2(uint32_t w) {
  uint32_t d;
  asm("{\n.reg .b16 lo, hi;\nmov.b32 {lo, hi}, %1;\ncvt.rn.f16x2.e4m3x2 %0, hi;\n}\n" : "=r"(d) : "r"(w));
  return d;
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}
// One MUFU instruction: 2^x, relative error 2^-22, 2^(-inf) = 0, results below 2^-126 flush to zero.
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
// lower 16 bits <- lo, upper <- hi
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void st_shared_u32x4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}


}  // namespace

// What a warp needs to fetch tiles of one item.
struct TileSrc {
  const uint8_t* Kb;         // rows of this (b, kv head) in the cache that is read
  const uint8_t* Vb;
  const uint8_t* k_new_row;  // fused append: source of row new_row
  const uint8_t* v_new_row;
  int j0, j1;                // key rows of the chunk
  int new_row;               // -1 when the chunk does not hold the new token
  int my_tiles;              // tiles of this warp's stream (tiles stream, stream + STREAMS, ... of the chunk)
  int tbl_off;               // paged full cache: offset of this batch row's block-table row, else -1
  int layer;                 // for the per-layer scales of 8-bit caches
};

// Shared memory: [rings: WARPS x NSTAGE x stage][merge: two 8 x 128 fp32 buffers,
// (max, sum) of every warp][work list].  A stage holds K half-tiles
// [2][TILE][128 B] then V half-tiles [2][TILE][128 B]; inside a half-tile the
// 16-byte column c of row r sits at column c ^ (r & 7).
//
// FP8 = true: the caches hold E4M3 bytes (rows of 128 B) with one scale per layer
// for K and one for V.  A ring stage then holds the raw bytes of a 32-key tile (K rows,
// then V rows); the MMA fragments are made from the bytes in registers, as f16, with one
// conversion instruction per byte pair (this GPU's warp-level MMAs take no 8-bit floats:
// the compiler expands them into the same conversions plus f16 MMAs, less well):
//   K: ldmatrix on the bytes hands thread (g, c) the four bytes d = 4c .. 4c+3 of
//      row g - the halves of that register are the f16 pairs of an A fragment for a d
//      order that Q's fragments simply follow;
//   V: the byte-transposing ldmatrix (16 x 16 bytes, two per instruction) hands it
//      V^T[d][four keys], again two f16 pairs of an A fragment (16 d x 16 keys); lane i
//      addresses the key that byte i stands for, chosen as the order in which movmatrix
//      delivers P.
// Q and P are f16 as well (P = 256 * 2^(t - M) as one f16 term: its 11 bits are far finer
// than E4M3's 4; O and the row sums both carry the factor 256, their ratio none).  The K
// scale is folded into the softmax scale and the V scale into the final normalisation.
// 16-byte column c of K row r sits at column c ^ (r & 7), of V row r at
// c ^ (r & 7) ^ (4 * ((r >> 3) & 1)): the eight rows of either ldmatrix phase fall into eight different bank groups.
//
// ROLES = 2 (query groups of 9..16 heads): the four warps work as two pairs.  The warps of a pair walk the same
// tiles through one shared ring (each copies half of every tile, a 64-thread named barrier per tile makes the
// copies visible and frees the stage that is refilled), warp 0 of the pair serves heads 0-7 of the group and warp
// 1 heads 8-15, so the chunk still crosses HBM, L2 and shared memory once.
// ROLES = 4 (groups of 17..32 heads): all four warps walk one ring of twice the depth (a quarter of
// every tile each, one 128-thread named barrier per tile); warp w serves heads 8w .. 8w + 7 - a warp beyond the
// group's last head computes on zeros and stores nothing - and no sums cross warps.
template <int TILE, int NSTAGE, int WARPS, int MINB, bool FP8, int DH, int ROLES>
__global__ void __launch_bounds__(WARPS * 32, MINB)
    decode_mma_kernel(DecodeArgs a, LayerTable kf, LayerTable vf, LayerTable ks, LayerTable vs) {
  static_assert(WARPS == 4, "the merge tree below is written for four warps");
  static_assert(DH == 128 || (DH == 64 && !FP8), "head_dim 128, or 64 with 16-bit caches");
  static_assert(ROLES == 1 || ROLES == 2 || ROLES == 4, "one, two or four warps per tile stream");
  constexpr bool PAIR = ROLES > 1;                    // several warps share a ring, eight heads of the group each
  constexpr int STREAMS = WARPS / ROLES;              // independent tile streams of the CTA
  constexpr int RSTAGES = NSTAGE;                     // ring stages of a stream
  constexpr int kD = DH;                       // head_dim
  constexpr int kSrcRowBytes = kD * 2;         // one row of q, k_new, v_new (bf16)
  constexpr int NK = kD / 16;                  // 16-wide k-steps of S = K Q^T = 16-row tiles of O^T
  constexpr int HALVES = kD / 64;              // 128-byte halves of a 16-bit row
  constexpr int VPR = kD / 8;                  // 16-byte vectors of a 16-bit row
  constexpr int MT = TILE / 16;                // 16-key MMA tiles per pipeline tile
  constexpr int HALF_BYTES = TILE * 128;       // one half-tile
  constexpr int STAGE_BYTES = 2 * HALVES * HALF_BYTES;  // K halves + V halves (16-bit layout)
  constexpr int kRowBytes = FP8 ? kD : 2 * kD;             // one cached K or V row
  constexpr int RAW_BYTES = 2 * TILE * kD;                 // FP8: K rows + V rows of a tile as stored
  constexpr int RING_STAGE = FP8 ? RAW_BYTES : STAGE_BYTES;  // what one ring stage holds
  constexpr int STREAM_BYTES = RSTAGES * RING_STAGE;
  constexpr int RING_BYTES = STREAMS * STREAM_BYTES;
  constexpr int MERGE_BYTES = 2 * 8 * kD * 4 + 2 * WARPS * 8 * 4;
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ int s_flag, s_next;

  const lt_shape& s = a.s;
  const int G = s.n_q_heads / s.n_kv_heads;
  float* sm_buf = reinterpret_cast<float*>(smem + RING_BYTES);  // [2][8][head_dim]
  float* sm_m = sm_buf + 2 * 8 * kD;                            // [WARPS][8]
  float* sm_l = sm_m + WARPS * 8;                               // [WARPS][8]
  // the previous launch of the stream is complete: lengths, counters and partial slots are ours (an overlapped
  // launch has its own and starts at once)
  if (!a.overlap) pdl_wait_prior_grid();
  WorkList wl;
  wl.carve(smem + RING_BYTES + MERGE_BYTES, a.layer_count, s.batch);
  wl.build(a, kf, vf, ks, vs);
  pdl_allow_next_grid();   // seq_lens has been read: the next launch may take SMs as this one's CTAs retire
  const int n_items = wl.total(a);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gp = lane >> 2, c = lane & 3;  // fragment row / column-pair index
  const int stream = warp / ROLES;  // tile stream of this warp
  const int role = warp % ROLES;    // which eight heads of the group this warp serves
  const uint32_t wsm = smem_u32(smem) + stream * STREAM_BYTES;
  auto stream_sync = [&]() {  // the threads that share a ring: the warp, or the 64 threads of a pair
    if constexpr (ROLES == 4) {
      asm volatile("bar.sync 1, 128;\n" ::: "memory");
    } else if constexpr (ROLES == 2) {
      if (stream == 0) asm volatile("bar.sync 1, 64;\n" ::: "memory");
      else asm volatile("bar.sync 2, 64;\n" ::: "memory");
    } else {
      __syncwarp();
    }
  };
  // lane-constant parts of the ldmatrix addresses
  const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8;  // K (A operand, not transposed)
  const int k_chk = lane >> 4;
  const int v_row = (lane & 7) + ((lane >> 4) & 1) * 8;  // V (A operand, transposed)
  const int v_chk = (lane >> 3) & 1;
  // 8-bit V: lane i addresses the key that byte i of the transposed 16-key block stands for (bytes 4c, 4c + 1
  // are keys 2c, 2c + 1 and bytes 4c + 2, 4c + 3 keys 2c + 8, 2c + 9: the order in which movmatrix delivers P)
  const int v8_key = 16 * (lane >> 4) + 2 * ((lane & 15) >> 2) + (lane & 1) + 8 * ((lane >> 1) & 1);
  const int v8_swz = (v8_key & 7) ^ ((v8_key >> 1) & 4);

  // d index of accumulator element (tile idx, row half) of this thread
  auto dmap = [&](int idx, int half) {
    return idx * 16 + gp + 8 * half;
  };
  auto make_src = [&](const WorkItem& w) {
    TileSrc t;
    // contiguous: base of this (b, kv head); paged: base of kv head h inside page 0 of the layer's pool
    const bool paged = !w.lazy && s.page_size > 0;
    const long long base_row = paged ? (long long)w.h * s.page_size
                                     : ((long long)w.b * s.n_kv_heads + w.h) * w.rows;
    t.Kb = (const uint8_t*)(w.lazy ? ks.p[w.l] : kf.p[w.l]) + base_row * kRowBytes;
    t.Vb = (const uint8_t*)(w.lazy ? vs.p[w.l] : vf.p[w.l]) + base_row * kRowBytes;
    t.tbl_off = paged ? w.b * s.pages_per_seq : -1;
    t.layer = w.l;
    t.j0 = w.j0;
    t.j1 = w.j1;
    t.new_row = w.new_row;
    t.k_new_row = nullptr;
    t.v_new_row = nullptr;
    if (w.new_row >= 0) {
      const long long src = (((long long)w.l * s.batch + w.b) * s.n_kv_heads + w.h) * kSrcRowBytes;
      t.k_new_row = (const uint8_t*)a.k_new + src;
      t.v_new_row = (const uint8_t*)a.v_new + src;
    }
    const int n_tiles = (w.j1 - w.j0 + TILE - 1) / TILE;
    t.my_tiles = (n_tiles > stream) ? (n_tiles - stream + STREAMS - 1) / STREAMS : 0;
    return t;
  };
  // copy this warp's idx-th tile of `t` into ring stage `stage` (no commit)
  // row of key `row` relative to t.Kb / t.Vb (a paged chunk starts on a multiple of 32, so a tile has one page)
  auto cache_row = [&](const TileSrc& t, int row) -> long long {
    if (t.tbl_off < 0) return row;
    const int page = s.block_table[t.tbl_off + row / s.page_size];
    return (long long)page * s.n_kv_heads * s.page_size + row % s.page_size;
  };
  // 16 bf16 values of a new row -> 16 E4M3 bytes with the layer's scale (same rounding as lt_kv_append)
  auto quantize16 = [&](const uint8_t* src32, float scale, uint32_t (&out)[4]) {
    const uint4 lo = *reinterpret_cast<const uint4*>(src32), hi = *reinterpret_cast<const uint4*>(src32 + 16);
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t packed = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t pair = w[2 * i + (e >> 1)];
        const float x = (e & 1) ? bf16_hi(pair) : bf16_lo(pair);
        packed |= (uint32_t)__nv_cvt_float_to_fp8(__fdiv_rn(x, scale), __NV_SATFINITE, __NV_E4M3) << (8 * e);
      }
      out[i] = packed;
    }
  };
  // Lane-constant parts of a tile copy.  One pass of the warp covers RPI rows; this lane's first row is f_row,
  // its later rows f_row + dr with dr a multiple of RPI, so that (row & 7) = (f_row & 7) ^ (dr & 7): the swizzled
  // offset of every pass is the first one xor a constant.
  constexpr int VPRX = FP8 ? 8 : VPR;             // 16-byte vectors of a cached row
  constexpr int RPI = 32 / VPRX;
  constexpr int FROWS = TILE / ROLES;             // rows of a tile this warp copies (the warps of a ring share them out)
  const int f_row = role * FROWS + lane / VPRX;
  const int f_p = lane % VPRX;
  const uint32_t f_goff = f_row * kRowBytes + f_p * 16;
  const uint32_t f_soff = FP8 ? f_row * kD + ((f_p ^ (f_row & 7)) << 4)
                              : (f_p >> 3) * HALF_BYTES + f_row * 128 + (((f_p & 7) ^ (f_row & 7)) << 4);
  const uint32_t f_soff_v = FP8 ? TILE * kD + f_row * kD + ((f_p ^ (f_row & 7) ^ ((f_row >> 1) & 4)) << 4)
                                : HALVES * HALF_BYTES + f_soff;
  auto fetch_tile = [&](const TileSrc& t, int idx, int stage) {
    const int key_base = t.j0 + (stream + idx * STREAMS) * TILE;
    const long long tile_row = cache_row(t, key_base);
    const uint32_t st = wsm + stage * RING_STAGE;
    if (key_base + TILE <= t.j1 && (t.new_row < key_base || t.new_row >= key_base + TILE)) {
      // every row of the tile is a cached row (the usual case): addresses are a base plus constants
      const uint8_t* kp = t.Kb + tile_row * kRowBytes + f_goff;
      const uint8_t* vp = t.Vb + tile_row * kRowBytes + f_goff;
#pragma unroll
      for (int i = 0; i < FROWS / RPI; ++i) {
        constexpr int kSRow = FP8 ? kD : 128;  // bytes between rows in a stage
        const int dr = RPI * i;
        const uint32_t x = (uint32_t)(dr & 7) << 4;
        const uint32_t xv = FP8 ? (uint32_t)((dr & 7) ^ ((dr >> 1) & 4)) << 4 : x;
        cp_async16(st + ((f_soff ^ x) + dr * kSRow), kp + (long long)dr * kRowBytes, 16);
        cp_async16(st + ((f_soff_v ^ xv) + dr * kSRow), vp + (long long)dr * kRowBytes, 16);
      }
    } else if constexpr (FP8) {
      // raw rows: 8 chunks of 16 bytes per row, K rows then V rows
#pragma unroll
      for (int i = 0; i < FROWS / 4; ++i) {
        const int r = role * FROWS + 4 * i + (lane >> 3), p = lane & 7;
        const int row = key_base + r;
        const bool valid = row < t.j1;
        const long long goff = (tile_row + (valid ? r : 0)) * kRowBytes + p * 16;
        const uint32_t soff = r * kD + ((p ^ (r & 7)) << 4);
        const uint32_t soff_v = TILE * kD + r * kD + ((p ^ (r & 7) ^ ((r >> 1) & 4)) << 4);
        if (row == t.new_row) {
          // the new token's row is quantised on the fly from k_new / v_new
          uint32_t q4[4];
          quantize16(t.k_new_row + p * 32, a.s.kv_scales[2 * t.layer], q4);
          st_shared_u32x4(st + soff, q4[0], q4[1], q4[2], q4[3]);
          quantize16(t.v_new_row + p * 32, a.s.kv_scales[2 * t.layer + 1], q4);
          st_shared_u32x4(st + soff_v, q4[0], q4[1], q4[2], q4[3]);
        } else {
          cp_async16(st + soff, t.Kb + goff, valid ? 16 : 0);
          cp_async16(st + soff_v, t.Vb + goff, valid ? 16 : 0);
        }
      }
    } else {
      constexpr int ROWS = TILE / ROLES;  // the warps of a ring copy an equal share of the tile each
#pragma unroll
      for (int i = 0; i < ROWS * VPR / 32; ++i) {
        const int r = role * ROWS + (32 / VPR) * i + lane / VPR;
        const int p = lane % VPR;
        const int row = key_base + r;
        const bool valid = row < t.j1;
        const long long goff = (tile_row + (valid ? r : 0)) * kRowBytes + p * 16;
        const uint32_t soff = (p >> 3) * HALF_BYTES + r * 128 + (((p & 7) ^ (r & 7)) << 4);
        const bool fresh = row == t.new_row;
        cp_async16(st + soff, fresh ? t.k_new_row + p * 16 : t.Kb + goff, valid ? 16 : 0);
        cp_async16(st + HALVES * HALF_BYTES + soff, fresh ? t.v_new_row + p * 16 : t.Vb + goff, valid ? 16 : 0);
      }
    }
  };
  // The CTA's first two items are fixed; later ones come from the device counter.
  int cur = blockIdx.x, nxt = blockIdx.x + gridDim.x;
  WorkItem w;
  TileSrc src_cur, src_nxt;
  src_cur.my_tiles = 0;
  src_nxt.my_tiles = 0;
  if (cur < n_items) {
    w = wl.item(a, cur);
    src_cur = make_src(w);
  }
  if (nxt < n_items) src_nxt = make_src(wl.item(a, nxt));

  // Every cp.async group is one "slot" of the warp's tile stream (a tile, or
  // nothing once the stream has run dry); slot k lives in ring stage k % NSTAGE.
  uint32_t issued = 0, consumed = 0;
  int la_in_next = 0;  // look-ahead cursor: 0 = in the current item, 1 = in the next one
  int la_idx = 0;      // tile index of the cursor inside that item
  int skip_after = 0;  // empty slots that follow the current item's tiles
  auto issue_slot = [&]() {
    if (la_in_next == 0 && la_idx >= src_cur.my_tiles) {
      la_in_next = 1;
      la_idx = 0;
    }
    const int stage = issued % RSTAGES;
    if (la_in_next == 0) fetch_tile(src_cur, la_idx, stage);
    else if (la_idx < src_nxt.my_tiles) fetch_tile(src_nxt, la_idx, stage);
    ++la_idx;
    ++issued;
    cp_async_commit();
  };

  while (cur < n_items) {
    const int l = w.l, b = w.b, h = w.h;
    // query heads served by this warp: the group, or this warp's eight of a pair's sixteen
    const int g0 = role * 8;
    const int Gn = PAIR ? max(0, min(8, G - role * 8)) : G;
    const int j1 = src_cur.j1;
    int fetched_next = 0;
    if (threadIdx.x == 0) fetched_next = 2 * gridDim.x + atomicAdd(a.work_counter, 1);

    // per-layer scales of 8-bit caches: K's goes into the softmax scale, V's into the normalisation
    float cs_l = a.cs, v_scale = 1.f;
    if constexpr (FP8) {
      cs_l = a.cs * a.s.kv_scales[2 * l];
      v_scale = a.s.kv_scales[2 * l + 1];
    }

    // fused append: store the new token's row into the cache
    if (src_cur.new_row >= 0 && warp == 0) {
      if constexpr (FP8) {
        if (lane < 16) {
          const bool is_k = lane < 8;
          uint32_t q4[4];
          quantize16((is_k ? src_cur.k_new_row : src_cur.v_new_row) + (lane & 7) * 32,
                     a.s.kv_scales[2 * l + (is_k ? 0 : 1)], q4);
          uint8_t* dp = const_cast<uint8_t*>(is_k ? src_cur.Kb : src_cur.Vb) +
                        cache_row(src_cur, src_cur.new_row) * kRowBytes + (lane & 7) * 16;
          *reinterpret_cast<uint4*>(dp) = make_uint4(q4[0], q4[1], q4[2], q4[3]);
        }
      } else {
        if (lane < 2 * VPR) {
          const uint8_t* sp = (lane < VPR ? src_cur.k_new_row : src_cur.v_new_row) + (lane % VPR) * 16;
          uint8_t* dp = const_cast<uint8_t*>(lane < VPR ? src_cur.Kb : src_cur.Vb) +
                        cache_row(src_cur, src_cur.new_row) * kRowBytes + (lane % VPR) * 16;
          *reinterpret_cast<uint4*>(dp) = *reinterpret_cast<const uint4*>(sp);
        }
      }
    }

    // Q fragments (B operand of S^T = K Q^T): head gp, d = 16*ks + 2c (+8).
    // 8-bit caches: K's bytes reach the MMA as f16 in the d order the byte ldmatrix delivers (k-step ks covers
    // d = 16 ks .. 16 ks + 15, this thread's four are 16 ks + 4c .. 4c+3), and q follows as f16 at one
    // power-of-two scale per head (bf16 -> f16 is exact inside f16's range, which the scale centres).
    uint32_t qf[NK][2];
    float q_scale0 = 1.f, q_scale1 = 1.f;  // scale of heads 2c and 2c + 1 (this thread's S columns)
    {
      const __nv_bfloat16* qp =
          (const __nv_bfloat16*)a.q + (((long long)l * s.batch + b) * s.n_q_heads + h * G + g0 + gp) * kD;
      if constexpr (FP8) {
        float x[NK][4];
        float amax = 0.f;
#pragma unroll
        for (int ks = 0; ks < NK; ++ks) {
          uint2 q4 = make_uint2(0u, 0u);
          if (gp < Gn) q4 = *reinterpret_cast<const uint2*>(qp + 16 * ks + 4 * c);
          x[ks][0] = bf16_lo(q4.x);
          x[ks][1] = bf16_hi(q4.x);
          x[ks][2] = bf16_lo(q4.y);
          x[ks][3] = bf16_hi(q4.y);
#pragma unroll
          for (int e = 0; e < 4; ++e) amax = fmaxf(amax, fabsf(x[ks][e]));
        }
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));  // the four lanes of a head hold its 128 values
        // power-of-two scale that puts the head's largest |q| into [1, 2): products with |K| <= 448 stay far
        // inside f16's range and values down to 2^-14 of the largest keep all their bits
        const int e2 = (amax > 0.f && amax < INFINITY) ? ilogbf(amax) : 0;
        const float inv = exp2f((float)-e2), scale = exp2f((float)e2);
#pragma unroll
        for (int ks = 0; ks < NK; ++ks) {
          qf[ks][0] = pack_f16(x[ks][0] * inv, x[ks][1] * inv);
          qf[ks][1] = pack_f16(x[ks][2] * inv, x[ks][3] * inv);
        }
        q_scale0 = __shfl_sync(0xffffffffu, scale, (2 * c) * 4);
        q_scale1 = __shfl_sync(0xffffffffu, scale, (2 * c + 1) * 4);
      } else {
#pragma unroll
        for (int ks8 = 0; ks8 < NK; ++ks8) {
          if (gp < Gn) {
            qf[ks8][0] = *reinterpret_cast<const uint32_t*>(qp + 16 * ks8 + 2 * c);
            qf[ks8][1] = *reinterpret_cast<const uint32_t*>(qp + 16 * ks8 + 8 + 2 * c);
          } else {
            qf[ks8][0] = 0u;
            qf[ks8][1] = 0u;
          }
        }
      }
    }

    const float cs0 = cs_l * q_scale0, cs1 = cs_l * q_scale1;  // per S column (head 2c, 2c + 1)
    float o[NK][4];
#pragma unroll
    for (int i = 0; i < NK; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) o[i][j] = 0.f;
    float M0 = -INFINITY, M1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // heads 2c and 2c+1

    while (issued - consumed < RSTAGES - 1) issue_slot();
    for (int it = 0; it < src_cur.my_tiles; ++it) {
      if constexpr (PAIR) {
        // one barrier per tile: behind it both warps' copies of this tile have landed and both are done with the
        // previous tile, whose stage the next slot refills
        cp_async_wait<RSTAGES - 2>();
        stream_sync();
        issue_slot();
      } else {
        __syncwarp();              // every lane is done reading the stage that is refilled next
        issue_slot();
        cp_async_wait<NSTAGE - 1>();
        __syncwarp();              // all lanes' copies of this tile have landed
      }
      const uint32_t st = wsm + (consumed % RSTAGES) * RING_STAGE;
      ++consumed;
      const int key_base = src_cur.j0 + (stream + it * STREAMS) * TILE;
      // a warp whose eight heads lie beyond the group (four roles, groups of 17..24) only copies its share of the tiles
      if (ROLES == 4 && Gn == 0) continue;

      // ---- S^T = K Q^T ------------------------------------------------------
      float sc[MT][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        sc[mt][0] = sc[mt][1] = sc[mt][2] = sc[mt][3] = 0.f;
        const int row = mt * 16 + k_row;
        if constexpr (FP8) {
          float sc2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int blk = 0; blk < 4; ++blk) {  // 32 d per ldmatrix: matrices (rows 0-7 | 8-15) x (chunk 2 blk | 2 blk + 1)
            uint32_t m[4];
            const int chunk = 2 * blk + k_chk;
            ldmatrix_x4(m, st + row * kD + ((chunk ^ (row & 7)) << 4));
            // a register holds bytes d = 4c .. 4c+3 of row g (m0, m2) or g + 8 (m1, m3): its halves are the
            // f16 pairs of the A fragment, contraction index 2c + j <-> d 4c + j, 2c + 8 + j <-> d 4c + 2 + j
            const uint32_t a0[4] = {e4m3_lo2_to_f16x2(m[0]), e4m3_lo2_to_f16x2(m[1]), e4m3_hi2_to_f16x2(m[0]),
                                    e4m3_hi2_to_f16x2(m[1])};
            const uint32_t a1[4] = {e4m3_lo2_to_f16x2(m[2]), e4m3_lo2_to_f16x2(m[3]), e4m3_hi2_to_f16x2(m[2]),
                                    e4m3_hi2_to_f16x2(m[3])};
            mma_f16(sc[mt], a0, qf[2 * blk][0], qf[2 * blk][1]);
            mma_f16(sc2, a1, qf[2 * blk + 1][0], qf[2 * blk + 1][1]);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) sc[mt][i] += sc2[i];
        } else {
          // two accumulators (even / odd k-steps): half the length of the dependent MMA chain
          float sc2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int ks8 = 0; ks8 < NK; ++ks8) {
            uint32_t af[4];
            const int chunk = 2 * (ks8 & 3) + k_chk;
            ldmatrix_x4(af, st + (ks8 >> 2) * HALF_BYTES + row * 128 + ((chunk ^ (row & 7)) << 4));
            if (ks8 & 1) mma_bf16(sc2, af, qf[ks8][0], qf[ks8][1]);
            else mma_bf16(sc[mt], af, qf[ks8][0], qf[ks8][1]);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) sc[mt][i] += sc2[i];
        }
      }
      // ---- scale, mask the ragged tail, tile max per head ---------------------
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const int key_lo = key_base + mt * 16 + gp;
        const bool v_lo = key_lo < j1, v_hi = key_lo + 8 < j1;
        sc[mt][0] = v_lo ? sc[mt][0] * cs0 : -INFINITY;
        sc[mt][1] = v_lo ? sc[mt][1] * cs1 : -INFINITY;
        sc[mt][2] = v_hi ? sc[mt][2] * cs0 : -INFINITY;
        sc[mt][3] = v_hi ? sc[mt][3] * cs1 : -INFINITY;
        mx0 = fmaxf(mx0, fmaxf(sc[mt][0], sc[mt][2]));
        mx1 = fmaxf(mx1, fmaxf(sc[mt][1], sc[mt][3]));
      }
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
      }
      const float Mn0 = fmaxf(M0, mx0), Mn1 = fmaxf(M1, mx1);
      const float corr0 = ex2(M0 - Mn0), corr1 = ex2(M1 - Mn1);
      M0 = Mn0;
      M1 = Mn1;
      // once the running maxima have settled the factors are exactly 1 for every lane: skip the rescale then
      if (__any_sync(0xffffffffu, (corr0 != 1.f) | (corr1 != 1.f))) {
        l0 *= corr0;
        l1 *= corr1;
#pragma unroll
        for (int i = 0; i < NK; ++i) {
          o[i][0] *= corr0;
          o[i][1] *= corr1;
          o[i][2] *= corr0;
          o[i][3] *= corr1;
        }
      }
      // ---- P = 2^(t - M), O^T += V^T P ---------------------------------------
      if constexpr (FP8) {
        static_assert(!FP8 || MT == 2, "one byte-transposing ldmatrix spans the 32 keys of a tile");
        const float Ms0 = Mn0 - 8.f, Ms1 = Mn1 - 8.f;  // P (and with it O and the row sums) carries the factor 256:
        uint32_t bh[MT][2];                            // small probabilities stay normal numbers in f16
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const float p0 = ex2(sc[mt][0] - Ms0), p1 = ex2(sc[mt][1] - Ms1);
          const float p2 = ex2(sc[mt][2] - Ms0), p3 = ex2(sc[mt][3] - Ms1);
          l0 += p0 + p2;
          l1 += p1 + p3;
          // thread (g, c) gets head g, keys 2c, 2c + 1 (bh[.][0]) and 2c + 8, 2c + 9 (bh[.][1]) of this 16-key block
          bh[mt][0] = movmatrix_trans(pack_f16(p0, p1));
          bh[mt][1] = movmatrix_trans(pack_f16(p2, p3));
        }
#pragma unroll
        for (int db = 0; db < NK; ++db) {  // 16 d per instruction = one 16-byte column of the V rows
          uint32_t r[4];
          ldmatrix_b8_x2_trans(r, st + TILE * kD + v8_key * kD + ((db ^ v8_swz) << 4));
          const uint32_t a0[4] = {e4m3_lo2_to_f16x2(r[0]), e4m3_lo2_to_f16x2(r[1]), e4m3_hi2_to_f16x2(r[0]),
                                  e4m3_hi2_to_f16x2(r[1])};
          const uint32_t a1[4] = {e4m3_lo2_to_f16x2(r[2]), e4m3_lo2_to_f16x2(r[3]), e4m3_hi2_to_f16x2(r[2]),
                                  e4m3_hi2_to_f16x2(r[3])};
          mma_f16(o[db], a0, bh[0][0], bh[0][1]);
          mma_f16(o[db], a1, bh[1][0], bh[1][1]);
        }
      } else {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const float p0 = ex2(sc[mt][0] - Mn0), p1 = ex2(sc[mt][1] - Mn1);
          const float p2 = ex2(sc[mt][2] - Mn0), p3 = ex2(sc[mt][3] - Mn1);
          l0 += p0 + p2;
          l1 += p1 + p3;
          // P for the B operand: a bf16 head and a bf16 residual
          const uint32_t hi01 = pack_bf16(p0, p1);
          const uint32_t hi23 = pack_bf16(p2, p3);
          const uint32_t bh0 = movmatrix_trans(hi01), bh1 = movmatrix_trans(hi23);
          const uint32_t bl0 = movmatrix_trans(pack_bf16(p0 - bf16_lo(hi01), p1 - bf16_hi(hi01)));
          const uint32_t bl1 = movmatrix_trans(pack_bf16(p2 - bf16_lo(hi23), p3 - bf16_hi(hi23)));
          const int row = mt * 16 + v_row;
#pragma unroll
          for (int dt = 0; dt < NK; ++dt) {
            uint32_t af[4];
            const int chunk = 2 * (dt & 3) + v_chk;
            ldmatrix_x4_trans(af, st + HALVES * HALF_BYTES + (dt >> 2) * HALF_BYTES + row * 128 +
                                      ((chunk ^ (row & 7)) << 4));
            mma_bf16(o[dt], af, bh0, bh1);
            mma_bf16(o[dt], af, bl0, bl1);
          }
        }
      }
    }
    // Slots that were issued for this item past its last tile are empty groups:
    // step over them.  The slots after those are the next item's first tiles,
    // already in flight.
    consumed += skip_after;

    // ---- merge the four warps: (w0 + w2) + (w1 + w3), fixed order ---------------
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      l0 += __shfl_xor_sync(0xffffffffu, l0, off);
      l1 += __shfl_xor_sync(0xffffffffu, l1, off);
    }
    if (gp == 0) {
      sm_m[warp * 8 + 2 * c] = M0;
      sm_m[warp * 8 + 2 * c + 1] = M1;
      sm_l[warp * 8 + 2 * c] = l0;
      sm_l[warp * 8 + 2 * c + 1] = l1;
    }
    if (threadIdx.x == 0) s_next = fetched_next;
    __syncthreads();  // (max, sum) of every warp and the next item index are visible
    const int after_next = s_next;
    // the warps whose results belong to the same heads: all four, or (pairs) the two of this warp's role
    constexpr int W0_STEP = ROLES;
    const int w_first = role;
    float Mx0 = -INFINITY, Mx1 = -INFINITY;
#pragma unroll
    for (int ww = w_first; ww < WARPS; ww += W0_STEP) {
      Mx0 = fmaxf(Mx0, sm_m[ww * 8 + 2 * c]);
      Mx1 = fmaxf(Mx1, sm_m[ww * 8 + 2 * c + 1]);
    }
    float ls0 = 0.f, ls1 = 0.f;
    if (Mx0 > -INFINITY)
#pragma unroll
      for (int ww = w_first; ww < WARPS; ww += W0_STEP) ls0 += exp2f(sm_m[ww * 8 + 2 * c] - Mx0) * sm_l[ww * 8 + 2 * c];
    if (Mx1 > -INFINITY)
#pragma unroll
      for (int ww = w_first; ww < WARPS; ww += W0_STEP)
        ls1 += exp2f(sm_m[ww * 8 + 2 * c + 1] - Mx1) * sm_l[ww * 8 + 2 * c + 1];
    {
      const float f0 = Mx0 > -INFINITY ? exp2f(M0 - Mx0) : 0.f;
      const float f1 = Mx1 > -INFINITY ? exp2f(M1 - Mx1) : 0.f;
#pragma unroll
      for (int i = 0; i < NK; ++i) {
        o[i][0] *= f0;
        o[i][1] *= f1;
        o[i][2] *= f0;
        o[i][3] *= f1;
      }
    }
    // rows of heads 2c (and 2c + 1 at + kD) of a warp's O in merge buffer `which`
    auto buf_at = [&](int which, int) { return sm_buf + which * (8 * kD) + (2 * c) * kD; };
    // (four roles: every warp holds the whole sum of its own eight heads, nothing to add)
    if (ROLES < 4 && warp >= 2) {
#pragma unroll
      for (int dt = 0; dt < NK; ++dt) {
        float* p = buf_at(warp - 2, dt);
        p[dmap(dt, 0)] = o[dt][0];
        p[kD + dmap(dt, 0)] = o[dt][1];
        p[dmap(dt, 1)] = o[dt][2];
        p[kD + dmap(dt, 1)] = o[dt][3];
      }
    }
    __syncthreads();
    if (ROLES < 4 && warp < 2) {
#pragma unroll
      for (int dt = 0; dt < NK; ++dt) {
        const float* p = buf_at(warp, dt);
        o[dt][0] += p[dmap(dt, 0)];
        o[dt][1] += p[kD + dmap(dt, 0)];
        o[dt][2] += p[dmap(dt, 1)];
        o[dt][3] += p[kD + dmap(dt, 1)];
      }
    }
    if constexpr (!PAIR) {
      __syncthreads();  // buffer 0 has been read by warp 0 before warp 1 overwrites it
      if (warp == 1) {
#pragma unroll
        for (int dt = 0; dt < NK; ++dt) {
          float* p = buf_at(0, dt);
          p[dmap(dt, 0)] = o[dt][0];
          p[kD + dmap(dt, 0)] = o[dt][1];
          p[dmap(dt, 1)] = o[dt][2];
          p[kD + dmap(dt, 1)] = o[dt][3];
        }
      }
      __syncthreads();
    }
    const bool single = w.nc <= 1;  // the whole (layer, b, kv head) is this one chunk
    // the warps that hold the item's sum: warp 0, or one warp per role with eight heads each
    if (warp < ROLES) {
      if constexpr (!PAIR) {
#pragma unroll
        for (int dt = 0; dt < NK; ++dt) {
          const float* p = buf_at(0, dt);
          o[dt][0] += p[dmap(dt, 0)];
          o[dt][1] += p[kD + dmap(dt, 0)];
          o[dt][2] += p[dmap(dt, 1)];
          o[dt][3] += p[kD + dmap(dt, 1)];
        }
      }
      if (single) {
        // no partials: normalise and write the output of heads 2c, 2c + 1 directly
        const long long ob = (((long long)l * s.batch + b) * s.n_q_heads + h * G + g0) * kD;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int g = 2 * c + e;
          if (g < Gn) {
            const float den = e ? ls1 : ls0;
#pragma unroll
            for (int dt = 0; dt < NK; ++dt) {
#pragma unroll
              for (int half = 0; half < 2; ++half) {
                const float num = o[dt][e + 2 * half];
                const float r = den > 0.f ? (num / den) * v_scale : 0.f;
                const long long oi = ob + (long long)g * kD + dmap(dt, half);
                if (a.out_dtype == LT_F32) ((float*)a.out)[oi] = r;
                else ((__nv_bfloat16*)a.out)[oi] = __float2bfloat16_rn(r);
              }
            }
          }
        }
      } else {
        const long long unit = partial_unit(a, w);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int g = 2 * c + e;
          if (g < Gn) {
            const long long pslot = unit * G + g0 + g;  // a slot holds the group's heads in order
            float* po = a.part_o + pslot * kD;
#pragma unroll
            for (int dt = 0; dt < NK; ++dt) {
              po[dmap(dt, 0)] = o[dt][e];
              po[dmap(dt, 1)] = o[dt][e + 2];
            }
            if (gp == 0) {
              a.part_ml[pslot * 2] = e ? Mx1 : Mx0;
              a.part_ml[pslot * 2 + 1] = e ? ls1 : ls0;
            }
          }
        }
      }
    }
    if (!single) {
      if (count_item_in(a, w, &s_flag)) combine_unit(a, w, reinterpret_cast<float2*>(sm_buf));
    }
    __syncthreads();  // merge buffers and flags are free for the next item

    // ---- move on: the next item becomes current ----------------------------------
    cur = nxt;
    nxt = after_next;
    const int pre = la_in_next ? la_idx : 0;  // slots already issued on behalf of the new current item
    src_cur = src_nxt;
    la_in_next = 0;
    la_idx = pre;
    skip_after = max(0, pre - src_cur.my_tiles);
    if (cur < n_items) w = wl.item(a, cur);
    src_nxt.my_tiles = 0;
    if (nxt < n_items) src_nxt = make_src(wl.item(a, nxt));
  }
  cp_async_wait<0>();
  finish_launch(a);
}
bool decode_mma_supported(const lt_shape& s) {
  // groups of 9..16: two warps per tile, eight heads each; 17..32: four warps per tile
  return s.dtype == LT_BF16 && (s.head_dim == 128 || s.head_dim == 64) &&
         (s.n_q_heads / s.n_kv_heads) <= 32;
}

template <int TILE, int NSTAGE, int WARPS, int MINB, bool FP8, int DH, int ROLES>
static cudaError_t launch_variant(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                                  const LayerTable& ks, const LayerTable& vs, cudaStream_t st) {
  constexpr int streams = WARPS / ROLES;
  constexpr int ring = FP8 ? streams * NSTAGE * TILE * 256 : streams * NSTAGE * TILE * 4 * DH;
  constexpr int merge = 2 * 8 * DH * 4 + 2 * WARPS * 8 * 4;
  static_assert(2 * 8 * DH * 4 >= kCombineStagePairs * 8, "the merge buffers double as the combine staging area");
  const int smem = ring + merge + worklist_smem_bytes(a.layer_count * a.s.batch, a.s.batch);
  auto kern = decode_mma_kernel<TILE, NSTAGE, WARPS, MINB, FP8, DH, ROLES>;
  // Per device, behind a lock (host threads may issue their first calls concurrently): the dynamic
  // shared-memory limit is raised once to the largest size any launch of this variant can ask for, and
  // the occupancy of each shared-memory size met so far is remembered (host time matters for per-layer callers).
  constexpr int kSmemMax = ring + merge + worklist_smem_bytes(kMaxWorkEntries, kMaxWorkEntries);
  constexpr int kSizes = 8;
  struct PerDevice {
    bool attr_set;
    int n, smem[kSizes], per_sm[kSizes];
  };
  static std::mutex mu;
  static PerDevice cache[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int per_sm = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    PerDevice& c = cache[dev];
    if (!c.attr_set) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
      if (e != cudaSuccess) return e;
      c.attr_set = true;
    }
    for (int i = 0; i < c.n; ++i)
      if (c.smem[i] == smem) per_sm = c.per_sm[i];
    if (per_sm == 0) {
      cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, WARPS * 32, smem);
      if (e != cudaSuccess) return e;
      if (per_sm < 1) return cudaErrorLaunchOutOfResources;
      const int slot = c.n < kSizes ? c.n++ : 0;  // a caller that cycles through many sizes just looks up again
      c.smem[slot] = smem;
      c.per_sm[slot] = per_sm;
    }
  }
  const int grid = persistent_grid(a, per_sm);
  return launch_decode_kernel(kern, grid, WARPS * 32, smem, st, a, kf, vf, ks, vs);
}

cudaError_t launch_decode_mma(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf, const LayerTable& ks,
                              const LayerTable& vs, cudaStream_t st) {
  const int G = a.s.n_q_heads / a.s.n_kv_heads;
  const bool pair = G > 8;   // groups of 9..16: two warps per tile, eight heads each
  const bool quad = G > 16;  // groups of 17..32: the four warps share one ring of twice the depth
  // 8-bit caches: raw stages of 32 keys (8 KB); a warp's three stages or a pair's six hold what the 16-bit ring holds
  if (a.s.kv_fp8) {
    if (quad) return launch_variant<32, 12, 4, 2, true, 128, 4>(a, kf, vf, ks, vs, st);
    return pair ? launch_variant<32, 6, 4, 2, true, 128, 2>(a, kf, vf, ks, vs, st)
                : launch_variant<32, 3, 4, 2, true, 128, 1>(a, kf, vf, ks, vs, st);
  }
  // head_dim 64: rows are half as long, so 32-key tiles keep the bytes in flight per warp (24 KB) the same
  if (a.s.head_dim == 64) {
    if (quad) return launch_variant<32, 12, 4, 2, false, 64, 4>(a, kf, vf, ks, vs, st);
    return pair ? launch_variant<32, 6, 4, 2, false, 64, 2>(a, kf, vf, ks, vs, st)
                : launch_variant<32, 3, 4, 2, false, 64, 1>(a, kf, vf, ks, vs, st);
  }
  if (quad) return launch_variant<32, 6, 4, 2, false, 128, 4>(a, kf, vf, ks, vs, st);
  return pair ? launch_variant<32, 3, 4, 2, false, 128, 2>(a, kf, vf, ks, vs, st)
              : launch_variant<16, 3, 4, 2, false, 128, 1>(a, kf, vf, ks, vs, st);
}

}  // namespace lt
