// Decode step, CUDA-core path (fp32 stacks, and bf16 stacks whose GQA group exceeds 16; head_dim 64 or
// 128).  Same persistent work-list structure, fused append and in-kernel merge as the tensor-core path.
//
// Partials of one (layer, b, kv head, chunk, head-in-group), log2 domain:
//   M = max_j t_j,  l = sum_j 2^(t_j - M),  o[d] = sum_j 2^(t_j - M) v_j[d]
// with t_j = scale * log2(e) * (q . k_j).
//
// A CTA of 128 threads walks the chunk in tiles of TK keys (16 KB of K rows and 16 KB of V rows per tile, two
// tiles in shared memory: the copies of the next tile run under the arithmetic of this one) and serves up to
// eight query heads of the group per pass over the chunk.  Phases of a tile, a CTA barrier between them:
//   scores   a thread owns one key and one slice of d and keeps the partial dot products of all eight heads:
//            its K values come as 16-byte vectors (rows are padded by 16 bytes, so the eight rows of a
//            quarter warp fall into different banks), q (times scale * log2 e) as broadcasts of the eight
//            heads' values of one d, [d][head] in shared memory: 32 multiply-adds per K vector.  The slices
//            of a key are then added and the scores masked.
//   softmax  a warp owns a head: tile maximum, new running maximum, p = 2^(t - M) stored [key][head],
//            running sum and the factor that rescales what was accumulated before.
//   values   a warp owns a quarter of the tile's keys, a lane D / 32 consecutive d of all eight heads:
//            one V vector and one broadcast of the key's eight probabilities per 8 x D / 32 multiply-adds.
// At the end of a pass the four warps' sums are added in a fixed order.  Every K and V byte is read from HBM
// once per pass; groups of more than eight heads take several passes.
#include <cuda_bf16.h>

#include "lt_decode_common.cuh"
#include "lt_internal.h"

namespace lt {

namespace {

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) {
  return x;
}
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) {
  return __bfloat162float(x);
}

__device__ __forceinline__ void copy16_async(void* smem_dst, const void* src, int src_bytes) {
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void copy_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void copy_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

__device__ __forceinline__ float bf_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

// the 16-byte vector at p as floats: four fp32 or eight bf16 values
__device__ __forceinline__ void load_vec16(const float* p, float (&x)[4]) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
}
__device__ __forceinline__ void load_vec16(const __nv_bfloat16* p, float (&x)[8]) {
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  x[0] = bf_lo(v.x); x[1] = bf_hi(v.x); x[2] = bf_lo(v.y); x[3] = bf_hi(v.y);
  x[4] = bf_lo(v.z); x[5] = bf_hi(v.z); x[6] = bf_lo(v.w); x[7] = bf_hi(v.w);
}
// DL (2 or 4) consecutive values of a V row
template <int DL>
__device__ __forceinline__ void load_vals(const float* p, float (&x)[DL]) {
  if constexpr (DL == 4) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  } else {
    const float2 v = *reinterpret_cast<const float2*>(p);
    x[0] = v.x; x[1] = v.y;
  }
}
template <int DL>
__device__ __forceinline__ void load_vals(const __nv_bfloat16* p, float (&x)[DL]) {
  if constexpr (DL == 4) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    x[0] = bf_lo(v.x); x[1] = bf_hi(v.x); x[2] = bf_lo(v.y); x[3] = bf_hi(v.y);
  } else {
    const uint32_t v = *reinterpret_cast<const uint32_t*>(p);
    x[0] = bf_lo(v); x[1] = bf_hi(v);
  }
}

constexpr int kGenericThreads = 128;
constexpr int kGenericHeads = 8;  // query heads per pass over the chunk

template <typename T, int D>
struct GenericGeometry {
  static constexpr int TK = 16384 / (D * (int)sizeof(T));   // keys per tile: 32, 64 or 128
  static constexpr int ROW = D * (int)sizeof(T);            // bytes of a cached row
  static constexpr int KROW = ROW + 16;                     // a K row in shared memory (padded)
  static constexpr int VEC = ROW / 16;                      // 16-byte vectors of a row
  static constexpr int EPV = 16 / (int)sizeof(T);           // elements of a 16-byte vector
  static constexpr int NS = kGenericThreads / TK;           // score phase: slices of d
  static constexpr int DS = D / NS;                         // score phase: d per thread
  static constexpr int DL = D / 32;                         // value phase: d per lane
  static constexpr int KW = TK / (kGenericThreads / 32);    // value phase: keys per warp
  static constexpr int kStage = TK * KROW + TK * ROW;       // K rows, then V rows
  static constexpr int kTiles = 2 * kStage;
  // floats after the tiles: q [D][8], slice partials [NS][TK][8], scores [TK][9], probabilities [TK][8], state [3][8]
  static constexpr int kFloats = D * 8 + NS * TK * 8 + TK * 9 + TK * 8 + 24;
  static constexpr int kFixedBytes = (kTiles + kFloats * 4 + 15) / 16 * 16;  // shared memory before the work list
  static_assert(TK >= 32 && TK <= kGenericThreads && kGenericThreads % TK == 0, "a thread per key of the tile");
  static_assert(DS % EPV == 0 && (DL == 2 || DL == 4), "geometry");
  static_assert(kTiles >= (kGenericThreads / 32) * kGenericHeads * D * 4, "the tiles hold the warps' sums at the end of a pass");
};

}  // namespace

template <typename T, int D>
__global__ void __launch_bounds__(kGenericThreads) decode_generic_kernel(DecodeArgs a, LayerTable kf, LayerTable vf,
                                                                         LayerTable ks, LayerTable vs) {
  using Geo = GenericGeometry<T, D>;
  constexpr int HB = kGenericHeads, TK = Geo::TK, ROW = Geo::ROW, KROW = Geo::KROW, VEC = Geo::VEC, EPV = Geo::EPV,
                NS = Geo::NS, DS = Geo::DS, DL = Geo::DL, KW = Geo::KW;
  static_assert(HB == 8, "the phases below are written for eight heads per pass");
  extern __shared__ __align__(16) uint8_t smem[];
  __shared__ int s_flag;
  __shared__ float2 s_ml[kCombineStagePairs];
  uint8_t* tiles = smem;                                             // [2][K rows TK x KROW | V rows TK x ROW]
  float* q_t = reinterpret_cast<float*>(smem + Geo::kTiles);         // [D][8]: q[head][d] times scale * log2 e
  float* part = q_t + D * 8;                                         // [NS][TK][8] dot products of the d slices
  float* sc = part + NS * TK * 8;                                    // [TK][9] scores (a row per key, padded)
  float* p_t = sc + TK * 9;                                          // [TK][8] probabilities
  float* st_M = p_t + TK * 8;                                        // [8] running maximum
  float* st_l = st_M + 8;                                            // [8] running sum
  float* st_corr = st_l + 8;                                         // [8] factor of this tile
  const lt_shape& s = a.s;
  const int G = s.n_q_heads / s.n_kv_heads;
  pdl_wait_prior_grid();
  pdl_allow_next_grid();
  WorkList wl;
  wl.carve(smem + Geo::kFixedBytes, a.layer_count, s.batch);
  wl.build(a, kf, vf, ks, vs);
  const int n_items = wl.total(a);
  const float cs = a.cs;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < TK * 8; i += kGenericThreads) p_t[i] = 0.f;  // columns of heads that a pass does not have stay 0

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const WorkItem w = wl.item(a, item);
    const int l = w.l, b = w.b, h = w.h;
    const long long bh = (long long)b * s.n_kv_heads + h;
    const T* Kl = (const T*)(w.lazy ? ks.p[l] : kf.p[l]);
    const T* Vl = (const T*)(w.lazy ? vs.p[l] : vf.p[l]);
    // element offset of cache row j of this (b, kv head): stream caches are contiguous, full caches may be paged
    auto row_off = [&](int j) { return (w.lazy ? bh * w.rows + j : full_cache_row(s, b, h, j)) * D; };
    const T* k_new_row = nullptr;
    const T* v_new_row = nullptr;
    if (w.new_row >= 0) {
      // fused append: this item owns the new token's row; it reads the row from k_new / v_new and stores it
      const long long src = (((long long)l * s.batch + b) * s.n_kv_heads + h) * D;
      k_new_row = (const T*)a.k_new + src;
      v_new_row = (const T*)a.v_new + src;
      T* kd = const_cast<T*>(Kl) + row_off(w.new_row);
      T* vd = const_cast<T*>(Vl) + row_off(w.new_row);
      for (int d = tid; d < D; d += blockDim.x) {
        kd[d] = k_new_row[d];
        vd[d] = v_new_row[d];
      }
    }
    const int n_tiles = (w.j1 - w.j0 + TK - 1) / TK;
    // copies of tile `it` into stage `it & 1` (rows past the chunk are filled with zeros)
    auto fetch_tile = [&](int it) {
      uint8_t* kt = tiles + (it & 1) * Geo::kStage;
      uint8_t* vt = kt + TK * KROW;
      for (int i = tid; i < TK * VEC; i += kGenericThreads) {
        const int r = i / VEC, p = i - r * VEC;
        const int j = w.j0 + it * TK + r;
        const bool valid = j < w.j1;
        const bool fresh = j == w.new_row;
        const long long ro = row_off(valid ? j : w.j0);
        const uint8_t* ksrc = reinterpret_cast<const uint8_t*>(fresh ? k_new_row : Kl + ro);
        const uint8_t* vsrc = reinterpret_cast<const uint8_t*>(fresh ? v_new_row : Vl + ro);
        copy16_async(kt + r * KROW + p * 16, ksrc + p * 16, valid ? 16 : 0);
        copy16_async(vt + r * ROW + p * 16, vsrc + p * 16, valid ? 16 : 0);
      }
    };
    const long long unit = partial_unit(a, w);

    for (int g0 = 0; g0 < G; g0 += HB) {  // one pass over the chunk per eight heads of the group
      const int HBn = min(HB, G - g0);
      const T* qp = (const T*)a.q + (((long long)l * s.batch + b) * s.n_q_heads + h * G + g0) * D;
      for (int i = tid; i < D * HB; i += kGenericThreads) {
        const int d = i >> 3, g = i & 7;
        q_t[i] = g < HBn ? to_f32<T>(qp[g * D + d]) * cs : 0.f;
      }
      if (tid < HB) {
        st_M[tid] = -INFINITY;
        st_l[tid] = 0.f;
        st_corr[tid] = 0.f;
      }
      float acc[HB][DL];
#pragma unroll
      for (int g = 0; g < HB; ++g)
#pragma unroll
        for (int e = 0; e < DL; ++e) acc[g][e] = 0.f;
      if (n_tiles > 0) fetch_tile(0);
      copy_commit();
      for (int it = 0; it < n_tiles; ++it) {
        if (it + 1 < n_tiles) fetch_tile(it + 1);
        copy_commit();
        copy_wait<1>();
        __syncthreads();  // tile `it` has landed for every thread; q and the state of this pass are visible
        const uint8_t* kt = tiles + (it & 1) * Geo::kStage;
        const T* vt = reinterpret_cast<const T*>(kt + TK * KROW);
        const int tile_j0 = w.j0 + it * TK;
        // ---- scores: one key, one slice of d, eight heads -------------------------------
        {
          const int key = tid % TK, sl = tid / TK;
          const T* krow = reinterpret_cast<const T*>(kt + key * KROW) + sl * DS;
          const float* qd = q_t + sl * DS * 8;
          float t[HB];
#pragma unroll
          for (int g = 0; g < HB; ++g) t[g] = 0.f;
#pragma unroll 2
          for (int v = 0; v < DS / EPV; ++v) {
            float kx[EPV];
            load_vec16(krow + v * EPV, kx);
#pragma unroll
            for (int e = 0; e < EPV; ++e) {
              const float4 qa = *reinterpret_cast<const float4*>(qd + (v * EPV + e) * 8);
              const float4 qb = *reinterpret_cast<const float4*>(qd + (v * EPV + e) * 8 + 4);
              t[0] = fmaf(kx[e], qa.x, t[0]);
              t[1] = fmaf(kx[e], qa.y, t[1]);
              t[2] = fmaf(kx[e], qa.z, t[2]);
              t[3] = fmaf(kx[e], qa.w, t[3]);
              t[4] = fmaf(kx[e], qb.x, t[4]);
              t[5] = fmaf(kx[e], qb.y, t[5]);
              t[6] = fmaf(kx[e], qb.z, t[6]);
              t[7] = fmaf(kx[e], qb.w, t[7]);
            }
          }
          if constexpr (NS == 1) {
            const bool valid = tile_j0 + key < w.j1;
#pragma unroll
            for (int g = 0; g < HB; ++g) sc[key * 9 + g] = valid ? t[g] : -INFINITY;
          } else {
            float4* dst = reinterpret_cast<float4*>(part + (sl * TK + key) * 8);
            dst[0] = make_float4(t[0], t[1], t[2], t[3]);
            dst[1] = make_float4(t[4], t[5], t[6], t[7]);
          }
        }
        if constexpr (NS > 1) {
          __syncthreads();
          // the slices of a key added in slice order; keys past the chunk are masked
          for (int i = tid; i < TK * 8; i += kGenericThreads) {
            const int key = i >> 3, g = i & 7;
            float t = part[i];
#pragma unroll
            for (int sl = 1; sl < NS; ++sl) t += part[sl * TK * 8 + i];
            sc[key * 9 + g] = tile_j0 + key < w.j1 ? t : -INFINITY;
          }
        }
        __syncthreads();
        // ---- softmax statistics: a warp per head --------------------------------------
        for (int g = warp; g < HBn; g += kGenericThreads / 32) {
          float v[TK / 32];
          float m = -INFINITY;
#pragma unroll
          for (int r = 0; r < TK / 32; ++r) {
            v[r] = sc[(lane + 32 * r) * 9 + g];
            m = fmaxf(m, v[r]);
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
          const float Mo = st_M[g];
          const float Mn = fmaxf(Mo, m);  // finite: a tile has at least one key of the chunk
          float sum = 0.f;
#pragma unroll
          for (int r = 0; r < TK / 32; ++r) {
            const float p = exp2f(v[r] - Mn);
            p_t[(lane + 32 * r) * 8 + g] = p;
            sum += p;
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
          if (lane == 0) {
            const float corr = exp2f(Mo - Mn);  // 0 on the first tile (Mo = -inf)
            st_corr[g] = corr;
            st_M[g] = Mn;
            st_l[g] = st_l[g] * corr + sum;
          }
        }
        __syncthreads();
        // ---- values: a quarter of the keys per warp, D / 32 consecutive d per lane, eight heads ----
        {
          const float4 ca = *reinterpret_cast<const float4*>(st_corr), cb = *reinterpret_cast<const float4*>(st_corr + 4);
          const float corr[HB] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
#pragma unroll
          for (int g = 0; g < HB; ++g)
#pragma unroll
            for (int e = 0; e < DL; ++e) acc[g][e] *= corr[g];
          const T* vcol = vt + (warp * KW) * D + lane * DL;
          const float* pk = p_t + (warp * KW) * 8;
#pragma unroll 4
          for (int k = 0; k < KW; ++k) {
            float vx[DL];
            load_vals<DL>(vcol + k * D, vx);
            const float4 pa = *reinterpret_cast<const float4*>(pk + k * 8);
            const float4 pb = *reinterpret_cast<const float4*>(pk + k * 8 + 4);
            const float p8[HB] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
#pragma unroll
            for (int g = 0; g < HB; ++g)
#pragma unroll
              for (int e = 0; e < DL; ++e) acc[g][e] = fmaf(p8[g], vx[e], acc[g][e]);
          }
        }
        __syncthreads();  // the stage, the scores and the probabilities are free for the tile after next
      }
      copy_wait<0>();
      // ---- the four warps' sums, added in a fixed order; partials of this pass's heads ----
      float* red = reinterpret_cast<float*>(tiles);  // [4 warps][8][D]: the tiles are idle now
#pragma unroll
      for (int g = 0; g < HB; ++g)
#pragma unroll
        for (int e = 0; e < DL; ++e) red[(warp * HB + g) * D + lane * DL + e] = acc[g][e];
      __syncthreads();
      for (int i = tid; i < HBn * D; i += kGenericThreads) {
        const float o = (red[i] + red[HB * D + i]) + (red[2 * HB * D + i] + red[3 * HB * D + i]);
        a.part_o[(unit * G + g0) * D + i] = o;  // heads g0 .. g0 + HBn - 1 are consecutive rows of the slot
      }
      if (tid < HBn) {
        float* pml = a.part_ml + (unit * G + g0 + tid) * 2;
        pml[0] = st_M[tid];
        pml[1] = st_l[tid];
      }
      __syncthreads();  // q, the state and the tiles are rewritten by the next pass
    }
    if (count_item_in(a, w, &s_flag)) combine_unit(a, w, s_ml);
    __syncthreads();
  }
  finish_launch(a);
}

template <typename T, int D>
static cudaError_t launch_generic_variant(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                                          const LayerTable& ks, const LayerTable& vs, cudaStream_t st) {
  using Geo = GenericGeometry<T, D>;
  const int smem = Geo::kFixedBytes + worklist_smem_bytes(a.layer_count * a.s.batch, a.s.batch);
  auto kern = decode_generic_kernel<T, D>;
  // the same upper bound on every call, so concurrent first calls from several host threads set the same value
  constexpr int kSmemMax = Geo::kFixedBytes + worklist_smem_bytes(kMaxWorkEntries, kMaxWorkEntries);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kGenericThreads, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  return launch_decode_kernel(kern, persistent_grid(a, per_sm), kGenericThreads, smem, st, a, kf, vf, ks, vs);
}

cudaError_t launch_decode_generic(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                                  const LayerTable& ks, const LayerTable& vs, cudaStream_t st) {
  const bool bf = a.s.dtype == LT_BF16;
  if (a.s.head_dim == 128) {
    return bf ? launch_generic_variant<__nv_bfloat16, 128>(a, kf, vf, ks, vs, st)
              : launch_generic_variant<float, 128>(a, kf, vf, ks, vs, st);
  }
  return bf ? launch_generic_variant<__nv_bfloat16, 64>(a, kf, vf, ks, vs, st)
            : launch_generic_variant<float, 64>(a, kf, vf, ks, vs, st);
}

}  // namespace lt
