// Decode step, CUDA-core path (fp32 stacks, and bf16 stacks whose GQA group exceeds 16; head_dim 64 or
// 128).  Same persistent work-list structure, fused append and in-kernel merge as the tensor-core path.
//
// Partials of one (layer, b, kv head, chunk, head-in-group), log2 domain:
//   M = max_j t_j,  l = sum_j 2^(t_j - M),  o[d] = sum_j 2^(t_j - M) v_j[d]
// with t_j = scale * log2(e) * (q . k_j).
//
// A CTA of 128 threads walks the chunk in tiles of TK keys (32 KB of K and V rows per tile, two tiles in
// shared memory: the copies of the next tile run under the arithmetic of this one) and serves up to eight
// query heads of the group per pass over the chunk.  Three phases per tile, a CTA barrier between them:
//   scores   a thread owns one key of the tile and a share of the heads.  It walks its K row starting at
//            element `key` and wrapping around, so the 32 lanes of a warp read 32 different banks although
//            their rows are a multiple of 128 bytes apart; q (pre-multiplied by scale * log2 e) is read
//            from shared memory at the same rotated index, one K element feeding every head of the thread.
//   softmax  a warp owns a head: tile maximum, new running maximum, p = 2^(t - M) written over the scores,
//            running sum and the factor that rescales what was accumulated before.
//   values   a thread owns four consecutive d of one or two heads: o = o * factor + sum_key p[key] v[key][d],
//            V rows read as 16-byte (fp32) or 8-byte (bf16) vectors, p as a broadcast.
// Every K and V byte is read from HBM once per pass; groups of more than eight heads take several passes.
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

// four consecutive values of a V row
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                     __uint_as_float(u.y & 0xffff0000u));
}

constexpr int kGenericThreads = 128;
constexpr int kGenericHeads = 8;           // query heads per pass over the chunk
constexpr int kGenericTileBytes = 32768;   // K rows + V rows of one tile

template <typename T, int D>
struct GenericGeometry {
  static constexpr int TK = kGenericTileBytes / (2 * D * (int)sizeof(T));  // keys per tile: 32, 64 or 128
  static constexpr int ROW = D * (int)sizeof(T);                           // bytes of a cached row
  static constexpr int VEC = ROW / 16;                                     // 16-byte vectors of a row
  static constexpr int NHG = kGenericThreads / TK;                         // score phase: head shares
  static constexpr int HPA = kGenericHeads / NHG;                          // score phase: heads per thread
  static constexpr int CG = D / 4;                                         // value phase: groups of four d
  static constexpr int HPC = kGenericHeads * CG / kGenericThreads;         // value phase: heads per thread
  static constexpr int kTiles = 2 * kGenericTileBytes;                     // two stages
  static constexpr int kFloats = kGenericHeads * D + kGenericHeads * TK + 3 * kGenericHeads;
  static constexpr int kFixedBytes = kTiles + kFloats * 4;                 // shared memory before the work list
  static_assert(TK >= 32 && TK <= kGenericThreads && kGenericThreads % TK == 0, "a thread per key of the tile");
  static_assert(HPA >= 1 && HPC >= 1 && kFixedBytes % 16 == 0, "geometry");
};

}  // namespace

template <typename T, int D>
__global__ void __launch_bounds__(kGenericThreads) decode_generic_kernel(DecodeArgs a, LayerTable kf, LayerTable vf,
                                                                         LayerTable ks, LayerTable vs) {
  using Geo = GenericGeometry<T, D>;
  constexpr int HB = kGenericHeads, TK = Geo::TK, ROW = Geo::ROW, VEC = Geo::VEC, HPA = Geo::HPA, CG = Geo::CG,
                HPC = Geo::HPC;
  extern __shared__ __align__(16) uint8_t smem[];
  __shared__ int s_flag;
  __shared__ float2 s_ml[kCombineStagePairs];
  uint8_t* tiles = smem;                                             // [2][K rows TK x ROW | V rows TK x ROW]
  float* q_s = reinterpret_cast<float*>(smem + Geo::kTiles);         // [HB][D], times scale * log2 e
  float* sc = q_s + HB * D;                                          // [HB][TK] scores, then probabilities
  float* st_M = sc + HB * TK;                                        // [HB] running maximum
  float* st_l = st_M + HB;                                           // [HB] running sum
  float* st_corr = st_l + HB;                                        // [HB] factor of this tile
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
      uint8_t* kt = tiles + (it & 1) * kGenericTileBytes;
      uint8_t* vt = kt + TK * ROW;
      for (int i = tid; i < TK * VEC; i += kGenericThreads) {
        const int r = i / VEC, p = i - r * VEC;
        const int j = w.j0 + it * TK + r;
        const bool valid = j < w.j1;
        const bool fresh = j == w.new_row;
        const long long ro = row_off(valid ? j : w.j0);
        const uint8_t* ksrc = reinterpret_cast<const uint8_t*>(fresh ? k_new_row : Kl + ro);
        const uint8_t* vsrc = reinterpret_cast<const uint8_t*>(fresh ? v_new_row : Vl + ro);
        copy16_async(kt + r * ROW + p * 16, ksrc + p * 16, valid ? 16 : 0);
        copy16_async(vt + r * ROW + p * 16, vsrc + p * 16, valid ? 16 : 0);
      }
    };
    const long long unit = partial_unit(a, w);

    for (int g0 = 0; g0 < G; g0 += HB) {  // one pass over the chunk per eight heads of the group
      const int HBn = min(HB, G - g0);
      const T* qp = (const T*)a.q + (((long long)l * s.batch + b) * s.n_q_heads + h * G + g0) * D;
      for (int i = tid; i < HB * D; i += kGenericThreads) q_s[i] = i < HBn * D ? to_f32<T>(qp[i]) * cs : 0.f;
      if (tid < HB) {
        st_M[tid] = -INFINITY;
        st_l[tid] = 0.f;
      }
      // value phase: this thread's four d and its heads
      const int cg = tid % CG, hs = tid / CG;
      float4 acc[HPC];
#pragma unroll
      for (int i = 0; i < HPC; ++i) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (n_tiles > 0) fetch_tile(0);
      copy_commit();
      for (int it = 0; it < n_tiles; ++it) {
        if (it + 1 < n_tiles) fetch_tile(it + 1);
        copy_commit();
        copy_wait<1>();
        __syncthreads();  // tile `it` has landed for every thread; q and the state of this pass are visible
        const T* kt = reinterpret_cast<const T*>(tiles + (it & 1) * kGenericTileBytes);
        const T* vt = kt + TK * D;
        // ---- scores ---------------------------------------------------------------
        {
          const int key = tid % TK, hg = tid / TK;
          if (hg * HPA < HBn) {  // a share whose heads do not exist in this pass has nothing to do
            const T* krow = kt + key * D;
            const float* qh = q_s + hg * HPA * D;
            float t[HPA];
#pragma unroll
            for (int i = 0; i < HPA; ++i) t[i] = 0.f;
#pragma unroll 8
            for (int dd = 0; dd < D; ++dd) {
              const int d = (dd + key) & (D - 1);
              const float kv = to_f32<T>(krow[d]);
#pragma unroll
              for (int i = 0; i < HPA; ++i) t[i] = fmaf(kv, qh[i * D + d], t[i]);
            }
            const bool valid = w.j0 + it * TK + key < w.j1;
#pragma unroll
            for (int i = 0; i < HPA; ++i) sc[(hg * HPA + i) * TK + key] = valid ? t[i] : -INFINITY;
          }
        }
        __syncthreads();
        // ---- softmax statistics: a warp per head --------------------------------------
        for (int g = warp; g < HBn; g += kGenericThreads / 32) {
          float v[TK / 32];
          float m = -INFINITY;
#pragma unroll
          for (int r = 0; r < TK / 32; ++r) {
            v[r] = sc[g * TK + lane + 32 * r];
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
            sc[g * TK + lane + 32 * r] = p;
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
        // ---- values ---------------------------------------------------------------
        if (hs * HPC < HBn) {
          const float* ph[HPC];
#pragma unroll
          for (int i = 0; i < HPC; ++i) {
            const int g = hs * HPC + i;
            const float corr = g < HBn ? st_corr[g] : 0.f;
            acc[i].x *= corr;
            acc[i].y *= corr;
            acc[i].z *= corr;
            acc[i].w *= corr;
            ph[i] = sc + g * TK;
          }
          const T* vcol = vt + cg * 4;
#pragma unroll 4
          for (int key = 0; key < TK; ++key) {
            const float4 v4 = load4(vcol + key * D);
#pragma unroll
            for (int i = 0; i < HPC; ++i) {
              const float p = ph[i][key];
              acc[i].x = fmaf(p, v4.x, acc[i].x);
              acc[i].y = fmaf(p, v4.y, acc[i].y);
              acc[i].z = fmaf(p, v4.z, acc[i].z);
              acc[i].w = fmaf(p, v4.w, acc[i].w);
            }
          }
        }
        __syncthreads();  // the stage and the probabilities are free for the tile after next
      }
      copy_wait<0>();
      // ---- partials of this pass's heads ---------------------------------------------
#pragma unroll
      for (int i = 0; i < HPC; ++i) {
        const int g = hs * HPC + i;
        if (g < HBn) *reinterpret_cast<float4*>(a.part_o + (unit * G + g0 + g) * D + cg * 4) = acc[i];
      }
      if (tid < HBn) {
        float* pml = a.part_ml + (unit * G + g0 + tid) * 2;
        pml[0] = st_M[tid];
        pml[1] = st_l[tid];
      }
      __syncthreads();  // q and the state are rewritten by the next pass
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
