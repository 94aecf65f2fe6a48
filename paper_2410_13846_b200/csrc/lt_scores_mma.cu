// Lazy ratio (Eq. 1), tensor-core path: bf16, head_dim 128.
//
// One CTA per (layer, batch row, kv head, key split, block of 256 query rows).
// The query rows of a kv head are its G heads x w_last tail queries, row
// r = g * w_last + t, which is one contiguous [G * w_last][128] matrix in
// q_tail.  Each of the 8 warps keeps 32 rows of Q in registers (A fragments)
// for the whole key range; K tiles of 64 keys stream through a 4-stage cp.async
// ring shared by the warps and are read with ldmatrix as the B operand of
// S = Q K^T (mma.sync m16n8k16, fp32 accumulate).  Only three numbers per row
// survive: running max, sum of exp over visible keys, sum of exp over visible
// window keys; no probabilities are written anywhere and K is read once.
// Each thread keeps statistics over the columns it owns and the four lanes of
// a row are merged once at the end, so the key loop has no shuffles.
#include <cuda_bf16.h>

#include "lt_internal.h"

namespace lt {

namespace {

constexpr int kD = 128;
constexpr int kRowBytes = 256;
constexpr int kTileKeys = 64;
constexpr int kStageBytes = kTileKeys * kRowBytes;  // 16 KB: halves [2][64][128 B]
constexpr int kHalfBytes = kTileKeys * 128;
constexpr int kStages = 4;
constexpr int kWarps = 8;
constexpr int kRowsPerCta = kWarps * 32;

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
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__host__ __device__ inline int split_len(int n_ctx, int n_splits) {
  int len = (n_ctx + n_splits - 1) / n_splits;
  return (len + 63) / 64 * 64;
}

}  // namespace

// grid (n_splits * row_blocks, B * Hkv, L); block 256.
__global__ void __launch_bounds__(kWarps * 32, 1) scores_mma_kernel(ScoreArgs a, LayerTable kf) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const lt_shape& s = a.s;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int T = a.w_last;
  const int M = G * T;  // query rows of this kv head
  const int sp = blockIdx.x % a.n_splits, rb = blockIdx.x / a.n_splits;
  const int b = blockIdx.y / s.n_kv_heads, h = blockIdx.y % s.n_kv_heads;
  const int l = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gp = lane >> 2, c = lane & 3;
  const int n_ctx = a.n_ctx;
  const int len = split_len(n_ctx, a.n_splits);
  const int k0 = sp * len;
  const int k1 = min(n_ctx, k0 + len);
  const int row0 = rb * kRowsPerCta + warp * 32;  // first row of this warp

  // rows of this thread: row0 + mt*16 + hf*8 + gp ; their query positions' last visible key
  int vis[4];  // last visible key index of row (mt*2+hf)
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = row0 + (i >> 1) * 16 + (i & 1) * 8 + gp;
    vis[i] = n_ctx - T + (r % T);
  }

  // ---- Q fragments (A operand), kept for the whole key range ------------------
  uint32_t qf[2][8][4];
  {
    const __nv_bfloat16* qb =
        (const __nv_bfloat16*)a.q_tail + ((((long long)l * s.batch + b) * s.n_q_heads + (long long)h * G) * T) * kD;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      const int r_lo = row0 + mt * 16 + gp, r_hi = r_lo + 8;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int d = 16 * ks + 2 * c;
        qf[mt][ks][0] = r_lo < M ? *reinterpret_cast<const uint32_t*>(qb + (long long)r_lo * kD + d) : 0u;
        qf[mt][ks][1] = r_hi < M ? *reinterpret_cast<const uint32_t*>(qb + (long long)r_hi * kD + d) : 0u;
        qf[mt][ks][2] = r_lo < M ? *reinterpret_cast<const uint32_t*>(qb + (long long)r_lo * kD + d + 8) : 0u;
        qf[mt][ks][3] = r_hi < M ? *reinterpret_cast<const uint32_t*>(qb + (long long)r_hi * kD + d + 8) : 0u;
      }
    }
  }

  const uint8_t* Kb = (const uint8_t*)kf.p[l] + ((long long)(b * s.n_kv_heads + h) * s.full_capacity) * kRowBytes;
  const int n_tiles = k1 > k0 ? (k1 - k0 + kTileKeys - 1) / kTileKeys : 0;
  const uint32_t sbase = smem_u32(smem);

  auto load_tile = [&](int t) {
    if (t < n_tiles) {
      const int kb = k0 + t * kTileKeys;
      const uint32_t st = sbase + (t % kStages) * kStageBytes;
#pragma unroll
      for (int i = 0; i < (kTileKeys * 16) / (kWarps * 32); ++i) {
        const int idx = i * (kWarps * 32) + threadIdx.x;
        const int r = idx >> 4, p = idx & 15;
        const int row = kb + r;
        const bool valid = row < k1;
        const long long goff = (long long)(valid ? row : (k1 - 1)) * kRowBytes + p * 16;
        cp_async16(st + (p >> 3) * kHalfBytes + r * 128 + (((p & 7) ^ (r & 7)) << 4), Kb + goff, valid ? 16 : 0);
      }
    }
    cp_async_commit();
  };

  float mx[4], sA[4], sW[4];  // per row (mt*2+hf): raw-logit max, sum exp, window sum exp (this thread's columns)
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    mx[i] = -INFINITY;
    sA[i] = 0.f;
    sW[i] = 0.f;
  }
  const float cs = a.cs;
  const int S = s.n_sink, win_lo = n_ctx - s.n_recent;  // window: j < S or j >= win_lo

#pragma unroll
  for (int i = 0; i < kStages - 1; ++i) load_tile(i);

  const int b_row = lane & 7, b_chk = lane >> 3;  // ldmatrix lane address parts

  for (int it = 0; it < n_tiles; ++it) {
    cp_async_wait<kStages - 2>();
    __syncthreads();
    load_tile(it + kStages - 1);
    const uint32_t st = sbase + (it % kStages) * kStageBytes;
    const int kb = k0 + it * kTileKeys;

    float sc[2][8][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) sc[mt][nt][0] = sc[mt][nt][1] = sc[mt][nt][2] = sc[mt][nt][3] = 0.f;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int row = nt * 8 + b_row;
#pragma unroll
      for (int kp = 0; kp < 4; ++kp) {
        uint32_t bf[4];
        const int chunk = 4 * kp + b_chk;  // 16-byte column 0..15 of the row
        ldmatrix_x4(bf, st + (chunk >> 3) * kHalfBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          mma_bf16(sc[mt][nt], qf[mt][2 * kp], bf[0], bf[1]);
          mma_bf16(sc[mt][nt], qf[mt][2 * kp + 1], bf[2], bf[3]);
        }
      }
    }

    // ---- classify the tile (uniform over the CTA) --------------------------------
    const int kend = kb + kTileKeys;
    const bool all_win = (kend <= S) || (kb >= win_lo);
    const bool no_win = (kb >= S) && (kend <= win_lo);
    const bool plain = (kend <= k1) && (kend - 1 <= n_ctx - T) && (all_win || no_win);
    if (plain) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int mt = i >> 1, e0 = (i & 1) * 2;
        float tm = sc[mt][0][e0];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) tm = fmaxf(tm, fmaxf(sc[mt][nt][e0], sc[mt][nt][e0 + 1]));
        const float mn = fmaxf(mx[i], tm);
        const float corr = exp2f((mx[i] - mn) * cs);
        const float off = -mn * cs;
        float ps = 0.f;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
          ps += exp2f(fmaf(sc[mt][nt][e0], cs, off)) + exp2f(fmaf(sc[mt][nt][e0 + 1], cs, off));
        sA[i] = sA[i] * corr + ps;
        sW[i] = sW[i] * corr + (all_win ? ps : 0.f);
        mx[i] = mn;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int mt = i >> 1, e0 = (i & 1) * 2;
        const int lim = min(vis[i], k1 - 1);  // last key this row may use in this split
        float tm = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int j = kb + nt * 8 + 2 * c + e;
            if (j <= lim) tm = fmaxf(tm, sc[mt][nt][e0 + e]);
          }
        const float mn = fmaxf(mx[i], tm);
        if (mn > -INFINITY) {
          const float corr = exp2f((mx[i] - mn) * cs);  // mx = -inf -> 0
          const float off = -mn * cs;
          float ps = 0.f, pw = 0.f;
#pragma unroll
          for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int j = kb + nt * 8 + 2 * c + e;
              if (j <= lim) {
                const float p = exp2f(fmaf(sc[mt][nt][e0 + e], cs, off));
                ps += p;
                if (j < S || j >= win_lo) pw += p;
              }
            }
          sA[i] = sA[i] * corr + ps;
          sW[i] = sW[i] * corr + pw;
          mx[i] = mn;
        }
      }
    }
  }
  cp_async_wait<0>();

  // ---- merge the four lanes of each row, write the split's statistics --------------
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float m = mx[i], A = sA[i], W = sW[i];
#pragma unroll
    for (int off = 1; off < 4; off <<= 1) {
      const float mo = __shfl_xor_sync(0xffffffffu, m, off);
      const float Ao = __shfl_xor_sync(0xffffffffu, A, off);
      const float Wo = __shfl_xor_sync(0xffffffffu, W, off);
      const float mn = fmaxf(m, mo);
      if (mn > -INFINITY) {
        const float w1 = exp2f((m - mn) * cs), w2 = exp2f((mo - mn) * cs);
        A = A * w1 + Ao * w2;
        W = W * w1 + Wo * w2;
      }
      m = mn;
    }
    const int r = row0 + (i >> 1) * 16 + (i & 1) * 8 + gp;
    if (c == 0 && r < M) {
      const int g = r / T, t = r - g * T;
      const long long rowid = (((long long)l * s.batch + b) * s.n_q_heads + h * G + g) * T + t;
      float* stp = a.stats + (rowid * a.n_splits + sp) * 3;
      stp[0] = m * cs;  // log2 domain, as the merge kernel expects (-inf when the split saw no key)
      stp[1] = A;
      stp[2] = W;
    }
  }
}

bool scores_mma_supported(const lt_shape& s, int /*w_last*/) { return s.dtype == LT_BF16 && s.head_dim == 128; }

cudaError_t launch_scores_mma(const ScoreArgs& a, const LayerTable& kf, cudaStream_t st) {
  const int G = a.s.n_q_heads / a.s.n_kv_heads;
  const int M = G * a.w_last;
  const int row_blocks = (M + kRowsPerCta - 1) / kRowsPerCta;
  constexpr int smem = kStages * kStageBytes;
  cudaError_t e = cudaFuncSetAttribute(scores_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  dim3 grid(a.n_splits * row_blocks, a.s.batch * a.s.n_kv_heads, a.s.n_layers);
  scores_mma_kernel<<<grid, kWarps * 32, smem, st>>>(a, kf);
  return cudaGetLastError();
}

}  // namespace lt
