// Decode attention, bandwidth path: bf16, head_dim 128, GQA group <= 8.
//
// One CTA per (layer, batch row, kv head, KV chunk) serves every query head of
// the group, so each cached K and V byte is read from HBM exactly once per step.
// Each warp streams its own tiles of the chunk through a private multi-stage
// cp.async ring in shared memory (16-byte vectors, fully coalesced rows, XOR
// swizzle of the 16-byte column so that ldmatrix is conflict-free) and needs no
// CTA-wide barrier until the final merge.
//
// Tensor-core mapping (mma.sync m16n8k16, bf16 in, fp32 accumulate):
//   S^T[key][head]  = K[key][d] . Q^T[d][head]      keys are M (16), heads are N (8)
//   O^T[d][head]   += V^T[d][key] . P[key][head]    d is M (8 tiles), keys are K
// K is the A operand through ldmatrix, V^T through ldmatrix.trans, Q sits in
// registers for the whole chunk, and P moves from the accumulator layout to the
// B layout with one movmatrix per 8x8 block.  P is split into a bf16 head and a
// bf16 residual (two MMAs) so that the probabilities keep ~16 bits.
#include <cuda_bf16.h>

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
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}
// lower 16 bits <- lo, upper <- hi
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

constexpr int kD = 128;
constexpr int kRowBytes = kD * 2;  // one K or V row

}  // namespace

// Shared memory of one warp and one stage: K half-tiles [2][TILE][128 B] then V
// half-tiles [2][TILE][128 B]; inside a half-tile the 16-byte column c of row r
// sits at column c ^ (r & 7).
template <int TILE, int NSTAGE, int WARPS, int MINB>
__global__ void __launch_bounds__(WARPS * 32, MINB)
    decode_mma_kernel(DecodeArgs a, LayerTable kf, LayerTable vf, LayerTable ks, LayerTable vs) {
  constexpr int MT = TILE / 16;                // 16-key MMA tiles per pipeline tile
  constexpr int HALF_BYTES = TILE * 128;       // one half-tile
  constexpr int STAGE_BYTES = 4 * HALF_BYTES;  // K halves + V halves
  extern __shared__ __align__(1024) uint8_t smem[];

  const lt_shape& s = a.s;
  const int l = a.layer_begin + blockIdx.z;
  const int bh = blockIdx.y;
  const int b = bh / s.n_kv_heads, h = bh - b * s.n_kv_heads;
  const int G = s.n_q_heads / s.n_kv_heads;
  const bool lazy = a.mask[l] != 0;
  const uint8_t* K = (const uint8_t*)(lazy ? ks.p[l] : kf.p[l]);
  const uint8_t* V = (const uint8_t*)(lazy ? vs.p[l] : vf.p[l]);
  const int rows = lazy ? s.n_sink + s.n_recent : s.full_capacity;
  int n = a.seq_lens[b];
  if (!K || !V) {
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(a.dev_err, LT_DEVERR_NULL_LAYER);
    return;
  }
  if (n > rows) {
    if (!lazy && threadIdx.x == 0 && blockIdx.x == 0) atomicOr(a.dev_err, LT_DEVERR_LEN_CLAMPED);
    n = rows;
  }
  if (n > a.n_chunks_launch * a.chunk_keys) {
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(a.dev_err, LT_DEVERR_LEN_CLAMPED);
    n = a.n_chunks_launch * a.chunk_keys;
  }
  const int j0 = blockIdx.x * a.chunk_keys;
  const int j1 = min(n, j0 + a.chunk_keys);
  if (j0 >= j1) return;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gp = lane >> 2, c = lane & 3;  // fragment row / column-pair index
  const uint8_t* Kb = K + (long long)bh * rows * kRowBytes;
  const uint8_t* Vb = V + (long long)bh * rows * kRowBytes;
  const uint32_t wsm = smem_u32(smem) + warp * (NSTAGE * STAGE_BYTES);

  // Q fragments (B operand of S^T = K Q^T): head gp, d = 16*ks + 2c (+8)
  uint32_t qf[8][2];
  {
    const __nv_bfloat16* qp =
        (const __nv_bfloat16*)a.q + (((long long)l * s.batch + b) * s.n_q_heads + h * G + gp) * kD;
#pragma unroll
    for (int ks8 = 0; ks8 < 8; ++ks8) {
      if (gp < G) {
        qf[ks8][0] = *reinterpret_cast<const uint32_t*>(qp + 16 * ks8 + 2 * c);
        qf[ks8][1] = *reinterpret_cast<const uint32_t*>(qp + 16 * ks8 + 8 + 2 * c);
      } else {
        qf[ks8][0] = 0u;
        qf[ks8][1] = 0u;
      }
    }
  }

  const int n_tiles = (j1 - j0 + TILE - 1) / TILE;  // tiles of this chunk
  // warp w owns tiles w, w + WARPS, ...
  auto issue_tile = [&](int my_idx) {
    const int t = warp + my_idx * WARPS;
    if (t < n_tiles) {
      const int key_base = j0 + t * TILE;
      const uint32_t st = wsm + (my_idx % NSTAGE) * STAGE_BYTES;
#pragma unroll
      for (int i = 0; i < TILE / 2; ++i) {
        const int r = 2 * i + (lane >> 4);
        const int p = lane & 15;
        const int row = key_base + r;
        const bool valid = row < j1;
        const long long goff = (long long)(valid ? row : (j1 - 1)) * kRowBytes + p * 16;
        const uint32_t soff = (p >> 3) * HALF_BYTES + r * 128 + (((p & 7) ^ (r & 7)) << 4);
        cp_async16(st + soff, Kb + goff, valid ? 16 : 0);
        cp_async16(st + 2 * HALF_BYTES + soff, Vb + goff, valid ? 16 : 0);
      }
    }
    cp_async_commit();
  };

  float o[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) o[i][j] = 0.f;
  float M0 = -INFINITY, M1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // heads 2c and 2c+1

  const int my_tiles = (n_tiles > warp) ? (n_tiles - warp + WARPS - 1) / WARPS : 0;
#pragma unroll
  for (int i = 0; i < NSTAGE - 1; ++i) issue_tile(i);

  // lane-constant parts of the ldmatrix addresses
  const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8;  // K (A operand, not transposed)
  const int k_chk = lane >> 4;
  const int v_row = (lane & 7) + ((lane >> 4) & 1) * 8;  // V (A operand, transposed)
  const int v_chk = (lane >> 3) & 1;

  for (int it = 0; it < my_tiles; ++it) {
    __syncwarp();              // every lane is done reading the stage that is refilled next
    issue_tile(it + NSTAGE - 1);
    cp_async_wait<NSTAGE - 1>();
    __syncwarp();              // all lanes' copies of tile `it` have landed
    const uint32_t st = wsm + (it % NSTAGE) * STAGE_BYTES;
    const int key_base = j0 + (warp + it * WARPS) * TILE;

    // ---- S^T = K Q^T ------------------------------------------------------
    float sc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      sc[mt][0] = sc[mt][1] = sc[mt][2] = sc[mt][3] = 0.f;
      const int row = mt * 16 + k_row;
#pragma unroll
      for (int ks8 = 0; ks8 < 8; ++ks8) {
        uint32_t af[4];
        const int chunk = 2 * (ks8 & 3) + k_chk;
        ldmatrix_x4(af, st + (ks8 >> 2) * HALF_BYTES + row * 128 + ((chunk ^ (row & 7)) << 4));
        mma_bf16(sc[mt], af, qf[ks8][0], qf[ks8][1]);
      }
    }
    // ---- scale, mask the ragged tail, tile max per head ---------------------
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const int key_lo = key_base + mt * 16 + gp;
      const bool v_lo = key_lo < j1, v_hi = key_lo + 8 < j1;
      sc[mt][0] = v_lo ? sc[mt][0] * a.cs : -INFINITY;
      sc[mt][1] = v_lo ? sc[mt][1] * a.cs : -INFINITY;
      sc[mt][2] = v_hi ? sc[mt][2] * a.cs : -INFINITY;
      sc[mt][3] = v_hi ? sc[mt][3] * a.cs : -INFINITY;
      mx0 = fmaxf(mx0, fmaxf(sc[mt][0], sc[mt][2]));
      mx1 = fmaxf(mx1, fmaxf(sc[mt][1], sc[mt][3]));
    }
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
    }
    const float Mn0 = fmaxf(M0, mx0), Mn1 = fmaxf(M1, mx1);
    const float corr0 = exp2f(M0 - Mn0), corr1 = exp2f(M1 - Mn1);
    M0 = Mn0;
    M1 = Mn1;
    l0 *= corr0;
    l1 *= corr1;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      o[i][0] *= corr0;
      o[i][1] *= corr1;
      o[i][2] *= corr0;
      o[i][3] *= corr1;
    }
    // ---- P = 2^(t - M), O^T += V^T P ---------------------------------------
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const float p0 = exp2f(sc[mt][0] - Mn0), p1 = exp2f(sc[mt][1] - Mn1);
      const float p2 = exp2f(sc[mt][2] - Mn0), p3 = exp2f(sc[mt][3] - Mn1);
      l0 += p0 + p2;
      l1 += p1 + p3;
      const uint32_t hi01 = pack_bf16(p0, p1), hi23 = pack_bf16(p2, p3);
      const uint32_t lo01 = pack_bf16(p0 - bf16_lo(hi01), p1 - bf16_hi(hi01));
      const uint32_t lo23 = pack_bf16(p2 - bf16_lo(hi23), p3 - bf16_hi(hi23));
      const uint32_t bh0 = movmatrix_trans(hi01), bh1 = movmatrix_trans(hi23);
      const uint32_t bl0 = movmatrix_trans(lo01), bl1 = movmatrix_trans(lo23);
      const int row = mt * 16 + v_row;
#pragma unroll
      for (int dt = 0; dt < 8; ++dt) {
        uint32_t af[4];
        const int chunk = 2 * (dt & 3) + v_chk;
        ldmatrix_x4_trans(af, st + 2 * HALF_BYTES + (dt >> 2) * HALF_BYTES + row * 128 + ((chunk ^ (row & 7)) << 4));
        mma_bf16(o[dt], af, bh0, bh1);
        mma_bf16(o[dt], af, bl0, bl1);
      }
    }
  }
  cp_async_wait<0>();

  // ---- warp totals, then merge the warps of the CTA through shared memory ----
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, off);
    l1 += __shfl_xor_sync(0xffffffffu, l1, off);
  }
  __syncthreads();  // every warp has drained its ring: the memory can be reused
  float* sm_m = reinterpret_cast<float*>(smem);  // [WARPS][8]
  float* sm_l = sm_m + WARPS * 8;                // [WARPS][8]
  float* sm_o = sm_l + WARPS * 8;                // [WARPS][8][128]
  if (gp == 0) {
    sm_m[warp * 8 + 2 * c] = M0;
    sm_m[warp * 8 + 2 * c + 1] = M1;
    sm_l[warp * 8 + 2 * c] = l0;
    sm_l[warp * 8 + 2 * c + 1] = l1;
  }
#pragma unroll
  for (int dt = 0; dt < 8; ++dt) {
    float* base = sm_o + (warp * 8 + 2 * c) * kD + dt * 16 + gp;
    base[0] = o[dt][0];
    base[kD] = o[dt][1];
    base[8] = o[dt][2];
    base[kD + 8] = o[dt][3];
  }
  __syncthreads();
  const long long unit = (((long long)l * s.batch + b) * s.n_kv_heads + h) * a.n_chunks_max + blockIdx.x;
  for (int idx = threadIdx.x; idx < G * kD; idx += WARPS * 32) {
    const int g = idx / kD, d = idx - g * kD;
    float Mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) Mx = fmaxf(Mx, sm_m[w * 8 + g]);
    float acc = 0.f, lsum = 0.f;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) {
      const float wgt = exp2f(sm_m[w * 8 + g] - Mx);
      acc += wgt * sm_o[(w * 8 + g) * kD + d];
      lsum += wgt * sm_l[w * 8 + g];
    }
    a.part_o[(unit * G + g) * kD + d] = acc;
    if (d == 0) {
      a.part_ml[(unit * G + g) * 2] = Mx;
      a.part_ml[(unit * G + g) * 2 + 1] = lsum;
    }
  }
}

bool decode_mma_supported(const lt_shape& s) {
  return s.dtype == LT_BF16 && s.head_dim == 128 && (s.n_q_heads / s.n_kv_heads) <= 8;
}

template <int TILE, int NSTAGE, int WARPS, int MINB>
static cudaError_t launch_variant(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf,
                                  const LayerTable& ks, const LayerTable& vs, cudaStream_t st) {
  constexpr int smem = WARPS * NSTAGE * TILE * 512;
  static_assert(smem >= WARPS * (16 + 8 * 128) * 4, "merge buffer must fit in the pipeline memory");
  auto kern = decode_mma_kernel<TILE, NSTAGE, WARPS, MINB>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  dim3 grid(a.n_chunks_launch, a.s.batch * a.s.n_kv_heads, a.layer_count);
  kern<<<grid, WARPS * 32, smem, st>>>(a, kf, vf, ks, vs);
  return cudaGetLastError();
}

cudaError_t launch_decode_mma(const DecodeArgs& a, const LayerTable& kf, const LayerTable& vf, const LayerTable& ks,
                              const LayerTable& vs, cudaStream_t st) {
  return launch_variant<16, 3, 4, 2>(a, kf, vf, ks, vs, st);
}

}  // namespace lt
