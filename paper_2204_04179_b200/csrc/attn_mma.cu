// Attention over short sequences (S <= 128 tokens, head width 32 or 64) with bf16 tensor-core
// products and fp32 softmax.  One block owns one (sequence, head): Q, K, V (and dO in the backward)
// live in shared memory (each once, row-major) for the whole block, a warp owns 16 query rows (forward, first half of the
// backward) or 16 key rows (second half of the backward), and score tiles never leave registers.
// The sequences are far shorter than a 128-row tcgen05 tile, and attention is ~2% of the encoder's
// flops, so this uses the warp-level m16n8k16 MMA; the kernel is bound by reading qkv once.
#include "layers.h"

namespace {

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float x, float y) {
  __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float quad_max(float v) {
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
  return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  return v + __shfl_xor_sync(0xffffffffu, v, 2);
}

// Fragment conventions of m16n8k16 (g = lane / 4, q = lane % 4):
//   A (16 x 16, row-major source X[m][k]):  a0 = X[g][2q..], a1 = X[g+8][2q..], a2 = X[g][2q+8..], a3 = X[g+8][2q+8..]
//   B (16 x 8, source stored as Y[n][k]):   b0 = Y[g][2q..], b1 = Y[g][2q+8..]
//   C (16 x 8):                             c0,c1 = C[g][2q, 2q+1], c2,c3 = C[g+8][2q, 2q+1]
// Where the contraction index is contiguous in shared memory (Q K^T, dO V^T) fragments are plain 32-bit
// loads.  Where it is the row index (P V, dS K, dS^T Q, P^T dO) the 8 x 8 tiles are read with
// ldmatrix.trans, so every matrix is kept once, row-major, with rows padded by 8 elements (conflict-free
// for both access kinds).

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, const bf16* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(smem_addr(p)));
}
__device__ __forceinline__ void ldsm_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, const bf16* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(smem_addr(p)));
}
// B fragments of two adjacent n-tiles (n0, n0+8) for the k-tile k0, from Y[n][k] (contraction index contiguous):
// (b0, b1) of tile n0 and (b2, b3) of tile n0 + 8
__device__ __forceinline__ void load_b_rows(const bf16* Y, int ld, int n0, int k0, int lane, uint32_t& b0, uint32_t& b1,
                                            uint32_t& b2, uint32_t& b3) {
  const int row = n0 + (lane & 7) + (lane >> 4) * 8, col = k0 + ((lane >> 3) & 1) * 8;
  ldsm_x4(b0, b1, b2, b3, Y + row * ld + col);
}
// A fragment (rows m0.., k-tile k0) of a row-major X[m][k]
__device__ __forceinline__ void load_a_rows(const bf16* X, int ld, int m0, int k0, int lane, uint32_t& a0, uint32_t& a1,
                                            uint32_t& a2, uint32_t& a3) {
  const int row = m0 + (lane & 7) + ((lane >> 3) & 1) * 8, col = k0 + (lane >> 4) * 8;
  ldsm_x4(a0, a1, a2, a3, X + row * ld + col);
}
// B fragments of two adjacent n-tiles (n0, n0+8) for the k-tile k0, from a row-major S[k][n] with row stride ld:
// (b0, b1) of tile n0 and (b2, b3) of tile n0 + 8
__device__ __forceinline__ void load_b_trans(const bf16* S, int ld, int k0, int n0, int lane, uint32_t& b0, uint32_t& b1,
                                             uint32_t& b2, uint32_t& b3) {
  const int row = k0 + (lane & 7) + ((lane >> 3) & 1) * 8, col = n0 + (lane >> 4) * 8;
  ldsm_x4_trans(b0, b1, b2, b3, S + row * ld + col);
}
// A fragment (m-tile m0, k-tile k0) of the transpose of a row-major S[k][m] with row stride ld
__device__ __forceinline__ void load_a_trans(const bf16* S, int ld, int k0, int m0, int lane, uint32_t& a0, uint32_t& a1,
                                             uint32_t& a2, uint32_t& a3) {
  const int row = k0 + (lane & 7) + (lane >> 4) * 8, col = m0 + ((lane >> 3) & 1) * 8;
  ldsm_x4_trans(a0, a1, a2, a3, S + row * ld + col);
}

// scores of 16 query rows against all SP keys: p[nt][0..3] for key tile nt, normalised probabilities on return.
// MASK = false: every key is visible to every row (S == SP, no causal mask), the per-element tests are left out.
// The 1/sqrt(dh) scale is folded into the exponent: exp(scale (s - max s)) = exp2(c s - c max s), c = scale log2(e).
// SKIP (causal launches): key tiles that no row of this query tile can see are not multiplied at all.
template <int SP, int DH, bool MASK, bool SKIP = false>
__device__ __forceinline__ void score_rows(const bf16* __restrict__ Qs, const bf16* __restrict__ Ks, int r0, int S, int causal,
                                           float scale, int g, int q, float (&p)[SP / 8][4]) {
  constexpr int LD = DH + 8;
#pragma unroll
  for (int nt = 0; nt < SP / 8; ++nt) p[nt][0] = p[nt][1] = p[nt][2] = p[nt][3] = 0.f;
  const int lane = g * 4 + q;
#pragma unroll
  for (int kt = 0; kt < DH / 16; ++kt) {
    uint32_t a0, a1, a2, a3;
    load_a_rows(Qs, LD, r0, kt * 16, lane, a0, a1, a2, a3);
#pragma unroll
    for (int nt = 0; nt < SP / 8; nt += 2) {
      if (!SKIP || nt * 8 <= r0 + 15) {        // later keys are masked for every row of the tile: their scores stay 0, then -inf
        uint32_t b0, b1, b2, b3;
        load_b_rows(Ks, LD, nt * 8, kt * 16, lane, b0, b1, b2, b3);
        mma16816(p[nt], a0, a1, a2, a3, b0, b1);
        mma16816(p[nt + 1], a0, a1, a2, a3, b2, b3);
      }
    }
  }
  const int i0 = r0 + g, i1 = r0 + g + 8;
  float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
  for (int nt = 0; nt < SP / 8; ++nt) {
    if (MASK) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int j = nt * 8 + 2 * q + (e & 1);
        const int i = (e < 2) ? i0 : i1;
        const bool ok = j < S && (!causal || j <= i);
        if (!ok) p[nt][e] = -INFINITY;
      }
    }
    m0 = fmaxf(m0, fmaxf(p[nt][0], p[nt][1]));
    m1 = fmaxf(m1, fmaxf(p[nt][2], p[nt][3]));
  }
  m0 = quad_max(m0);
  m1 = quad_max(m1);
  if (m0 == -INFINITY) m0 = 0.f;        // no key is visible to this (padded) row
  if (m1 == -INFINITY) m1 = 0.f;
  const float c = scale * 1.4426950408889634f;
  const float mc0 = m0 * c, mc1 = m1 * c;
  float l0 = 0.f, l1 = 0.f;
#pragma unroll
  for (int nt = 0; nt < SP / 8; ++nt) {
    p[nt][0] = fast_exp2(fmaf(p[nt][0], c, -mc0)); p[nt][1] = fast_exp2(fmaf(p[nt][1], c, -mc0));
    p[nt][2] = fast_exp2(fmaf(p[nt][2], c, -mc1)); p[nt][3] = fast_exp2(fmaf(p[nt][3], c, -mc1));
    l0 += p[nt][0] + p[nt][1];
    l1 += p[nt][2] + p[nt][3];
  }
  l0 = quad_sum(l0);
  l1 = quad_sum(l1);
  const float r0i = l0 > 0.f ? 1.f / l0 : 0.f, r1i = l1 > 0.f ? 1.f / l1 : 0.f;
#pragma unroll
  for (int nt = 0; nt < SP / 8; ++nt) {
    p[nt][0] *= r0i; p[nt][1] *= r0i;
    p[nt][2] *= r1i; p[nt][3] *= r1i;
  }
}

// rows [0, S) of one head's slice of a [tokens, ld] bf16 matrix -> shared memory, row-major; rows S..SP-1 are zero.
// The copies are asynchronous (16 bytes each, no registers in between): loads_done() before the tile is read.
template <int SP, int DH>
__device__ __forceinline__ void load_head(const bf16* __restrict__ src, int64_t ld, int S, bf16* __restrict__ dst) {
  constexpr int LD = DH + 8;
  for (int i = threadIdx.x; i < SP * (DH / 8); i += blockDim.x) {
    const int s = i / (DH / 8), c = (i - s * (DH / 8)) * 8;
    if (s < S) {
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst + s * LD + c)), "l"(src + (int64_t)s * ld + c)
                   : "memory");
    } else {
      *reinterpret_cast<uint4*>(dst + s * LD + c) = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}
__device__ __forceinline__ void loads_done() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
  __syncthreads();
}
// rows [row_begin, row_end) (below S) of a shared-memory tile -> one head's slice of a [tokens, ld] matrix, 16 bytes
// per thread, whole 128-byte (64-byte for DH = 32) row pieces per eight (four) threads
template <int DH>
__device__ __forceinline__ void store_rows(const bf16* __restrict__ src, int row_begin, int row_end, int S, bf16* __restrict__ dst,
                                           int64_t ld, int tid, int nthreads) {
  constexpr int LD = DH + 8;
  if (row_end > S) row_end = S;
  for (int i = tid; i < (row_end - row_begin) * (DH / 8); i += nthreads) {
    const int s = row_begin + i / (DH / 8), c = (i % (DH / 8)) * 8;
    *reinterpret_cast<uint4*>(dst + (int64_t)s * ld + c) = *reinterpret_cast<const uint4*>(src + s * LD + c);
  }
}
// the C-layout registers of a 16 x DH tile (rows r0 + g and r0 + g + 8) -> bf16 in a shared-memory tile
template <int DH>
__device__ __forceinline__ void stage_tile(const float (&o)[DH / 8][4], bf16* __restrict__ dst, int r0, int g, int q) {
  constexpr int LD = DH + 8;
#pragma unroll
  for (int nt = 0; nt < DH / 8; ++nt) {
    const int c = nt * 8 + 2 * q;
    *reinterpret_cast<uint32_t*>(dst + (r0 + g) * LD + c) = pack2(o[nt][0], o[nt][1]);
    *reinterpret_cast<uint32_t*>(dst + (r0 + g + 8) * LD + c) = pack2(o[nt][2], o[nt][3]);
  }
}

// acc[nt] += A(16 x SP, from the C-layout registers x) * S[k][n] (row-major, SP x DH)
// LIMIT: the columns of x from n_rows on are zero (keys a causal tile cannot see), their 16-row tiles are skipped.
template <int SP, int DH, bool LIMIT = false>
__device__ __forceinline__ void mma_regs_times_rows(const float (&x)[SP / 8][4], const bf16* S, int lane,
                                                    float (&acc)[DH / 8][4], int n_rows = 0) {
  constexpr int LD = DH + 8;
#pragma unroll
  for (int kt = 0; kt < SP / 16; ++kt) {
    if (LIMIT && kt * 16 >= n_rows) continue;
    const uint32_t a0 = pack2(x[2 * kt][0], x[2 * kt][1]), a1 = pack2(x[2 * kt][2], x[2 * kt][3]);
    const uint32_t a2 = pack2(x[2 * kt + 1][0], x[2 * kt + 1][1]), a3 = pack2(x[2 * kt + 1][2], x[2 * kt + 1][3]);
#pragma unroll
    for (int nt = 0; nt < DH / 8; nt += 2) {
      uint32_t b0, b1, b2, b3;
      load_b_trans(S, LD, kt * 16, nt * 8, lane, b0, b1, b2, b3);
      mma16816(acc[nt], a0, a1, a2, a3, b0, b1);
      mma16816(acc[nt + 1], a0, a1, a2, a3, b2, b3);
    }
  }
}

// NW warps per block; CAUSAL launches skip the tiles above the diagonal.
template <int SP, int DH, int NW, bool CAUSAL>
__global__ void __launch_bounds__(NW * 32) attn_fwd_mma_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ out, int S, int d,
                                                           int n_heads, int causal, float scale,
                                                           const int32_t* __restrict__ seq_len,
                                                           const int32_t* __restrict__ seq_off,
                                                           const int32_t* __restrict__ seq_list) {
  constexpr int LD = DH + 8;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  bf16* Qs = reinterpret_cast<bf16*>(smem_raw);
  bf16* Ks = Qs + SP * LD;
  bf16* Vs = Ks + SP * LD;
  const int64_t seq = seq_list ? seq_list[blockIdx.x / n_heads] : blockIdx.x / n_heads;   // this launch's share of the sequences
  const int h = blockIdx.x % n_heads;
  int64_t row0 = seq * S;
  if (seq_off) {                                  // packed rows: this sequence is rows seq_off .. + seq_len, no padding
    row0 = seq_off[seq];
    S = seq_len[seq];
  }
  const bf16* base = qkv + row0 * 3 * (int64_t)d + h * DH;
  load_head<SP, DH>(base, 3 * (int64_t)d, S, Qs);
  load_head<SP, DH>(base + d, 3 * (int64_t)d, S, Ks);
  load_head<SP, DH>(base + 2 * d, 3 * (int64_t)d, S, Vs);
  loads_done();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, q = lane & 3;
  bf16* ob = out + row0 * (int64_t)d + h * DH;
  const int Sv = seq_len ? seq_len[seq] : S;      // keys that are text; the rows after them are padding
  for (int r0 = warp * 16; r0 < S; r0 += NW * 16) {
    float p[SP / 8][4];
    if (!CAUSAL && Sv == SP) score_rows<SP, DH, false>(Qs, Ks, r0, Sv, causal, scale, g, q, p);
    else score_rows<SP, DH, true, CAUSAL>(Qs, Ks, r0, Sv, causal, scale, g, q, p);
    float o[DH / 8][4];
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    mma_regs_times_rows<SP, DH, CAUSAL>(p, Vs, lane, o, r0 + 16);              // O = P V
    // the 16 rows of Q are this warp's alone and no longer needed: O goes through them so that it leaves in whole rows
    __syncwarp();
    stage_tile<DH>(o, Qs, r0, g, q);
    __syncwarp();
    store_rows<DH>(Qs, r0, r0 + 16, S, ob, d, lane, 32);
  }
}

template <int SP, int DH, int NW, bool CAUSAL>
__global__ void __launch_bounds__(NW * 32) attn_bwd_mma_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ dctx,
                                                           bf16* __restrict__ dqkv, float* __restrict__ colpart, int S, int d,
                                                           int n_heads, int causal, float scale,
                                                           const int32_t* __restrict__ seq_len,
                                                           const int32_t* __restrict__ seq_off,
                                                           const int32_t* __restrict__ seq_list) {
  constexpr int LD = DH + 8, LP = SP + 8;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  bf16* Qs = reinterpret_cast<bf16*>(smem_raw);   // [SP][DH+8]
  bf16* Ks = Qs + SP * LD;
  bf16* Vs = Ks + SP * LD;
  bf16* dOs = Vs + SP * LD;
  bf16* Ps = dOs + SP * LD;                       // [query i][key j], [SP][SP+8]
  bf16* dSs = Ps + SP * LP;
  const int64_t seq = seq_list ? seq_list[blockIdx.x / n_heads] : blockIdx.x / n_heads;
  const int h = blockIdx.x % n_heads;
  int64_t row0 = seq * S;
  if (seq_off) {
    row0 = seq_off[seq];
    S = seq_len[seq];
  }
  const bf16* base = qkv + row0 * 3 * (int64_t)d + h * DH;
  load_head<SP, DH>(base, 3 * (int64_t)d, S, Qs);
  load_head<SP, DH>(base + d, 3 * (int64_t)d, S, Ks);
  load_head<SP, DH>(base + 2 * d, 3 * (int64_t)d, S, Vs);
  load_head<SP, DH>(dctx + row0 * (int64_t)d + h * DH, d, S, dOs);
  loads_done();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, q = lane & 3;
  bf16* dq = dqkv + row0 * 3 * (int64_t)d + h * DH;
  const int Sv = seq_len ? seq_len[seq] : S;
  // ---- first half: 16 query rows per warp: P, dS (kept in shared memory), dQ (kept in registers as bf16 pairs) ----
  constexpr int NIT = (SP + 16 * NW - 1) / (16 * NW);
  uint32_t dqp[NIT][DH / 8][2];
#pragma unroll
  for (int it = 0; it < NIT; ++it) {
    const int r0 = warp * 16 + it * (16 * NW);
    if (r0 < SP) {
      float p[SP / 8][4];
      if (!CAUSAL && Sv == SP) score_rows<SP, DH, false>(Qs, Ks, r0, Sv, causal, scale, g, q, p);
      else score_rows<SP, DH, true, CAUSAL>(Qs, Ks, r0, Sv, causal, scale, g, q, p);
      float dp[SP / 8][4];
#pragma unroll
      for (int nt = 0; nt < SP / 8; ++nt) dp[nt][0] = dp[nt][1] = dp[nt][2] = dp[nt][3] = 0.f;
#pragma unroll
      for (int kt = 0; kt < DH / 16; ++kt) {        // dP = dO V^T
        uint32_t a0, a1, a2, a3;
        load_a_rows(dOs, LD, r0, kt * 16, lane, a0, a1, a2, a3);
#pragma unroll
        for (int nt = 0; nt < SP / 8; nt += 2) {
          if (!CAUSAL || nt * 8 <= r0 + 15) {   // the probabilities of keys out of sight are zero: dP there is not needed
            uint32_t b0, b1, b2, b3;
            load_b_rows(Vs, LD, nt * 8, kt * 16, lane, b0, b1, b2, b3);
            mma16816(dp[nt], a0, a1, a2, a3, b0, b1);
            mma16816(dp[nt + 1], a0, a1, a2, a3, b2, b3);
          }
        }
      }
      float d0 = 0.f, d1 = 0.f;
#pragma unroll
      for (int nt = 0; nt < SP / 8; ++nt) {
        d0 += p[nt][0] * dp[nt][0] + p[nt][1] * dp[nt][1];
        d1 += p[nt][2] * dp[nt][2] + p[nt][3] * dp[nt][3];
      }
      d0 = quad_sum(d0);
      d1 = quad_sum(d1);
#pragma unroll
      for (int nt = 0; nt < SP / 8; ++nt) {         // dS = P (dP - delta) / sqrt(dh)
        dp[nt][0] = p[nt][0] * (dp[nt][0] - d0) * scale; dp[nt][1] = p[nt][1] * (dp[nt][1] - d0) * scale;
        dp[nt][2] = p[nt][2] * (dp[nt][2] - d1) * scale; dp[nt][3] = p[nt][3] * (dp[nt][3] - d1) * scale;
        const int j = nt * 8 + 2 * q;
        *reinterpret_cast<uint32_t*>(Ps + (r0 + g) * LP + j) = pack2(p[nt][0], p[nt][1]);
        *reinterpret_cast<uint32_t*>(Ps + (r0 + g + 8) * LP + j) = pack2(p[nt][2], p[nt][3]);
        *reinterpret_cast<uint32_t*>(dSs + (r0 + g) * LP + j) = pack2(dp[nt][0], dp[nt][1]);
        *reinterpret_cast<uint32_t*>(dSs + (r0 + g + 8) * LP + j) = pack2(dp[nt][2], dp[nt][3]);
      }
      float o[DH / 8][4];
#pragma unroll
      for (int nt = 0; nt < DH / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
      mma_regs_times_rows<SP, DH, CAUSAL>(dp, Ks, lane, o, r0 + 16);             // dQ = dS K
#pragma unroll
      for (int nt = 0; nt < DH / 8; ++nt) {
        dqp[it][nt][0] = pack2(o[nt][0], o[nt][1]);
        dqp[it][nt][1] = pack2(o[nt][2], o[nt][3]);
      }
    }
  }
  __syncthreads();
  // ---- second half: 16 key rows per warp: dK = dS^T Q, dV = P^T dO; K and V are no longer read, so the results
  // ---- replace this warp's rows of them
  for (int j0 = warp * 16; j0 < S; j0 += NW * 16) {
    float dk[DH / 8][4], dv[DH / 8][4];
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) {
      dk[nt][0] = dk[nt][1] = dk[nt][2] = dk[nt][3] = 0.f;
      dv[nt][0] = dv[nt][1] = dv[nt][2] = dv[nt][3] = 0.f;
    }
#pragma unroll
    for (int kt = 0; kt < SP / 16; ++kt) {        // contraction over query rows i = kt*16 ..
      if (CAUSAL && kt * 16 + 15 < j0) continue;  // queries before these keys cannot see them: P and dS are zero there
      uint32_t s0, s1, s2, s3, p0, p1, p2, p3;
      load_a_trans(dSs, LP, kt * 16, j0, lane, s0, s1, s2, s3);
      load_a_trans(Ps, LP, kt * 16, j0, lane, p0, p1, p2, p3);
#pragma unroll
      for (int nt = 0; nt < DH / 8; nt += 2) {
        uint32_t b0, b1, b2, b3;
        load_b_trans(Qs, LD, kt * 16, nt * 8, lane, b0, b1, b2, b3);
        mma16816(dk[nt], s0, s1, s2, s3, b0, b1);
        mma16816(dk[nt + 1], s0, s1, s2, s3, b2, b3);
        load_b_trans(dOs, LD, kt * 16, nt * 8, lane, b0, b1, b2, b3);
        mma16816(dv[nt], p0, p1, p2, p3, b0, b1);
        mma16816(dv[nt + 1], p0, p1, p2, p3, b2, b3);
      }
    }
    stage_tile<DH>(dk, Ks, j0, g, q);
    stage_tile<DH>(dv, Vs, j0, g, q);
  }
  __syncthreads();                                 // Q is no longer read either: dQ replaces it
#pragma unroll
  for (int it = 0; it < NIT; ++it) {
    const int r0 = warp * 16 + it * (16 * NW);
    if (r0 < SP) {
#pragma unroll
      for (int nt = 0; nt < DH / 8; ++nt) {
        const int c = nt * 8 + 2 * q;
        *reinterpret_cast<uint32_t*>(Qs + (r0 + g) * LD + c) = dqp[it][nt][0];
        *reinterpret_cast<uint32_t*>(Qs + (r0 + g + 8) * LD + c) = dqp[it][nt][1];
      }
    }
  }
  __syncthreads();
  store_rows<DH>(Qs, 0, S, S, dq, 3 * (int64_t)d, threadIdx.x, blockDim.x);
  store_rows<DH>(Ks, 0, S, S, dq + d, 3 * (int64_t)d, threadIdx.x, blockDim.x);
  store_rows<DH>(Vs, 0, S, S, dq + 2 * d, 3 * (int64_t)d, threadIdx.x, blockDim.x);
  if (colpart) {
    // column sums of the three gradient tiles as stored (bf16), rows in ascending order: row `seq` of the partial
    // sums of the bias gradient of the Q, K, V projection
    for (int c = threadIdx.x; c < 3 * DH; c += blockDim.x) {
      const int which = c / DH, col = c - which * DH;
      const bf16* M = Qs + which * (SP * LD) + col;
      float a = 0.f;
      for (int r = 0; r < S; ++r) a += __bfloat162float(M[r * LD]);
      colpart[seq * 3 * (int64_t)d + which * d + h * DH + col] = a;
    }
  }
}

template <int SP, int DH>
gram_status launch_fwd(gram_ctx* ctx, const bf16* qkv, bf16* out, int64_t n_seq, int S, int d, int n_heads, int causal,
                       const int32_t* seq_len, const int32_t* seq_off, const int32_t* seq_list, cudaStream_t st) {
  constexpr size_t smem = (size_t)3 * SP * (DH + 8) * 2;
  constexpr int NW = SP >= 96 ? 8 : 4;                // one 16-row query tile per warp up to 128 rows
  auto kern = causal ? attn_fwd_mma_kernel<SP, DH, NW, true> : attn_fwd_mma_kernel<SP, DH, NW, false>;
  if (smem > 48 * 1024) GRAM_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<(unsigned)(n_seq * n_heads), NW * 32, smem, st>>>(qkv, out, S, d, n_heads, causal, 1.f / sqrtf((float)DH), seq_len, seq_off, seq_list);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
template <int SP, int DH>
gram_status launch_bwd(gram_ctx* ctx, const bf16* qkv, const bf16* dctx, bf16* dqkv, float* colpart, int64_t n_seq, int S, int d,
                       int n_heads, int causal, const int32_t* seq_len, const int32_t* seq_off, const int32_t* seq_list,
                       cudaStream_t st) {
  constexpr size_t smem = ((size_t)4 * SP * (DH + 8) + (size_t)2 * SP * (SP + 8)) * 2;
  static_assert(smem <= 227 * 1024, "attention backward tile exceeds shared memory");
  constexpr int NW = SP >= 96 ? 8 : 4;
  auto kern = causal ? attn_bwd_mma_kernel<SP, DH, NW, true> : attn_bwd_mma_kernel<SP, DH, NW, false>;
  if (smem > 48 * 1024) GRAM_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<(unsigned)(n_seq * n_heads), NW * 32, smem, st>>>(qkv, dctx, dqkv, colpart, S, d, n_heads, causal, 1.f / sqrtf((float)DH), seq_len, seq_off, seq_list);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

}  // namespace

bool attention_mma_supported(int S, int d, int n_heads) {
  const int dh = n_heads > 0 ? d / n_heads : 0;
  return S >= 1 && S <= 128 && (dh == 32 || dh == 64) && dh * n_heads == d && d % 8 == 0;
}

#define ATTN_DISPATCH(FN, ...)                                                      \
  do {                                                                              \
    const int dh = d / n_heads;                                                     \
    if (dh == 64) {                                                                 \
      if (S <= 32) return FN<32, 64>(__VA_ARGS__);                                  \
      if (S <= 64) return FN<64, 64>(__VA_ARGS__);                                  \
      if (S <= 96) return FN<96, 64>(__VA_ARGS__);                                  \
      return FN<128, 64>(__VA_ARGS__);                                              \
    } else {                                                                        \
      if (S <= 32) return FN<32, 32>(__VA_ARGS__);                                  \
      if (S <= 64) return FN<64, 32>(__VA_ARGS__);                                  \
      if (S <= 96) return FN<96, 32>(__VA_ARGS__);                                  \
      return FN<128, 32>(__VA_ARGS__);                                              \
    }                                                                               \
  } while (0)

gram_status attention_forward_mma(gram_ctx* ctx, const void* qkv, void* out, int64_t n_seq, int S, int d, int n_heads,
                                  int causal, const int32_t* seq_len, const int32_t* seq_off, const int32_t* seq_list,
                                  cudaStream_t st) {
  ATTN_DISPATCH(launch_fwd, ctx, (const bf16*)qkv, (bf16*)out, n_seq, S, d, n_heads, causal, seq_len, seq_off, seq_list, st);
}
gram_status attention_backward_mma(gram_ctx* ctx, const void* qkv, const void* dctx, void* dqkv, float* colpart, int64_t n_seq,
                                   int S, int d, int n_heads, int causal, const int32_t* seq_len, const int32_t* seq_off,
                                   const int32_t* seq_list, cudaStream_t st) {
  ATTN_DISPATCH(launch_bwd, ctx, (const bf16*)qkv, (const bf16*)dctx, (bf16*)dqkv, colpart, n_seq, S, d, n_heads, causal, seq_len, seq_off, seq_list, st);
}
