// Non-GEMM layers: embedding, LayerNorm, attention over short sequences, pooling, bias-gradient
// column sums, the task heads.  All reductions that feed parameter gradients run in a fixed order
// (per-warp registers -> ordered block sum -> ordered sum over blocks), so results are bit-stable.
#include "gemm.h"
#include "layers.h"

namespace {

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const bf16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(bf16* p, float v) { *p = __float2bfloat16(v); }
__device__ __forceinline__ float2 ld2(const float* p) { return *reinterpret_cast<const float2*>(p); }
__device__ __forceinline__ float2 ld2(const bf16* p) {
  return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
}
__device__ __forceinline__ void st2(float* p, float2 v) { *reinterpret_cast<float2*>(p) = v; }
__device__ __forceinline__ void st2(bf16* p, float2 v) {
  *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(v.x, v.y);
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ---------------------------------------------------------------------------- embedding
__global__ void embed_fwd_kernel(const int32_t* __restrict__ item_tokens, const int32_t* __restrict__ items,
                                 int32_t first_item, int64_t n_tok, int32_t n_items_total, int l_t, int vocab, int d,
                                 const float* __restrict__ tok_emb, const float* __restrict__ pos_emb,
                                 float* __restrict__ z0, int32_t* __restrict__ tok_ids,
                                 const int32_t* __restrict__ seq_len, const int32_t* __restrict__ seq_off, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nw = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t t = w; t < n_tok; t += nw) {
    const int64_t u = t / l_t;
    const int s = (int)(t - u * l_t);
    int32_t item = items ? items[u] : first_item + (int32_t)u;
    if (item < 0 || item >= n_items_total) { gram_device_fail(status, GRAM_ERR_ID_RANGE); item = 0; }
    int32_t tok = item_tokens[(int64_t)item * l_t + s];
    if (tok < 0 || tok >= vocab) { gram_device_fail(status, GRAM_ERR_ID_RANGE); tok = 0; }
    int64_t row = t;
    if (seq_off) {                               // packed rows: item u owns rows seq_off[u] .. + seq_len[u], no padding
      if (s >= seq_len[u]) continue;
      row = (int64_t)seq_off[u] + s;
    }
    if (lane == 0) tok_ids[row] = tok;
    const float* te = tok_emb + (int64_t)tok * d;
    const float* pe = pos_emb + (int64_t)s * d;
    for (int c = 2 * lane; c < d; c += 64) {
      float2 a = ld2(te + c), b = ld2(pe + c);
      st2(z0 + row * d + c, make_float2(a.x + b.x, a.y + b.y));
    }
  }
}

// ---------------------------------------------------------------------------- LayerNorm
__device__ __forceinline__ float4 ld4f(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void st4t(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void st4t(bf16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
}

// a warp per row; lane l owns columns 4*(l + 32*i) .. +3 for i < NQ (d <= 128*NQ, d % 4 == 0)
template <typename T, int NQ>
__global__ void __launch_bounds__(256) ln_fwd_kernel(const float* __restrict__ z, const float* __restrict__ g,
                                                     const float* __restrict__ b, T* __restrict__ y,
                                                     float* __restrict__ mean, float* __restrict__ rstd, int64_t rows,
                                                     int d) {
  const int lane = threadIdx.x & 31;
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nw = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t r = w; r < rows; r += nw) {
    float4 v[NQ];
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < NQ; ++i) {
      const int c = 4 * (lane + 32 * i);
      v[i] = (c < d) ? ld4f(z + r * d + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
    }
    const float mu = warp_sum(s) / d;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < NQ; ++i) {
      const int c = 4 * (lane + 32 * i);
      if (c < d) {
        const float a0 = v[i].x - mu, a1 = v[i].y - mu, a2 = v[i].z - mu, a3 = v[i].w - mu;
        q += (a0 * a0 + a1 * a1) + (a2 * a2 + a3 * a3);
      }
    }
    const float rs = rsqrtf(warp_sum(q) / d + kLnEps);
#pragma unroll
    for (int i = 0; i < NQ; ++i) {
      const int c = 4 * (lane + 32 * i);
      if (c < d) {
        const float4 gg = ld4f(g + c), bb = ld4f(b + c);
        st4t(y + r * d + c, make_float4((v[i].x - mu) * rs * gg.x + bb.x, (v[i].y - mu) * rs * gg.y + bb.y,
                                        (v[i].z - mu) * rs * gg.z + bb.z, (v[i].w - mu) * rs * gg.w + bb.w));
      }
    }
    if (lane == 0) {
      mean[r] = mu;
      rstd[r] = rs;
    }
  }
}

template <typename T, int NQ>
__global__ void __launch_bounds__(256, 2) ln_bwd_kernel(const float* __restrict__ dy, const float* __restrict__ z,
                                                        const float* __restrict__ mean, const float* __restrict__ rstd,
                                                        const float* __restrict__ g, float* __restrict__ dz,
                                                        T* __restrict__ dz_b, float* __restrict__ part, int64_t rows,
                                                        int d, int want_col) {
  // [3][d]: dgamma, dbeta and the column sums of dz of this block; then [d]: gamma; then, when the column sums
  // are wanted, one float4 per (warp, i, lane): each thread's running column sums (registers are all taken)
  extern __shared__ float sacc[];
  float* sgam = sacc + 3 * d;
  float4* scol = reinterpret_cast<float4*>(sgam + d) + (threadIdx.x >> 5) * (NQ * 32) + (threadIdx.x & 31);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwb = blockDim.x >> 5;
  const int64_t w = (int64_t)blockIdx.x * nwb + warp;
  const int64_t nw = (int64_t)gridDim.x * nwb;
  for (int i = threadIdx.x; i < d; i += blockDim.x) sgam[i] = g[i];
  for (int i = threadIdx.x; i < 3 * d; i += blockDim.x) sacc[i] = 0.f;
  __syncthreads();
  float4 ag[NQ], ab[NQ];
#pragma unroll
  for (int i = 0; i < NQ; ++i) {
    ag[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    ab[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (want_col) scol[i * 32] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int64_t r = w; r < rows; r += nw) {
    const float mu = mean[r], rs = rstd[r];
    float4 xh[NQ], dd[NQ];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < NQ; ++i) {
      const int c = 4 * (lane + 32 * i);
      if (c < d) {
        const float4 zz = ld4f(z + r * d + c);
        dd[i] = ld4f(dy + r * d + c);
        xh[i] = make_float4((zz.x - mu) * rs, (zz.y - mu) * rs, (zz.z - mu) * rs, (zz.w - mu) * rs);
      } else {
        xh[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        dd[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int i = 0; i < NQ; ++i) {
      const int c = 4 * (lane + 32 * i);
      const float4 gg = (c < d) ? *reinterpret_cast<const float4*>(sgam + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      ag[i].x += dd[i].x * xh[i].x; ag[i].y += dd[i].y * xh[i].y; ag[i].z += dd[i].z * xh[i].z; ag[i].w += dd[i].w * xh[i].w;
      ab[i].x += dd[i].x; ab[i].y += dd[i].y; ab[i].z += dd[i].z; ab[i].w += dd[i].w;
      dd[i].x *= gg.x; dd[i].y *= gg.y; dd[i].z *= gg.z; dd[i].w *= gg.w;     // dy * gamma
      s1 += (dd[i].x + dd[i].y) + (dd[i].z + dd[i].w);
      s2 += (dd[i].x * xh[i].x + dd[i].y * xh[i].y) + (dd[i].z * xh[i].z + dd[i].w * xh[i].w);
    }
    s1 = warp_sum(s1) / d;
    s2 = warp_sum(s2) / d;
#pragma unroll
    for (int i = 0; i < NQ; ++i) {
      const int c = 4 * (lane + 32 * i);
      if (c < d) {
        const float4 o = make_float4(rs * (dd[i].x - s1 - xh[i].x * s2), rs * (dd[i].y - s1 - xh[i].y * s2),
                                     rs * (dd[i].z - s1 - xh[i].z * s2), rs * (dd[i].w - s1 - xh[i].w * s2));
        st4t(dz + r * d + c, o);
        if (dz_b) st4t(dz_b + r * d + c, o);
        if (want_col) {
          float4 t = scol[i * 32];
          t.x += o.x; t.y += o.y; t.z += o.z; t.w += o.w;
          scol[i * 32] = t;
        }
      }
    }
  }
  for (int ww = 0; ww < nwb; ++ww) {       // warps add in ascending order
    if (warp == ww) {
#pragma unroll
      for (int i = 0; i < NQ; ++i) {
        const int c = 4 * (lane + 32 * i);
        if (c < d) {
          sacc[c] += ag[i].x; sacc[c + 1] += ag[i].y; sacc[c + 2] += ag[i].z; sacc[c + 3] += ag[i].w;
          sacc[d + c] += ab[i].x; sacc[d + c + 1] += ab[i].y; sacc[d + c + 2] += ab[i].z; sacc[d + c + 3] += ab[i].w;
          if (want_col) {
            const float4 t = scol[i * 32];
            sacc[2 * d + c] += t.x; sacc[2 * d + c + 1] += t.y; sacc[2 * d + c + 2] += t.z; sacc[2 * d + c + 3] += t.w;
          }
        }
      }
    }
    __syncthreads();
  }
  for (int i = threadIdx.x; i < 3 * d; i += blockDim.x) part[(int64_t)blockIdx.x * 3 * d + i] = sacc[i];
}

// out[c] += scale * sum_b part[b*stride + c]   (two outputs when out2 != null: second half of each partial row).
// A block owns 32 columns; its 8 warps take the partial rows b = w, w+8, ... and their sums are added in
// ascending w, so the order of additions is fixed.
__global__ void __launch_bounds__(256) reduce_partials_kernel(const float* __restrict__ part, int nblocks, int64_t stride,
                                                              int n, float* __restrict__ out, float* __restrict__ out2,
                                                              float scale) {
  __shared__ float sa[8][32], sb[8][32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  float a = 0.f, b = 0.f;
  if (c < n) {
    for (int k = w; k < nblocks; k += 8) {
      a += part[(int64_t)k * stride + c];
      if (out2) b += part[(int64_t)k * stride + n + c];
    }
  }
  sa[w][lane] = a;
  sb[w][lane] = b;
  __syncthreads();
  if (w == 0 && c < n) {
    float ta = sa[0][lane], tb = sb[0][lane];
#pragma unroll
    for (int k = 1; k < 8; ++k) { ta += sa[k][lane]; tb += sb[k][lane]; }
    out[c] += ta * scale;
    if (out2) out2[c] += tb * scale;
  }
}

// ---------------------------------------------------------------------------- attention
// One block per (sequence, head).  Rows of Q, K, V live in shared memory as fp32 with a padded
// stride; a warp owns one query row at a time, with keys spread over lanes (S <= 128).
template <typename T>
__global__ void __launch_bounds__(128) attn_fwd_kernel(const T* __restrict__ qkv, T* __restrict__ out, int S, int d,
                                                       int n_heads, int causal, float scale,
                                                       const int32_t* __restrict__ seq_len,
                                                       const int32_t* __restrict__ seq_off) {
  extern __shared__ float sm[];
  const int dh = d / n_heads, ld = dh + 1;
  int64_t row0 = (int64_t)(blockIdx.x / n_heads) * S;
  if (seq_off) {                                  // packed rows: this sequence is rows seq_off .. + seq_len
    row0 = seq_off[blockIdx.x / n_heads];
    S = seq_len[blockIdx.x / n_heads];
  }
  float* Q = sm;
  float* K = Q + S * ld;
  float* V = K + S * ld;
  const int64_t seq = blockIdx.x / n_heads;
  const int h = blockIdx.x % n_heads;
  const int Sv = seq_len ? seq_len[seq] : S;          // keys that are text; rows past them are padding
  const T* base = qkv + row0 * 3 * (int64_t)d + h * dh;
  for (int i = threadIdx.x; i < S * dh; i += blockDim.x) {
    const int s = i / dh, c = i - s * dh;
    const T* p = base + (int64_t)s * 3 * d + c;
    Q[s * ld + c] = ldf(p);
    K[s * ld + c] = ldf(p + d);
    V[s * ld + c] = ldf(p + 2 * d);
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwb = blockDim.x >> 5;
  for (int i = warp; i < S; i += nwb) {
    float p[4];
    float m = -INFINITY;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int j = lane + 32 * jj;
      float sc = -INFINITY;
      if (j < Sv && (!causal || j <= i)) {
        float acc = 0.f;
        for (int c = 0; c < dh; ++c) acc += Q[i * ld + c] * K[j * ld + c];
        sc = acc * scale;
      }
      p[jj] = sc;
      m = fmaxf(m, sc);
    }
    m = warp_max(m);
    float l = 0.f;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      p[jj] = (p[jj] == -INFINITY) ? 0.f : __expf(p[jj] - m);
      l += p[jj];
    }
    l = warp_sum(l);
    const float inv = 1.f / l;
    const int jmax = min(causal ? i + 1 : S, Sv);
    float o0 = 0.f, o1 = 0.f;      // columns lane and lane + 32 (dh <= 64)
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      for (int l2 = 0; l2 < 32; ++l2) {
        const int j = jj * 32 + l2;
        if (j >= jmax) break;
        const float pj = __shfl_sync(0xffffffffu, p[jj], l2);
        if (lane < dh) o0 += pj * V[j * ld + lane];
        if (lane + 32 < dh) o1 += pj * V[j * ld + lane + 32];
      }
    }
    T* o = out + (row0 + i) * (int64_t)d + h * dh;
    if (lane < dh) stf(o + lane, o0 * inv);
    if (lane + 32 < dh) stf(o + lane + 32, o1 * inv);
  }
}

template <typename T>
__global__ void __launch_bounds__(128) attn_bwd_kernel(const T* __restrict__ qkv, const T* __restrict__ dctx,
                                                       T* __restrict__ dqkv, int S, int d, int n_heads, int causal,
                                                       float scale, const int32_t* __restrict__ seq_len,
                                                       const int32_t* __restrict__ seq_off) {
  extern __shared__ float sm[];
  int64_t row0 = (int64_t)(blockIdx.x / n_heads) * S;
  if (seq_off) {
    row0 = seq_off[blockIdx.x / n_heads];
    S = seq_len[blockIdx.x / n_heads];
  }
  const int dh = d / n_heads, ld = dh + 1, lp = S + 1;
  float* Q = sm;
  float* K = Q + S * ld;
  float* V = K + S * ld;
  float* dO = V + S * ld;
  float* Pm = dO + S * ld;       // [S][S+1] probabilities
  float* dS = Pm + S * lp;       // [S][S+1] gradient of the scaled scores
  const int64_t seq = blockIdx.x / n_heads;
  const int h = blockIdx.x % n_heads;
  const T* base = qkv + row0 * 3 * (int64_t)d + h * dh;
  const T* dbase = dctx + row0 * (int64_t)d + h * dh;
  const int Sv = seq_len ? seq_len[seq] : S;
  for (int i = threadIdx.x; i < S * dh; i += blockDim.x) {
    const int s = i / dh, c = i - s * dh;
    const T* p = base + (int64_t)s * 3 * d + c;
    Q[s * ld + c] = ldf(p);
    K[s * ld + c] = ldf(p + d);
    V[s * ld + c] = ldf(p + 2 * d);
    dO[s * ld + c] = ldf(dbase + (int64_t)s * d + c);
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwb = blockDim.x >> 5;
  T* dbq = dqkv + row0 * 3 * (int64_t)d + h * dh;
  // phase 1: one query row per warp: probabilities, dS, and dQ
  for (int i = warp; i < S; i += nwb) {
    float p[4], dp[4];
    float m = -INFINITY;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int j = lane + 32 * jj;
      float sc = -INFINITY, g = 0.f;
      if (j < Sv && (!causal || j <= i)) {
        float acc = 0.f;
        for (int c = 0; c < dh; ++c) {
          acc += Q[i * ld + c] * K[j * ld + c];
          g += dO[i * ld + c] * V[j * ld + c];
        }
        sc = acc * scale;
      }
      p[jj] = sc;
      dp[jj] = g;
      m = fmaxf(m, sc);
    }
    m = warp_max(m);
    float l = 0.f;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      p[jj] = (p[jj] == -INFINITY) ? 0.f : __expf(p[jj] - m);
      l += p[jj];
    }
    l = warp_sum(l);
    const float inv = 1.f / l;
    float delta = 0.f;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      p[jj] *= inv;
      delta += p[jj] * dp[jj];
    }
    delta = warp_sum(delta);
    float ds[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int j = lane + 32 * jj;
      ds[jj] = p[jj] * (dp[jj] - delta) * scale;
      if (j < S) {
        Pm[i * lp + j] = p[jj];
        dS[i * lp + j] = ds[jj];
      }
    }
    const int jmax = min(causal ? i + 1 : S, Sv);
    float o0 = 0.f, o1 = 0.f;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      for (int l2 = 0; l2 < 32; ++l2) {
        const int j = jj * 32 + l2;
        if (j >= jmax) break;
        const float dsj = __shfl_sync(0xffffffffu, ds[jj], l2);
        if (lane < dh) o0 += dsj * K[j * ld + lane];
        if (lane + 32 < dh) o1 += dsj * K[j * ld + lane + 32];
      }
    }
    T* o = dbq + (int64_t)i * 3 * d;
    if (lane < dh) stf(o + lane, o0);
    if (lane + 32 < dh) stf(o + lane + 32, o1);
  }
  __syncthreads();
  // phase 2: one key row per warp: dK[j] = sum_i dS[i][j] Q[i], dV[j] = sum_i P[i][j] dO[i]
  for (int j = warp; j < S; j += nwb) {
    float k0 = 0.f, k1 = 0.f, v0 = 0.f, v1 = 0.f;
    const int i0 = causal ? j : 0;
    for (int i = i0; i < S; ++i) {
      const float a = dS[i * lp + j], b = Pm[i * lp + j];
      if (lane < dh) { k0 += a * Q[i * ld + lane]; v0 += b * dO[i * ld + lane]; }
      if (lane + 32 < dh) { k1 += a * Q[i * ld + lane + 32]; v1 += b * dO[i * ld + lane + 32]; }
    }
    T* o = dbq + (int64_t)j * 3 * d;
    if (lane < dh) { stf(o + d + lane, k0); stf(o + 2 * d + lane, v0); }
    if (lane + 32 < dh) { stf(o + d + lane + 32, k1); stf(o + 2 * d + lane + 32, v1); }
  }
}

// ---------------------------------------------------------------------------- column sums
// grid (column slabs of 64, row blocks); each warp sums rows warp, warp+8, ... of the block's range
template <typename T>
__global__ void __launch_bounds__(256) colsum_kernel(const T* __restrict__ X, int64_t rows, int N, int64_t rows_per_block,
                                                     float* __restrict__ part) {
  __shared__ float2 sw[8][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = blockIdx.x * 64 + 2 * lane;
  const int64_t r0 = (int64_t)blockIdx.y * rows_per_block, r1 = min(r0 + rows_per_block, rows);
  float2 acc = make_float2(0.f, 0.f);
  if (c < N) {
    for (int64_t r = r0 + warp; r < r1; r += 8) {
      float2 v = ld2(X + r * N + c);
      acc.x += v.x;
      acc.y += v.y;
    }
  }
  sw[warp][lane] = acc;
  __syncthreads();
  if (warp == 0 && c < N) {
    float2 t = sw[0][lane];
#pragma unroll
    for (int w = 1; w < 8; ++w) { t.x += sw[w][lane].x; t.y += sw[w][lane].y; }
    part[(int64_t)blockIdx.y * N + c] = t.x;
    part[(int64_t)blockIdx.y * N + c + 1] = t.y;
  }
}

// blockIdx.y owns the groups [y * per, (y + 1) * per) and leaves their sum in part[y][period * d]; with one chunk
// (part == null) the sum is added to out directly
__global__ void periodic_rowsum_kernel(const float* __restrict__ X, int64_t n_groups, int64_t per, int period, int d,
                                       float* __restrict__ out, float* __restrict__ part,
                                       const int32_t* __restrict__ seq_len, const int32_t* __restrict__ seq_off) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)period * d) return;
  const int s = (int)(i / d), c = (int)(i - (int64_t)s * d);
  const int64_t u0 = (int64_t)blockIdx.y * per, u1 = min(u0 + per, n_groups);
  float acc = 0.f;
  if (seq_off) {                                   // packed rows: group u has seq_len[u] rows starting at seq_off[u]
    for (int64_t u = u0; u < u1; ++u)
      if (s < seq_len[u]) acc += X[((int64_t)seq_off[u] + s) * d + c];
  } else {
    for (int64_t u = u0; u < u1; ++u) acc += X[(u * period + s) * d + c];
  }
  if (part) part[(int64_t)blockIdx.y * period * d + i] = acc;
  else out[i] += acc;
}

// ---------------------------------------------------------------------------- pooling
__device__ __forceinline__ float stream_at(const StreamRef& x, int64_t row, int c, int d) {
  float v = x.z[row * d + c];
  if (x.mean) v = (v - x.mean[row]) * x.rstd[row] * x.gamma[c] + x.beta[c];
  return v;
}
__global__ void pool_fwd_kernel(StreamRef x, float* __restrict__ H, int64_t n, int l_t, int d, int pooling,
                                const int32_t* __restrict__ seq_len, const int32_t* __restrict__ seq_off) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n * d) return;
  const int64_t u = i / d;
  const int c = (int)(i - u * d);
  const int64_t row0 = seq_off ? (int64_t)seq_off[u] : u * l_t;
  if (pooling == GRAM_POOL_CLS) {
    H[i] = stream_at(x, row0, c, d);
  } else {
    const int len = seq_len ? seq_len[u] : l_t;      // mean over the tokens that are text
    float acc = 0.f;
    for (int s = 0; s < len; ++s) acc += stream_at(x, row0 + s, c, d);
    H[i] = acc / len;
  }
}
__global__ void pool_bwd_kernel(const float* __restrict__ G, float* __restrict__ dx, int64_t n, int l_t, int d, int pooling,
                                const int32_t* __restrict__ seq_len, const int32_t* __restrict__ seq_off) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n * l_t * d) return;
  const int64_t t = i / d;
  const int c = (int)(i - t * d);
  const int64_t u = t / l_t;
  const int s = (int)(t - u * l_t);
  float v;
  if (pooling == GRAM_POOL_CLS) v = (s == 0) ? G[u * d + c] : 0.f;
  else {
    const int len = seq_len ? seq_len[u] : l_t;
    v = s < len ? G[u * d + c] / len : 0.f;
  }
  if (seq_off) {                                   // packed rows: the padding slots have no row
    if (s < seq_len[u]) dx[((int64_t)seq_off[u] + s) * d + c] = v;
    return;
  }
  dx[i] = v;
}

// additive-attention pooling, one block per item: scores a_s = q . tanh(pre[s, :]) over the item's rows, alpha = softmax,
// H[u, :] = sum_s alpha_s x[s, :]; alpha is kept for the backward pass
template <typename T>
__global__ void __launch_bounds__(128) pool_additive_fwd_kernel(StreamRef x, const T* __restrict__ pre, const float* __restrict__ q,
                                                                float* __restrict__ H, float* __restrict__ alpha, int l_t, int d,
                                                                int pa, const int32_t* __restrict__ seq_len,
                                                                const int32_t* __restrict__ seq_off) {
  __shared__ float sa[128];
  const int64_t u = blockIdx.x;
  const int64_t row0 = seq_off ? (int64_t)seq_off[u] : u * l_t;
  const int S = seq_len ? seq_len[u] : l_t;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int s = warp; s < S; s += 4) {
    float acc = 0.f;
    for (int j = lane; j < pa; j += 32) acc += q[j] * tanhf(ldf(pre + (row0 + s) * pa + j));
    acc = warp_sum(acc);
    if (lane == 0) sa[s] = acc;
  }
  __syncthreads();
  if (warp == 0) {                      // softmax over the S <= 128 scores
    float m = -INFINITY;
    for (int s = lane; s < S; s += 32) m = fmaxf(m, sa[s]);
    m = warp_max(m);
    float l = 0.f;
    for (int s = lane; s < S; s += 32) { const float e = __expf(sa[s] - m); sa[s] = e; l += e; }
    l = warp_sum(l);
    const float inv = 1.f / l;
    for (int s = lane; s < S; s += 32) { sa[s] *= inv; alpha[row0 + s] = sa[s]; }
  }
  __syncthreads();
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float acc = 0.f;
    for (int s = 0; s < S; ++s) acc += sa[s] * stream_at(x, row0 + s, c, d);
    H[u * d + c] = acc;
  }
}

// backward of the above for the cotangent G[u, :]: dx[s, :] = alpha_s G (the part that does not go through the scores),
// dpre[s, j] = da_s q_j (1 - tanh^2 pre[s, j]) with da = alpha (dalpha - sum alpha dalpha), dalpha_s = G . x[s, :];
// qpart[u, j] = sum_s da_s tanh(pre[s, j]) (summed over items by the caller, in order)
template <typename T>
__global__ void __launch_bounds__(128) pool_additive_bwd_kernel(StreamRef x, const T* __restrict__ pre, const float* __restrict__ q,
                                                                const float* __restrict__ alpha, const float* __restrict__ G,
                                                                float* __restrict__ dx, T* __restrict__ dpre,
                                                                float* __restrict__ qpart, int l_t, int d, int pa,
                                                                const int32_t* __restrict__ seq_len,
                                                                const int32_t* __restrict__ seq_off) {
  __shared__ float sda[128], sal[128];
  __shared__ float sdelta;
  const int64_t u = blockIdx.x;
  const int64_t row0 = seq_off ? (int64_t)seq_off[u] : u * l_t;
  const int S = seq_len ? seq_len[u] : l_t;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int s = warp; s < S; s += 4) {
    float acc = 0.f;
    for (int c = lane; c < d; c += 32) acc += G[u * d + c] * stream_at(x, row0 + s, c, d);
    acc = warp_sum(acc);
    if (lane == 0) { sda[s] = acc; sal[s] = alpha[row0 + s]; }
  }
  __syncthreads();
  if (warp == 0) {
    float dl = 0.f;
    for (int s = lane; s < S; s += 32) dl += sal[s] * sda[s];
    dl = warp_sum(dl);
    if (lane == 0) sdelta = dl;
  }
  __syncthreads();
  for (int s = threadIdx.x; s < S; s += blockDim.x) sda[s] = sal[s] * (sda[s] - sdelta);
  __syncthreads();
  for (int j = threadIdx.x; j < pa; j += blockDim.x) {
    const float qj = q[j];
    float acc = 0.f;
    for (int s = 0; s < S; ++s) {
      const float t = tanhf(ldf(pre + (row0 + s) * pa + j));
      stf(dpre + (row0 + s) * pa + j, sda[s] * qj * (1.f - t * t));
      acc += sda[s] * t;
    }
    qpart[u * pa + j] = acc;
  }
  for (int64_t i = threadIdx.x; i < (int64_t)S * d; i += blockDim.x) {
    const int s = (int)(i / d), c = (int)(i - (int64_t)s * d);
    dx[(row0 + s) * d + c] = sal[s] * G[u * d + c];
  }
}

// ---------------------------------------------------------------------------- KT task input / head
// ET: element type of the encodings.  index (may be null): the encoding of position p is row index[p] of E (the gather
// of stage 3 done where its result is consumed: E is then the matrix of encodings per item, n_rows of them).
template <typename T, typename ET>
__global__ void kt_input_fwd_kernel(const ET* __restrict__ E, const int32_t* __restrict__ index, int64_t n_rows,
                                    const float* __restrict__ pos, const float* __restrict__ resp,
                                    const int32_t* __restrict__ labels, float* __restrict__ x, T* __restrict__ x_b, int64_t P,
                                    int L, int d, int32_t* status) {
  const int64_t p = blockIdx.x;                  // one block per position
  const int n = (int)(p % L);
  int prev = (n == 0) ? 2 : labels[p - 1];
  prev = prev < 0 ? 2 : (prev > 1 ? (n == 0 ? 2 : 1) : prev);      // after a padded position (label -1): only at padded rows
  int64_t row = p;
  if (index) {
    row = index[p];
    if (row < 0 || row >= n_rows) {
      if (threadIdx.x == 0) gram_device_fail(status, GRAM_ERR_ID_RANGE);
      row = 0;
    }
  }
  const ET* e = E + row * d;
  const float* pe = pos + (int64_t)n * d;
  const float* re = resp + (int64_t)prev * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const float v = ldf(e + c) + pe[c] + re[c];
    x[p * d + c] = v;
    stf(x_b + p * d + c, v);
  }
}
// one thread per column: dE = dx (when dE is not null); dpos[n, c] += sum_b; dresp[r, c] += sum over positions with prev == r
__global__ void kt_input_bwd_kernel(const float* __restrict__ dx, const int32_t* __restrict__ labels, float* __restrict__ dE,
                                    float* __restrict__ dpos, float* __restrict__ dresp, int B, int L, int d) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  const int n = blockIdx.y;
  if (c >= d) return;
  float ap = 0.f, r0 = 0.f, r1 = 0.f, r2 = 0.f;
  constexpr int UB = 8;                          // histories per round: their loads are issued together
  for (int b0 = 0; b0 < B; b0 += UB) {
    float v[UB];
    int prev[UB];
#pragma unroll
    for (int k = 0; k < UB; ++k) {
      const int64_t p = (int64_t)(b0 + k) * L + n;
      const bool ok = b0 + k < B;
      v[k] = ok ? dx[p * d + c] : 0.f;
      prev[k] = (ok && n > 0) ? labels[p - 1] : 2;
    }
#pragma unroll
    for (int k = 0; k < UB; ++k) {              // sums in ascending history order
      if (b0 + k < B) {
        if (dE) dE[((int64_t)(b0 + k) * L + n) * d + c] = v[k];
        ap += v[k];
        if (prev[k] == 0) r0 += v[k]; else if (prev[k] == 1) r1 += v[k]; else r2 += v[k];
      }
    }
  }
  dpos[(int64_t)n * d + c] += ap;
  // per-position partial of dresp, reduced over n by the caller: part[n][3][d]
  dresp[((int64_t)n * 3 + 0) * d + c] = r0;
  dresp[((int64_t)n * 3 + 1) * d + c] = r1;
  dresp[((int64_t)n * 3 + 2) * d + c] = r2;
}

// warp per position; per-block partials: [d] for dw, then loss and db.  A warp keeps the sums of its own rows in
// registers (d <= 1024); the warps' sums are added in warp order at the end, so the order of additions is fixed.
template <typename T>
__global__ void __launch_bounds__(256) kt_head_kernel(StreamRef y, const float* __restrict__ w,
                                                      const float* __restrict__ bias, const int32_t* __restrict__ labels,
                                                      float* __restrict__ dy, T* __restrict__ dy_b,
                                                      float* __restrict__ part, int64_t P, int d, int64_t pstride,
                                                      const int32_t* __restrict__ n_real) {
  extern __shared__ float sacc[];            // [warps][d + 2]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwb = blockDim.x >> 5;
  const float b0 = bias[0], invP = 1.f / (float)max(*n_real, 1);   // the mean runs over the real predictions
  // rows are dealt to blocks in contiguous ranges, and inside a block to warps round-robin
  const int64_t per = (P + gridDim.x - 1) / gridDim.x;
  const int64_t r0 = (int64_t)blockIdx.x * per, r1 = min(r0 + per, P);
  float acc_w[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) acc_w[i] = 0.f;
  float acc_loss = 0.f, acc_db = 0.f;
  for (int64_t r = r0 + warp; r < r1; r += nwb) {
    float yv[32];
    float acc = 0.f;
    const bool ln = y.mean != nullptr;             // the stream's LayerNorm, its row statistics read once
    const float mu = ln ? y.mean[r] : 0.f, rs = ln ? y.rstd[r] : 1.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int c = lane + 32 * i;
      yv[i] = 0.f;
      if (c < d) {
        const float v = y.z[r * d + c];
        yv[i] = ln ? (v - mu) * rs * y.gamma[c] + y.beta[c] : v;
        acc += yv[i] * w[c];
      }
    }
    const float z = warp_sum(acc) + b0;
    const int32_t li = labels[r];
    const float lab = (float)li;
    float dzl = 0.f;
    if (li >= 0) {                          // label -1: padding at the end of a history, not predicted
      acc_loss += fmaxf(z, 0.f) + log1pf(__expf(-fabsf(z))) - lab * z;
      dzl = (1.f / (1.f + __expf(-z)) - lab) * invP;
    }
    acc_db += dzl;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int c = lane + 32 * i;
      if (c < d) {
        dy[r * d + c] = dzl * w[c];
        if (dy_b) stf(dy_b + r * d + c, dzl * w[c]);
        acc_w[i] += dzl * yv[i];
      }
    }
  }
  float* mine = sacc + (size_t)warp * (d + 2);
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    const int c = lane + 32 * i;
    if (c < d) mine[c] = acc_w[i];
  }
  if (lane == 0) { mine[d] = acc_loss; mine[d + 1] = acc_db; }
  __syncthreads();
  for (int i = threadIdx.x; i < d + 2; i += blockDim.x) {
    float a = 0.f;
    for (int ww = 0; ww < nwb; ++ww) a += sacc[(size_t)ww * (d + 2) + i];
    part[(int64_t)blockIdx.x * pstride + i] = a;
  }
}

__global__ void kt_head_reduce_kernel(const float* __restrict__ part, int nblocks, int64_t pstride, int d,
                                      const int32_t* __restrict__ n_real, float* __restrict__ dw, float* __restrict__ db,
                                      float* __restrict__ loss) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= d + 2) return;
  const float invP = 1.f / (float)max(*n_real, 1);
  float a = 0.f;
  for (int k = 0; k < nblocks; ++k) a += part[(int64_t)k * pstride + c];
  if (c < d) dw[c] += a;
  else if (c == d) loss[0] = a * invP;
  else db[0] += a;
}

// positions with a label >= 0 (integer adds: the count does not depend on their order); *n_real must start at zero
__global__ void count_real_kernel(const int32_t* __restrict__ labels, int64_t P, int32_t* __restrict__ n_real) {
  int32_t c = 0;
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < P; p += (int64_t)gridDim.x * blockDim.x) c += labels[p] >= 0;
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(n_real, c);
}

// ---------------------------------------------------------------------------- NR task (per user)
// pre[b, n, :] = E[b, n, :] wa^T + ba is given.  One block per user.
template <typename T>
__global__ void __launch_bounds__(256) nr_user_kernel(const float* __restrict__ E, const T* __restrict__ pre,
                                                      const float* __restrict__ qa, float* __restrict__ dE,
                                                      T* __restrict__ dpre, float* __restrict__ part, int L, int n_cand,
                                                      int d, int d_a, float invB, const int32_t* __restrict__ labels) {
  extern __shared__ float sm[];
  const int n_hist = L - n_cand;
  float* a = sm;                 // [L] scores / alpha
  float* da = a + L;             // [L]
  float* u = da + L;             // [d]
  float* du = u + d;             // [d]
  float* sc = du + d;            // [n_cand] scores, then ds
  const int b = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwb = blockDim.x >> 5;
  const float* Eb = E + (int64_t)b * L * d;
  const T* pb = pre + (int64_t)b * L * d_a;
  for (int n = warp; n < n_hist; n += nwb) {
    float acc = 0.f;
    for (int k = lane; k < d_a; k += 32) acc += qa[k] * tanhf(ldf(pb + (int64_t)n * d_a + k));
    acc = warp_sum(acc);
    if (labels && labels[(int64_t)b * L + n] < 0) acc = -INFINITY;       // a slot without a click takes no part
    if (lane == 0) a[n] = acc;
  }
  __syncthreads();
  if (warp == 0) {               // softmax over the history
    float m = -INFINITY;
    for (int n = lane; n < n_hist; n += 32) m = fmaxf(m, a[n]);
    m = warp_max(m);
    if (m == -INFINITY) m = 0.f;                                           // no click at all: every weight is zero
    float l = 0.f;
    for (int n = lane; n < n_hist; n += 32) l += __expf(a[n] - m);
    l = warp_sum(l);
    const float inv = l > 0.f ? 1.f / l : 0.f;
    for (int n = lane; n < n_hist; n += 32) a[n] = __expf(a[n] - m) * inv;
  }
  __syncthreads();
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float acc = 0.f;
    for (int n = 0; n < n_hist; ++n) acc += a[n] * ldf(Eb + (int64_t)n * d + c);
    u[c] = acc;
  }
  __syncthreads();
  for (int j = warp; j < n_cand; j += nwb) {
    float acc = 0.f;
    for (int c = lane; c < d; c += 32) acc += u[c] * ldf(Eb + (int64_t)(n_hist + j) * d + c);
    acc = warp_sum(acc);
    if (lane == 0) sc[j] = acc;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = -INFINITY;
    for (int j = 0; j < n_cand; ++j) m = fmaxf(m, sc[j]);
    float l = 0.f;
    for (int j = 0; j < n_cand; ++j) l += expf(sc[j] - m);
    part[(int64_t)b * (d_a + 1) + d_a] = -(sc[0] - m - logf(l));       // this user's loss
    for (int j = 0; j < n_cand; ++j) sc[j] = (expf(sc[j] - m) / l - (j == 0 ? 1.f : 0.f)) * invB;   // ds
  }
  __syncthreads();
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float acc = 0.f;
    for (int j = 0; j < n_cand; ++j) {
      acc += sc[j] * ldf(Eb + (int64_t)(n_hist + j) * d + c);
      dE[((int64_t)b * L + n_hist + j) * d + c] = sc[j] * u[c];          // gradient of the candidates
    }
    du[c] = acc;
  }
  __syncthreads();
  for (int n = warp; n < n_hist; n += nwb) {     // d alpha_n = du . h_n
    float acc = 0.f;
    for (int c = lane; c < d; c += 32) acc += du[c] * ldf(Eb + (int64_t)n * d + c);
    acc = warp_sum(acc);
    if (lane == 0) da[n] = acc;
  }
  __syncthreads();
  if (warp == 0) {
    float s = 0.f;
    for (int n = lane; n < n_hist; n += 32) s += a[n] * da[n];
    s = warp_sum(s);
    for (int n = lane; n < n_hist; n += 32) da[n] = a[n] * (da[n] - s);   // gradient of the scores a_n
  }
  __syncthreads();
  for (int i = threadIdx.x; i < n_hist * d; i += blockDim.x) {            // direct part of dh_n
    const int n = i / d, c = i - n * d;
    dE[((int64_t)b * L + n) * d + c] = a[n] * du[c];
  }
  for (int k = threadIdx.x; k < d_a; k += blockDim.x) {
    float gq = 0.f;
    for (int n = 0; n < L; ++n) {
      float v = 0.f;
      if (n < n_hist) {
        const float t = tanhf(ldf(pb + (int64_t)n * d_a + k));
        gq += da[n] * t;
        v = da[n] * qa[k] * (1.f - t * t);
      }
      stf(dpre + ((int64_t)b * L + n) * d_a + k, v);
    }
    part[(int64_t)b * (d_a + 1) + k] = gq;
  }
}

__global__ void nr_reduce_kernel(const float* __restrict__ part, int B, int d_a, float invB, float* __restrict__ dqa,
                                 float* __restrict__ loss) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k > d_a) return;
  float a = 0.f;
  for (int b = 0; b < B; ++b) a += part[(int64_t)b * (d_a + 1) + k];
  if (k < d_a) dqa[k] += a;
  else loss[0] = a * invB;
}

// ---------------------------------------------------------------------------- NR task: the clicked items as packed sequences
// One block.  User b's clicked slots (the history positions whose label is not negative) become sequence b of a packed
// layout: seq_len[b] = their number, seq_off = its exclusive prefix sum, rows[seq_off[b] + k] = position of the k-th clicked
// slot, pos2row[position] = its packed row (-1 for empty slots and candidates).  rows[r] = -1 for the unused tail r >= total.
__global__ void __launch_bounds__(1024) nr_layout_kernel(const int32_t* __restrict__ labels, int B, int L, int n_hist,
                                                         int32_t* __restrict__ seq_len, int32_t* __restrict__ seq_off,
                                                         int32_t* __restrict__ rows, int32_t* __restrict__ pos2row) {
  __shared__ int32_t total;
  if (threadIdx.x == 0) total = 0;
  __syncthreads();
  for (int b = 0; b < B; ++b) {                  // users in order: a few dozen to a few hundred per batch
    const int32_t base = total;
    __syncthreads();
    int32_t placed = 0;
    for (int n0 = 0; n0 < L; n0 += 1024) {
      const int n = n0 + (int)threadIdx.x;
      const bool hist = n < n_hist, clicked = hist && (!labels || labels[(int64_t)b * L + n] >= 0);
      // rank of this slot among the clicked ones of the user: block-wide count of clicked slots before it
      __shared__ int32_t wsum[32];
      const uint32_t vote = __ballot_sync(0xffffffffu, clicked);
      const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
      if (lane == 0) wsum[warp] = __popc(vote);
      __syncthreads();
      int32_t before = placed;
      for (int w = 0; w < warp; ++w) before += wsum[w];
      int32_t all = 0;
      for (int w = 0; w < 32; ++w) all += wsum[w];
      const int32_t rank = before + __popc(vote & ((1u << lane) - 1u));
      if (n < L) pos2row[(int64_t)b * L + n] = clicked ? base + rank : -1;
      if (clicked) rows[base + rank] = b * L + n;
      placed += all;
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      seq_len[b] = placed;
      seq_off[b] = base;
      total = base + placed;
    }
    __syncthreads();
  }
  const int32_t t = total;
  if (threadIdx.x == 0) seq_off[B] = t;
  for (int64_t r = t + threadIdx.x; r < (int64_t)B * n_hist; r += blockDim.x) rows[r] = -1;
}

// out[r, :] = src[rows[r], :] (zero rows where rows[r] < 0), fp32, and an operand-typed copy when out_b is given
template <typename T>
__global__ void nr_pack_kernel(const float* __restrict__ src, const int32_t* __restrict__ rows, int64_t n, int d,
                               float* __restrict__ out, T* __restrict__ out_b) {
  const int64_t r = blockIdx.x;
  const int32_t p = rows[r];
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const float v = p >= 0 ? src[(int64_t)p * d + c] : 0.f;
    out[r * d + c] = v;
    if (out_b) stf(out_b + r * d + c, v);
  }
}

// out[p, :] = y(pos2row[p], :) where the position has a packed row, else other[p, :]; y is a view of the residual stream
__global__ void nr_select_kernel(StreamRef y, const int32_t* __restrict__ pos2row, const float* __restrict__ other, int64_t P, int d,
                                 float* __restrict__ out) {
  const int64_t p = blockIdx.x;
  const int32_t r = pos2row[p];
  if (r < 0) {
    for (int c = threadIdx.x; c < d; c += blockDim.x) out[p * d + c] = other[p * d + c];
    return;
  }
  const bool ln = y.mean != nullptr;
  const float mu = ln ? y.mean[r] : 0.f, rs = ln ? y.rstd[r] : 1.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const float v = y.z[(int64_t)r * d + c];
    out[p * d + c] = ln ? (v - mu) * rs * y.gamma[c] + y.beta[c] : v;
  }
}

// ---------------------------------------------------------------------------- element-wise
__global__ void f32_to_bf16_kernel(const float* __restrict__ in, bf16* __restrict__ out, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    out[i] = __float2bfloat16(in[i]);
}
__global__ void bf16_to_f32_kernel(const bf16* __restrict__ in, float* __restrict__ out, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    out[i] = __bfloat162float(in[i]);
}
// gate (may be null): a device word; nothing is updated when it is not zero (an error met earlier in the step)
__global__ void sgd_kernel(float* __restrict__ w, const float* __restrict__ g, float lr, size_t n, const int32_t* __restrict__ gate) {
  if (gate && *gate) return;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    w[i] -= lr * g[i];
}
template <typename T>
__global__ void scatter_rows_kernel(const float* __restrict__ src, const int32_t* __restrict__ index, int64_t n, int d,
                                    int64_t n_dst_rows, T* __restrict__ dst, int32_t* status) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n * d) return;
  const int64_t u = i / d;
  const int c = (int)(i - u * d);
  const int32_t r = index[u];
  if (r < 0 || r >= n_dst_rows) { gram_device_fail(status, GRAM_ERR_ID_RANGE); return; }
  stf(dst + (int64_t)r * d + c, src[i]);
}

// rows of `words` 32-bit words copied between two layouts whose rows are in_stride / out_stride words apart
// in_rows / out_rows (may be null): row r of that side is row in_rows[r] / out_rows[r] instead of r
__global__ void strided_rows_kernel(const uint32_t* __restrict__ in, uint32_t* __restrict__ out, int64_t n, int64_t in_stride,
                                    int64_t out_stride, int words, const int32_t* __restrict__ in_rows,
                                    const int32_t* __restrict__ out_rows) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n * words) return;
  const int64_t r = i / words;
  const int c = (int)(i - r * words);
  const int64_t ri = in_rows ? in_rows[r] : r, ro = out_rows ? out_rows[r] : r;
  out[ro * out_stride + c] = in[ri * in_stride + c];
}

// lengths and first rows of the sequences of one encoder pass: seq_len[u] = item_len[item(u)] (clamped to 1..l_t),
// seq_off = its exclusive prefix sum, seq_off[n] = total rows.  One block; item(u) = items[u] or first_item + u.
__global__ void __launch_bounds__(1024) seq_layout_kernel(const int32_t* __restrict__ item_len, const int32_t* __restrict__ items,
                                                          int32_t first_item, int32_t n, int32_t n_items_total, int l_t,
                                                          int32_t* __restrict__ seq_len, int32_t* __restrict__ seq_off,
                                                          int32_t* __restrict__ group_list, int32_t* __restrict__ info,
                                                          int32_t* status) {
  __shared__ int32_t sw[33];
  __shared__ int32_t carry_s;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int32_t base = 0; base < n; base += 1024) {
    const int32_t u = base + threadIdx.x;
    int32_t len = 0;
    if (u < n) {
      int32_t item = items ? items[u] : first_item + u;
      if (item < 0 || item >= n_items_total) { gram_device_fail(status, GRAM_ERR_ID_RANGE); item = 0; }
      len = item_len[item];
      len = len < 1 ? 1 : (len > l_t ? l_t : len);
      seq_len[u] = len;
    }
    // inclusive scan over the block
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int32_t incl = len;
    for (int o = 1; o < 32; o <<= 1) {
      const int32_t t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) sw[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int32_t w = sw[lane], wi = w;
      for (int o = 1; o < 32; o <<= 1) {
        const int32_t t = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += t;
      }
      sw[lane] = wi - w;
      if (lane == 31) sw[32] = wi;
    }
    __syncthreads();
    const int32_t carry = carry_s;
    if (u < n) seq_off[u] = carry + sw[warp] + incl - len;
    __syncthreads();
    if (threadIdx.x == 0) carry_s = carry + sw[32];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    seq_off[n] = carry_s;
    info[4] = carry_s;
  }
  __syncthreads();
  // the sequence numbers grouped by length (1..32, 33..64, 65..96, 97.. rows), ascending inside a group
  int32_t placed = 0;
  for (int gi = 0; gi < 4; ++gi) {
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (int32_t base = 0; base < n; base += 1024) {
      const int32_t u = base + threadIdx.x;
      int32_t in = 0;
      if (u < n) {
        const int32_t b = (seq_len[u] - 1) >> 5;
        in = (b > 3 ? 3 : b) == gi;
      }
      const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
      const uint32_t vote = __ballot_sync(0xffffffffu, in);
      if (lane == 0) sw[warp] = __popc(vote);
      __syncthreads();
      if (warp == 0) {
        int32_t w = sw[lane], wi = w;
        for (int o = 1; o < 32; o <<= 1) {
          const int32_t t = __shfl_up_sync(0xffffffffu, wi, o);
          if (lane >= o) wi += t;
        }
        sw[lane] = wi - w;
        if (lane == 31) sw[32] = wi;
      }
      __syncthreads();
      const int32_t carry = carry_s;
      if (in) group_list[placed + carry + sw[warp] + __popc(vote & ((1u << lane) - 1u))] = u;
      __syncthreads();
      if (threadIdx.x == 0) carry_s = carry + sw[32];
      __syncthreads();
    }
    if (threadIdx.x == 0) info[gi] = carry_s;
    placed += carry_s;
    __syncthreads();
  }
}

inline int grid_for(int64_t n, int threads, int cap) {
  int64_t b = (n + threads - 1) / threads;
  if (b > cap) b = cap;
  if (b < 1) b = 1;
  return (int)b;
}

template <typename F> gram_status set_smem(gram_ctx* ctx, F kern, size_t bytes) {
  if (bytes > 227 * 1024) return gram_set_error(ctx, "a sequence is too long for the attention kernel's shared memory"), GRAM_ERR_UNSUPPORTED;
  if (bytes > 48 * 1024) GRAM_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
  return GRAM_OK;
}

}  // namespace

#define DISPATCH_T(dtype, ...)             \
  if ((dtype) == GRAM_F32) { typedef float T; __VA_ARGS__; } else { typedef bf16 T; __VA_ARGS__; }

#define DISPATCH_NQ(d, ...)                                                    \
  if ((d) <= 128) { constexpr int NQ = 1; __VA_ARGS__; }                       \
  else if ((d) <= 256) { constexpr int NQ = 2; __VA_ARGS__; }                  \
  else if ((d) <= 512) { constexpr int NQ = 4; __VA_ARGS__; }                  \
  else if ((d) <= 768) { constexpr int NQ = 6; __VA_ARGS__; }                  \
  else { constexpr int NQ = 8; __VA_ARGS__; }

gram_status embed_forward(gram_ctx* ctx, const int32_t* item_tokens, const int32_t* items, int32_t first_item,
                          int32_t n_chunk, int32_t n_items_total, int l_t, int vocab, int d, const float* tok_emb,
                          const float* pos_emb, float* z0, int32_t* tok_ids, const int32_t* seq_len, const int32_t* seq_off,
                          cudaStream_t st) {
  const int64_t n_tok = (int64_t)n_chunk * l_t;
  if (n_tok == 0) return GRAM_OK;
  const int blocks = grid_for(n_tok * 32, 256, kNumSMs * 8);
  ProfScope prof(ctx, GRAM_K_EMBED_POOL, 8.0 * (double)n_tok * d, 1, st);
  embed_fwd_kernel<<<blocks, 256, 0, st>>>(item_tokens, items, first_item, n_tok, n_items_total, l_t, vocab, d, tok_emb,
                                           pos_emb, z0, tok_ids, seq_len, seq_off, gram_status_word(ctx));
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status layernorm_forward(gram_ctx* ctx, int dtype, const float* z, const float* gamma, const float* beta, void* y,
                              float* mean, float* rstd, int64_t rows, int d, cudaStream_t st) {
  if (rows == 0) return GRAM_OK;
  if (d > 1024 || (d & 3)) return gram_set_error(ctx, "LayerNorm: d must be a multiple of 4 and at most 1024"), GRAM_ERR_UNSUPPORTED;
  const int blocks = grid_for(rows * 32, 256, kNumSMs * 8);
  ProfScope prof(ctx, GRAM_K_LAYERNORM, (double)rows * d * (4.0 + (dtype == GRAM_BF16 ? 2.0 : 4.0)), 1, st, "ln_fwd");
  DISPATCH_T(dtype, DISPATCH_NQ(d, ln_fwd_kernel<T, NQ><<<blocks, 256, 0, st>>>(z, gamma, beta, (T*)y, mean, rstd, rows, d)));
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status layernorm_backward(gram_ctx* ctx, int dtype, const float* dy, const float* z, const float* mean,
                               const float* rstd, const float* gamma, float* dz, void* dz_b, float* dgamma,
                               float* dbeta, float* dcol, float* scratch, int64_t rows, int d, cudaStream_t st) {
  if (rows == 0) return GRAM_OK;
  if (d > 1024 || (d & 3)) return gram_set_error(ctx, "LayerNorm: d must be a multiple of 4 and at most 1024"), GRAM_ERR_UNSUPPORTED;
  int cap = (int)(kRedScratchBytes / ((size_t)3 * d * sizeof(float)));
  if (cap > kNumSMs * 8) cap = kNumSMs * 8;
  // at least sixteen rows per warp where the row count allows it: a block's fixed work (clearing and writing 3 d partial
  // sums, which the reduction kernels then read) is otherwise most of a call on a few ten thousand rows
  int64_t want = (rows + 127) / 128;
  if (want < kNumSMs) want = kNumSMs;
  if (want > cap) want = cap;
  const int blocks = grid_for(rows * 32, 256, (int)want);
  const int nq = d <= 128 ? 1 : d <= 256 ? 2 : d <= 512 ? 4 : d <= 768 ? 6 : 8;   // float4 per lane: the kernel's NQ
  const size_t smem = (size_t)4 * d * sizeof(float) + (dcol ? (size_t)8 * nq * 32 * sizeof(float4) : 0);
  ProfScope prof(ctx, GRAM_K_LAYERNORM, (double)rows * d * (12.0 + (dz_b ? (dtype == GRAM_BF16 ? 2.0 : 4.0) : 0.0)), dcol ? 3 : 2, st, "ln_bwd");
  DISPATCH_T(dtype, DISPATCH_NQ(d, ln_bwd_kernel<T, NQ><<<blocks, 256, smem, st>>>(dy, z, mean, rstd, gamma, dz, (T*)dz_b, scratch, rows, d, dcol ? 1 : 0)));
  reduce_partials_kernel<<<ceil_div(d, 32), 256, 0, st>>>(scratch, blocks, (int64_t)3 * d, d, dgamma, dbeta, 1.f);
  if (dcol) reduce_partials_kernel<<<ceil_div(d, 32), 256, 0, st>>>(scratch + 2 * d, blocks, (int64_t)3 * d, d, dcol, nullptr, 1.f);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status attention_forward(gram_ctx* ctx, int dtype, const void* qkv, void* out, float* lse, int64_t rows, int64_t n_seq, int S,
                              int d, int n_heads, int causal, const int32_t* seq_len, const int32_t* seq_off,
                              const SeqGroups* groups, cudaStream_t st) {
  if (n_seq == 0) return GRAM_OK;
  const int dh = d / n_heads;
  if (dh * n_heads != d) return gram_set_error(ctx, "attention: d is not a multiple of the head count"), GRAM_ERR_ARG;
  const float scale = 1.f / sqrtf((float)dh);
  ProfScope prof(ctx, GRAM_K_ATTENTION, 4.0 * (double)n_seq * n_heads * S * S * dh, 1, st, "attn_fwd");
  if (dtype == GRAM_BF16 && attention_tc_supported(S, d, n_heads)) {
    if (!groups || !seq_off) return attention_forward_tc(ctx, qkv, out, lse, rows, n_seq, S, d, n_heads, causal, seq_len, seq_off, nullptr, st);
    int32_t first = 0;
    for (int gi = 0; gi < 4; ++gi) {                 // one launch per length group, with the smallest slot that fits
      const int bound = gi < 3 ? (S < 32 * (gi + 1) ? S : 32 * (gi + 1)) : S;
      if (groups->count[gi] > 0)
        GRAM_TRY(attention_forward_tc(ctx, qkv, out, lse, rows, groups->count[gi], bound, d, n_heads, causal, seq_len, seq_off,
                                      groups->list + first, st));
      first += groups->count[gi];
    }
    return GRAM_OK;
  }
  if (S > 128 || dh > 64) return gram_set_error(ctx, "attention: this element type and head width need S <= 128 and head width <= 64"), GRAM_ERR_UNSUPPORTED;
  const size_t smem = (size_t)3 * S * (dh + 1) * sizeof(float);
  if (dtype == GRAM_BF16 && attention_mma_supported(S, d, n_heads)) {
    if (!groups || !seq_off) return attention_forward_mma(ctx, qkv, out, n_seq, S, d, n_heads, causal, seq_len, seq_off, nullptr, st);
    int32_t first = 0;
    for (int gi = 0; gi < 4; ++gi) {                 // one launch per length group, with the smallest tile that fits
      if (groups->count[gi] > 0)
        GRAM_TRY(attention_forward_mma(ctx, qkv, out, groups->count[gi], S < 32 * (gi + 1) ? S : 32 * (gi + 1), d, n_heads,
                                       causal, seq_len, seq_off, groups->list + first, st));
      first += groups->count[gi];
    }
    return GRAM_OK;
  }
  DISPATCH_T(dtype, {
    GRAM_TRY(set_smem(ctx, attn_fwd_kernel<T>, smem));
    attn_fwd_kernel<T><<<(unsigned)(n_seq * n_heads), 128, smem, st>>>((const T*)qkv, (T*)out, S, d, n_heads, causal, scale, seq_len, seq_off);
  });
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status attention_backward(gram_ctx* ctx, int dtype, const void* qkv, const void* dctx, const void* octx, const float* lse,
                               float* delta, void* dqkv, float* colpart, int64_t colpart_cap_rows, int64_t* colpart_rows_used,
                               int64_t rows, int64_t n_seq, int S, int d, int n_heads, int causal, const int32_t* seq_len,
                               const int32_t* seq_off, const SeqGroups* groups, cudaStream_t st) {
  if (colpart_rows_used) *colpart_rows_used = 0;
  if (n_seq == 0) return GRAM_OK;
  const int dh = d / n_heads;
  if (dh * n_heads != d) return gram_set_error(ctx, "attention: d is not a multiple of the head count"), GRAM_ERR_ARG;
  const float scale = 1.f / sqrtf((float)dh);
  ProfScope prof(ctx, GRAM_K_ATTENTION, 10.0 * (double)n_seq * n_heads * S * S * dh, 1, st, "attn_bwd");
  const bool grouped = groups && seq_off;
  if (dtype == GRAM_BF16 && attention_tc_supported(S, d, n_heads)) {
    auto bound = [&](int gi) { return gi < 3 ? (S < 32 * (gi + 1) ? S : 32 * (gi + 1)) : S; };
    int64_t need = 0;
    if (!grouped) need = attention_tc_colpart_rows(n_seq, S);
    else for (int gi = 0; gi < 4; ++gi) need += groups->count[gi] > 0 ? attention_tc_colpart_rows(groups->count[gi], bound(gi)) : 0;
    float* cp = (colpart && need <= colpart_cap_rows) ? colpart : nullptr;      // partial column sums only when they fit
    if (cp && colpart_rows_used) *colpart_rows_used = need;
    if (!grouped)
      return attention_backward_tc(ctx, qkv, dctx, octx, lse, delta, dqkv, cp, 0, rows, n_seq, S, d, n_heads, causal, seq_len, seq_off, nullptr, st);
    int32_t first = 0;
    int64_t row0 = 0;
    for (int gi = 0; gi < 4; ++gi) {
      if (groups->count[gi] > 0) {
        GRAM_TRY(attention_backward_tc(ctx, qkv, dctx, octx, lse, delta, dqkv, cp, row0, rows, groups->count[gi], bound(gi), d, n_heads,
                                       causal, seq_len, seq_off, groups->list + first, st));
        row0 += attention_tc_colpart_rows(groups->count[gi], bound(gi));
      }
      first += groups->count[gi];
    }
    return GRAM_OK;
  }
  if (S > 128 || dh > 64) return gram_set_error(ctx, "attention: this element type and head width need S <= 128 and head width <= 64"), GRAM_ERR_UNSUPPORTED;
  const size_t smem = ((size_t)4 * S * (dh + 1) + (size_t)2 * S * (S + 1)) * sizeof(float);
  if (dtype == GRAM_BF16 && attention_mma_supported(S, d, n_heads)) {
    float* cp = (colpart && n_seq <= colpart_cap_rows) ? colpart : nullptr;    // one row of partial sums per sequence
    if (cp && colpart_rows_used) *colpart_rows_used = n_seq;
    if (!grouped)
      return attention_backward_mma(ctx, qkv, dctx, dqkv, cp, n_seq, S, d, n_heads, causal, seq_len, seq_off, nullptr, st);
    int32_t first = 0;
    for (int gi = 0; gi < 4; ++gi) {
      if (groups->count[gi] > 0)
        GRAM_TRY(attention_backward_mma(ctx, qkv, dctx, dqkv, cp, groups->count[gi], S < 32 * (gi + 1) ? S : 32 * (gi + 1), d,
                                        n_heads, causal, seq_len, seq_off, groups->list + first, st));
      first += groups->count[gi];
    }
    return GRAM_OK;
  }
  DISPATCH_T(dtype, {
    GRAM_TRY(set_smem(ctx, attn_bwd_kernel<T>, smem));
    attn_bwd_kernel<T><<<(unsigned)(n_seq * n_heads), 128, smem, st>>>((const T*)qkv, (const T*)dctx, (T*)dqkv, S, d, n_heads, causal, scale, seq_len, seq_off);
  });
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

// fold[g][c] = sum of part[r][c] over the rows r = g, g + G, g + 2G, ... (G = gridDim.y), warps taking every
// eighth of them and adding their sums in ascending order
__global__ void __launch_bounds__(256) fold_partials_kernel(const float* __restrict__ part, int64_t nrows, int n,
                                                            float* __restrict__ fold) {
  __shared__ float sa[8][32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  const int64_t G = gridDim.y;
  float a = 0.f;
  if (c < n) {
    for (int64_t r = blockIdx.y + (int64_t)w * G; r < nrows; r += 8 * G) a += part[r * n + c];
  }
  sa[w][lane] = a;
  __syncthreads();
  if (w == 0 && c < n) {
    float t = sa[0][lane];
#pragma unroll
    for (int k = 1; k < 8; ++k) t += sa[k][lane];
    fold[(int64_t)blockIdx.y * n + c] = t;
  }
}

gram_status colsum_from_partials(gram_ctx* ctx, const float* part, int64_t nrows, int N, float* out, float* scratch,
                                 cudaStream_t st) {
  if (nrows == 0 || N == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_COLSUM, (double)nrows * N * 4.0, 2, st, "colsum_partials");
  int G = 32;                                             // rows of the folded matrix (fixed: the order of additions depends on it)
  if ((size_t)G * N * sizeof(float) > kRedScratchBytes) G = (int)(kRedScratchBytes / ((size_t)N * sizeof(float)));
  if (G < 1) return gram_set_error(ctx, "column sums: N too large for the reduction scratch"), GRAM_ERR_UNSUPPORTED;
  fold_partials_kernel<<<dim3((unsigned)ceil_div(N, 32), (unsigned)G), 256, 0, st>>>(part, nrows, N, scratch);
  reduce_partials_kernel<<<ceil_div(N, 32), 256, 0, st>>>(scratch, G, (int64_t)N, N, out, nullptr, 1.f);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status colsum_accumulate(gram_ctx* ctx, int dtype, const void* X, int64_t rows, int N, float* out, float* scratch,
                              cudaStream_t st) {
  if (rows == 0 || N == 0) return GRAM_OK;
  if (N & 1) return gram_set_error(ctx, "column sum: N must be even"), GRAM_ERR_UNSUPPORTED;
  int64_t rb = ceil_div64(rows, 64);
  const int64_t cap = (int64_t)(kRedScratchBytes / sizeof(float)) / N;
  if (rb > 256) rb = 256;
  if (rb > cap) rb = cap;
  const int64_t per = ceil_div64(rows, rb);
  rb = ceil_div64(rows, per);
  dim3 grid((unsigned)ceil_div(N, 64), (unsigned)rb);
  ProfScope prof(ctx, GRAM_K_COLSUM, (double)rows * N * (dtype == GRAM_BF16 ? 2.0 : 4.0), 2, st, "colsum");
  DISPATCH_T(dtype, colsum_kernel<T><<<grid, 256, 0, st>>>((const T*)X, rows, N, per, scratch));
  reduce_partials_kernel<<<ceil_div(N, 32), 256, 0, st>>>(scratch, (int)rb, (int64_t)N, N, out, nullptr, 1.f);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status periodic_rowsum_accumulate(gram_ctx* ctx, const float* X, int64_t n_groups, int period, int d, float* out,
                                       float* scratch, const int32_t* seq_len, const int32_t* seq_off, cudaStream_t st) {
  if (n_groups == 0) return GRAM_OK;
  const int64_t n = (int64_t)period * d;
  // the groups are cut into chunks that are summed side by side; the chunk sums are then added in ascending order
  int64_t chunks = n_groups / 64;
  const int64_t fit = (int64_t)(kRedScratchBytes / sizeof(float)) / n;
  if (chunks > 64) chunks = 64;
  if (chunks > fit) chunks = fit;
  if (chunks < 2 || !scratch || n > INT32_MAX) chunks = 1;
  const int64_t per = ceil_div64(n_groups, chunks);
  ProfScope prof(ctx, GRAM_K_EMBED_POOL, 4.0 * (double)n_groups * period * d, chunks > 1 ? 2 : 1, st);
  dim3 grid((unsigned)ceil_div64(n, 128), (unsigned)chunks);
  periodic_rowsum_kernel<<<grid, 128, 0, st>>>(X, n_groups, per, period, d, out, chunks > 1 ? scratch : nullptr, seq_len, seq_off);
  if (chunks > 1) reduce_partials_kernel<<<ceil_div((int)n, 32), 256, 0, st>>>(scratch, (int)chunks, n, (int)n, out, nullptr, 1.f);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status pool_forward(gram_ctx* ctx, const StreamRef& x, float* H, int64_t n, int l_t, int d, int pooling,
                         const int32_t* seq_len, const int32_t* seq_off, cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_EMBED_POOL, 4.0 * (double)n * d * (pooling == GRAM_POOL_CLS ? 2 : l_t + 1), 1, st);
  pool_fwd_kernel<<<(unsigned)ceil_div64(n * d, 256), 256, 0, st>>>(x, H, n, l_t, d, pooling, seq_len, seq_off);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status pool_backward(gram_ctx* ctx, const float* G, float* dx, int64_t n, int l_t, int d, int pooling,
                          const int32_t* seq_len, const int32_t* seq_off, cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_EMBED_POOL, 4.0 * (double)n * d * (l_t + 1), 1, st);
  pool_bwd_kernel<<<(unsigned)ceil_div64(n * l_t * d, 256), 256, 0, st>>>(G, dx, n, l_t, d, pooling, seq_len, seq_off);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status kt_input_forward(gram_ctx* ctx, int dtype, const void* E, int e_bf16, const int32_t* index, int64_t n_rows,
                             const float* pos, const float* resp, const int32_t* labels, float* x, void* x_b, int B, int L,
                             int d, cudaStream_t st) {
  const int64_t P = (int64_t)B * L;
  if (P == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_TASK_HEAD, (double)P * d * ((e_bf16 ? 6.0 : 8.0) + (dtype == GRAM_BF16 ? 2.0 : 4.0)), 1, st);
  const int threads = d >= 256 ? 256 : 64;
  int32_t* sw = gram_status_word(ctx);
  if (e_bf16) {
    DISPATCH_T(dtype, kt_input_fwd_kernel<T, bf16><<<(unsigned)P, threads, 0, st>>>((const bf16*)E, index, n_rows, pos, resp, labels, x, (T*)x_b, P, L, d, sw));
  } else {
    DISPATCH_T(dtype, kt_input_fwd_kernel<T, float><<<(unsigned)P, threads, 0, st>>>((const float*)E, index, n_rows, pos, resp, labels, x, (T*)x_b, P, L, d, sw));
  }
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status kt_head(gram_ctx* ctx, int dtype, const StreamRef& y, const float* w, const float* b, const int32_t* labels,
                    float* dy, void* dy_b, float* dw, float* db, float* loss, float* scratch, int32_t* n_real, int64_t P,
                    int d, cudaStream_t st) {
  if (P == 0) return GRAM_OK;
  int blocks = (int)ceil_div64(P, 64);
  if (blocks > kRedBlocks) blocks = kRedBlocks;
  const int64_t pstride = d + 2;
  if (d > 1024) return gram_set_error(ctx, "kt head: d must be at most 1024"), GRAM_ERR_UNSUPPORTED;
  const size_t smem = (size_t)8 * (d + 2) * sizeof(float);
  ProfScope prof(ctx, GRAM_K_TASK_HEAD, 12.0 * (double)P * d, 3, st);
  GRAM_CUDA(ctx, cudaMemsetAsync(n_real, 0, sizeof(int32_t), st));
  count_real_kernel<<<grid_for(P, 256, kNumSMs), 256, 0, st>>>(labels, P, n_real);
  DISPATCH_T(dtype, kt_head_kernel<T><<<blocks, 256, smem, st>>>(y, w, b, labels, dy, (T*)dy_b, scratch, P, d, pstride, n_real));
  kt_head_reduce_kernel<<<ceil_div(d + 2, 256), 256, 0, st>>>(scratch, blocks, pstride, d, n_real, dw, db, loss);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

// dE = dx, dpos += column sums over b, dresp += sums by previous response; scratch holds [L][3][d]
gram_status kt_input_backward(gram_ctx* ctx, const float* dx, const int32_t* labels, float* dE, float* dpos,
                              float* dresp, float* scratch, int B, int L, int d, cudaStream_t st) {
  if (B == 0) return GRAM_OK;
  if ((size_t)L * 3 * d * sizeof(float) > kRedScratchBytes) return gram_set_error(ctx, "kt task: L*d too large for the reduction scratch"), GRAM_ERR_UNSUPPORTED;
  dim3 grid((unsigned)ceil_div(d, 128), (unsigned)L);
  ProfScope prof(ctx, GRAM_K_TASK_HEAD, 8.0 * (double)B * L * d, 2, st);
  kt_input_bwd_kernel<<<grid, 128, 0, st>>>(dx, labels, dE, dpos, scratch, B, L, d);
  reduce_partials_kernel<<<ceil_div(3 * d, 32), 256, 0, st>>>(scratch, L, (int64_t)3 * d, 3 * d, dresp, nullptr, 1.f);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status nr_user(gram_ctx* ctx, int dtype, const float* E, const void* pre, const float* qa, float* dE,
                           void* dpre, float* dqa, float* loss, float* scratch, const int32_t* labels, int B, int L, int n_cand,
                           int d, int d_a, cudaStream_t st) {
  if (B == 0) return GRAM_OK;
  if (n_cand <= 0 || n_cand >= L) return gram_set_error(ctx, "nr task: need 0 < n_cand < L"), GRAM_ERR_ARG;
  const size_t smem = ((size_t)2 * L + 2 * d + n_cand) * sizeof(float);
  ProfScope prof(ctx, GRAM_K_TASK_HEAD, (double)B * L * (8.0 * d + 4.0 * d_a), 2, st);
  DISPATCH_T(dtype, {
    GRAM_TRY(set_smem(ctx, nr_user_kernel<T>, smem));
    nr_user_kernel<T><<<B, 256, smem, st>>>(E, (const T*)pre, qa, dE, (T*)dpre, scratch, L, n_cand, d, d_a, 1.f / (float)B, labels);
  });
  nr_reduce_kernel<<<ceil_div(d_a + 1, 256), 256, 0, st>>>(scratch, B, d_a, 1.f / (float)B, dqa, loss);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status nr_layout(gram_ctx* ctx, const int32_t* labels, int B, int L, int n_hist, int32_t* seq_len, int32_t* seq_off,
                      int32_t* rows, int32_t* pos2row, cudaStream_t st) {
  if (B == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_TASK_HEAD, 12.0 * (double)B * L, 1, st);
  nr_layout_kernel<<<1, 1024, 0, st>>>(labels, B, L, n_hist, seq_len, seq_off, rows, pos2row);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
gram_status nr_pack(gram_ctx* ctx, int dtype, const float* src, const int32_t* rows, int64_t n, int d, float* out, void* out_b,
                    cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_TASK_HEAD, (double)n * d * (8.0 + (out_b ? (dtype == GRAM_BF16 ? 2.0 : 4.0) : 0.0)), 1, st);
  DISPATCH_T(dtype, nr_pack_kernel<T><<<(unsigned)n, d >= 256 ? 256 : 64, 0, st>>>(src, rows, n, d, out, (T*)out_b));
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
gram_status nr_select(gram_ctx* ctx, const StreamRef& y, const int32_t* pos2row, const float* other, int64_t P, int d, float* out,
                      cudaStream_t st) {
  if (P == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_TASK_HEAD, 8.0 * (double)P * d, 1, st);
  nr_select_kernel<<<(unsigned)P, d >= 256 ? 256 : 64, 0, st>>>(y, pos2row, other, P, d, out);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status convert_f32_to_bf16(gram_ctx* ctx, const float* in, bf16* out, size_t n, cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_OTHER, 6.0 * (double)n, 1, st);
  f32_to_bf16_kernel<<<grid_for((int64_t)n, 256, kNumSMs * 16), 256, 0, st>>>(in, out, n);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
gram_status convert_to_f32(gram_ctx* ctx, int dtype, const void* in, float* out, size_t n, cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  if (dtype == GRAM_F32) GRAM_CUDA(ctx, cudaMemcpyAsync(out, in, n * sizeof(float), cudaMemcpyDeviceToDevice, st));
  else {
    ProfScope prof(ctx, GRAM_K_OTHER, 6.0 * (double)n, 1, st);
    bf16_to_f32_kernel<<<grid_for((int64_t)n, 256, kNumSMs * 16), 256, 0, st>>>((const bf16*)in, out, n);
  }
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
// Adam (Kingma & Ba, Algorithm 1) on four values per thread; c1, c2: the bias corrections 1 / (1 - beta^t)
template <bool WB>
__global__ void __launch_bounds__(256) adam_kernel(float* __restrict__ w, const float* __restrict__ g, float* __restrict__ m,
                                                   float* __restrict__ v, bf16* __restrict__ wb, size_t n, float rate,
                                                   float beta1, float beta2, float eps, float c1, float c2,
                                                   const int32_t* __restrict__ gate) {
  if (gate && *gate) return;                    // an error met earlier in the step: no update
  const size_t n4 = n >> 2;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    float4 ww = reinterpret_cast<float4*>(w)[i];
    const float4 gg = __ldcs(reinterpret_cast<const float4*>(g) + i);
    float4 mm = reinterpret_cast<float4*>(m)[i], vv = reinterpret_cast<float4*>(v)[i];
    float* pw = &ww.x; const float* pg = &gg.x; float* pm = &mm.x; float* pv = &vv.x;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      pm[k] = beta1 * pm[k] + (1.f - beta1) * pg[k];
      pv[k] = beta2 * pv[k] + (1.f - beta2) * pg[k] * pg[k];
      pw[k] -= rate * (pm[k] * c1) / (sqrtf(pv[k] * c2) + eps);
    }
    reinterpret_cast<float4*>(w)[i] = ww;
    reinterpret_cast<float4*>(m)[i] = mm;
    reinterpret_cast<float4*>(v)[i] = vv;
    if (WB) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(ww.x, ww.y), hi = __floats2bfloat162_rn(ww.z, ww.w);
      uint2 o;
      o.x = *reinterpret_cast<uint32_t*>(&lo);
      o.y = *reinterpret_cast<uint32_t*>(&hi);
      reinterpret_cast<uint2*>(wb)[i] = o;
    }
  }
  // the last n % 4 values
  for (size_t i = (n4 << 2) + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const float gi = g[i];
    const float mi = beta1 * m[i] + (1.f - beta1) * gi;
    const float vi = beta2 * v[i] + (1.f - beta2) * gi * gi;
    const float wi = w[i] - rate * (mi * c1) / (sqrtf(vi * c2) + eps);
    m[i] = mi; v[i] = vi; w[i] = wi;
    if (WB) wb[i] = __float2bfloat16(wi);
  }
}

gram_status adam_update(gram_ctx* ctx, float* w, const float* g, float* m, float* v, void* wb, size_t n, int64_t t, float rate,
                        float beta1, float beta2, float eps, cudaStream_t st, const int32_t* gate) {
  if (n == 0) return GRAM_OK;
  if (t < 1) return gram_set_error(ctx, "Adam: the update count starts at 1"), GRAM_ERR_ARG;
  if (((uintptr_t)w | (uintptr_t)g | (uintptr_t)m | (uintptr_t)v) % 16 || (wb && (uintptr_t)wb % 8))
    return gram_set_error(ctx, "Adam: buffers must be 16-byte aligned"), GRAM_ERR_UNSUPPORTED;
  const float c1 = (float)(1.0 / (1.0 - pow((double)beta1, (double)t)));
  const float c2 = (float)(1.0 / (1.0 - pow((double)beta2, (double)t)));
  ProfScope prof(ctx, GRAM_K_OPTIMIZER, (double)n * (28.0 + (wb ? 2.0 : 0.0)), 1, st, "adam");
  const int grid = grid_for((int64_t)((n + 3) / 4), 256, kNumSMs * 8);
  if (wb) adam_kernel<true><<<grid, 256, 0, st>>>(w, g, m, v, (bf16*)wb, n, rate, beta1, beta2, eps, c1, c2, gate);
  else adam_kernel<false><<<grid, 256, 0, st>>>(w, g, m, v, nullptr, n, rate, beta1, beta2, eps, c1, c2, gate);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status sgd_update(gram_ctx* ctx, float* w, const float* g, float lr, size_t n, cudaStream_t st, const int32_t* gate) {
  if (n == 0 || lr == 0.f) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_OPTIMIZER, 12.0 * (double)n, 1, st, "sgd");
  sgd_kernel<<<grid_for((int64_t)n, 256, kNumSMs * 16), 256, 0, st>>>(w, g, lr, n, gate);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
gram_status scatter_rows(gram_ctx* ctx, int dtype, const float* src, const int32_t* index, int64_t n, int d,
                         int64_t n_dst_rows, void* dst, cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_OTHER, (double)n * d * (4.0 + (dtype == GRAM_BF16 ? 2.0 : 4.0)), 1, st);
  DISPATCH_T(dtype, scatter_rows_kernel<T><<<(unsigned)ceil_div64(n * d, 256), 256, 0, st>>>(src, index, n, d, n_dst_rows, (T*)dst, gram_status_word(ctx)));
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status take_strided_rows(gram_ctx* ctx, const void* in, int64_t n, int64_t stride, const int32_t* rows, int d,
                              int elem_bytes, void* out, cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  if ((d * elem_bytes) % 4) return gram_set_error(ctx, "row copy: rows must be whole 32-bit words"), GRAM_ERR_ARG;
  const int words = d * elem_bytes / 4;
  ProfScope prof(ctx, GRAM_K_OTHER, 2.0 * (double)n * d * elem_bytes, 1, st);
  strided_rows_kernel<<<(unsigned)ceil_div64(n * words, 256), 256, 0, st>>>((const uint32_t*)in, (uint32_t*)out, n,
                                                                          rows ? words : stride * words, words, words, rows,
                                                                          nullptr);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
gram_status put_strided_rows(gram_ctx* ctx, const void* in, int64_t n, int64_t stride, const int32_t* rows, int d,
                             int elem_bytes, void* out, cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  if ((d * elem_bytes) % 4) return gram_set_error(ctx, "row copy: rows must be whole 32-bit words"), GRAM_ERR_ARG;
  const int words = d * elem_bytes / 4;
  ProfScope prof(ctx, GRAM_K_OTHER, 2.0 * (double)n * d * elem_bytes, 1, st);
  strided_rows_kernel<<<(unsigned)ceil_div64(n * words, 256), 256, 0, st>>>((const uint32_t*)in, (uint32_t*)out, n, words,
                                                                          rows ? words : stride * words, words, nullptr, rows);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status sequence_layout(gram_ctx* ctx, const int32_t* item_len, const int32_t* items, int32_t first_item, int32_t n,
                            int32_t n_items_total, int l_t, int32_t* seq_len, int32_t* seq_off, int32_t* group_list,
                            int32_t* info, cudaStream_t st) {
  if (n <= 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_EMBED_POOL, 12.0 * (double)n, 1, st);
  seq_layout_kernel<<<1, 1024, 0, st>>>(item_len, items, first_item, n, n_items_total, l_t, seq_len, seq_off, group_list, info,
                                        gram_status_word(ctx));
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status pool_additive_forward(gram_ctx* ctx, int dtype, const StreamRef& x, const void* pre, const float* q, float* H,
                                  float* alpha, int64_t n, int l_t, int d, int pa, const int32_t* seq_len, const int32_t* seq_off,
                                  cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  if (l_t > 128) return gram_set_error(ctx, "additive pooling: at most 128 tokens per item"), GRAM_ERR_UNSUPPORTED;
  ProfScope prof(ctx, GRAM_K_EMBED_POOL, 4.0 * (double)n * l_t * (d + pa), 1, st);
  DISPATCH_T(dtype, pool_additive_fwd_kernel<T><<<(unsigned)n, 128, 0, st>>>(x, (const T*)pre, q, H, alpha, l_t, d, pa, seq_len, seq_off));
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
gram_status pool_additive_backward(gram_ctx* ctx, int dtype, const StreamRef& x, const void* pre, const float* q,
                                   const float* alpha, const float* G, float* dx, void* dpre, float* dq, float* scratch,
                                   int64_t n, int l_t, int d, int pa, const int32_t* seq_len, const int32_t* seq_off,
                                   cudaStream_t st) {
  if (n == 0) return GRAM_OK;
  if ((size_t)n * pa * sizeof(float) > kRedScratchBytes)
    return gram_set_error(ctx, "additive pooling: %lld items x %d exceed the reduction scratch", (long long)n, pa), GRAM_ERR_WORKSPACE;
  ProfScope prof(ctx, GRAM_K_EMBED_POOL, 4.0 * (double)n * l_t * (2 * d + 2 * pa), 2, st);
  DISPATCH_T(dtype, pool_additive_bwd_kernel<T><<<(unsigned)n, 128, 0, st>>>(x, (const T*)pre, q, alpha, G, dx, (T*)dpre, scratch, l_t, d,
                                                                            pa, seq_len, seq_off));
  reduce_partials_kernel<<<ceil_div(pa, 32), 256, 0, st>>>(scratch, (int)n, pa, pa, dq, nullptr, 1.f);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
