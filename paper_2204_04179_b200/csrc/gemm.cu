// Matrix products.  bf16: a persistent, warp-specialised tcgen05 kernel (one TMA producer warp, one
// MMA-issuing warp, eight epilogue warps; operands staged in 128-byte-swizzled shared memory by TMA,
// fp32 accumulators double-buffered in tensor memory so that the epilogue of one tile overlaps the
// main loop of the next).  fp32: a plain tiled CUDA-core kernel for the small fp32 configuration.
#include <cuda.h>
#include <stdlib.h>

#include "gemm.h"
#include "tc_common.cuh"

namespace {
using namespace tc;

// ============================================================================================
// fp32 CUDA-core kernel: C(m, n) = sum_k A(m, k) * B(n, k), generic strides
// ============================================================================================
struct EpiDev {
  const float* bias;
  const float* res;
  const float* res_mean;
  const float* res_rstd;
  const float* res_gamma;
  const float* res_beta;
  void* pre;
  const void* dgelu_pre;
  void* copy_out;
  float* colsum_part;
  int gelu;
  int accumulate;
};

template <typename CT> __device__ __forceinline__ float ld_c(const CT* p);
template <> __device__ __forceinline__ float ld_c<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld_c<bf16>(const bf16* p) { return __bfloat162float(*p); }
template <typename CT> __device__ __forceinline__ void st_c(CT* p, float v);
template <> __device__ __forceinline__ void st_c<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void st_c<bf16>(bf16* p, float v) { *p = __float2bfloat16(v); }

// one element; CT is C's type, OT the operands' type
template <typename CT, typename OT>
__device__ __forceinline__ void epilogue_store(const EpiDev& e, CT* C, int64_t ldc, int64_t m, int n, float acc) {
  float v = acc + (e.bias ? e.bias[n] : 0.f);
  const int64_t o = m * ldc + n;
  if (e.gelu) {
    if (e.pre) st_c<OT>(reinterpret_cast<OT*>(e.pre) + o, gelu_grad_f(v));
    v = gelu_f(v);
  }
  if (e.dgelu_pre) v *= ld_c<OT>(reinterpret_cast<const OT*>(e.dgelu_pre) + o);
  if (e.res) {
    float r = e.res[o];
    if (e.res_mean) r = (r - e.res_mean[m]) * e.res_rstd[m] * e.res_gamma[n] + e.res_beta[n];
    v += r;
  }
  if (e.accumulate) v += ld_c<CT>(C + o);
  st_c<CT>(C + o, v);
  if (e.copy_out) st_c<OT>(reinterpret_cast<OT*>(e.copy_out) + o, v);
}

// four consecutive columns n..n+3 of row m (n, ldc multiples of 4): the unit of the coalesced epilogue
__device__ __forceinline__ void ld4(const float* p, float (&x)[4]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
}
__device__ __forceinline__ void ld4(const bf16* p, float (&x)[4]) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  const float2 f0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
  const float2 f1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
  x[0] = f0.x; x[1] = f0.y; x[2] = f1.x; x[3] = f1.y;
}
__device__ __forceinline__ void st4(float* p, const float (&x)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
}
__device__ __forceinline__ void st4(bf16* p, const float (&x)[4]) {
  __nv_bfloat162 h0 = __floats2bfloat162_rn(x[0], x[1]), h1 = __floats2bfloat162_rn(x[2], x[3]);
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
}

// GELU and its derivative for the tensor-core epilogue.  erf comes from the rational approximation
// 7.1.26 of Abramowitz & Stegun, erf(y) = 1 - (a1 t + ... + a5 t^5) exp(-y^2), t = 1 / (1 + p y), whose
// absolute error is below 1.5e-7: far under the bf16 resolution of the values that are stored.  With
// y = |x| / sqrt(2) the exponential exp(-x^2 / 2) is also the Gaussian density the derivative needs.
__device__ __forceinline__ void gelu_parts(float x, float& cdf, float& pdf) {
  const float ax = fabsf(x);
  float ex, t;                                            // flush-to-zero forms: one MUFU each, no range fix-up
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(ex) : "f"(x * x * -0.72134752f));            // exp(-x^2 / 2)
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f * 0.70710678f, ax, 1.f)));
  const float poly = t * (0.254829592f + t * (-0.284496736f + t * (1.421413741f + t * (-1.453152027f + t * 1.061405429f))));
  const float erf_abs = 1.f - poly * ex;                  // erf(|x| / sqrt 2)
  cdf = 0.5f * (1.f + copysignf(erf_abs, x));
  pdf = 0.39894228f * ex;
}

// The same for two values at a time with the packed fp32 instructions of sm_100 (two lanes of one 64-bit
// register): x holds the two pre-activations; on return g = gelu(x), dg = gelu'(x).  Half the instruction
// slots of the scalar form, which is what bounds the epilogue of the first feed-forward product.
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t f2_const(float c) {
  const uint64_t u = (uint64_t)__float_as_uint(c);
  return u | (u << 32);
}
__device__ __forceinline__ void gelu_pair(uint64_t x, uint64_t& g, uint64_t& dg) {
  float e0, e1, y0, y1;
  f2_unpack(f2_mul(f2_mul(x, x), f2_const(-0.72134752f)), e0, e1);
  asm("ex2.approx.ftz.f32 %0, %0;" : "+f"(e0));                          // exp(-x^2 / 2)
  asm("ex2.approx.ftz.f32 %0, %0;" : "+f"(e1));
  const uint64_t ex = f2_pack(e0, e1);
  f2_unpack(f2_fma(x & 0x7FFFFFFF7FFFFFFFull, f2_const(0.3275911f * 0.70710678f), f2_const(1.f)), y0, y1);
  asm("rcp.approx.ftz.f32 %0, %0;" : "+f"(y0));
  asm("rcp.approx.ftz.f32 %0, %0;" : "+f"(y1));
  const uint64_t t = f2_pack(y0, y1);
  uint64_t p = f2_fma(t, f2_const(1.061405429f), f2_const(-1.453152027f));
  p = f2_fma(p, t, f2_const(1.421413741f));
  p = f2_fma(p, t, f2_const(-0.284496736f));
  p = f2_fma(p, t, f2_const(0.254829592f));
  p = f2_mul(p, t);
  const uint64_t h = f2_fma(f2_mul(p, ex), f2_const(-0.5f), f2_const(0.5f));    // erf(|x| / sqrt 2) / 2
  const uint64_t cdf = f2_add(h | (x & 0x8000000080000000ull), f2_const(0.5f));   // 1/2 + sign(x) * h
  g = f2_mul(x, cdf);
  dg = f2_fma(f2_mul(x, ex), f2_const(0.39894228f), cdf);
}
__device__ __forceinline__ uint32_t f2_to_bf16x2(uint64_t v) {
  float lo, hi;
  f2_unpack(v, lo, hi);
  return pack_bf16x2(lo, hi);
}

// what one lane reads before it may store anything for its 4 columns of one row: the residual, the
// saved GELU derivative or the old value of C (the tensor-core path takes at most one of the three)
struct EpiLoads {
  float aux[4];
};
template <typename CT>
__device__ __forceinline__ void epilogue_load4(const EpiDev& e, const CT* C, int64_t ldc, int64_t m, int n, EpiLoads& L) {
  const int64_t o = m * ldc + n;
  if (e.res) ld4(e.res + o, L.aux);
  else if (e.dgelu_pre) ld4(reinterpret_cast<const bf16*>(e.dgelu_pre) + o, L.aux);
  else if (e.accumulate) ld4(reinterpret_cast<const float*>(C) + o, L.aux);      // accumulation is offered for fp32 C only
}
template <typename CT>
__device__ __forceinline__ void epilogue_store4(const EpiDev& e, CT* C, int64_t ldc, int64_t m, int n, float (&v)[4],
                                                const EpiLoads& L, const float (&bias)[4], const float (&gam)[4],
                                                const float (&bet)[4], float mu, float rs) {
  const int64_t o = m * ldc + n;
  if (e.bias) {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] += bias[i];
  }
  if (e.gelu) {
    float dg[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float c, p;
      gelu_parts(v[i], c, p);
      dg[i] = c + v[i] * p;        // gelu'(v), kept for the backward pass
      v[i] = v[i] * c;             // gelu(v)
    }
    if (e.pre) st4(reinterpret_cast<bf16*>(e.pre) + o, dg);
  }
  if (e.res) {
    if (e.res_mean) {
#pragma unroll
      for (int i = 0; i < 4; ++i) v[i] += (L.aux[i] - mu) * rs * gam[i] + bet[i];
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) v[i] += L.aux[i];
    }
  } else if (e.dgelu_pre) {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] *= L.aux[i];
  } else if (e.accumulate) {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] += L.aux[i];
  }
  st4(C + o, v);
  if (e.copy_out) st4(reinterpret_cast<bf16*>(e.copy_out) + o, v);
}

constexpr int ST = 64, SK = 16;
__global__ void __launch_bounds__(256) gemm_f32_kernel(const float* __restrict__ A, int64_t sam, int64_t sak,
                                                       const float* __restrict__ B, int64_t sbn, int64_t sbk,
                                                       float* __restrict__ C, int64_t ldc, int64_t M, int N, int64_t K,
                                                       EpiDev e) {
  __shared__ float As[SK][ST + 1];
  __shared__ float Bs[SK][ST + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int64_t m0 = (int64_t)blockIdx.y * ST;
  const int n0 = blockIdx.x * ST;
  float acc[4][4] = {};
  for (int64_t k0 = 0; k0 < K; k0 += SK) {
    for (int i = threadIdx.x; i < ST * SK; i += 256) {
      int r, k;
      if (sak == 1) { r = i / SK; k = i % SK; } else { k = i / ST; r = i % ST; }
      As[k][r] = (m0 + r < M && k0 + k < K) ? A[(m0 + r) * sam + (k0 + k) * sak] : 0.f;
    }
    for (int i = threadIdx.x; i < ST * SK; i += 256) {
      int r, k;
      if (sbk == 1) { r = i / SK; k = i % SK; } else { k = i / ST; r = i % ST; }
      Bs[k][r] = (n0 + r < N && k0 + k < K) ? B[(int64_t)(n0 + r) * sbn + (k0 + k) * sbk] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < SK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty + 16 * i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx + 16 * j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * b[j];
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int64_t m = m0 + ty + 16 * i;
      int n = n0 + tx + 16 * j;
      if (m < M && n < N) epilogue_store<float, float>(e, C, ldc, m, n, acc[i][j]);
    }
}

// ============================================================================================
// bf16 tcgen05 kernel
// ============================================================================================
constexpr int BM = 128, BK = 64;
constexpr int EPI_WARPS = 8;
constexpr int TC_THREADS = 64 + 32 * EPI_WARPS;   // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue
constexpr int STAGE_LD = 32;                     // a warp's 32 x 32 fp32 transpose buffer (swizzled, no padding)
// A warp's 32 x 32 fp32 transpose buffer: rows of eight 16-byte slots, slot j of row r stored at j ^ (r & 7).
// Row-per-thread writes and eight-lanes-per-row reads are then both free of bank conflicts.
__device__ __forceinline__ void stage_write_row(float* stage, int lane, const uint32_t (&v)[32]) {
  float4* s4 = reinterpret_cast<float4*>(stage) + lane * 8;
#pragma unroll
  for (int j = 0; j < 8; ++j)
    s4[j ^ (lane & 7)] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                     __uint_as_float(v[4 * j + 3]));
}
__device__ __forceinline__ float4 stage_read(const float* stage, int row, int slot) {
  return reinterpret_cast<const float4*>(stage)[row * 8 + (slot ^ (row & 7))];
}

struct TcArgs {
  void* C;
  int64_t ldc;
  int64_t M;
  int32_t N;
  int32_t num_kb;          // k-blocks of 64 over the whole K
  int32_t n_tiles_m, n_tiles_n, splits, kb_per_split;
  int64_t split_stride;    // elements between the partial outputs of two splits
  EpiDev epi;
  int32_t* status;
};

template <int BN> struct TcCfg {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : (BN == 128 ? 6 : 8);
  static constexpr int TMEM_COLS = 2 * BN;           // two accumulator buffers
  static constexpr int EPI_BYTES = EPI_WARPS * 32 * STAGE_LD * 4;   // per-warp transpose buffers of the epilogue
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// The epilogue of one output tile for one epilogue warp: rows row0 .. row0+31 (TMEM lanes q*32..), columns
// [half*BN/PARTS, (half+1)*BN/PARTS) of tile column tn.  A warp may read only its quarter of the TMEM lanes; PARTS warps
// share a quarter and split the columns.  Each 32 x 32 block is loaded one row per thread, turned through a
// padded shared-memory buffer, and then handled four rows per instruction with eight lanes per row, so that
// global loads and stores of a row are contiguous 128-byte pieces.  Returns false if the bounded wait for the
// accumulator gave up.
// DG: the epilogue is only "multiply by the saved GELU derivative, store bf16" (backward of the
// feed-forward layer); the derivative's values for the whole tile are then fetched into registers
// while the main loop of that tile is still running, which hides their HBM latency.
// Epilogue variants fixed at compile time (the general one reads the EpiDev flags at run time):
//   EPI_DG    multiply by the saved GELU derivative, bf16 out (values prefetched during the main loop)
//   EPI_BIAS  (+ bias), bf16 or fp32 out
//   EPI_GELU  + bias, GELU, saved derivative, both bf16
//   EPI_RES   (+ bias) + fp32 residual (LayerNorm on the fly when res_mean is set), fp32 out (+ bf16 copy)
//   EPI_RES_TS  the same without the bf16 copy, residual in and result out by bulk tensor copies (pair kernel)
enum { EPI_GENERAL = 0, EPI_DG = 1, EPI_BIAS = 2, EPI_GELU = 3, EPI_RES = 4, EPI_RES_TS = 5 };

template <int BN, typename CT, int MODE, int PARTS = 2>
__device__ __forceinline__ bool epilogue_tile(const TcArgs& a, CT* Cs, int64_t row0, int tn, int half, int q, int lane,
                                              float* stage, uint32_t tmem_base, int buf, uint32_t tfull_addr,
                                              uint32_t parity, volatile int* abort_flag) {
  if constexpr (MODE == EPI_DG) {
    uint2 pf[BN / (32 * PARTS)][8];                       // packed bf16: 4 columns of one row per entry
    const int sub = lane >> 3, slot = lane & 7;
    const int64_t rows_left = a.M - (row0 + sub);
    const int64_t step = 4 * a.ldc;
    const int ncol0 = tn * BN + half * (BN / PARTS) + slot * 4;
    const int64_t o0 = (row0 + sub) * a.ldc + ncol0;
    const bf16* pre = reinterpret_cast<const bf16*>(a.epi.dgelu_pre) + o0;
#pragma unroll
    for (int blk = 0; blk < BN / (32 * PARTS); ++blk) {
      const bool col_ok = ncol0 + blk * 32 < a.N;
#pragma unroll
      for (int rr = 0; rr < 8; ++rr)
        pf[blk][rr] = (col_ok && rr * 4 < rows_left) ? *reinterpret_cast<const uint2*>(pre + blk * 32 + rr * step) : make_uint2(0u, 0u);
    }
    if (!mbar_wait(tfull_addr, parity, abort_flag)) return false;
    tc_fence_after();
#pragma unroll
    for (int blk = 0; blk < BN / (32 * PARTS); ++blk) {
      const int c0 = half * (BN / PARTS) + blk * 32;
      uint32_t v[32];
      tc_ld32_issue(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), v);
      tc_ld32_wait(v);
      stage_write_row(stage, lane, v);
      __syncwarp();
      if (ncol0 + blk * 32 < a.N) {
        CT* cp = Cs + o0 + blk * 32;
#pragma unroll
        for (int rr = 0; rr < 8; ++rr) {
          if (rr * 4 < rows_left) {
            const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pf[blk][rr].x));
            const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pf[blk][rr].y));
            const float4 t = stage_read(stage, rr * 4 + sub, slot);
            const float x[4] = {t.x * g0.x, t.y * g0.y, t.z * g1.x, t.w * g1.y};
            st4(cp, x);
          }
          cp += step;
        }
      }
      __syncwarp();
    }
    tc_fence_before();
    return true;
  } else if constexpr (MODE == EPI_RES) {
    // fp32 result = accumulator (+ bias) + residual (LayerNorm applied where it is read), plus an optional bf16 copy.
    // The residual is 4 bytes per element from HBM, and eight warps per SM keep too few loads in flight to hide its
    // latency if every 32-column block waits for its own: the loads of a block are therefore issued one block ahead,
    // the first block's before the wait for the accumulator.
    constexpr int NBLK = BN / PARTS / 32;
    const int sub = lane >> 3, slot = lane & 7;
    const int64_t rows_left = a.M - (row0 + sub);         // row rr*4 + sub exists iff rr*4 < rows_left
    const int64_t step = 4 * a.ldc;
    const int nbase = tn * BN + half * (BN / PARTS) + slot * 4;
    const int64_t obase = (row0 + sub) * a.ldc + nbase;
    float4 rnext[8];
    auto load_res = [&](int blk, float4 (&dst)[8]) {
      const bool col_ok = nbase + blk * 32 < a.N;
      const float* rp = a.epi.res + obase + blk * 32;
#pragma unroll
      for (int rr = 0; rr < 8; ++rr)
        dst[rr] = (col_ok && rr * 4 < rows_left) ? __ldcs(reinterpret_cast<const float4*>(rp + rr * step)) : make_float4(0.f, 0.f, 0.f, 0.f);
    };
    load_res(0, rnext);
    float mu_l = 0.f, rs_l = 1.f;
    const bool ln = a.epi.res_mean != nullptr;
    if (ln && row0 + lane < a.M) {
      mu_l = a.epi.res_mean[row0 + lane];
      rs_l = a.epi.res_rstd[row0 + lane];
    }
    if (!mbar_wait(tfull_addr, parity, abort_flag)) return false;
    tc_fence_after();
#pragma unroll 1
    for (int blk = 0; blk < NBLK; ++blk) {
      float4 r4[8];
#pragma unroll
      for (int rr = 0; rr < 8; ++rr) r4[rr] = rnext[rr];
      if (blk + 1 < NBLK) load_res(blk + 1, rnext);
      uint32_t v[32];
      tc_ld32_issue(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + half * (BN / PARTS) + blk * 32), v);
      tc_ld32_wait(v);
      stage_write_row(stage, lane, v);
      __syncwarp();
      const int n = nbase + blk * 32;
      const bool col_ok = n < a.N;                          // lanes of a warp may differ here when N is not a multiple of 32
      float b4[4] = {0.f, 0.f, 0.f, 0.f}, g4[4] = {0.f, 0.f, 0.f, 0.f}, be4[4] = {0.f, 0.f, 0.f, 0.f};
      if (col_ok) {
        if (a.epi.bias) ld4(a.epi.bias + n, b4);
        if (ln) {
          ld4(a.epi.res_gamma + n, g4);
          ld4(a.epi.res_beta + n, be4);
        }
      }
      CT* cp = Cs + obase + blk * 32;
      bf16* qp = a.epi.copy_out ? reinterpret_cast<bf16*>(a.epi.copy_out) + obase + blk * 32 : nullptr;
#pragma unroll
      for (int rr = 0; rr < 8; ++rr) {
        const int rl = rr * 4 + sub;
        // every lane takes part in the shuffles, whatever its columns
        const float mu = __shfl_sync(0xffffffffu, mu_l, rl), rs = __shfl_sync(0xffffffffu, rs_l, rl);
        if (col_ok && rr * 4 < rows_left) {
          const float4 t = stage_read(stage, rl, slot);
          float x[4] = {t.x + b4[0], t.y + b4[1], t.z + b4[2], t.w + b4[3]};
          if (ln) {
            x[0] += (r4[rr].x - mu) * rs * g4[0] + be4[0];
            x[1] += (r4[rr].y - mu) * rs * g4[1] + be4[1];
            x[2] += (r4[rr].z - mu) * rs * g4[2] + be4[2];
            x[3] += (r4[rr].w - mu) * rs * g4[3] + be4[3];
          } else {
            x[0] += r4[rr].x; x[1] += r4[rr].y; x[2] += r4[rr].z; x[3] += r4[rr].w;
          }
          st4(cp, x);
          if (qp) st4(qp, x);
        }
        cp += step;
        if (qp) qp += step;
      }
      __syncwarp();
    }
    tc_fence_before();
    return true;
  } else if constexpr (MODE == EPI_BIAS || MODE == EPI_GELU) {
    if (!mbar_wait(tfull_addr, parity, abort_flag)) return false;
    tc_fence_after();
    const int sub = lane >> 3, slot = lane & 7;
    const int64_t rows_left = a.M - (row0 + sub);         // row rr*4 + sub exists iff rr*4 < rows_left
#pragma unroll 1
    for (int c0 = half * (BN / PARTS); c0 < (half + 1) * (BN / PARTS); c0 += 32) {
      uint32_t v[32];
      tc_ld32_issue(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), v);
      tc_ld32_wait(v);
      stage_write_row(stage, lane, v);
      __syncwarp();
      const int n = tn * BN + c0 + slot * 4;
      if (n < a.N) {                                      // N is a multiple of 8
        float b4[4] = {0.f, 0.f, 0.f, 0.f};
        if (a.epi.bias) ld4(a.epi.bias + n, b4);
        const int64_t o0 = (row0 + sub) * a.ldc + n;      // element offset of this lane's first row
        const int64_t step = 4 * a.ldc;
        if constexpr (MODE == EPI_BIAS) {
          CT* cp = Cs + o0;
#pragma unroll
          for (int rr = 0; rr < 8; ++rr) {
            if (rr * 4 < rows_left) {
              const float4 t = stage_read(stage, rr * 4 + sub, slot);
              const float x[4] = {t.x + b4[0], t.y + b4[1], t.z + b4[2], t.w + b4[3]};
              st4(cp, x);
            }
            cp += step;
          }
        } else if constexpr (MODE == EPI_GELU) {
          CT* cp = Cs + o0;
          bf16* pp = reinterpret_cast<bf16*>(a.epi.pre) + o0;
#pragma unroll
          for (int rr = 0; rr < 8; ++rr) {
            if (rr * 4 < rows_left) {
              const float4 t = stage_read(stage, rr * 4 + sub, slot);
              float x[4] = {t.x + b4[0], t.y + b4[1], t.z + b4[2], t.w + b4[3]};
              float dg[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                float c, p;
                gelu_parts(x[i], c, p);
                dg[i] = c + x[i] * p;
                x[i] *= c;
              }
              st4(cp, x);
              st4(pp, dg);
            }
            cp += step;
            pp += step;
          }
        }
      }
      __syncwarp();
    }
    tc_fence_before();
    return true;
  } else {
    if (!mbar_wait(tfull_addr, parity, abort_flag)) return false;
    tc_fence_after();
    float mu_l = 0.f, rs_l = 1.f;               // LayerNorm statistics of row row0 + lane
    if (a.epi.res_mean && row0 + lane < a.M) {
      mu_l = a.epi.res_mean[row0 + lane];
      rs_l = a.epi.res_rstd[row0 + lane];
    }
#pragma unroll 1
    for (int c0 = half * (BN / PARTS); c0 < (half + 1) * (BN / PARTS); c0 += 32) {
      uint32_t v[32];
      tc_ld32_issue(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), v);
      tc_ld32_wait(v);
      stage_write_row(stage, lane, v);
      __syncwarp();
      const int n = tn * BN + c0 + (lane & 7) * 4;
      const bool col_ok = n < a.N;                // N is a multiple of 8
      float bias4[4] = {0.f, 0.f, 0.f, 0.f}, gam4[4] = {0.f, 0.f, 0.f, 0.f}, bet4[4] = {0.f, 0.f, 0.f, 0.f};
      if (col_ok) {
        if (a.epi.bias) ld4(a.epi.bias + n, bias4);
        if (a.epi.res_mean) {
          ld4(a.epi.res_gamma + n, gam4);
          ld4(a.epi.res_beta + n, bet4);
        }
      }
      // global loads of four rows are issued before the first store of those rows
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        EpiLoads L[4];
#pragma unroll
        for (int r4 = 0; r4 < 4; ++r4) {
          const int64_t m = row0 + (hh * 4 + r4) * 4 + (lane >> 3);
          if (m < a.M && col_ok) epilogue_load4<CT>(a.epi, Cs, a.ldc, m, n, L[r4]);
        }
#pragma unroll
        for (int r4 = 0; r4 < 4; ++r4) {
          const int rl = (hh * 4 + r4) * 4 + (lane >> 3);
          const float mu = __shfl_sync(0xffffffffu, mu_l, rl), rs = __shfl_sync(0xffffffffu, rs_l, rl);
          const int64_t m = row0 + rl;
          if (m < a.M && col_ok) {
            const float4 t = stage_read(stage, rl, lane & 7);
            float x[4] = {t.x, t.y, t.z, t.w};
            epilogue_store4<CT>(a.epi, Cs, a.ldc, m, n, x, L[r4], bias4, gam4, bet4, mu, rs);
          }
        }
      }
      __syncwarp();
    }
    tc_fence_before();
    return true;
  }
}

template <int BN, bool A_K, bool B_K, typename CT, int MODE = EPI_GENERAL>
__global__ void __launch_bounds__(TC_THREADS, 1) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA,
                                                               const __grid_constant__ CUtensorMap tmB, TcArgs a) {
  using Cfg = TcCfg<BN>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;                 // swizzled tiles need 1024-byte alignment
  uint8_t* gen_tiles = smem_raw + (tiles - raw);
  float* epi_stage = reinterpret_cast<float*>(gen_tiles + STAGES * Cfg::STAGE_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_tiles + STAGES * Cfg::STAGE_BYTES + Cfg::EPI_BYTES);
  const uint32_t bar0 = tiles + STAGES * Cfg::STAGE_BYTES + Cfg::EPI_BYTES;
  // barrier slots: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]; then tmem base, abort flag
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), 32 * EPI_WARPS);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)Cfg::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int64_t total = (int64_t)a.n_tiles_m * a.n_tiles_n * a.splits;
  bool failed = false;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int64_t t = blockIdx.x; t < total && !failed; t += gridDim.x) {
        const int split = (int)(t / ((int64_t)a.n_tiles_m * a.n_tiles_n));
        const int64_t r = t - (int64_t)split * a.n_tiles_m * a.n_tiles_n;
        const int tm = (int)(r / a.n_tiles_n), tn = (int)(r % a.n_tiles_n);
        const int kb0 = split * a.kb_per_split, kb1 = min(kb0 + a.kb_per_split, a.num_kb);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { failed = true; break; }
          mbar_expect_tx(full_bar(s), Cfg::STAGE_BYTES);
          const uint32_t sa = tiles + s * Cfg::STAGE_BYTES, sb = sa + Cfg::A_BYTES;
          if (A_K) {
            tma_load_2d(sa, &tmA, kb * BK, tm * BM, full_bar(s));
          } else {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) tma_load_2d(sa + i * 8192, &tmA, tm * BM + i * 64, kb * BK, full_bar(s));
          }
          if (B_K) {
            tma_load_2d(sb, &tmB, kb * BK, tn * BN, full_bar(s));
          } else {
#pragma unroll
            for (int i = 0; i < BN / 64; ++i) tma_load_2d(sb + i * 8192, &tmB, tn * BN + i * 64, kb * BK, full_bar(s));
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
      if (failed) {
        *abort_flag = 1;
        gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_K ? 0u : 1u) << 15) |
                                 ((B_K ? 0u : 1u) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      int s = 0;
      uint32_t ph = 0;
      int64_t it = 0;
      for (int64_t t = blockIdx.x; t < total && !failed; t += gridDim.x, ++it) {
        const int split = (int)(t / ((int64_t)a.n_tiles_m * a.n_tiles_n));
        const int kb0 = split * a.kb_per_split, kb1 = min(kb0 + a.kb_per_split, a.num_kb);
        const int buf = (int)(it & 1);
        if (!mbar_wait(tempty_bar(buf), (uint32_t)((it >> 1) & 1) ^ 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(buf * BN);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t sa = tiles + s * Cfg::STAGE_BYTES, sb = sa + Cfg::A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = A_K ? make_desc(sa + k * 32, 16, 1024) : make_desc(sa + k * 2048, 8192, 1024);
            const uint64_t db = B_K ? make_desc(sb + k * 32, 16, 1024) : make_desc(sb + k * 2048, 8192, 1024);
            tc_mma(tmem_d, da, db, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(s));            // the stage is free once these MMAs have read it
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (failed) break;
        tc_commit(tfull_bar(buf));            // accumulator complete
      }
      if (failed) {
        *abort_flag = 1;
        gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
      }
    }
  } else {
    // ------------------------------ epilogue warps ----------------------------
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    float* stage = epi_stage + ew * (32 * STAGE_LD);
    CT* C = reinterpret_cast<CT*>(a.C);
    int64_t it = 0;
    for (int64_t t = blockIdx.x; t < total && !failed; t += gridDim.x, ++it) {
      const int split = (int)(t / ((int64_t)a.n_tiles_m * a.n_tiles_n));
      const int64_t r = t - (int64_t)split * a.n_tiles_m * a.n_tiles_n;
      const int tm = (int)(r / a.n_tiles_n), tn = (int)(r % a.n_tiles_n);
      const int buf = (int)(it & 1);
      const int64_t row0 = (int64_t)tm * BM + q * 32;
      CT* Cs = C + (int64_t)split * a.split_stride;
      if (!epilogue_tile<BN, CT, MODE>(a, Cs, row0, tn, half, q, lane, stage, tmem_base, buf, tfull_bar(buf),
                                     (uint32_t)((it >> 1) & 1), abort_flag)) {
        failed = true;
        break;
      }
      mbar_arrive(tempty_bar(buf));           // all epilogue threads free the accumulator buffer
    }
    if (failed && lane == 0) {
      *abort_flag = 1;
      gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
    }
  }

  // ------------------------------ teardown --------------------------------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // a wait gave up: let copies and MMAs already issued drain (bounded) before memory is released
    if (warp == 0 && lane == 0) {
      for (int s = 0; s < STAGES; ++s) {
        uint64_t t0 = clock64();
        while (!mbar_try(full_bar(s), 0) && !mbar_try(full_bar(s), 1) && clock64() - t0 < WAIT_LIMIT_CYCLES / 64) {}
      }
    }
    if (warp == 1 && lane == 0) {
      uint64_t t0 = clock64();
      while (clock64() - t0 < WAIT_LIMIT_CYCLES / 64) {}
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS)
                 : "memory");
  }
}

// ============================================================================================
// The same product on pairs of SMs (tcgen05 cta_group::2): a cluster of two CTAs owns a 256 x 256
// output tile.  Each CTA stages its own 128 rows of A and its own 128 of the tile's 256 columns of B,
// the leader CTA (cluster rank 0) issues one M256 N256 K16 MMA per step that reads both CTAs' shared
// memory, and each CTA's tensor memory receives its 128 rows of the result.  Per CTA and k-block this
// moves 32 KB through shared memory instead of 48 KB, which is what bounds the single-CTA kernel.
// Protocol: each CTA's TMA loads signal the leader's "full" barrier (two arrivals with their byte
// counts); the leader's commits arrive on the "empty" and "accumulator full" barriers of both CTAs
// (one plain commit per CTA); the epilogue warps of both CTAs arrive on the leader's
// "accumulator empty" barrier.  Every wait is bounded as in the single-CTA kernel; the CTAs meet at a
// cluster barrier before they exit so that neither releases shared or tensor memory the other may
// still touch.
// ============================================================================================
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_expect_tx_remote(uint32_t cluster_bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1,
                                                 uint32_t cluster_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t cluster_bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(accum)
      : "memory");
}

// Epilogue of the pair kernel for bf16 results (EPI_BIAS, EPI_GELU, EPI_DG): one warp owns rows row0 .. row0+31
// and NB blocks of 32 columns from global column col0 (tile column c_local).  A thread keeps its own row: 32
// accumulators from tensor memory per block, the arithmetic, 64 bytes of bf16 written into a 32-row x 64-column
// box in shared memory (128-byte rows whose 16-byte pieces are XOR-swizzled as the 128-byte swizzle of the
// tensor map expects, which also keeps the writes free of bank conflicts).  Two blocks fill a box, and lane 0
// hands it to a bulk tensor store, which writes whole 128-byte lines and clips the box at the matrix edges.
// EPI_GELU fills a second box with the derivative; EPI_DG (NB = 2) first fetches the box of the saved derivative
// with a bulk tensor load (issued before the wait for the accumulator), multiplies in place and stores the same
// box.  The accumulator buffer is handed back as soon as the last block has been read.  sbuf: 4 KB (8 KB for
// EPI_GELU), 1024-byte aligned, private to the warp.  Returns false if a bounded wait gave up.
template <int MODE, int NB>
__device__ __forceinline__ bool epilogue_tile_ts(const TcArgs& a, const CUtensorMap* tmC, const CUtensorMap* tmP, int32_t row0,
                                                 int32_t col0, int c_local, int q, int lane, uint32_t sbuf,
                                                 uint32_t tmem_base, int buf, uint32_t tfull_addr, uint32_t parity,
                                                 volatile int* abort_flag, uint32_t tempty_remote, uint32_t ld_bar,
                                                 uint32_t ld_parity) {
  static_assert(MODE != EPI_DG || NB == 2, "the derivative's box is fetched once per tile");
  const uint32_t swz = (uint32_t)(lane & 7);
  const uint32_t srow = sbuf + (uint32_t)lane * 128u;
  if constexpr (MODE == EPI_DG) {
    if (lane == 0) {
      bulk_wait_read_all();                                // the last tile's store has read the box
      mbar_expect_tx(ld_bar, 4096);
      tma_load_2d(sbuf, tmP, col0, row0, ld_bar);
    }
    __syncwarp();
  }
  if (!mbar_wait(tfull_addr, parity, abort_flag)) return false;
  tc_fence_after();
  if constexpr (MODE == EPI_DG) {
    if (!mbar_wait(ld_bar, ld_parity, abort_flag)) return false;
  }
  const bool rows_ok = row0 < a.M;                         // a box that starts below the matrix is not stored
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    uint32_t v[32];
    tc_ld32_issue(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 256 + c_local + b * 32), v);
    tc_ld32_wait(v);
    if (b == NB - 1) {                                     // every value of this tile is in registers now
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(tempty_remote);
    }
    const int nbx = col0 + (b >> 1) * 64;                  // first column of the box
    const int n = col0 + b * 32;
    if (nbx >= a.N || !rows_ok) continue;
    const uint32_t p0 = (uint32_t)(b & 1) * 4u;            // this block's first 16-byte piece of the row
    uint32_t oc[16];
    if constexpr (MODE == EPI_DG) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint4 g4 = lds128(srow + (((p0 + (uint32_t)c) ^ swz) << 4));
        const uint32_t gw[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 gg = unpack_bf16x2(gw[i]);
          oc[4 * c + i] = pack_bf16x2(__uint_as_float(v[8 * c + 2 * i]) * gg.x, __uint_as_float(v[8 * c + 2 * i + 1]) * gg.y);
        }
      }
#pragma unroll
      for (int c = 0; c < 4; ++c)
        sts128(srow + (((p0 + (uint32_t)c) ^ swz) << 4), oc[4 * c], oc[4 * c + 1], oc[4 * c + 2], oc[4 * c + 3]);
    } else {
      uint32_t op[MODE == EPI_GELU ? 16 : 1];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (a.epi.bias && n + 4 * j < a.N) b4 = __ldg(reinterpret_cast<const float4*>(a.epi.bias + n + 4 * j));
        if constexpr (MODE == EPI_GELU) {
          uint64_t g0, g1, d0, d1;
          gelu_pair(f2_add(f2_pack(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1])), f2_pack(b4.x, b4.y)), g0, d0);
          gelu_pair(f2_add(f2_pack(__uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])), f2_pack(b4.z, b4.w)), g1, d1);
          oc[2 * j] = f2_to_bf16x2(g0);
          oc[2 * j + 1] = f2_to_bf16x2(g1);
          op[2 * j] = f2_to_bf16x2(d0);
          op[2 * j + 1] = f2_to_bf16x2(d1);
        } else {
          oc[2 * j] = pack_bf16x2(__uint_as_float(v[4 * j]) + b4.x, __uint_as_float(v[4 * j + 1]) + b4.y);
          oc[2 * j + 1] = pack_bf16x2(__uint_as_float(v[4 * j + 2]) + b4.z, __uint_as_float(v[4 * j + 3]) + b4.w);
        }
      }
      if ((b & 1) == 0) {                                  // the last store from the box(es) has read them
        if (lane == 0) bulk_wait_read_all();
        __syncwarp();
      }
#pragma unroll
      for (int c = 0; c < 4; ++c)
        sts128(srow + (((p0 + (uint32_t)c) ^ swz) << 4), oc[4 * c], oc[4 * c + 1], oc[4 * c + 2], oc[4 * c + 3]);
      if constexpr (MODE == EPI_GELU) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
          sts128(srow + 4096u + (((p0 + (uint32_t)c) ^ swz) << 4), op[4 * c], op[4 * c + 1], op[4 * c + 2], op[4 * c + 3]);
      }
    }
    if (b & 1) {
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        tma_store_2d(tmC, sbuf, nbx, row0);
        if constexpr (MODE == EPI_GELU) tma_store_2d(tmP, sbuf + 4096, nbx, row0);
        bulk_commit();
      }
      if constexpr (MODE == EPI_DG) {
        if (a.epi.colsum_part) {
          // column sums of the box as stored (rows and columns outside the matrix hold zeros): lane c adds
          // columns 2c, 2c+1 over the 32 rows in ascending order and writes row (row0 / 32) of the partial sums
          float s0 = 0.f, s1 = 0.f;
          const uint32_t piece = (uint32_t)(lane >> 2), word = (uint32_t)(lane & 3) * 4u;
#pragma unroll 8
          for (uint32_t r = 0; r < 32; ++r) {
            uint32_t w;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(sbuf + r * 128u + ((piece ^ (r & 7u)) << 4) + word) : "memory");
            const float2 f = unpack_bf16x2(w);
            s0 += f.x;
            s1 += f.y;
          }
          const int cc = nbx + 2 * lane;
          if (cc < a.N) *reinterpret_cast<float2*>(a.epi.colsum_part + (int64_t)(row0 >> 5) * a.N + cc) = make_float2(s0, s1);
          __syncwarp();                                    // every lane has read the box before it is refilled
        }
      }
    }
  }
  return true;
}

// Epilogue of the pair kernel for the fp32 residual products (EPI_RES_TS): result = accumulator (+ bias) + residual,
// the residual being the fp32 stream or LayerNorm of it applied where it is read.  One warp owns rows row0 .. row0+31
// and four blocks of 32 columns from global column col0.  The residual is 4 bytes per element from HBM and the result
// 4 bytes back: both travel as 32-row x 32-column boxes (128-byte rows, 128-byte swizzle) by bulk tensor copies, so the
// warp issues no global load or store of its own and many boxes are in flight per SM.  A thread keeps its own row: 32
// accumulators from tensor memory, its row of the residual box from shared memory, the sum written back in place,
// and lane 0 hands the box to a bulk tensor store.  Three boxes per warp rotate (block k of the warp's running count
// uses box k % 3 and load barrier k % 3): the loads of a tile's first two blocks are issued before the wait for the
// accumulator, that of block b + 2 after the store of block b has been committed and the store before it has read its box.
// sbuf: 12 KB, 1024-byte aligned, private to the warp; nb: the warp's running block count.
__device__ __forceinline__ bool epilogue_tile_res(const TcArgs& a, const CUtensorMap* tmC, const CUtensorMap* tmR, int32_t row0,
                                                  int32_t col0, int c_local, int q, int lane, uint32_t sbuf, uint32_t tmem_base,
                                                  int buf, uint32_t tfull_addr, uint32_t parity, volatile int* abort_flag,
                                                  uint32_t tempty_remote, uint32_t ld_bar0, uint32_t& nb) {
  int nv = 0;                                               // blocks of this warp that lie inside the matrix
  if (row0 < a.M) {
    nv = (a.N - col0 + 31) / 32;
    nv = nv < 0 ? 0 : (nv > 4 ? 4 : nv);
  }
  auto request = [&](int b) {                               // residual box of block b of this tile -> box (nb + b) % 3
    const uint32_t k = nb + (uint32_t)b;
    const uint32_t bar = ld_bar0 + 8u * (k % 3u);
    mbar_expect_tx(bar, 4096);
    tma_load_2d(sbuf + (k % 3u) * 4096u, tmR, col0 + 32 * b, row0, bar);
  };
  if (lane == 0 && nv > 0) {
    bulk_wait_read_but_one();                               // every store but the latest has read its box
    request(0);
    if (nv > 1) request(1);
  }
  const bool ln = a.epi.res_mean != nullptr;
  float mu = 0.f, rs = 1.f;
  if (ln && row0 + lane < a.M) {
    mu = a.epi.res_mean[row0 + lane];
    rs = a.epi.res_rstd[row0 + lane];
  }
  if (!mbar_wait(tfull_addr, parity, abort_flag)) return false;
  tc_fence_after();
  if (nv == 0) {
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive_remote(tempty_remote);
    return true;
  }
  const uint32_t swz = (uint32_t)(lane & 7);
#pragma unroll 1
  for (int b = 0; b < nv; ++b) {
    const uint32_t k = nb + (uint32_t)b;
    const uint32_t box = sbuf + (k % 3u) * 4096u, srow = box + (uint32_t)lane * 128u;
    uint32_t v[32];
    tc_ld32_issue(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 256 + c_local + b * 32), v);
    tc_ld32_wait(v);
    if (b == nv - 1) {                                      // every value of this tile is in registers now
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(tempty_remote);
    }
    if (!mbar_wait(ld_bar0 + 8u * (k % 3u), (k / 3u) & 1u, abort_flag)) return false;
    const int n = col0 + b * 32;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const uint32_t addr = srow + ((((uint32_t)c) ^ swz) << 4);
      const uint4 ru = lds128(addr);
      float x[4] = {__uint_as_float(v[4 * c]), __uint_as_float(v[4 * c + 1]), __uint_as_float(v[4 * c + 2]), __uint_as_float(v[4 * c + 3])};
      const float r[4] = {__uint_as_float(ru.x), __uint_as_float(ru.y), __uint_as_float(ru.z), __uint_as_float(ru.w)};
      if (n + 4 * c < a.N) {                                // N is a multiple of 8: a piece of four columns is in or out
        if (a.epi.bias) {
          const float4 b4 = __ldg(reinterpret_cast<const float4*>(a.epi.bias + n + 4 * c));
          x[0] += b4.x; x[1] += b4.y; x[2] += b4.z; x[3] += b4.w;
        }
        if (ln) {
          const float4 g4 = __ldg(reinterpret_cast<const float4*>(a.epi.res_gamma + n + 4 * c));
          const float4 e4 = __ldg(reinterpret_cast<const float4*>(a.epi.res_beta + n + 4 * c));
          x[0] += (r[0] - mu) * rs * g4.x + e4.x;
          x[1] += (r[1] - mu) * rs * g4.y + e4.y;
          x[2] += (r[2] - mu) * rs * g4.z + e4.z;
          x[3] += (r[3] - mu) * rs * g4.w + e4.w;
        } else {
          x[0] += r[0]; x[1] += r[1]; x[2] += r[2]; x[3] += r[3];
        }
      }
      sts128(addr, __float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
      tma_store_2d(tmC, box, n, row0);
      bulk_commit();
      if (b + 2 < nv) {
        bulk_wait_read_but_one();                           // the store of block b - 1 has read the box that block b + 2 takes
        request(b + 2);
      }
    }
    __syncwarp();
  }
  nb += (uint32_t)nv;
  return true;
}

// EW epilogue warps per CTA: 8 (two per TMEM lane quarter) or, for the light epilogues whose register use allows
// it, 16 (four per quarter, 64 columns each) with one pipeline stage fewer
// bytes of private shared memory per epilogue warp: one 4 KB store box, two for the GELU epilogue (value and derivative),
// three fp32 boxes for the residual epilogue
template <typename CT, int MODE> constexpr int warp_bytes() {
  return (sizeof(CT) == 4 && MODE == EPI_RES_TS) ? 12288 : ((sizeof(CT) == 2 && MODE == EPI_GELU) ? 8192 : 4096);
}
template <int EW, int WARP_BYTES = 4096> struct Tc2Cfg {
  static constexpr int BN = 256;                       // columns of the pair's tile
  static constexpr int A_BYTES = BM * BK * 2;          // this CTA's 128 rows of A
  static constexpr int B_BYTES = (BN / 2) * BK * 2;    // this CTA's 128 columns of B
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int EPI_BYTES = EW * WARP_BYTES;    // the epilogue warps' private buffers
  static constexpr int STAGES = (232448 - 1024 - 512 - EPI_BYTES) / STAGE_BYTES;   // 6 with 32 KB of buffers, 5 with 64 KB
  static constexpr int TMEM_COLS = 2 * BN;
  static constexpr int THREADS = 64 + 32 * EW;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 + 512;
};

// n_tiles_m counts 256-row tiles here.  tmC / tmP: maps of the bf16 result and of the GELU-derivative matrix
// (boxes of 32 rows x 64 columns, 128-byte swizzle) for the variants whose epilogue uses bulk tensor stores; unused otherwise.
template <bool A_K, bool B_K, typename CT, int MODE = EPI_GENERAL, int EW = EPI_WARPS>
__global__ void __launch_bounds__(64 + 32 * EW, 1) gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                  const __grid_constant__ CUtensorMap tmB,
                                                                  const __grid_constant__ CUtensorMap tmC,
                                                                  const __grid_constant__ CUtensorMap tmP, TcArgs a) {
  constexpr bool RS = sizeof(CT) == 4 && MODE == EPI_RES_TS;       // fp32 residual epilogue through bulk tensor copies
  constexpr bool TS = RS || (sizeof(CT) == 2 && ((EW == 16 && MODE == EPI_DG) || MODE == EPI_BIAS || MODE == EPI_GELU));
  constexpr int WARP_BYTES = warp_bytes<CT, MODE>();
  using Cfg = Tc2Cfg<EW, WARP_BYTES>;
  constexpr int BN = Cfg::BN, STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;       // the same offset in both CTAs of the pair
  uint8_t* gen_tiles = smem_raw + (tiles - raw);
  float* epi_stage = reinterpret_cast<float*>(gen_tiles + STAGES * Cfg::STAGE_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_tiles + STAGES * Cfg::STAGE_BYTES + Cfg::EPI_BYTES);
  const uint32_t bar0 = tiles + STAGES * Cfg::STAGE_BYTES + Cfg::EPI_BYTES;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };                       // used in the leader
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };           // one per CTA
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };       // one per CTA
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };  // used in the leader
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  auto ld_bar = [&](int w) { return bar0 + 8u * (2 * STAGES + 6 + w); };      // one per epilogue warp (EPI_DG loads), three for EPI_RES_TS

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 2);              // the two CTAs' producers, each with its byte count
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), 2 * EW);          // one arrival per epilogue warp of either CTA
    }
    if (TS) {
      for (int w = 0; w < (RS ? 3 * EW : EW); ++w) mbar_init(ld_bar(w), 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)Cfg::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                           // both CTAs' barriers exist before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int64_t total = (int64_t)a.n_tiles_m * a.n_tiles_n * a.splits;
  const int64_t cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  bool failed = false;

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------------------
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      const uint32_t lead_bar0 = map_to_cta(bar0, 0);          // the leader's barrier block, as seen from this CTA
      for (int64_t t = cluster_id; t < total && !failed; t += n_clusters) {
        const int split = (int)(t / ((int64_t)a.n_tiles_m * a.n_tiles_n));
        const int64_t r = t - (int64_t)split * a.n_tiles_m * a.n_tiles_n;
        const int tm = (int)(r / a.n_tiles_n), tn = (int)(r % a.n_tiles_n);
        const int kb0 = split * a.kb_per_split, kb1 = min(kb0 + a.kb_per_split, a.num_kb);
        const int m0 = tm * 2 * BM + (int)rank * BM;            // this CTA's rows of A
        const int n0 = tn * BN + (int)rank * (BN / 2);          // this CTA's columns of B
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { failed = true; break; }
          const uint32_t lead_full = lead_bar0 + 8u * s;           // the leader's full_bar(s)
          mbar_arrive_expect_tx_remote(lead_full, Cfg::STAGE_BYTES);
          const uint32_t sa = tiles + s * Cfg::STAGE_BYTES, sb = sa + Cfg::A_BYTES;
          if (A_K) {
            tma_load_2d_pair(sa, &tmA, kb * BK, m0, lead_full);
          } else {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) tma_load_2d_pair(sa + i * 8192, &tmA, m0 + i * 64, kb * BK, lead_full);
          }
          if (B_K) {
            tma_load_2d_pair(sb, &tmB, kb * BK, n0, lead_full);
          } else {
#pragma unroll
            for (int i = 0; i < BN / 128; ++i) tma_load_2d_pair(sb + i * 8192, &tmB, n0 + i * 64, kb * BK, lead_full);
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
      if (failed) {
        *abort_flag = 1;
        gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA only) ----------------------------
    if (leader && lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_K ? 0u : 1u) << 15) |
                                 ((B_K ? 0u : 1u) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
      int s = 0;
      uint32_t ph = 0;
      int64_t it = 0;
      // This thread shares its scheduler with four busy epilogue warps, so the loop is kept to a few instructions
      // per k-block: the descriptors of stage 0 are built once (a later stage or k-step only adds to the 14-bit
      // address field, which cannot overflow inside shared memory), and so are the barrier addresses of both CTAs.
      const uint64_t da0 = A_K ? make_desc(tiles, 16, 1024) : make_desc(tiles, 8192, 1024);
      const uint64_t db0 = B_K ? make_desc(tiles + Cfg::A_BYTES, 16, 1024) : make_desc(tiles + Cfg::A_BYTES, 8192, 1024);
      constexpr uint32_t ka = (A_K ? 32 : 2048) >> 4, kbs = (B_K ? 32 : 2048) >> 4;
      const uint32_t rbar0 = map_to_cta(bar0, 0), rbar1 = map_to_cta(bar0, 1);
      for (int64_t t = cluster_id; t < total && !failed; t += n_clusters, ++it) {
        const int split = (int)(t / ((int64_t)a.n_tiles_m * a.n_tiles_n));
        const int kb0 = split * a.kb_per_split, kb1 = min(kb0 + a.kb_per_split, a.num_kb);
        const int buf = (int)(it & 1);
        if (!mbar_wait(tempty_bar(buf), (uint32_t)((it >> 1) & 1) ^ 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(buf * BN);
        uint32_t acc = 0u;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t soff = (uint32_t)(s * (Cfg::STAGE_BYTES >> 4));
          const uint64_t da = da0 + soff, db = db0 + soff;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            tc_mma_pair(tmem_d, da + (uint64_t)(k * ka), db + (uint64_t)(k * kbs), idesc, acc);
            acc = 1u;
          }
          const uint32_t eb = 8u * (uint32_t)(STAGES + s);  // empty_bar(s): the stage is free in both CTAs once these MMAs are done
          tc_commit_pair(rbar0 + eb);
          tc_commit_pair(rbar1 + eb);
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (failed) break;
        const uint32_t fb = 8u * (uint32_t)(2 * STAGES + buf);   // tfull_bar(buf): accumulator complete in both CTAs
        tc_commit_pair(rbar0 + fb);
        tc_commit_pair(rbar1 + fb);
      }
      if (failed) {
        *abort_flag = 1;
        gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
      }
    }
  } else {
    // ------------------------------ epilogue warps (both CTAs) ------------------------------
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    float* stage = epi_stage + ew * (32 * STAGE_LD);
    CT* C = reinterpret_cast<CT*>(a.C);
    int64_t it = 0;
    uint32_t res_blocks = 0;                      // EPI_RES_TS: this warp's running count of 32-column blocks
    for (int64_t t = cluster_id; t < total && !failed; t += n_clusters, ++it) {
      const int split = (int)(t / ((int64_t)a.n_tiles_m * a.n_tiles_n));
      const int64_t r = t - (int64_t)split * a.n_tiles_m * a.n_tiles_n;
      const int tm = (int)(r / a.n_tiles_n), tn = (int)(r % a.n_tiles_n);
      const int buf = (int)(it & 1);
      const int64_t row0 = (int64_t)tm * 2 * BM + (int64_t)rank * BM + q * 32;
      if constexpr (RS) {
        if (!epilogue_tile_res(a, &tmC, &tmP, (int32_t)row0, tn * BN + half * 128, half * 128, q, lane,
                               tiles + STAGES * Cfg::STAGE_BYTES + (uint32_t)(ew * WARP_BYTES), tmem_base, buf, tfull_bar(buf),
                               (uint32_t)((it >> 1) & 1), abort_flag, map_to_cta(tempty_bar(buf), 0), ld_bar(3 * ew), res_blocks)) {
          failed = true;
          break;
        }
      } else if constexpr (TS) {
        constexpr int NB = 32 / EW;               // blocks of 32 columns per warp
        const bool ok = epilogue_tile_ts<MODE, NB>(a, &tmC, &tmP, (int32_t)row0, tn * BN + half * (NB * 32), half * (NB * 32), q, lane,
                                    tiles + STAGES * Cfg::STAGE_BYTES + (uint32_t)(ew * WARP_BYTES), tmem_base, buf, tfull_bar(buf),
                                    (uint32_t)((it >> 1) & 1), abort_flag, map_to_cta(tempty_bar(buf), 0), ld_bar(ew),
                                    (uint32_t)(it & 1));
        if (!ok) {
          failed = true;
          break;
        }
      } else {
        CT* Cs = C + (int64_t)split * a.split_stride;
        if (!epilogue_tile<BN, CT, MODE, EW / 4>(a, Cs, row0, tn, half, q, lane, stage, tmem_base, buf, tfull_bar(buf),
                                                 (uint32_t)((it >> 1) & 1), abort_flag)) {
          failed = true;
          break;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(map_to_cta(tempty_bar(buf), 0));
      }
    }
    if (TS && lane == 0) bulk_wait_all();       // this warp's stores are complete before the CTA may exit
    if (failed && lane == 0) {
      *abort_flag = 1;
      gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
    }
  }

  // ------------------------------ teardown --------------------------------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (warp == 1 && lane == 0) {           // let copies and MMAs already issued drain (bounded)
      uint64_t t0 = clock64();
      while (clock64() - t0 < WAIT_LIMIT_CYCLES / 64) {}
    }
    __syncthreads();
  }
  cluster_sync_all();                        // the peer no longer reads this CTA's memory or signals its barriers
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS)
                 : "memory");
  }
}

// out[i] (+)= sum over splits of part[s][i], in ascending s; then the epilogue
template <typename CT>
__global__ void splitk_reduce_kernel(const float* __restrict__ part, int splits, int64_t split_stride, int64_t M, int N,
                                     CT* __restrict__ C, int64_t ldc, EpiDev e) {
  const int64_t n_el = M * N;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_el; i += (int64_t)gridDim.x * blockDim.x) {
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) acc += part[(int64_t)s * split_stride + i];
    const int64_t m = i / N;
    const int n = (int)(i - m * N);
    epilogue_store<CT, bf16>(e, C, ldc, m, n, acc);
  }
}

// ------------------------------ host side --------------------------------------------------
template <int BN, bool A_K, bool B_K, typename CT, int MODE = EPI_GENERAL>
cudaError_t launch_tc(const CUtensorMap& ma, const CUtensorMap& mb, const TcArgs& args, int grid, cudaStream_t st) {
  auto kern = gemm_tc_kernel<BN, A_K, B_K, CT, MODE>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<BN>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  kern<<<grid, TC_THREADS, TcCfg<BN>::SMEM_BYTES, st>>>(ma, mb, args);
  return cudaGetLastError();
}

template <int BN, typename CT>
cudaError_t launch_tc_major(bool a_k, bool b_k, const CUtensorMap& ma, const CUtensorMap& mb, const TcArgs& args, int grid,
                            cudaStream_t st) {
  if (a_k && b_k) return launch_tc<BN, true, true, CT>(ma, mb, args, grid, st);
  if (a_k && !b_k) return launch_tc<BN, true, false, CT>(ma, mb, args, grid, st);
  if (!a_k && b_k) return launch_tc<BN, false, true, CT>(ma, mb, args, grid, st);
  return launch_tc<BN, false, false, CT>(ma, mb, args, grid, st);
}

template <bool A_K, bool B_K, typename CT, int MODE = EPI_GENERAL, int EW = EPI_WARPS>
cudaError_t launch_tc2(const CUtensorMap& ma, const CUtensorMap& mb, const TcArgs& args, int grid, cudaStream_t st,
                       const CUtensorMap* mc = nullptr, const CUtensorMap* mp = nullptr) {
  using Tc2 = Tc2Cfg<EW, warp_bytes<CT, MODE>()>;
  auto kern = gemm_tc2_kernel<A_K, B_K, CT, MODE, EW>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Tc2::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(Tc2::THREADS);
  cfg.dynamicSmemBytes = Tc2::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, ma, mb, mc ? *mc : ma, mp ? *mp : (mc ? *mc : ma), args);
}
template <typename CT>
cudaError_t launch_tc2_major(bool a_k, bool b_k, const CUtensorMap& ma, const CUtensorMap& mb, const TcArgs& args, int grid,
                             cudaStream_t st) {
  if (a_k && b_k) return launch_tc2<true, true, CT>(ma, mb, args, grid, st);
  if (a_k && !b_k) return launch_tc2<true, false, CT>(ma, mb, args, grid, st);
  if (!a_k && b_k) return launch_tc2<false, true, CT>(ma, mb, args, grid, st);
  return launch_tc2<false, false, CT>(ma, mb, args, grid, st);
}

}  // namespace

static bool pair_enabled_env() {
  static const bool on = []() { const char* v = getenv("GRAM_GEMM_PAIR"); return !(v && v[0] == '0'); }();
  return on;
}
// GRAM_GEMM_RES_TS=0 in the environment keeps the register path of the fp32 residual epilogue (for comparisons)
static bool res_ts_env() {
  static const bool on = []() { const char* v = getenv("GRAM_GEMM_RES_TS"); return !(v && v[0] == '0'); }();
  return on;
}
bool gemm_fused_colsum(int dtype, int64_t M, int N) {
  const bool bn256 = (N % 256 == 0 || N > 1024);
  return dtype == GRAM_BF16 && pair_enabled_env() && bn256 && M >= 2 * BM && M < ((int64_t)1 << 31) && get_encode_fn() != nullptr;
}

gram_status gemm_ws_alloc(gram_ctx* ctx, GemmWorkspace* ws, size_t splitk_bytes) {
  ws->splitk_bytes = splitk_bytes;
  if (splitk_bytes) GRAM_CUDA(ctx, cudaMalloc(&ws->splitk, splitk_bytes));
  return GRAM_OK;
}
void gemm_ws_free(GemmWorkspace* ws) {
  cudaFree(ws->splitk);
  *ws = GemmWorkspace();
}

gram_status gemm_launch(gram_ctx* ctx, GemmWorkspace* ws, int dtype, const void* A, int a_kmajor, int64_t lda,
                        const void* B, int b_kmajor, int64_t ldb, void* C, int c_f32, int64_t ldc, int64_t M, int N,
                        int64_t K, const GemmEpilogue& epi, int allow_splitk, cudaStream_t st) {
  if (M < 0 || N < 0 || K < 0) return gram_set_error(ctx, "gemm: negative size"), GRAM_ERR_ARG;
  if (M == 0 || N == 0) return GRAM_OK;
  if (!A || !B || !C) return gram_set_error(ctx, "gemm: null operand"), GRAM_ERR_ARG;
  EpiDev e{epi.bias, epi.res, epi.res_mean, epi.res_rstd, epi.res_gamma, epi.res_beta, epi.pre, epi.dgelu_pre, epi.copy_out,
           epi.colsum_part, epi.gelu, epi.accumulate};
  if (dtype == GRAM_F32) {
    if (!c_f32) return gram_set_error(ctx, "gemm: fp32 operands need an fp32 result"), GRAM_ERR_UNSUPPORTED;
    ProfScope prof(ctx, GRAM_K_GEMM, 2.0 * (double)M * N * (double)K, 1, st, epi.tag ? epi.tag : "gemm_f32");
    dim3 grid((unsigned)ceil_div(N, ST), (unsigned)ceil_div64(M, ST));
    gemm_f32_kernel<<<grid, 256, 0, st>>>((const float*)A, a_kmajor ? lda : 1, a_kmajor ? 1 : lda, (const float*)B,
                                          b_kmajor ? ldb : 1, b_kmajor ? 1 : ldb, (float*)C, ldc, M, N, K, e);
    GRAM_LAUNCH_CHECK(ctx);
    return GRAM_OK;
  }
  // ---- bf16 on the tensor cores ----
  if ((lda % 8) || (ldb % 8) || ((uintptr_t)A % 16) || ((uintptr_t)B % 16) || ((uintptr_t)C % 16) || (ldc % 8) ||
      K == 0)
    return gram_set_error(ctx, "gemm: bf16 operands need 16-byte aligned rows (sizes multiples of 8)"), GRAM_ERR_UNSUPPORTED;
  if (e.accumulate && !c_f32) return gram_set_error(ctx, "gemm: accumulation needs an fp32 result"), GRAM_ERR_UNSUPPORTED;
  if ((e.res != nullptr) + (e.dgelu_pre != nullptr) + (e.accumulate != 0) > 1)
    return gram_set_error(ctx, "gemm: at most one of residual, GELU derivative and accumulation per product"), GRAM_ERR_UNSUPPORTED;
  if ((N % 8) || (e.bias && ((uintptr_t)e.bias % 16)) || (e.res_gamma && (((uintptr_t)e.res_gamma % 16) || ((uintptr_t)e.res_beta % 16))))
    return gram_set_error(ctx, "gemm: N must be a multiple of 8 and the epilogue's vectors 16-byte aligned"), GRAM_ERR_UNSUPPORTED;
  const int BNsel = (N % 256 == 0 || N > 1024) ? 256 : (N > 64 ? 128 : 64);
  // pairs of SMs (256 x 256 tiles) when the problem has full-height tiles; GRAM_GEMM_PAIR=0 keeps single CTAs
  const bool pair = pair_enabled_env() && BNsel == 256 && M >= 2 * BM;
  CUtensorMap ma, mb;
  bool ok;
  if (a_kmajor) ok = make_map(&ma, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK, BM);
  else ok = make_map(&ma, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, 64, BK);
  if (b_kmajor) ok = ok && make_map(&mb, B, (uint64_t)K, (uint64_t)N, (uint64_t)ldb, BK, (uint32_t)(pair ? BNsel / 2 : BNsel));
  else ok = ok && make_map(&mb, B, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, 64, BK);
  if (!ok) return gram_set_error(ctx, "gemm: cuTensorMapEncodeTiled failed"), GRAM_ERR_CUDA;

  TcArgs args;
  args.M = M;
  args.N = N;
  args.num_kb = (int32_t)ceil_div64(K, BK);
  args.n_tiles_m = (int32_t)ceil_div64(M, pair ? 2 * BM : BM);
  args.n_tiles_n = ceil_div(N, BNsel);
  args.status = gram_status_word(ctx);
  const int64_t tiles = (int64_t)args.n_tiles_m * args.n_tiles_n;
  const int units = pair ? kNumSMs / 2 : kNumSMs;        // CTAs, or CTA pairs, that run at once
  int splits = 1;
  if (allow_splitk && tiles < units && args.num_kb >= 16 && ws && ws->splitk) {
    // between 2 and 4 work units per CTA (pair); among those, the count that leaves the last wave fullest
    const int64_t per = (int64_t)M * N * (int64_t)sizeof(float);
    int lo = (int)((2 * units + tiles - 1) / tiles), hi = (int)((4 * units + tiles - 1) / tiles);
    int cap = args.num_kb / 8;
    if ((int64_t)cap * per > (int64_t)ws->splitk_bytes) cap = (int)(ws->splitk_bytes / per);
    if (hi > cap) hi = cap;
    if (lo > hi) lo = hi;
    double best = -1.0;
    for (int sp = lo; sp <= hi && sp >= 1; ++sp) {
      const int64_t total = tiles * sp;
      const double fill = (double)total / (double)(ceil_div64(total, units) * units);
      if (fill > best + 1e-9) { best = fill; splits = sp; }
    }
    if (splits < 1) splits = 1;
  }
  args.kb_per_split = ceil_div(args.num_kb, splits);
  splits = ceil_div(args.num_kb, args.kb_per_split);
  args.splits = splits;
  cudaError_t err;
  ProfScope prof(ctx, GRAM_K_GEMM, 2.0 * (double)M * N * (double)K, splits > 1 ? 2 : 1, st, epi.tag ? epi.tag : "gemm");
  const int grid = pair ? 2 * (int)((tiles * splits < units) ? tiles * splits : units)
                        : (int)((tiles * splits < kNumSMs) ? tiles * splits : kNumSMs);
  if (splits > 1) {
    args.C = ws->splitk;
    args.ldc = N;
    args.split_stride = (int64_t)M * N;
    args.epi = EpiDev{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, 0};
    if (pair && !a_kmajor && !b_kmajor) err = launch_tc2<false, false, float, EPI_BIAS>(ma, mb, args, grid, st);
    else if (pair) err = launch_tc2_major<float>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
    else if (BNsel == 256) err = launch_tc_major<256, float>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
    else if (BNsel == 128) err = launch_tc_major<128, float>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
    else err = launch_tc_major<64, float>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
    if (err != cudaSuccess) return gram_set_error(ctx, "gemm launch failed: %s", cudaGetErrorString(err)), GRAM_ERR_CUDA;
    int rb = (int)ceil_div64(M * N, 256);
    if (rb > kNumSMs * 8) rb = kNumSMs * 8;
    if (c_f32) splitk_reduce_kernel<float><<<rb, 256, 0, st>>>(ws->splitk, splits, (int64_t)M * N, M, N, (float*)C, ldc, e);
    else splitk_reduce_kernel<bf16><<<rb, 256, 0, st>>>(ws->splitk, splits, (int64_t)M * N, M, N, (bf16*)C, ldc, e);
    GRAM_LAUNCH_CHECK(ctx);
    return GRAM_OK;
  }
  args.C = C;
  args.ldc = ldc;
  args.split_stride = 0;
  args.epi = e;
  if (e.colsum_part && !(pair && e.dgelu_pre && !c_f32))
    return gram_set_error(ctx, "gemm: column-sum partials need the paired GELU-derivative variant"), GRAM_ERR_UNSUPPORTED;
  const bool dg_only = e.dgelu_pre && !e.bias && !e.res && !e.accumulate && !e.copy_out && !e.gelu && !c_f32 && a_kmajor &&
                       !b_kmajor;
  const bool others = e.gelu || e.dgelu_pre || e.res || e.accumulate || e.copy_out || e.pre;
  const bool m_bias = !others;
  const bool m_gelu = e.gelu && e.pre && !e.dgelu_pre && !e.res && !e.accumulate && !e.copy_out && !c_f32 && a_kmajor && b_kmajor;
  const bool m_res = e.res && !e.gelu && !e.dgelu_pre && !e.accumulate && !e.pre && c_f32 && a_kmajor;
  if (pair) {
    // bf16 results leave through bulk tensor stores: maps of C and of the GELU-derivative matrix (boxes of 32 rows x 64 columns)
    const void* aux = e.gelu ? e.pre : e.dgelu_pre;
    const bool ts = !c_f32 && M < (int64_t)1 << 31 && (!aux || (uintptr_t)aux % 16 == 0);
    CUtensorMap mc, mp;
    bool ts_ok = ts && make_map(&mc, C, (uint64_t)N, (uint64_t)M, (uint64_t)ldc, 64, 32);
    if (ts_ok && aux) ts_ok = make_map(&mp, aux, (uint64_t)N, (uint64_t)M, (uint64_t)ldc, 64, 32);
    const CUtensorMap* pc = &mc;
    const CUtensorMap* pp = aux ? &mp : &mc;
    // the fp32 residual products with a short reduction (K <= 1024: the output projection of attention), where the epilogue's
    // memory traffic outlasts the main loop: result and residual as fp32 boxes of 32 rows x 32 columns through bulk tensor
    // copies (no bf16 copy on this path).  With longer K the register path keeps six pipeline stages instead of four and
    // is the faster one (measured: 1279 against 1175 TFLOP/s at K = 3072).
    CUtensorMap mcf, mrf;
    const bool rs_ok = m_res && !e.copy_out && K <= 1024 && res_ts_env() && M < (int64_t)1 << 31 && (uintptr_t)e.res % 16 == 0 &&
                       make_map_f32(&mcf, C, (uint64_t)N, (uint64_t)M, (uint64_t)ldc, 32, 32) &&
                       make_map_f32(&mrf, e.res, (uint64_t)N, (uint64_t)M, (uint64_t)ldc, 32, 32);
    if (e.colsum_part && !(dg_only && ts_ok))
      return gram_set_error(ctx, "gemm: column-sum partials need the GELU-derivative variant with bulk stores"), GRAM_ERR_UNSUPPORTED;
    if (dg_only && ts_ok) err = launch_tc2<true, false, bf16, EPI_DG, 16>(ma, mb, args, grid, st, pc, pp);
    else if (m_gelu && ts_ok) err = launch_tc2<true, true, bf16, EPI_GELU, 8>(ma, mb, args, grid, st, pc, pp);
    else if (m_res && rs_ok && b_kmajor) err = launch_tc2<true, true, float, EPI_RES_TS>(ma, mb, args, grid, st, &mcf, &mrf);
    else if (m_res && rs_ok && !b_kmajor) err = launch_tc2<true, false, float, EPI_RES_TS>(ma, mb, args, grid, st, &mcf, &mrf);
    else if (m_res && b_kmajor) err = launch_tc2<true, true, float, EPI_RES>(ma, mb, args, grid, st);
    else if (m_res && !b_kmajor) err = launch_tc2<true, false, float, EPI_RES>(ma, mb, args, grid, st);
    else if (m_bias && a_kmajor && b_kmajor && ts_ok) err = launch_tc2<true, true, bf16, EPI_BIAS, 8>(ma, mb, args, grid, st, pc, pp);
    else if (m_bias && a_kmajor && !b_kmajor && ts_ok) err = launch_tc2<true, false, bf16, EPI_BIAS, 8>(ma, mb, args, grid, st, pc, pp);
    else if (c_f32) err = launch_tc2_major<float>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
    else err = launch_tc2_major<bf16>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
  } else if (dg_only) {
    if (BNsel == 256) err = launch_tc<256, true, false, bf16, EPI_DG>(ma, mb, args, grid, st);
    else if (BNsel == 128) err = launch_tc<128, true, false, bf16, EPI_DG>(ma, mb, args, grid, st);
    else err = launch_tc<64, true, false, bf16, EPI_DG>(ma, mb, args, grid, st);
  } else if (c_f32) {
    if (BNsel == 256) err = launch_tc_major<256, float>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
    else if (BNsel == 128) err = launch_tc_major<128, float>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
    else err = launch_tc_major<64, float>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
  } else {
    if (BNsel == 256) err = launch_tc_major<256, bf16>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
    else if (BNsel == 128) err = launch_tc_major<128, bf16>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
    else err = launch_tc_major<64, bf16>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
  }
  if (err != cudaSuccess) return gram_set_error(ctx, "gemm launch failed: %s", cudaGetErrorString(err)), GRAM_ERR_CUDA;
  return GRAM_OK;
}
