// Matrix products.  bf16: a persistent, warp-specialised tcgen05 kernel (one TMA producer warp, one
// MMA-issuing warp, eight epilogue warps; operands staged in 128-byte-swizzled shared memory by TMA,
// fp32 accumulators double-buffered in tensor memory so that the epilogue of one tile overlaps the
// main loop of the next).  fp32: a plain tiled CUDA-core kernel for the small fp32 configuration.
#include <cuda.h>

#include "gemm.h"

namespace {

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
  const float ex = __expf(-0.5f * x * x);
  const float t = __fdividef(1.f, 1.f + 0.3275911f * 0.70710678f * ax);
  const float poly = t * (0.254829592f + t * (-0.284496736f + t * (1.421413741f + t * (-1.453152027f + t * 1.061405429f))));
  const float erf_abs = 1.f - poly * ex;                  // erf(|x| / sqrt 2)
  cdf = 0.5f * (1.f + copysignf(erf_abs, x));
  pdf = 0.39894228f * ex;
}

// what one lane reads before it may store anything for its 4 columns of one row
struct EpiLoads {
  float res[4];
  float pre[4];
  float acc[4];
};
template <typename CT>
__device__ __forceinline__ void epilogue_load4(const EpiDev& e, const CT* C, int64_t ldc, int64_t m, int n, EpiLoads& L) {
  const int64_t o = m * ldc + n;
  if (e.res) ld4(e.res + o, L.res);
  if (e.dgelu_pre) ld4(reinterpret_cast<const bf16*>(e.dgelu_pre) + o, L.pre);
  if (e.accumulate) ld4(reinterpret_cast<const float*>(C) + o, L.acc);      // accumulation is offered for fp32 C only
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
  if (e.dgelu_pre) {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] *= L.pre[i];
  }
  if (e.res) {
    if (e.res_mean) {
#pragma unroll
      for (int i = 0; i < 4; ++i) v[i] += (L.res[i] - mu) * rs * gam[i] + bet[i];
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) v[i] += L.res[i];
    }
  }
  if (e.accumulate) {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] += L.acc[i];
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
constexpr int STAGE_LD = 33;                     // padded row of a warp's 32 x 32 transpose buffer
constexpr uint64_t WAIT_LIMIT_CYCLES = 4000000000ull;   // ~2 s: a wait that long has failed

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
// bounded wait: false when the limit ran out or another role has already given up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  uint64_t t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 0xFFF) == 0) {
      if (*abort_flag) return false;
      uint64_t now = clock64();
      if (t0 == 0) t0 = now;
      else if (now - t0 > WAIT_LIMIT_CYCLES) return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(accum)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a 128-byte-swizzled operand tile (bf16).
//   K-major tile  [rows][64 k]:  8-row groups 1024 bytes apart (stride offset), leading offset unused (1).
//   MN-major tile [64 k][64 mn] per 8 KB box: 8-k groups 1024 bytes apart (stride offset); the next 64
//   mn-elements start one box later (leading offset = box bytes).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;     // descriptor version of this architecture
  d |= (uint64_t)2 << 61;     // 128-byte swizzle
  return d;
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

// DG: the epilogue is only "multiply by the saved GELU derivative, store bf16" (backward of the
// feed-forward layer); the derivative's values for the whole tile are then fetched into registers
// while the main loop of that tile is still running, which hides their HBM latency.
template <int BN, bool A_K, bool B_K, typename CT, bool DG = false>
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
    // A warp may read only its quarter of the TMEM lanes (rows q*32..q*32+31 of the tile); two warps
    // share a quarter and split the columns.  Each 32 x 32 block is loaded one row per thread, turned
    // through a padded shared-memory buffer, and then handled four rows per instruction with eight
    // lanes per row, so that global loads and stores of a row are contiguous 128-byte pieces.
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
      if constexpr (DG) {
        uint2 pf[BN / 64][8];                       // packed bf16: 4 columns of one row per entry
        const bf16* pre = reinterpret_cast<const bf16*>(a.epi.dgelu_pre);
#pragma unroll
        for (int blk = 0; blk < BN / 64; ++blk) {
          const int n = tn * BN + half * (BN / 2) + blk * 32 + (lane & 7) * 4;
#pragma unroll
          for (int rr = 0; rr < 8; ++rr) {
            const int64_t m = row0 + rr * 4 + (lane >> 3);
            pf[blk][rr] = (m < a.M && n < a.N) ? *reinterpret_cast<const uint2*>(pre + m * a.ldc + n) : make_uint2(0u, 0u);
          }
        }
        if (!mbar_wait(tfull_bar(buf), (uint32_t)((it >> 1) & 1), abort_flag)) { failed = true; break; }
        tc_fence_after();
#pragma unroll
        for (int blk = 0; blk < BN / 64; ++blk) {
          const int c0 = half * (BN / 2) + blk * 32;
          uint32_t v[32];
          tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), v);
#pragma unroll
          for (int j = 0; j < 32; ++j) stage[lane * STAGE_LD + j] = __uint_as_float(v[j]);
          __syncwarp();
          const int n = tn * BN + c0 + (lane & 7) * 4;
#pragma unroll
          for (int rr = 0; rr < 8; ++rr) {
            const int rl = rr * 4 + (lane >> 3);
            const int64_t m = row0 + rl;
            if (m < a.M && n < a.N) {
              const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pf[blk][rr].x));
              const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pf[blk][rr].y));
              float x[4];
              x[0] = stage[rl * STAGE_LD + (lane & 7) * 4 + 0] * g0.x;
              x[1] = stage[rl * STAGE_LD + (lane & 7) * 4 + 1] * g0.y;
              x[2] = stage[rl * STAGE_LD + (lane & 7) * 4 + 2] * g1.x;
              x[3] = stage[rl * STAGE_LD + (lane & 7) * 4 + 3] * g1.y;
              st4(Cs + m * a.ldc + n, x);
            }
          }
          __syncwarp();
        }
        tc_fence_before();
        mbar_arrive(tempty_bar(buf));
        continue;
      }
      if (!mbar_wait(tfull_bar(buf), (uint32_t)((it >> 1) & 1), abort_flag)) { failed = true; break; }
      tc_fence_after();
      float mu_l = 0.f, rs_l = 1.f;               // LayerNorm statistics of row row0 + lane
      if (a.epi.res_mean && row0 + lane < a.M) {
        mu_l = a.epi.res_mean[row0 + lane];
        rs_l = a.epi.res_rstd[row0 + lane];
      }
#pragma unroll 1
      for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
        uint32_t v[32];
        tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), v);
#pragma unroll
        for (int j = 0; j < 32; ++j) stage[lane * STAGE_LD + j] = __uint_as_float(v[j]);
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
              float x[4];
#pragma unroll
              for (int k = 0; k < 4; ++k) x[k] = stage[rl * STAGE_LD + (lane & 7) * 4 + k];
              epilogue_store4<CT>(a.epi, Cs, a.ldc, m, n, x, L[r4], bias4, gam4, bet4, mu, rs);
            }
          }
        }
        __syncwarp();
      }
      tc_fence_before();
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
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D bf16 tensor map: `inner` contiguous elements per row, `outer` rows `ld` elements apart
bool make_map(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t ld, uint32_t box_inner,
              uint32_t box_outer) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t es[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, bool A_K, bool B_K, typename CT, bool DG = false>
cudaError_t launch_tc(const CUtensorMap& ma, const CUtensorMap& mb, const TcArgs& args, int grid, cudaStream_t st) {
  auto kern = gemm_tc_kernel<BN, A_K, B_K, CT, DG>;
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

}  // namespace

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
           epi.gelu, epi.accumulate};
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
  if ((N % 8) || (e.bias && ((uintptr_t)e.bias % 16)) || (e.res_gamma && (((uintptr_t)e.res_gamma % 16) || ((uintptr_t)e.res_beta % 16))))
    return gram_set_error(ctx, "gemm: N must be a multiple of 8 and the epilogue's vectors 16-byte aligned"), GRAM_ERR_UNSUPPORTED;
  const int BNsel = (N % 256 == 0 || N > 1024) ? 256 : (N > 64 ? 128 : 64);
  CUtensorMap ma, mb;
  bool ok;
  if (a_kmajor) ok = make_map(&ma, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK, BM);
  else ok = make_map(&ma, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, 64, BK);
  if (b_kmajor) ok = ok && make_map(&mb, B, (uint64_t)K, (uint64_t)N, (uint64_t)ldb, BK, (uint32_t)BNsel);
  else ok = ok && make_map(&mb, B, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, 64, BK);
  if (!ok) return gram_set_error(ctx, "gemm: cuTensorMapEncodeTiled failed"), GRAM_ERR_CUDA;

  TcArgs args;
  args.M = M;
  args.N = N;
  args.num_kb = (int32_t)ceil_div64(K, BK);
  args.n_tiles_m = (int32_t)ceil_div64(M, BM);
  args.n_tiles_n = ceil_div(N, BNsel);
  args.status = gram_status_word(ctx);
  const int64_t tiles = (int64_t)args.n_tiles_m * args.n_tiles_n;
  int splits = 1;
  if (allow_splitk && tiles < kNumSMs && args.num_kb >= 16 && ws && ws->splitk) {
    splits = (int)((2 * kNumSMs + tiles - 1) / tiles);
    if (splits > args.num_kb / 8) splits = args.num_kb / 8;
    const int64_t per = (int64_t)M * N * (int64_t)sizeof(float);
    if ((int64_t)splits * per > (int64_t)ws->splitk_bytes) splits = (int)(ws->splitk_bytes / per);
    if (splits < 1) splits = 1;
  }
  args.kb_per_split = ceil_div(args.num_kb, splits);
  splits = ceil_div(args.num_kb, args.kb_per_split);
  args.splits = splits;
  cudaError_t err;
  ProfScope prof(ctx, GRAM_K_GEMM, 2.0 * (double)M * N * (double)K, splits > 1 ? 2 : 1, st, epi.tag ? epi.tag : "gemm");
  const int grid = (int)((tiles * splits < kNumSMs) ? tiles * splits : kNumSMs);
  if (splits > 1) {
    args.C = ws->splitk;
    args.ldc = N;
    args.split_stride = (int64_t)M * N;
    args.epi = EpiDev{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, 0};
    if (BNsel == 256) err = launch_tc_major<256, float>(a_kmajor, b_kmajor, ma, mb, args, grid, st);
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
  const bool dg_only = e.dgelu_pre && !e.bias && !e.res && !e.accumulate && !e.copy_out && !e.gelu && !c_f32 && a_kmajor &&
                       !b_kmajor;
  if (dg_only) {
    if (BNsel == 256) err = launch_tc<256, true, false, bf16, true>(ma, mb, args, grid, st);
    else if (BNsel == 128) err = launch_tc<128, true, false, bf16, true>(ma, mb, args, grid, st);
    else err = launch_tc<64, true, false, bf16, true>(ma, mb, args, grid, st);
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
