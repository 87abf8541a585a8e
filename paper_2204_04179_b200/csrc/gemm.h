// Matrix products of the encoder and task module.
#pragma once
#include "gram_internal.h"

// What happens to an accumulator element acc(m, n) before it is stored to C(m, n):
//   v = acc + bias[n]
//   gelu:       pre(m, n) = gelu'(v) (if pre != null);  v = gelu(v)   (forward of the feed-forward layer;
//               the derivative shares erf and the exponential with the value, so it is saved here)
//   dgelu_pre:  v = v * dgelu_pre(m, n)                               (backward through the GELU)
//   res:        v += r(m, n), r = res(m, n), or, when res_mean != null, LayerNorm applied on the fly:
//               r = (res(m, n) - res_mean[m]) * res_rstd[m] * res_gamma[n] + res_beta[n]
//               (the fp32 residual stream: a layer's input is the LayerNorm of the previous fp32 sum)
//   accumulate: v += C(m, n)                                          (fp32 C only)
//   copy_out:   copy_out(m, n) = v as well                            (operand-typed copy of the result)
//   colsum_part: with dgelu_pre on the tensor cores only (see gemm_fused_colsum): row i of this fp32
//               [ceil(M / 32), N] matrix receives the column sums of rows 32 i .. 32 i + 31 of the stored
//               (rounded) result, i.e. the partial sums of the bias gradient of the layer below
// res is fp32; pre, dgelu_pre and copy_out have the operands' element type (bf16 on the tensor
// cores, float in the fp32 kernel).  All of them share C's leading dimension.
struct GemmEpilogue {
  const float* bias = nullptr;
  const float* res = nullptr;
  const float* res_mean = nullptr;
  const float* res_rstd = nullptr;
  const float* res_gamma = nullptr;
  const float* res_beta = nullptr;
  void* pre = nullptr;
  const void* dgelu_pre = nullptr;
  void* copy_out = nullptr;
  float* colsum_part = nullptr;
  int gelu = 0;
  int accumulate = 0;
  const char* tag = nullptr;   // names the call site in profiles (host side only)
};

struct GemmWorkspace {
  float* splitk = nullptr;      // partial products of split-K launches
  size_t splitk_bytes = 0;
};

// C[M, N] = op(A) x op(B)^T with fp32 accumulation.
//   a_kmajor: A is [M, K] (lda elements between rows), else [K, M].
//   b_kmajor: B is [N, K] (ldb), else [K, N].
//   dtype GRAM_F32: A, B float (plain CUDA cores).  GRAM_BF16: A, B bf16 on the tensor cores
//   (tcgen05 with TMA-fed shared-memory operands and the accumulator in tensor memory).
//   c_f32: C (and the epilogue's matrices) float, else bf16.  For GRAM_F32, c_f32 must be 1.
//   allow_splitk: the K range may be cut into parts that are added in a fixed order.
gram_status gemm_launch(gram_ctx* ctx, GemmWorkspace* ws, int dtype, const void* A, int a_kmajor, int64_t lda,
                        const void* B, int b_kmajor, int64_t ldb, void* C, int c_f32, int64_t ldc, int64_t M, int N,
                        int64_t K, const GemmEpilogue& epi, int allow_splitk, cudaStream_t st);

// true when gemm_launch(dtype, ..., M, N, ...) with dgelu_pre set runs the variant that can fill colsum_part
bool gemm_fused_colsum(int dtype, int64_t M, int N);

gram_status gemm_ws_alloc(gram_ctx* ctx, GemmWorkspace* ws, size_t splitk_bytes);
void gemm_ws_free(GemmWorkspace* ws);

__host__ __device__ inline float gelu_f(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }
__host__ __device__ inline float gelu_grad_f(float x) {
  // d/dx [x * Phi(x)] = Phi(x) + x * phi(x)
  const float cdf = 0.5f * (1.0f + erff(x * 0.70710678118654752f));
  const float pdf = 0.39894228040143268f * expf(-0.5f * x * x);
  return cdf + x * pdf;
}
