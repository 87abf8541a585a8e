// Non-GEMM layers of the encoder and the task module.  `dtype` selects the element type T of
// activations (GRAM_F32: float, GRAM_BF16: bf16); parameters and their gradients are always fp32.
#pragma once
#include "gram_internal.h"

constexpr float kLnEps = 1e-5f;
constexpr int kRedBlocks = 592;            // upper bound on blocks that leave partial sums (4 per SM)
// bytes of the reduction scratch: kRedBlocks partial rows of up to 2*4096 floats
constexpr size_t kRedScratchBytes = (size_t)kRedBlocks * 2 * 4096 * sizeof(float);

// z0[t, :] = tok_emb[token(t), :] + pos_emb[t % l_t, :], token(t) = item_tokens[items[t / l_t], t % l_t];
// tok_ids[t] = token(t).  items == null means items[u] = first_item + u.
gram_status embed_forward(gram_ctx* ctx, int dtype, const int32_t* item_tokens, const int32_t* items, int32_t first_item,
                          int32_t n_items_chunk, int32_t n_items_total, int l_t, int vocab, int d, const float* tok_emb,
                          const float* pos_emb, void* z0, int32_t* tok_ids, cudaStream_t st);

gram_status layernorm_forward(gram_ctx* ctx, int dtype, const void* z, const float* gamma, const float* beta, void* y,
                              float* mean, float* rstd, int64_t rows, int d, cudaStream_t st);
// dz = LayerNorm backward of dy at input z; dgamma += sum_rows dy * xhat; dbeta += sum_rows dy
gram_status layernorm_backward(gram_ctx* ctx, int dtype, const void* dy, const void* z, const float* mean,
                               const float* rstd, const float* gamma, void* dz, float* dgamma, float* dbeta,
                               float* scratch, int64_t rows, int d, cudaStream_t st);

// softmax(Q K^T / sqrt(dh)) V per (sequence, head); qkv is [n_seq*S, 3d] (Q | K | V), ctx [n_seq*S, d]
gram_status attention_forward(gram_ctx* ctx, int dtype, const void* qkv, void* out, int64_t n_seq, int S, int d,
                              int n_heads, int causal, cudaStream_t st);
gram_status attention_backward(gram_ctx* ctx, int dtype, const void* qkv, const void* dctx, void* dqkv, int64_t n_seq,
                               int S, int d, int n_heads, int causal, cudaStream_t st);

// out[n] += sum_rows X[r, n]
gram_status colsum_accumulate(gram_ctx* ctx, int dtype, const void* X, int64_t rows, int N, float* out, float* scratch,
                              cudaStream_t st);
// out[s, :] += sum_u X[u*period + s, :]  (s < period)
gram_status periodic_rowsum_accumulate(gram_ctx* ctx, int dtype, const void* X, int64_t n_groups, int period, int d,
                                       float* out, cudaStream_t st);

// H[u, :] = mean_s x[u*l_t + s, :] (mean) or x[u*l_t, :] (cls); H has type T
gram_status pool_forward(gram_ctx* ctx, int dtype, const void* x, void* H, int64_t n, int l_t, int d, int pooling,
                         cudaStream_t st);
// dx[u*l_t + s, :] from G[u, :] (fp32)
gram_status pool_backward(gram_ctx* ctx, int dtype, const float* G, void* dx, int64_t n, int l_t, int d, int pooling,
                          cudaStream_t st);

// knowledge-tracing task input: x[b, n, :] = E[b, n, :] + pos[n, :] + resp[prev(b, n), :],
// prev(b, 0) = 2, prev(b, n) = labels[b, n-1]
gram_status kt_input_forward(gram_ctx* ctx, int dtype, const void* E, const float* pos, const float* resp,
                             const int32_t* labels, void* x, int B, int L, int d, cudaStream_t st);
// dE (fp32) = dx; dpos[n] += sum_b dx[b, n]; dresp[r] += sum over positions with prev == r
gram_status kt_input_backward(gram_ctx* ctx, int dtype, const void* dx, const int32_t* labels, float* dE, float* dpos,
                              float* dresp, float* scratch, int B, int L, int d, cudaStream_t st);
// logit = y . w + b; loss = mean BCE; dy = (sigmoid(logit) - label) / (B*L) * w; dw, db accumulate
gram_status kt_head(gram_ctx* ctx, int dtype, const void* y, const float* w, const float* b, const int32_t* labels,
                    void* dy, float* dw, float* db, float* loss, float* scratch, int64_t P, int d, cudaStream_t st);

// news-recommendation task, the part between the matrix products (one block per user):
// given pre = E wa^T + ba [B*L, d_a], computes additive attention over the first L - n_cand encodings,
// dot-product scores with the candidates and softmax cross-entropy on candidate 0 (averaged over B);
// writes the direct part of dE (fp32 [B*L, d]), dpre (type T, zero rows for candidates), dqa +=, loss.
gram_status nr_user(gram_ctx* ctx, int dtype, const void* E, const void* pre, const float* qa, float* dE, void* dpre,
                    float* dqa, float* loss, float* scratch, int B, int L, int n_cand, int d, int d_a, cudaStream_t st);

// element-wise helpers
gram_status convert_f32_to_bf16(gram_ctx* ctx, const float* in, bf16* out, size_t n, cudaStream_t st);
gram_status convert_to_f32(gram_ctx* ctx, int dtype, const void* in, float* out, size_t n, cudaStream_t st);
gram_status sgd_update(gram_ctx* ctx, float* w, const float* g, float lr, size_t n, cudaStream_t st);
// dst[index[u], :] = src[u, :]
gram_status scatter_rows(gram_ctx* ctx, int dtype, const void* src, const int32_t* index, int64_t n, int d,
                         int64_t n_dst_rows, void* dst, cudaStream_t st);
