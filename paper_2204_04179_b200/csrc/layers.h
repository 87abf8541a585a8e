// Non-GEMM layers of the encoder and the task module.  `dtype` selects the element type T of
// activations (GRAM_F32: float, GRAM_BF16: bf16); parameters and their gradients are always fp32.
#pragma once
#include "gram_internal.h"

constexpr float kLnEps = 1e-5f;
constexpr int kRedBlocks = 592;            // upper bound on blocks that leave partial sums (4 per SM)
// bytes of the reduction scratch: kRedBlocks partial rows of up to 2*4096 floats
constexpr size_t kRedScratchBytes = (size_t)kRedBlocks * 2 * 4096 * sizeof(float);

// Packed sequences grouped by length for the tensor-core attention kernels, whose tile height is a template
// argument: list (device) holds the sequence numbers with 1..32 rows first, then 33..64, 65..96, 97..128;
// count (host) says how many there are of each.  A launch per group uses the smallest tile that fits.
struct SeqGroups {
  const int32_t* list = nullptr;
  int32_t count[4] = {0, 0, 0, 0};
};

// A row-major [rows, d] view of the fp32 residual stream: either the values themselves (mean == null)
// or LayerNorm of them, applied where they are read: (z - mean[row]) * rstd[row] * gamma[c] + beta[c].
struct StreamRef {
  const float* z = nullptr;
  const float* mean = nullptr;
  const float* rstd = nullptr;
  const float* gamma = nullptr;
  const float* beta = nullptr;
};

// z0[t, :] = tok_emb[token(t), :] + pos_emb[t % l_t, :] (fp32), token(t) = item_tokens[items[t / l_t], t % l_t];
// tok_ids[t] = token(t).  items == null means items[u] = first_item + u.  seq_len / seq_off (both or neither): packed
// rows for texts of different lengths: item u's tokens 0 .. seq_len[u]-1 go to rows seq_off[u] .. and its padding
// slots get no row at all.
gram_status embed_forward(gram_ctx* ctx, const int32_t* item_tokens, const int32_t* items, int32_t first_item,
                          int32_t n_items_chunk, int32_t n_items_total, int l_t, int vocab, int d, const float* tok_emb,
                          const float* pos_emb, float* z0, int32_t* tok_ids, const int32_t* seq_len, const int32_t* seq_off,
                          cudaStream_t st);
// seq_len[u] = item_len[item(u)] for the n items of an encoder pass and seq_off = its exclusive prefix sum
// (seq_off[n] = rows in total)
// Also: group_list [n] = the sequence numbers grouped by length (SeqGroups), info[0..3] = the size of each group,
// info[4] = rows in total (device words the caller reads back).
gram_status sequence_layout(gram_ctx* ctx, const int32_t* item_len, const int32_t* items, int32_t first_item, int32_t n,
                            int32_t n_items_total, int l_t, int32_t* seq_len, int32_t* seq_off, int32_t* group_list,
                            int32_t* info, cudaStream_t st);

// y = LayerNorm(z): z is the fp32 stream, y the operand-typed copy the next matrix product reads
gram_status layernorm_forward(gram_ctx* ctx, int dtype, const float* z, const float* gamma, const float* beta, void* y,
                              float* mean, float* rstd, int64_t rows, int d, cudaStream_t st);
// dz = LayerNorm backward of dy at input z (fp32, plus an operand-typed copy dz_b when not null);
// dgamma += sum_rows dy * xhat; dbeta += sum_rows dy; dcol += sum_rows dz when dcol is not null (the bias
// gradient of the product whose output gradient dz is)
gram_status layernorm_backward(gram_ctx* ctx, int dtype, const float* dy, const float* z, const float* mean,
                               const float* rstd, const float* gamma, float* dz, void* dz_b, float* dgamma,
                               float* dbeta, float* dcol, float* scratch, int64_t rows, int d, cudaStream_t st);

// softmax(Q K^T / sqrt(dh)) V per (sequence, head); qkv is [n_seq*S, 3d] (Q | K | V), ctx [n_seq*S, d].
// seq_len (may be null): only the first seq_len[s] rows of sequence s are keys; the rows after them are padding,
// whose outputs are finite and never read, and whose gradients are zero.  seq_off (may be null, needs seq_len): packed
// rows, sequence s is rows seq_off[s] .. seq_off[s] + seq_len[s] (at most S of them) and there is no padding.
// groups (may be null, packed rows only): the sequences grouped by length, see SeqGroups.
// rows: token rows in use (n_seq * S, or the packed total).  lse (may be null): fp32 [n_heads, rows], receives per row and
// head the base-2 logarithm of the softmax denominator plus the scaled row maximum (what the tensor-core backward reads
// instead of recomputing the row statistics); written by the tcgen05 kernel only.
gram_status attention_forward(gram_ctx* ctx, int dtype, const void* qkv, void* out, float* lse, int64_t rows, int64_t n_seq, int S,
                              int d, int n_heads, int causal, const int32_t* seq_len, const int32_t* seq_off,
                              const SeqGroups* groups, cudaStream_t st);
// octx: the forward pass's output; lse: its row statistics; delta: scratch fp32 [n_heads, rows] (the last three are read by
// the tcgen05 kernels only; octx and delta only for sequences of more than 128 rows).
// colpart (may be null): fp32 partial column sums of dqkv, the partial sums of the bias gradient of the Q, K, V projection:
// the tensor-core kernels fill one row of 3d sums per tile (tcgen05) or per sequence (warp-level kernel) when those rows
// number at most colpart_cap_rows, and report the count in *colpart_rows_used (0: nothing was written, sum dqkv instead).
gram_status attention_backward(gram_ctx* ctx, int dtype, const void* qkv, const void* dctx, const void* octx, const float* lse,
                               float* delta, void* dqkv, float* colpart, int64_t colpart_cap_rows, int64_t* colpart_rows_used,
                               int64_t rows, int64_t n_seq, int S, int d, int n_heads, int causal, const int32_t* seq_len,
                               const int32_t* seq_off, const SeqGroups* groups, cudaStream_t st);

// the tcgen05 kernels behind the two calls above (bf16, head width 64, sequences of any length)
bool attention_tc_supported(int S, int d, int n_heads);
gram_status attention_forward_tc(gram_ctx* ctx, const void* qkv, void* out, float* lse, int64_t rows, int64_t n_seq, int S, int d,
                                 int n_heads, int causal, const int32_t* seq_len, const int32_t* seq_off, const int32_t* seq_list,
                                 cudaStream_t st);
int64_t attention_tc_colpart_rows(int64_t n_seq, int S);
gram_status attention_backward_tc(gram_ctx* ctx, const void* qkv, const void* dctx, const void* octx, const float* lse, float* delta,
                                  void* dqkv, float* colpart, int64_t colpart_row0, int64_t rows, int64_t n_seq, int S, int d,
                                  int n_heads, int causal, const int32_t* seq_len, const int32_t* seq_off, const int32_t* seq_list,
                                  cudaStream_t st);
// the warp-level tensor-core kernels (bf16, S <= 128, head width 32 or 64)
bool attention_mma_supported(int S, int d, int n_heads);
gram_status attention_forward_mma(gram_ctx* ctx, const void* qkv, void* out, int64_t n_seq, int S, int d, int n_heads,
                                  int causal, const int32_t* seq_len, const int32_t* seq_off, const int32_t* seq_list,
                                  cudaStream_t st);
gram_status attention_backward_mma(gram_ctx* ctx, const void* qkv, const void* dctx, void* dqkv, float* colpart, int64_t n_seq, int S, int d,
                                   int n_heads, int causal, const int32_t* seq_len, const int32_t* seq_off,
                                   const int32_t* seq_list, cudaStream_t st);

// out[n] += sum_rows X[r, n]   (X operand-typed)
// out[c] += sum over the nrows rows of part[., c] (fp32 [nrows, N]; partial column sums left by a fused producer)
gram_status colsum_from_partials(gram_ctx* ctx, const float* part, int64_t nrows, int N, float* out, float* scratch,
                                 cudaStream_t st);
gram_status colsum_accumulate(gram_ctx* ctx, int dtype, const void* X, int64_t rows, int N, float* out, float* scratch,
                              cudaStream_t st);
// out[s, :] += sum_u X[u*period + s, :]  (s < period; X fp32)
// packed rows (seq_len, seq_off not null): out[s, :] += sum over the groups u with s < seq_len[u] of X[seq_off[u] + s, :]
// scratch (may be null): kRedScratchBytes of reduction scratch, lets the groups be summed in parallel chunks
gram_status periodic_rowsum_accumulate(gram_ctx* ctx, const float* X, int64_t n_groups, int period, int d, float* out,
                                       float* scratch, const int32_t* seq_len, const int32_t* seq_off, cudaStream_t st);

// H[u, :] = mean_s x[u*l_t + s, :] (mean; over the first seq_len[u] tokens when seq_len is given) or x[u*l_t, :] (cls), fp32
gram_status pool_forward(gram_ctx* ctx, const StreamRef& x, float* H, int64_t n, int l_t, int d, int pooling,
                         const int32_t* seq_len, const int32_t* seq_off, cudaStream_t st);
// dx[u*l_t + s, :] from G[u, :] (both fp32); with seq_off the rows of item u are seq_off[u] + s
gram_status pool_backward(gram_ctx* ctx, const float* G, float* dx, int64_t n, int l_t, int d, int pooling,
                          const int32_t* seq_len, const int32_t* seq_off, cudaStream_t st);

// knowledge-tracing task input: x[b, n, :] = e(b, n) + pos[n, :] + resp[prev(b, n), :] (fp32, and an
// operand-typed copy x_b), prev(b, 0) = 2, prev(b, n) = labels[b, n-1].  e(b, n) = E[b*L + n, :] when index is null,
// else E[index[b*L + n], :] with E holding n_rows rows (the gather of stage 3 fused into this load); e_bf16: E's rows
// are bf16 (the Multi-step encoding cache) instead of fp32.
gram_status kt_input_forward(gram_ctx* ctx, int dtype, const void* E, int e_bf16, const int32_t* index, int64_t n_rows,
                             const float* pos, const float* resp, const int32_t* labels, float* x, void* x_b, int B, int L,
                             int d, cudaStream_t st);
// dE = dx (skipped when dE is null: the caller then reads dx itself as the gradient with respect to the encodings);
// dpos[n] += sum_b dx[b, n]; dresp[r] += sum over positions with prev == r
gram_status kt_input_backward(gram_ctx* ctx, const float* dx, const int32_t* labels, float* dE, float* dpos,
                              float* dresp, float* scratch, int B, int L, int d, cudaStream_t st);
// logit = y . w + b; loss = mean BCE over the positions with a label >= 0 (label -1: padding at the end of a history,
// not predicted); dy = (sigmoid(logit) - label) / (their number) * w, zero at padded positions (fp32, and an
// operand-typed copy dy_b when not null); dw, db accumulate; n_real: one device word of scratch for that number
gram_status kt_head(gram_ctx* ctx, int dtype, const StreamRef& y, const float* w, const float* b, const int32_t* labels,
                    float* dy, void* dy_b, float* dw, float* db, float* loss, float* scratch, int32_t* n_real, int64_t P,
                    int d, cudaStream_t st);

// news-recommendation task, the part between the matrix products (one block per user):
// given pre = E wa^T + ba [B*L, d_a] (operand-typed), computes additive attention over the first L - n_cand
// encodings, dot-product scores with the candidates and softmax cross-entropy on candidate 0 (averaged over
// B; history slots whose label is negative hold no click and take no part, labels may be null); writes the direct
// part of dE (fp32 [B*L, d]), dpre (operand-typed, zero rows for candidates), dqa +=, loss.
gram_status nr_user(gram_ctx* ctx, int dtype, const float* E, const void* pre, const float* qa, float* dE, void* dpre,
                    float* dqa, float* loss, float* scratch, const int32_t* labels, int B, int L, int n_cand, int d, int d_a,
                    cudaStream_t st);

// News task with self-attention layers over the clicked items (Appendix D): the clicked history slots of every user as
// packed sequences.  nr_layout: seq_len [B], seq_off [B + 1], rows [B * n_hist] (position of each packed row, -1 in the
// unused tail), pos2row [B * L] (packed row of each position, -1 for empty slots and candidates); labels may be null (every
// slot clicked).  nr_pack: out[r] = src[rows[r]] or a zero row, fp32 plus an operand-typed copy (out_b may be null).
// nr_select: out[p] = y[pos2row[p]] where that is a row, else other[p].
gram_status nr_layout(gram_ctx* ctx, const int32_t* labels, int B, int L, int n_hist, int32_t* seq_len, int32_t* seq_off,
                      int32_t* rows, int32_t* pos2row, cudaStream_t st);
gram_status nr_pack(gram_ctx* ctx, int dtype, const float* src, const int32_t* rows, int64_t n, int d, float* out, void* out_b,
                    cudaStream_t st);
gram_status nr_select(gram_ctx* ctx, const StreamRef& y, const int32_t* pos2row, const float* other, int64_t P, int d, float* out,
                      cudaStream_t st);

// element-wise helpers
gram_status convert_f32_to_bf16(gram_ctx* ctx, const float* in, bf16* out, size_t n, cudaStream_t st);
gram_status convert_to_f32(gram_ctx* ctx, int dtype, const void* in, float* out, size_t n, cudaStream_t st);
// gate (may be null): a device word; the update is skipped when it is not zero
gram_status sgd_update(gram_ctx* ctx, float* w, const float* g, float lr, size_t n, cudaStream_t st, const int32_t* gate = nullptr);
// one Adam update at count t >= 1 (Kingma & Ba, Algorithm 1); wb (may be null): bf16 copy of the new parameters
gram_status adam_update(gram_ctx* ctx, float* w, const float* g, float* m, float* v, void* wb, size_t n, int64_t t, float rate,
                        float beta1, float beta2, float eps, cudaStream_t st, const int32_t* gate = nullptr);
// dst[index[u], :] = src[u, :] (src fp32, dst operand-typed)
gram_status scatter_rows(gram_ctx* ctx, int dtype, const float* src, const int32_t* index, int64_t n, int d,
                         int64_t n_dst_rows, void* dst, cudaStream_t st);
// out[r, :] = in[row(r), :] for r < n, row(r) = rows[r] when rows is given, else r * stride; elem_bytes-byte elements
gram_status take_strided_rows(gram_ctx* ctx, const void* in, int64_t n, int64_t stride, const int32_t* rows, int d,
                              int elem_bytes, void* out, cudaStream_t st);
// out[row(r), :] = in[r, :] for r < n; the other rows of out are left as they are
gram_status put_strided_rows(gram_ctx* ctx, const void* in, int64_t n, int64_t stride, const int32_t* rows, int d,
                             int elem_bytes, void* out, cudaStream_t st);
// Additive-attention pooling over an item's tokens: given pre = x Wa^T + ba [rows, pa] (operand-typed),
// a_s = q . tanh(pre[s]), alpha = softmax over the item's tokens (saved, fp32 [rows]), H[u] = sum_s alpha_s x[s].
gram_status pool_additive_forward(gram_ctx* ctx, int dtype, const StreamRef& x, const void* pre, const float* q, float* H,
                                  float* alpha, int64_t n, int l_t, int d, int pa, const int32_t* seq_len, const int32_t* seq_off,
                                  cudaStream_t st);
// Its backward for the cotangent G [n, d]: dx (fp32 [rows, d], overwritten) receives the part alpha_s G, dpre (operand-typed
// [rows, pa]) the gradient with respect to pre, dq += the gradient of q; scratch: kRedScratchBytes.
gram_status pool_additive_backward(gram_ctx* ctx, int dtype, const StreamRef& x, const void* pre, const float* q,
                                   const float* alpha, const float* G, float* dx, void* dpre, float* dq, float* scratch,
                                   int64_t n, int l_t, int d, int pa, const int32_t* seq_len, const int32_t* seq_off,
                                   cudaStream_t st);
