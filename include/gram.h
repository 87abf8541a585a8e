/* gram.h - C ABI of the GRAM deduplicated encode/accumulate training step (CUDA, sm_100a).
 *
 * GRAM (gradient accumulation for content-based collaborative filtering) trains
 * a content encoder CE and a task module CF (Section 3) without running CE once
 * per interaction: per mini-batch it encodes every *unique* item once, sums the
 * task module's gradients over the occurrences of each item, and runs CE's
 * backward once per unique item (Section 4.1, Fig. 1, Algorithm 1).
 *
 * Conventions for every call
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller
 *     owns every buffer it passes; the context owns parameters, gradients,
 *     workspaces, the Multi-step table and cache.  Nothing passed in is kept
 *     after the call returns unless stated.
 *   - `stream` is a cudaStream_t passed as a plain pointer (NULL = the default
 *     stream).  Work is stream-ordered; calls return without synchronising
 *     unless stated.  A context is not thread-safe.
 *   - Item IDs are int32 in [0, n_items).  Matrices are row-major.
 *   - Every call returns a gram_status and never throws, aborts or traps.  An
 *     error found on the device (an ID out of range) is recorded in the context
 *     and returned by the next synchronising call (gram_sync, gram_step*).
 *   - Outputs are fully overwritten, except the Multi-step table, which
 *     accumulates by definition until gram_window_reset.
 */
#ifndef GRAM_H_
#define GRAM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gram_ctx gram_ctx;
typedef void* gram_stream;              /* a cudaStream_t */

typedef enum gram_status {
  GRAM_OK = 0,
  GRAM_ERR_ARG = 1,                     /* null pointer, negative or inconsistent size */
  GRAM_ERR_ID_RANGE = 2,                /* an item or token ID outside its range */
  GRAM_ERR_WORKSPACE = 3,               /* sizes exceed what the context was created for */
  GRAM_ERR_UNSUPPORTED = 4,             /* a shape the kernels do not cover */
  GRAM_ERR_CUDA = 5,                    /* a CUDA runtime call failed; see gram_last_error */
  GRAM_ERR_TIMEOUT = 6                  /* a bounded device-side wait ran out */
} gram_status;

enum { GRAM_F32 = 0, GRAM_BF16 = 1 };                 /* element types */
/* item pooling: mean over the tokens, token 0, or additive attention over the tokens (Appendix D; width d_a):
 * a_s = q . tanh(W x_s + b), alpha = softmax(a), h = sum_s alpha_s x_s */
enum { GRAM_POOL_MEAN = 0, GRAM_POOL_CLS = 1, GRAM_POOL_ADDITIVE = 2 };
enum { GRAM_TASK_NONE = 0, GRAM_TASK_KT = 1, GRAM_TASK_NR = 2 };
enum { GRAM_MODULE_CE = 0, GRAM_MODULE_TASK = 1 };
enum { GRAM_OPT_SGD = 0, GRAM_OPT_ADAM = 1 };
/* Multi-step GRAM (Section 4.2, Algorithm 1 with N > 1), how a window treats the content representations:
 * GRAM_MULTI_TABLE: the task module reads the unchanged cached encodings during the whole window, the
 *   gradients of Eq. 6 go to a separate per-item table, and the encoder's cotangent is table[i].
 * GRAM_MULTI_PSEUDO_TARGET: the other reading of Section 4.3 and Algorithm 1, step 3 (Eqs. 6 and 9), in which an
 *   item's representation is itself a trainable embedding that later steps keep using: the task module reads
 *   the pseudo-target h~_i = cache[i] - table[i], i.e. the cached encoding minus every gradient the item
 *   has received so far in the window (Eq. 6, SGD with learning rate 1), and the encoder regresses
 *   towards it with the pseudo-loss of Eq. 9: its cotangent is CE(c_i; theta) - h~_i, which carries the
 *   staleness CE(c_i; theta) - cache[i] of the cache besides the accumulated gradients.  The cache is
 *   kept in fp32 in this variant whatever the context's dtype: pseudo-targets differ from the
 *   encodings by gradient-sized amounts that bf16 would round away. */
enum { GRAM_MULTI_TABLE = 0, GRAM_MULTI_PSEUDO_TARGET = 1 };

/* Shapes of the two modules and of the batches a context serves.
 * CE (Section 3.2; Appendix D: attention layers of width 768): token + position
 * embedding, LayerNorm, n_layers post-LayerNorm transformer layers (multi-head
 * attention, erf-GELU feed-forward), pooled to one d-vector per item.
 * CF (Section 3.1): task = KT: x_n = E[b,n] + pos[n] + resp[r_{n-1}], task_layers
 * causal layers (attention only when task_attn_only != 0), a linear head and
 * binary cross-entropy averaged over B*L predictions; task = NR: task_layers
 * self-attention layers (not causal) over the clicked items of a user (Appendix D
 * uses one; 0 = none), then additive
 * attention (width d_a) over the first L - n_cand encodings, dot-product scores
 * with the n_cand candidates, softmax cross-entropy on candidate 0 averaged
 * over B.  A context with n_layers == 0 and task == GRAM_TASK_NONE serves only
 * the index and accumulation calls.
 * Texts and histories longer than 128 rows need dtype = GRAM_BF16 with heads of
 * width 64 (d / n_heads, d / task_heads); other contexts return
 * GRAM_ERR_UNSUPPORTED from the attention of such a sequence.
 * dtype = GRAM_BF16: matrix products and attention take bf16 operands with fp32
 * accumulation; the residual stream, LayerNorm statistics, encodings,
 * parameters and their gradients stay fp32.  GRAM_F32: everything fp32. */
typedef struct gram_config {
  int32_t dtype;
  int32_t n_items, l_t, vocab;
  int32_t d, n_heads, d_ff, n_layers, pooling;
  int32_t task, task_layers, task_heads, task_d_ff, task_attn_only, d_a, n_cand;
  int32_t B_max, L;            /* largest batch: B_max histories of L positions */
  int64_t P_max;               /* largest number of positions for the index/accumulate calls (0 = B_max*L) */
  int32_t d_max;               /* widest row for gather/accumulate (0 = d) */
  int32_t K;                   /* Multi-step window length (Section 4.2); 1 = Single-step */
  int32_t ce_micro_batch;      /* items per encoder pass, bounds activation memory (Section 6.3); 0 = all at once */
  float lr_task;               /* SGD step applied to the task parameters after every gram_step (0 = none) */
  float lr_ce;                 /* SGD step applied to the encoder parameters after an encoder pass (0 = none) */
  int32_t optimizer;           /* GRAM_OPT_SGD: plain steps of lr_task / lr_ce.  GRAM_OPT_ADAM: Adam with the Noam
                                  learning-rate scheme (Appendix D); lr_task / lr_ce are then the peak rates */
  int32_t noam_warmup;         /* updates until the peak rate; <= 0: constant rate */
  float adam_beta1, adam_beta2, adam_eps;   /* <= 0: 0.9, 0.999, 1e-8 */
  int32_t multistep_variant;   /* K > 1: GRAM_MULTI_TABLE or GRAM_MULTI_PSEUDO_TARGET */
  int32_t refresh_after_update; /* K > 1: after the encoder update at the end of a window, encode the touched items once
                                   more with the new parameters and store those encodings in the cache (Algorithm 1,
                                   Eq. 4 produces h with the parameters of the current step); 0: the cache keeps the
                                   forward values of the encoder pass, one update old */
  int32_t defer_update;        /* != 0: gram_step computes gradients and applies no update; the caller calls
                                  gram_optimizer_step itself, e.g. after averaging the gradients over data-parallel
                                  replicas (Section 5.1 trains with distributed data parallelism).  Not with
                                  refresh_after_update, which encodes with the updated parameters inside the step */
} gram_config;

typedef struct gram_step_report {
  float loss;                  /* task loss of this step (Eq. 8) */
  int32_t n_positions;         /* P = B*L interactions in the batch */
  int32_t n_unique;            /* |B_I|, unique items in the batch */
  float boost_ratio;           /* R = P / n_unique (Section 4.4) */
  int32_t n_touched;           /* Multi-step: items touched so far in the window (Single-step: n_unique) */
  int32_t encoder_pass;        /* 1 if this step ran the encoder backward (always for K = 1, every K-th step else) */
  int32_t n_encoded;           /* items the encoder ran on in this step */
  float ms_dedup, ms_encode, ms_gather, ms_task, ms_accumulate, ms_backward, ms_total;  /* device time per stage */
} gram_step_report;

/* --- life cycle ---------------------------------------------------------- */

/* Allocates everything a context will ever need (parameters, gradients,
 * activations for one micro-batch, workspaces, Multi-step table / bitmap /
 * cache when K > 1); no later call allocates.  *out is NULL on failure. */
gram_status gram_create(const gram_config* cfg, gram_ctx** out);
gram_status gram_destroy(gram_ctx* ctx);
/* Waits for the stream and returns any error recorded on the device. */
gram_status gram_sync(gram_ctx* ctx, gram_stream stream);
/* Text of the last error of this context (valid until the next call on it). */
const char* gram_last_error(const gram_ctx* ctx);

/* Number of fp32 parameters of a module.  The flat layout is, for CE:
 * tok_emb[vocab,d] pos_emb[l_t,d] emb_ln_g[d] emb_ln_b[d], then per layer
 * wqkv[3d,d] bqkv[3d] wo[d,d] bo[d] ln1_g ln1_b w1[d_ff,d] b1[d_ff] w2[d,d_ff]
 * b2[d] ln2_g ln2_b, then for GRAM_POOL_ADDITIVE pool_wa[d_a,d] pool_ba[d_a] pool_qa[d_a]; for KT: pos[L,d] resp[3,d], the layers (attention-only
 * layers hold wqkv bqkv wo bo), head_w[d] head_b[1]; for NR: the task_layers
 * layers, then wa[d_a,d] ba[d_a] qa[d_a].  Rows 0..d-1 of wqkv produce Q, the next d K, the last d V; head h
 * owns columns h*d/n_heads .. of each. */
gram_status gram_param_count(const gram_ctx* ctx, int module, size_t* n);
gram_status gram_set_params(gram_ctx* ctx, int module, const float* h_params, size_t n);
gram_status gram_get_params(gram_ctx* ctx, int module, float* h_params, size_t n);
/* Gradients of the last gram_step / gram_encoder_backward / gram_task, same layout (synchronises). */
gram_status gram_get_grads(gram_ctx* ctx, int module, float* h_grads, size_t n);
gram_status gram_zero_grads(gram_ctx* ctx, int module, gram_stream stream);
/* Device address and length of a module's fp32 gradient buffer (same layout as the parameters).  The buffer
 * belongs to the context and lives as long as it; a data-parallel trainer all-reduces it in place between
 * gram_step (with defer_update) and gram_optimizer_step (Section 5.1).  Work queued on the stream that ran the
 * step must have finished, or be ordered, before another stream touches the buffer. */
gram_status gram_grads_device(gram_ctx* ctx, int module, float** d_grads, size_t* n);
/* The configured update of one module from its current gradients (what gram_step applies by itself): an SGD step,
 * or one Adam update at the module's next update count with the Noam rate of that count.  For callers that drive
 * the stages one by one. */
gram_status gram_optimizer_step(gram_ctx* ctx, int module, gram_stream stream);
/* Clears the Adam moment estimates and update counts of both modules (a context starts cleared). */
gram_status gram_optimizer_reset(gram_ctx* ctx, gram_stream stream);
/* Token IDs c_i of every item (Table 1), int32 [n_items, l_t], copied to the device. */
gram_status gram_set_item_tokens(gram_ctx* ctx, const int32_t* h_tokens);
/* Texts of different lengths (Table 3 lists 5 to 271 tokens per item; Appendix D pads or truncates to a maximum):
 * h_lengths int32 [n_items], item i's text is its first h_lengths[i] tokens (1 .. l_t), the remaining slots of its
 * row of h_tokens are padding whose values are never used.  The encoder then attends over the text tokens only and
 * mean pooling averages over them; an item encodes exactly as it would in a model whose l_t is its own length.
 * On the device the token rows of an encoder pass are then packed (item after item, no rows for padding), so a pass
 * costs the sum of its items' lengths, not n * l_t; the pass reads that sum back from the device once (it
 * synchronises the stream).  NULL restores texts of exactly l_t tokens (the state after gram_create). */
gram_status gram_set_item_lengths(gram_ctx* ctx, const int32_t* h_lengths);

/* --- the five stages (Algorithm 1; Fig. 1) -------------------------------- */

/* Stage 1, the unique-item set B_I of a mini-batch (Table 1) and the map from
 * occurrences to items (Fig. 1).  d_ids int32 [P].  Outputs:
 *   d_unique  [>= min(P, n_items)]  distinct IDs, ascending (first U valid)
 *   d_inverse [P]   d_unique[d_inverse[p]] == d_ids[p]
 *   d_perm    [P]   positions grouped by item, ascending inside a group (stable sort order)
 *   d_seg_off [>= min(P, n_items) + 1]  group u is d_perm[d_seg_off[u] .. d_seg_off[u+1])
 *   d_n_unique [1]  U
 * Radix sort on the low ceil(log2 n_items) key bits, then a run-length pass.
 * An ID outside [0, n_items) records GRAM_ERR_ID_RANGE (outputs then unspecified). */
gram_status gram_dedup(gram_ctx* ctx, const int32_t* d_ids, int64_t P, int32_t n_items,
                       int32_t* d_unique, int32_t* d_inverse, int32_t* d_perm, int32_t* d_seg_off,
                       int32_t* d_n_unique, gram_stream stream);

/* Stage 2, Eq. 4: d_H[u, :] = CE(tokens of item d_items[u]) for u < U, once per
 * unique item.  d_item_tokens int32 [n_items, l_t] (NULL = the context's copy).
 * d_H is fp32 [U, d] for either dtype (the residual stream stays fp32; bf16 is
 * the element type of the matrix products' operands).  save_activations != 0
 * keeps what gram_encoder_backward needs (U must then fit one micro-batch). */
gram_status gram_encode_unique(gram_ctx* ctx, const int32_t* d_item_tokens, const int32_t* d_items, int32_t U,
                               float* d_H, int save_activations, gram_stream stream);

/* Failure detection: every wait of one thread block on another (the tile look-back of gram_dedup, the pipeline
 * barriers of the matrix products) has a poll limit, after which the kernel records GRAM_ERR_TIMEOUT in the context,
 * writes nothing more and returns, so that a stuck wait costs about a second instead of the device.  This call shows
 * it: it launches the dedup's run-length kernel with a predecessor tile that never runs.  It returns GRAM_OK once the
 * launch is queued; the next gram_sync takes about a second and returns GRAM_ERR_TIMEOUT; the context stays usable.
 * (No counterpart in the paper.) */
gram_status gram_selftest_bounded_wait(gram_ctx* ctx, gram_stream stream);

/* Stage 3 (Section 4.3: the encoder's output h_i is handed to the task module, which completes the forward pass
 * with it; Fig. 1 draws the copies): d_E[p, :] = d_src[d_index[p], :] for p < P.  Single-step: src = H,
 * index = inverse.  Multi-step: src = the encoding cache, index = ids.
 * Rows are d elements of `dtype`; n_src_rows bounds the index (ID_RANGE else). */
gram_status gram_gather(gram_ctx* ctx, const void* d_src, int64_t n_src_rows, const int32_t* d_index, int64_t P,
                        int32_t d, int dtype, void* d_E, gram_stream stream);

/* Stage 4, Single-step (Eq. 6: with SGD of rate 1 the change of an item's
 * encoding is the sum of dL/dE over its occurrences):
 *   d_G[u, :] = sum over j in [d_seg_off[u], d_seg_off[u+1]) of d_dE[d_perm[j], :]
 * fp32 [P, d] -> fp32 [U, d].  The order of additions is fixed by (P, U,
 * d_seg_off) alone, so repeated calls give bit-identical results. */
gram_status gram_accumulate(gram_ctx* ctx, const float* d_dE, const int32_t* d_perm, const int32_t* d_seg_off,
                            int64_t P, int32_t U, int32_t d, float* d_G, gram_stream stream);

/* Stage 4, Multi-step (Section 4.2): the same sums are added into the per-item
 * table, d_table[d_unique[u], :] += sum, fp32 [n_items, d], and bit d_unique[u]
 * of d_touched_bits (uint32 [ceil(n_items/32)]) is set.  NULL table/bits select
 * the context's own (K > 1). */
gram_status gram_accumulate_multistep(gram_ctx* ctx, const float* d_dE, const int32_t* d_perm,
                                      const int32_t* d_seg_off, const int32_t* d_unique, int64_t P, int32_t U,
                                      int32_t d, int32_t n_items, float* d_table, uint32_t* d_touched_bits,
                                      gram_stream stream);
/* Ascending list of the set bits: d_list [>= n_items], d_count [1]. */
gram_status gram_touched_list(gram_ctx* ctx, const uint32_t* d_touched_bits, int32_t n_items, int32_t* d_list,
                              int32_t* d_count, gram_stream stream);

/* Task module forward and backward (Eq. 5 and the gradient of Eq. 8 with
 * respect to the encodings): d_E fp32 [B, L, d], d_labels int32 [B, L] ->
 * d_dE fp32 [B*L, d], d_loss fp32 [1]; task parameter gradients are
 * overwritten in the context.  Labels are 0 or 1.  For GRAM_TASK_KT a history
 * shorter than L ends in padding (Appendix D: sequences are cut or padded to a
 * maximum length): its padded positions carry label -1 and any valid item ID,
 * are not predicted, receive a zero row of d_dE, and the loss is the mean over
 * the real predictions of the batch.  For GRAM_TASK_NR a user with fewer
 * clicks than history slots marks the empty slots (any of the first
 * L - n_cand positions) with label -1; they take no part in the user vector
 * and receive a zero row of d_dE; at least one slot per user must hold a click.
 * The same holds for gram_step. */
gram_status gram_task(gram_ctx* ctx, const float* d_E, const int32_t* d_labels, int32_t B, float* d_dE,
                      float* d_loss, gram_stream stream);

/* Stage 5, Eq. 7: encoder parameter gradients += sum over u of J_u^T d_G[u, :],
 * one VJP per unique item, using the activations saved by the last
 * gram_encode_unique(save_activations = 1) over the same items. */
gram_status gram_encoder_backward(gram_ctx* ctx, const float* d_G, const int32_t* d_items, int32_t U,
                                  gram_stream stream);

/* --- the whole step -------------------------------------------------------- */

/* One training step (Algorithm 1) on a batch of B histories: d_ids, d_labels
 * int32 [B, L].  K = 1: dedup, encode unique, gather, task forward/backward,
 * accumulate, encoder backward; gradients of both modules are left in the
 * context.  K > 1: encodings come from the cache (gram_cache_fill first), the
 * sums go to the table, and every K-th call runs the encoder forward and
 * backward over the touched items in micro-batches, refreshes their cache
 * rows and clears the window.  Task parameters take the configured update of
 * rate lr_task, encoder parameters one of lr_ce after an encoder pass (none of
 * it with defer_update).  Synchronises; fills *report (may be NULL).
 * A batch with an item ID outside [0, n_items) returns GRAM_ERR_ID_RANGE and
 * leaves parameters, optimiser state, table, touched bits, cache and the
 * position in the window exactly as they were.  Host waits per call: K = 1:
 * one after the dedup (U sizes the encoder pass) and one at the end; K > 1: one
 * at the end, plus one on the K-th step for the number of touched items. */
gram_status gram_step(gram_ctx* ctx, const int32_t* d_ids, const int32_t* d_labels, int32_t B,
                      gram_step_report* report, gram_stream stream);
/* The same with HOST buffers: copies ids and labels to the device, runs the
 * step, copies the loss back. */
gram_status gram_step_host(gram_ctx* ctx, const int32_t* h_ids, const int32_t* h_labels, int32_t B,
                           gram_step_report* report, gram_stream stream);

/* Multi-step: encode every item with the current parameters into the cache. */
gram_status gram_cache_fill(gram_ctx* ctx, gram_stream stream);
/* Multi-step: zero the table and the touched bitmap, restart the window. */
gram_status gram_window_reset(gram_ctx* ctx, gram_stream stream);
/* Multi-step state, copied to host: table fp32 [n_items, d], touched uint32
 * [ceil(n_items/32)], cache fp32 [n_items, d] (converted).  NULL skips one. */
gram_status gram_get_window(gram_ctx* ctx, float* h_table, uint32_t* h_touched, float* h_cache);

/* --- checkpoint / resume (the paper keeps the checkpoint of the best validation epoch, Appendix D) ------------------
 * Everything a context holds besides what the caller gave it: parameters (gram_get_params / gram_set_params), the
 * optimiser's state, and for K > 1 the open window.  Exported by one context and imported into another context of the
 * same configuration, training continues bit for bit.  All calls synchronise. */
/* Multi-step: gram_get_window plus the number of steps already taken in the open window (0 .. K-1). */
gram_status gram_state_export(gram_ctx* ctx, float* h_table, uint32_t* h_touched, float* h_cache, int32_t* steps_in_window);
/* Multi-step: the reverse.  Arrays as in gram_get_window (NULL leaves that part as it is); the cache is rounded to the
 * context's cache type (bf16 contexts with GRAM_MULTI_TABLE), so values that came from gram_state_export are restored
 * exactly. */
gram_status gram_state_import(gram_ctx* ctx, const float* h_table, const uint32_t* h_touched, const float* h_cache,
                              int32_t steps_in_window);
/* Optimiser state of one module: update count, and for GRAM_OPT_ADAM the two moment estimates in the parameters'
 * layout (h_m, h_v fp32 [gram_param_count]; ignored and may be NULL for GRAM_OPT_SGD). */
gram_status gram_optimizer_export(gram_ctx* ctx, int module, float* h_m, float* h_v, int64_t* updates);
gram_status gram_optimizer_import(gram_ctx* ctx, int module, const float* h_m, const float* h_v, int64_t updates);

/* --- measurement -------------------------------------------------------------
 * Kernel kinds for gram_profile_read. */
enum { GRAM_K_GEMM = 0, GRAM_K_ATTENTION = 1, GRAM_K_LAYERNORM = 2, GRAM_K_COLSUM = 3, GRAM_K_EMBED_POOL = 4,
       GRAM_K_DEDUP = 5, GRAM_K_GATHER = 6, GRAM_K_ACCUMULATE = 7, GRAM_K_TASK_HEAD = 8, GRAM_K_OTHER = 9,
       GRAM_K_OPTIMIZER = 10, GRAM_K_COUNT = 11 };
/* enable != 0: from now on every kernel group the library launches is bracketed by
 * CUDA events on its stream (a few microseconds of host time per group); 0 turns
 * it off.  Either way the totals are cleared. */
gram_status gram_profile(gram_ctx* ctx, int enable);
/* Synchronises the device and returns, for one kind, the totals since the last
 * gram_profile call: device milliseconds, algorithmic work (flops for
 * GRAM_K_GEMM and GRAM_K_ATTENTION, bytes for the others) and kernel launches. */
gram_status gram_profile_read(gram_ctx* ctx, int kind, double* ms, double* work, int64_t* launches);
/* The same totals per call site, as text: one line "tag kind ms work launches"
 * per tag (the matrix products are tagged by their role, e.g. fwd_ffn1). */
gram_status gram_profile_dump(gram_ctx* ctx, char* h_text, size_t n);
/* Kernels this context has launched since it was created (counted always). */
gram_status gram_launch_count(const gram_ctx* ctx, int64_t* launches);

/* --- the segmented sum without any allocation ----------------------------------
 * (The paper has no counterpart to this call; it exists for the sake of callers.)
 * Same result as gram_accumulate, d_G[u, :] = sum of d_dE[d_perm[j], :] over
 * j in [d_seg_off[u], d_seg_off[u+1]), for code that is not allowed to allocate
 * device memory: a plug-in running inside a host application that owns the
 * allocator, a library called between the steps of a memory-planned job, a
 * real-time loop.  It needs no context (creating one allocates): the partial
 * sums that cross work-unit boundaries go to a fixed array inside the library
 * image, about 4.9 MB, which every GPU that loads the library holds until the
 * process exits.  The call uses no cudaMalloc/cudaFree and no allocating
 * library routine; inputs and outputs are the caller's.
 *   - Limits: d <= 1024 columns (a multiple of 4), P <= 2^31-1.  Larger sizes
 *     return GRAM_ERR_WORKSPACE and a message in h_err.
 *   - The first call on each device looks up the array's device address (with
 *     that device current); make that first call before any stream capture.
 *   - All calls on a device share the one array: two calls that may run on the
 *     GPU at the same time (different streams, different threads) race.  Order
 *     them on one stream or with events.
 *   - The order of additions differs from gram_accumulate's (fewer work units),
 *     so results agree to rounding, not bit for bit; they are bit-identical
 *     from call to call.  A position in d_perm outside [0, P) is read as row 0
 *     and is not reported.
 * h_err (may be NULL) receives a message of at most err_len bytes on failure. */
gram_status gram_accumulate_static(const float* d_dE, const int32_t* d_perm, const int32_t* d_seg_off, int64_t P,
                                   int32_t U, int32_t d, float* d_G, gram_stream stream, char* h_err, size_t err_len);

/* --- a building block, exported so that it can be tested on its own --------
 * C[M, N] = A x B with bf16 operands and fp32 accumulation on the tensor cores.
 * a_kmajor != 0: A is [M, K] row-major, else [K, M] row-major; b_kmajor != 0:
 * B is [N, K] row-major, else [K, N] row-major.  C is fp32 [M, N] when
 * c_f32 != 0, else bf16.  d_bias (fp32 [N]) may be NULL.  accumulate != 0
 * adds to C instead of overwriting (fp32 C only).  M, N, K multiples of 8. */
gram_status gram_gemm_bf16(gram_ctx* ctx, const void* d_A, int a_kmajor, const void* d_B, int b_kmajor, void* d_C,
                           int c_f32, const float* d_bias, int accumulate, int64_t M, int32_t N, int64_t K,
                           gram_stream stream);

/* The same product followed by one of the fused epilogues the encoder's layers use (Appendix D: attention layers of
 * width 768; each epilogue replaces a separate pass over the [M, N] result):
 *   v = acc + d_bias[n]
 *   gelu != 0:        d_gelu_grad_out(m, n) = gelu'(v) (bf16, may be NULL);  v = gelu(v)     (erf form)
 *   d_gelu_grad_in:   v *= d_gelu_grad_in(m, n) (bf16)
 *   d_res:            v += d_res(m, n) (fp32), or, when d_res_mean is given, LayerNorm applied where it is read:
 *                     v += (d_res(m, n) - d_res_mean[m]) * d_res_rstd[m] * d_res_gamma[n] + d_res_beta[n]
 *   accumulate != 0:  v += C(m, n)                                                   (fp32 C only)
 *   d_copy_bf16:      bf16 copy of the stored result
 * At most one of d_res, d_gelu_grad_in and accumulate per call.  All [M, N] matrices share C's leading
 * dimension N.  e == NULL is a plain product. */
typedef struct gram_gemm_epilogue {
  const float* d_bias;
  const float* d_res;
  const float* d_res_mean;
  const float* d_res_rstd;
  const float* d_res_gamma;
  const float* d_res_beta;
  void* d_gelu_grad_out;
  const void* d_gelu_grad_in;
  void* d_copy_bf16;
  int32_t gelu, accumulate;
} gram_gemm_epilogue;
gram_status gram_gemm_bf16_epilogue(gram_ctx* ctx, const void* d_A, int a_kmajor, const void* d_B, int b_kmajor, void* d_C,
                                    int c_f32, const gram_gemm_epilogue* e, int64_t M, int32_t N, int64_t K,
                                    gram_stream stream);

/* --- the optimiser's two pieces, exported so that they can be tested on their own (Appendix D: Adam under the
 * Noam learning-rate scheme) ----------------------------------------------
 * gram_noam_rate (host only): *h_rate = peak * min(t / warmup, sqrt(warmup / t)) for update t >= 1, the Noam curve
 * scaled so that its maximum, at t = warmup, is `peak`; warmup <= 0 gives the constant `peak`.
 * gram_adam_update: one Adam update of n fp32 parameters in place at update count t >= 1:
 *   m = beta1 m + (1 - beta1) g;  v = beta2 v + (1 - beta2) g^2;
 *   w -= rate * (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps)
 * d_w, d_g, d_m, d_v: device fp32 [n], 16-byte aligned; d_w_bf16 (may be NULL): device bf16 [n] that receives the
 * rounded new parameters (the copy the tensor cores read).  The two bias corrections are formed on the host in
 * double precision. */
gram_status gram_noam_rate(int64_t t, float peak, int32_t warmup, float* h_rate);
gram_status gram_adam_update(gram_ctx* ctx, float* d_w, const float* d_g, float* d_m, float* d_v, size_t n, int64_t t,
                             float rate, float beta1, float beta2, float eps, void* d_w_bf16, gram_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* GRAM_H_ */
