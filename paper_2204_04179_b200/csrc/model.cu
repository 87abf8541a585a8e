// The two modules (content encoder CE, task module CF) and the training step that ties the five
// stages together (Algorithm 1): parameter layout, activation arenas, forward and backward passes
// composed from gemm.cu / layers.cu / the index kernels, Single-step and Multi-step drivers.
#include <new>
#include <vector>

#include "gemm.h"
#include "layers.h"
#include "model.h"

namespace {

struct LayerOff {
  size_t wqkv, bqkv, wo, bo, ln1g, ln1b, w1, b1, w2, b2, ln2g, ln2b;
};

struct Module {
  size_t n = 0;
  float* w = nullptr;      // fp32 parameters
  float* g = nullptr;      // fp32 gradients
  bf16* wb = nullptr;      // bf16 copy of the parameters (bf16 contexts), refreshed when stale
  bool wb_stale = true;
  float *am = nullptr, *av = nullptr;   // Adam moment estimates (contexts created with GRAM_OPT_ADAM)
  int64_t updates = 0;     // updates applied so far (the count Adam's bias corrections and the Noam rate take)
};

// saved per layer.  fp32: the residual sums z1, z2 (attention-only layers: outf) and LayerNorm statistics;
// operand-typed (bf16 on the tensor cores): what the matrix products and attention read
struct LayerActs {
  void *qkv, *ctx, *h1, *u, *g, *out;
  float *z1, *z2, *outf;
  float *mean1, *rstd1, *mean2, *rstd2;
  float* lse;                              // [heads, rows] softmax row statistics of the attention (tensor-core kernels)
};

// a run of post-LayerNorm transformer layers over sequences of S tokens
struct Stack {
  int d = 0, heads = 0, d_ff = 0, n_layers = 0, attn_only = 0, causal = 0;
  int64_t cap = 0;                         // tokens the buffers hold
  const int32_t* seq_len = nullptr;        // per sequence: rows that are text (null: all S); set per pass
  const int32_t* seq_off = nullptr;        // packed rows: first row of each sequence (null: sequence s starts at row s*S)
  int64_t packed_rows = 0;                 // packed rows: rows in total (0: n_seq * S)
  SeqGroups groups;                        // packed rows: the sequences grouped by length
  bool grouped = false;
  std::vector<LayerOff> off;
  std::vector<LayerActs> acts;
  // backward scratch: the gradient stream (fp32, two buffers) and operand-typed branch gradients
  float *curf = nullptr, *othf = nullptr;
  void *dzb = nullptr, *dqkv = nullptr, *du = nullptr, *dctx = nullptr;
  float* cpart = nullptr;                  // column-sum partials written by fused producers
  size_t cpart_elems = 0;
  float* delta = nullptr;                  // [heads, rows] scratch of the attention backward over long sequences
};

struct Arena {
  char* base = nullptr;
  size_t off = 0;
  void* take(size_t bytes) {
    off = (off + 255) & ~(size_t)255;
    void* p = base ? base + off : nullptr;
    off += bytes;
    return p;
  }
};

size_t layer_layout(LayerOff* o, size_t at, int d, int d_ff, int attn_only) {
  o->wqkv = at; at += (size_t)3 * d * d;
  o->bqkv = at; at += (size_t)3 * d;
  o->wo = at; at += (size_t)d * d;
  o->bo = at; at += d;
  if (!attn_only) {
    o->ln1g = at; at += d;
    o->ln1b = at; at += d;
    o->w1 = at; at += (size_t)d_ff * d;
    o->b1 = at; at += d_ff;
    o->w2 = at; at += (size_t)d * d_ff;
    o->b2 = at; at += d;
    o->ln2g = at; at += d;
    o->ln2b = at; at += d;
  }
  return at;
}

}  // namespace

struct Model {
  gram_ctx* ctx = nullptr;
  gram_config cfg;
  int dtype = GRAM_F32;
  size_t esz = 4;
  Module ce, task;
  // encoder
  size_t o_tok = 0, o_pos = 0, o_elng = 0, o_elnb = 0;
  // additive-attention pooling (GRAM_POOL_ADDITIVE): parameters, saved scores and the encoder output they pool
  size_t o_pwa = 0, o_pba = 0, o_pqa = 0;
  void *pool_pre = nullptr, *pool_dpre = nullptr;
  float* pool_alpha = nullptr;
  StreamRef pool_x;
  const void* pool_xb = nullptr;
  Stack enc;
  // With token-0 pooling only row 0 of every item's last-layer output is ever read, so the row-wise part of the
  // last layer (output projection, feed-forward, both LayerNorms) runs on those rows alone: `tail` holds their
  // activations and scratch (one row per item), tail_* the layer's input stream at those rows.
  bool cls_tail = false;
  Stack tail;
  float *tail_z = nullptr, *tail_mean = nullptr, *tail_rstd = nullptr;
  float* z0 = nullptr;               // token + position embedding, fp32
  void* x0 = nullptr;                // its LayerNorm, operand-typed
  float *mean0 = nullptr, *rstd0 = nullptr;
  int32_t *tok_ids = nullptr, *tok_unique = nullptr, *tok_inverse = nullptr, *tok_perm = nullptr, *tok_seg = nullptr,
          *tok_nu = nullptr;
  int32_t* item_len = nullptr;       // [n_items] tokens of each item that are text (variable-length texts), else null
  int32_t* item_len_buf = nullptr;   // its storage
  int32_t* seq_len = nullptr;        // [mb] the same for the items of the current encoder pass
  int32_t* seq_off = nullptr;        // [mb + 1] first packed row of each of them; [n] = rows of the pass
  int32_t* seq_groups = nullptr;     // [mb] their numbers grouped by length (for the attention kernels' tile sizes)
  int32_t* seq_info = nullptr;       // [8] group sizes and the row total, read back by the host
  int64_t saved_rows = 0;            // token rows of the last encoder pass (packed when the texts differ in length)
  int32_t mb = 0;                    // items per encoder pass
  int32_t saved_n = -1;              // items whose activations the last encoder pass saved (-1: none)
  // task
  size_t t_pos = 0, t_resp = 0, t_headw = 0, t_headb = 0, t_wa = 0, t_ba = 0, t_qa = 0;
  Stack tk;
  float* tx = nullptr;               // task input stream, fp32
  void *txb = nullptr, *pre = nullptr, *dpre = nullptr;
  // news task with self-attention layers over the clicked items: their packed layout, and the encodings after the layers
  int32_t *nr_len = nullptr, *nr_off = nullptr, *nr_rows = nullptr, *nr_pos2row = nullptr;
  float *nr_E2 = nullptr, *nr_dE2 = nullptr;
  // step buffers
  int32_t* item_tokens = nullptr;
  int32_t *ids = nullptr, *labels = nullptr, *unique = nullptr, *inverse = nullptr, *perm = nullptr, *seg_off = nullptr,
          *n_unique = nullptr;
  int32_t u_cap = 0;
  float *H = nullptr, *E = nullptr;  // encodings per unique item / per position, fp32
  void* Eb = nullptr;                // operand-typed copy of E (NR products; Multi-step gather from the cache)
  float *dE = nullptr, *G = nullptr, *loss = nullptr, *red = nullptr;
  int32_t* n_real = nullptr;         // predictions of the batch that are not padding
  // Multi-step window
  float* table = nullptr;
  uint32_t* touched = nullptr;
  void* cache = nullptr;
  int cache_dtype = GRAM_F32;        // element type of the cache: the context's, or fp32 with pseudo-targets
  bool pseudo = false;               // Multi-step with pseudo-targets (GRAM_MULTI_PSEUDO_TARGET)
  int32_t *tlist = nullptr, *tcount = nullptr;
  int step_in_window = 0;
  char* arena = nullptr;
  size_t arena_bytes = 0;
  cudaEvent_t ev[8] = {};
  int32_t* h_pinned = nullptr;       // [16] pinned host words for small read-backs
};

// the Noam curve scaled to peak at update `warmup` (Appendix D; Vaswani et al. 2017, Eq. 3)
double noam_rate(int64_t t, double peak, int warmup) {
  if (warmup <= 0) return peak;
  const double x = (double)t, w = (double)warmup;
  const double up = x / w, down = sqrt(w / x);
  return peak * (up < down ? up : down);
}


namespace {

void stack_buffers(Arena& a, Stack& s, size_t esz) {
  s.acts.resize(s.n_layers);
  const size_t T = (size_t)s.cap, d = s.d, f = s.d_ff;
  for (int l = 0; l < s.n_layers; ++l) {
    LayerActs& x = s.acts[l];
    x.qkv = a.take(T * 3 * d * esz);
    x.ctx = a.take(T * d * esz);
    x.out = a.take(T * d * esz);
    x.lse = (float*)a.take(T * (size_t)(s.heads > 0 ? s.heads : 1) * 4);
    if (s.attn_only) {
      x.outf = (float*)a.take(T * d * 4);
    } else {
      x.z1 = (float*)a.take(T * d * 4);
      x.h1 = a.take(T * d * esz);
      x.u = a.take(T * f * esz);
      x.g = a.take(T * f * esz);
      x.z2 = (float*)a.take(T * d * 4);
      x.mean1 = (float*)a.take(T * 4);
      x.rstd1 = (float*)a.take(T * 4);
      x.mean2 = (float*)a.take(T * 4);
      x.rstd2 = (float*)a.take(T * 4);
    }
  }
  s.curf = (float*)a.take(T * d * 4);
  s.othf = (float*)a.take(T * d * 4);
  s.dzb = a.take(T * d * esz);
  s.dqkv = a.take(T * 3 * d * esz);
  s.dctx = a.take(T * d * esz);
  s.du = s.attn_only ? nullptr : a.take(T * f * esz);
  s.cpart_elems = ((T + 31) / 32) * (f > 3 * d ? f : 3 * d);     // [ceil(T / 32)][d_ff] or [sequences][3 d]
  s.cpart = (float*)a.take(s.cpart_elems * 4);
  s.delta = (float*)a.take(T * (size_t)(s.heads > 0 ? s.heads : 1) * 4);
}

void layout_buffers(Model* m, Arena& a) {
  const gram_config& c = m->cfg;
  const size_t esz = m->esz, d = c.d;
  const int64_t P = (int64_t)c.B_max * c.L;
  if (c.n_layers > 0) {
    const size_t T = (size_t)m->mb * c.l_t;
    m->z0 = (float*)a.take(T * d * 4);
    m->x0 = a.take(T * d * esz);
    m->mean0 = (float*)a.take(T * 4);
    m->rstd0 = (float*)a.take(T * 4);
    m->tok_ids = (int32_t*)a.take(T * 4);
    const size_t tu = T < (size_t)c.vocab ? T : (size_t)c.vocab;
    m->tok_unique = (int32_t*)a.take(tu * 4);
    m->tok_inverse = (int32_t*)a.take(T * 4);
    m->tok_perm = (int32_t*)a.take(T * 4);
    m->tok_seg = (int32_t*)a.take((tu + 1) * 4);
    m->tok_nu = (int32_t*)a.take(4);
    m->item_len_buf = (int32_t*)a.take((size_t)c.n_items * 4);
    m->seq_len = (int32_t*)a.take((size_t)m->mb * 4);
    m->seq_off = (int32_t*)a.take(((size_t)m->mb + 1) * 4);
    m->seq_groups = (int32_t*)a.take((size_t)m->mb * 4);
    m->seq_info = (int32_t*)a.take(8 * 4);
    stack_buffers(a, m->enc, esz);
    if (c.pooling == GRAM_POOL_ADDITIVE) {
      m->pool_pre = a.take(T * c.d_a * esz);
      m->pool_dpre = a.take(T * c.d_a * esz);
      m->pool_alpha = (float*)a.take(T * 4);
    }
    if (m->cls_tail) {
      stack_buffers(a, m->tail, esz);
      m->tail_z = (float*)a.take((size_t)m->mb * d * 4);
      m->tail_mean = (float*)a.take((size_t)m->mb * 4);
      m->tail_rstd = (float*)a.take((size_t)m->mb * 4);
    }
    m->item_tokens = (int32_t*)a.take((size_t)c.n_items * c.l_t * 4);
  }
  if (c.task != GRAM_TASK_NONE) {
    if (c.task == GRAM_TASK_KT) {
      m->tx = (float*)a.take((size_t)P * d * 4);
      m->txb = a.take((size_t)P * d * esz);
      stack_buffers(a, m->tk, esz);
    } else {
      m->pre = a.take((size_t)P * c.d_a * esz);
      m->dpre = a.take((size_t)P * c.d_a * esz);
      if (c.task_layers > 0) {
        const size_t Th = (size_t)m->tk.cap;
        m->tx = (float*)a.take(Th * d * 4);
        m->txb = a.take(Th * d * esz);
        stack_buffers(a, m->tk, esz);
        m->nr_len = (int32_t*)a.take((size_t)c.B_max * 4);
        m->nr_off = (int32_t*)a.take(((size_t)c.B_max + 1) * 4);
        m->nr_rows = (int32_t*)a.take(Th * 4);
        m->nr_pos2row = (int32_t*)a.take((size_t)P * 4);
        m->nr_E2 = (float*)a.take((size_t)P * d * 4);
        m->nr_dE2 = (float*)a.take((size_t)P * d * 4);
      }
    }
  }
  m->ids = (int32_t*)a.take((size_t)P * 4);
  m->labels = (int32_t*)a.take((size_t)P * 4);
  m->unique = (int32_t*)a.take((size_t)m->u_cap * 4);
  m->inverse = (int32_t*)a.take((size_t)P * 4);
  m->perm = (int32_t*)a.take((size_t)P * 4);
  m->seg_off = (int32_t*)a.take(((size_t)m->u_cap + 1) * 4);
  m->n_unique = (int32_t*)a.take(4);
  const size_t hrows = (size_t)(m->u_cap > m->mb ? m->u_cap : m->mb);
  m->H = (float*)a.take(hrows * d * 4);
  m->G = (float*)a.take(hrows * d * 4);
  m->E = (float*)a.take((size_t)P * d * 4);
  m->Eb = a.take((size_t)P * d * esz);
  m->dE = (float*)a.take((size_t)P * d * 4);
  m->loss = (float*)a.take(4);
  m->n_real = (int32_t*)a.take(4);
  m->red = (float*)a.take(kRedScratchBytes);
  if (c.K > 1) {
    m->table = (float*)a.take((size_t)c.n_items * d * 4);
    m->touched = (uint32_t*)a.take((size_t)((c.n_items + 31) / 32) * 4);
    m->cache = a.take((size_t)c.n_items * d * (m->cache_dtype == GRAM_BF16 ? 2 : 4));
    m->tlist = (int32_t*)a.take((size_t)c.n_items * 4);
    m->tcount = (int32_t*)a.take(4);
  }
}

gram_status module_alloc(gram_ctx* ctx, Module* mod, size_t n, bool want_bf16, bool want_adam) {
  mod->n = n;
  if (n == 0) return GRAM_OK;
  GRAM_CUDA(ctx, cudaMalloc(&mod->w, n * 4));
  GRAM_CUDA(ctx, cudaMalloc(&mod->g, n * 4));
  GRAM_CUDA(ctx, cudaMemset(mod->w, 0, n * 4));
  GRAM_CUDA(ctx, cudaMemset(mod->g, 0, n * 4));
  if (want_adam) {
    GRAM_CUDA(ctx, cudaMalloc(&mod->am, n * 4));
    GRAM_CUDA(ctx, cudaMalloc(&mod->av, n * 4));
    GRAM_CUDA(ctx, cudaMemset(mod->am, 0, n * 4));
    GRAM_CUDA(ctx, cudaMemset(mod->av, 0, n * 4));
  }
  if (want_bf16) GRAM_CUDA(ctx, cudaMalloc(&mod->wb, n * 2));
  mod->wb_stale = true;
  return GRAM_OK;
}

gram_status refresh_bf16(Model* m, Module& mod, cudaStream_t st) {
  if (m->dtype == GRAM_BF16 && mod.wb_stale && mod.n) {
    GRAM_TRY(convert_f32_to_bf16(m->ctx, mod.w, mod.wb, mod.n, st));
    mod.wb_stale = false;
  }
  return GRAM_OK;
}

// the weight matrix at `off` in the element type the matrix products take
inline const void* W(const Model* m, const Module& mod, size_t off) {
  return m->dtype == GRAM_BF16 ? (const void*)(mod.wb + off) : (const void*)(mod.w + off);
}
inline void* at(const Model* m, void* p, size_t elems) { return (char*)p + elems * m->esz; }

// Y[T, N] = X[T, K] W[N, K]^T (+ epilogue); y_f32: Y is the fp32 stream, else operand-typed
gram_status mm_fwd(Model* m, const void* X, const void* Wt, void* Y, bool y_f32, int64_t T, int N, int K,
                   const GemmEpilogue& e, cudaStream_t st) {
  return gemm_launch(m->ctx, gram_gemm_ws(m->ctx), m->dtype, X, 1, K, Wt, 1, K, Y, (y_f32 || m->dtype == GRAM_F32) ? 1 : 0, N, T,
                     N, K, e, 0, st);
}
// dX[T, K] = dY[T, N] W[N, K] (+ epilogue)
gram_status mm_dx(Model* m, const void* dY, const void* Wt, void* dX, bool x_f32, int64_t T, int N, int K,
                  const GemmEpilogue& e, cudaStream_t st) {
  return gemm_launch(m->ctx, gram_gemm_ws(m->ctx), m->dtype, dY, 1, N, Wt, 0, K, dX, (x_f32 || m->dtype == GRAM_F32) ? 1 : 0, K, T,
                     K, N, e, 0, st);
}
// dW[N, K] += dY[T, N]^T X[T, K]   (fp32 result, the token dimension may be split)
gram_status mm_dw(Model* m, const void* dY, const void* X, float* dW, int64_t T, int N, int K, cudaStream_t st,
                  const char* tag = "dw") {
  GemmEpilogue e;
  e.accumulate = 1;
  e.tag = tag;
  return gemm_launch(m->ctx, gram_gemm_ws(m->ctx), m->dtype, dY, 0, N, X, 0, K, dW, 1, K, N, K, T, e, 1, st);
}

void set_res(GemmEpilogue& e, const StreamRef& x) {
  e.res = x.z;
  e.res_mean = x.mean;
  e.res_rstd = x.rstd;
  e.res_gamma = x.gamma;
  e.res_beta = x.beta;
}

// ---- one transformer layer in two parts, forward --------------------------------------------
// the attention part over whole sequences: qkv = x Wqkv^T + bqkv, ctx = softmax(Q K^T / sqrt(dh)) V
gram_status layer_attention_forward(Model* m, Module& mod, Stack& s, int l, const void* xb, int64_t n_seq, int S, cudaStream_t st) {
  const int64_t T = s.packed_rows ? s.packed_rows : n_seq * S;
  const LayerOff& o = s.off[l];
  LayerActs& a = s.acts[l];
  GemmEpilogue e;
  e.bias = mod.w + o.bqkv;
  e.tag = "fwd_qkv";
  GRAM_TRY(mm_fwd(m, xb, W(m, mod, o.wqkv), a.qkv, false, T, 3 * s.d, s.d, e, st));
  return attention_forward(m->ctx, m->dtype, a.qkv, a.ctx, a.lse, T, n_seq, S, s.d, s.heads, s.causal, s.seq_len, s.seq_off,
                           s.grouped ? &s.groups : nullptr, st);
}

// the row-wise rest of the layer over T rows: output projection + residual, LayerNorm, feed-forward + residual,
// LayerNorm.  x: the layer's input stream at those rows; ctx_in: the attention output at those rows; a: where the
// activations of these rows are kept.  The rows need not be whole sequences.
gram_status layer_rest_forward(Model* m, Module& mod, const LayerOff& o, LayerActs& a, int d, int f, int attn_only,
                               const StreamRef& x, const void* ctx_in, int64_t T, cudaStream_t st, StreamRef* x_out,
                               const void** xb_out) {
  gram_ctx* ctx = m->ctx;
  GemmEpilogue e;
  e.bias = mod.w + o.bo;
  e.tag = "fwd_attn_out";
  set_res(e, x);
  if (attn_only) {
    e.copy_out = a.out;
    GRAM_TRY(mm_fwd(m, ctx_in, W(m, mod, o.wo), a.outf, true, T, d, d, e, st));       // out = x + ctx Wo^T + bo
    *x_out = StreamRef();
    x_out->z = a.outf;
  } else {
    GRAM_TRY(mm_fwd(m, ctx_in, W(m, mod, o.wo), a.z1, true, T, d, d, e, st));         // z1 = x + ctx Wo^T + bo
    GRAM_TRY(layernorm_forward(ctx, m->dtype, a.z1, mod.w + o.ln1g, mod.w + o.ln1b, a.h1, a.mean1, a.rstd1, T, d, st));
    e = GemmEpilogue();
    e.bias = mod.w + o.b1;
    e.gelu = 1;
    e.pre = a.u;
    e.tag = "fwd_ffn1";
    GRAM_TRY(mm_fwd(m, a.h1, W(m, mod, o.w1), a.g, false, T, f, d, e, st));          // v = h1 W1^T + b1: g = gelu(v), u = gelu'(v)
    e = GemmEpilogue();
    e.bias = mod.w + o.b2;
    e.tag = "fwd_ffn2";
    StreamRef h1;
    h1.z = a.z1; h1.mean = a.mean1; h1.rstd = a.rstd1; h1.gamma = mod.w + o.ln1g; h1.beta = mod.w + o.ln1b;
    set_res(e, h1);
    GRAM_TRY(mm_fwd(m, a.g, W(m, mod, o.w2), a.z2, true, T, d, f, e, st));           // z2 = LN1(z1) + g W2^T + b2
    GRAM_TRY(layernorm_forward(ctx, m->dtype, a.z2, mod.w + o.ln2g, mod.w + o.ln2b, a.out, a.mean2, a.rstd2, T, d, st));
    *x_out = StreamRef();
    x_out->z = a.z2; x_out->mean = a.mean2; x_out->rstd = a.rstd2; x_out->gamma = mod.w + o.ln2g; x_out->beta = mod.w + o.ln2b;
  }
  *xb_out = a.out;
  return GRAM_OK;
}

// x_in: the fp32 input stream; x_in_b: its operand-typed copy.  *out / *out_b: the same pair for the output of
// layer n_full - 1.  Layers [0, n_full) run completely; when n_full < n_layers, layer n_full runs its attention
// part only (its ctx is left in s.acts[n_full].ctx) and *out / *out_b describe that layer's input.
gram_status stack_forward(Model* m, Module& mod, Stack& s, const StreamRef& x_in, const void* x_in_b, int64_t n_seq, int S,
                          cudaStream_t st, StreamRef* out, const void** out_b, int n_full = -1) {
  const int64_t T = s.packed_rows ? s.packed_rows : n_seq * S;
  if (n_full < 0) n_full = s.n_layers;
  StreamRef x = x_in;
  const void* xb = x_in_b;
  for (int l = 0; l < n_full; ++l) {
    GRAM_TRY(layer_attention_forward(m, mod, s, l, xb, n_seq, S, st));
    GRAM_TRY(layer_rest_forward(m, mod, s.off[l], s.acts[l], s.d, s.d_ff, s.attn_only, x, s.acts[l].ctx, T, st, &x, &xb));
  }
  if (n_full < s.n_layers) GRAM_TRY(layer_attention_forward(m, mod, s, n_full, xb, n_seq, S, st));
  *out = x;
  *out_b = xb;
  return GRAM_OK;
}

// ---- the same two parts, backward -----------------------------------------------------------
// Rows part.  On entry *cur holds the gradient with respect to the layer's output at T rows (for an attention-only
// layer s.dzb holds its operand-typed copy as well); s supplies the scratch (dzb, du, dctx, cpart), a the saved
// activations of those rows.  On return s.dctx holds the gradient with respect to the attention output, *oth the
// gradient that reaches the layer's input through the residual connection (fp32), and *cur is free.
gram_status layer_rest_backward(Model* m, Module& mod, const LayerOff& o, Stack& s, LayerActs& a, int64_t T, float** cur_io,
                                float** oth_io, cudaStream_t st) {
  const int d = s.d, f = s.d_ff;
  gram_ctx* ctx = m->ctx;
  float* red = m->red;
  float* cur = *cur_io;
  float* oth = *oth_io;
  GemmEpilogue e;
  if (!s.attn_only) {
    // out = LN2(z2), z2 = h1 + W2 gelu(u) + b2, u = W1 h1 + b1, h1 = LN1(z1), z1 = x + Wo ctx + bo
    GRAM_TRY(layernorm_backward(ctx, m->dtype, cur, a.z2, a.mean2, a.rstd2, mod.w + o.ln2g, oth, s.dzb, mod.g + o.ln2g,
                                mod.g + o.ln2b, mod.g + o.b2, red, T, d, st));         // oth, dzb = dz2; db2 += its column sums
    GRAM_TRY(mm_dw(m, s.dzb, a.g, mod.g + o.w2, T, d, f, st, "dw_ffn2"));
    e = GemmEpilogue();
    e.dgelu_pre = a.u;
    e.tag = "dx_ffn2_dgelu";
    const bool fused_b1 = gemm_fused_colsum(m->dtype, T, f);                           // the product's epilogue also adds up its columns
    if (fused_b1) e.colsum_part = s.cpart;
    GRAM_TRY(mm_dx(m, s.dzb, W(m, mod, o.w2), s.du, false, T, d, f, e, st));           // du = (dz2 W2) * gelu'(v), the saved u
    if (fused_b1) GRAM_TRY(colsum_from_partials(ctx, s.cpart, (T + 31) / 32, f, mod.g + o.b1, red, st));
    else GRAM_TRY(colsum_accumulate(ctx, m->dtype, s.du, T, f, mod.g + o.b1, red, st));
    GRAM_TRY(mm_dw(m, s.du, a.h1, mod.g + o.w1, T, f, d, st, "dw_ffn1"));
    e = GemmEpilogue();
    e.res = oth;
    e.tag = "dx_ffn1";
    GRAM_TRY(mm_dx(m, s.du, W(m, mod, o.w1), cur, true, T, f, d, e, st));              // cur = dh1 = du W1 + dz2
    GRAM_TRY(layernorm_backward(ctx, m->dtype, cur, a.z1, a.mean1, a.rstd1, mod.w + o.ln1g, oth, s.dzb, mod.g + o.ln1g,
                                mod.g + o.ln1b, mod.g + o.bo, red, T, d, st));         // oth, dzb = dz1; dbo += its column sums
  } else {
    float* t = cur; cur = oth; oth = t;                                                // oth = d(out), dzb its copy
    GRAM_TRY(colsum_accumulate(ctx, m->dtype, s.dzb, T, d, mod.g + o.bo, red, st));
  }
  GRAM_TRY(mm_dw(m, s.dzb, a.ctx, mod.g + o.wo, T, d, d, st, "dw_attn_out"));
  e = GemmEpilogue();
  e.tag = "dx_attn_out";
  GRAM_TRY(mm_dx(m, s.dzb, W(m, mod, o.wo), s.dctx, false, T, d, d, e, st));
  *cur_io = cur;
  *oth_io = oth;
  return GRAM_OK;
}

// Attention part over whole sequences.  s.dctx: gradient with respect to the attention output; oth: the residual
// part of the gradient with respect to the layer's input.  Writes cur = dqkv Wqkv + oth, the gradient with respect
// to the layer's input; copy_b: the layer below reads it as an operand as well (attention-only stacks).
gram_status layer_attention_backward(Model* m, Module& mod, Stack& s, int l, const void* xb_l, int64_t n_seq, int S, float* cur,
                                     const float* oth, bool copy_b, cudaStream_t st) {
  const int64_t T = s.packed_rows ? s.packed_rows : n_seq * S;
  const int d = s.d;
  gram_ctx* ctx = m->ctx;
  const LayerOff& o = s.off[l];
  LayerActs& a = s.acts[l];
  // the tensor-core kernels also add up dqkv's columns, as partial sums that fit the scratch or not at all
  int64_t part_rows = 0;
  GRAM_TRY(attention_backward(ctx, m->dtype, a.qkv, s.dctx, a.ctx, a.lse, s.delta, s.dqkv, s.cpart,
                              (int64_t)(s.cpart_elems / ((size_t)3 * d)), &part_rows, T, n_seq, S, d, s.heads, s.causal, s.seq_len,
                              s.seq_off, s.grouped ? &s.groups : nullptr, st));
  if (part_rows > 0) GRAM_TRY(colsum_from_partials(ctx, s.cpart, part_rows, 3 * d, mod.g + o.bqkv, m->red, st));
  else GRAM_TRY(colsum_accumulate(ctx, m->dtype, s.dqkv, T, 3 * d, mod.g + o.bqkv, m->red, st));
  GRAM_TRY(mm_dw(m, s.dqkv, xb_l, mod.g + o.wqkv, T, 3 * d, d, st, "dw_qkv"));
  GemmEpilogue e;
  e.res = oth;
  e.tag = "dx_qkv";
  if (copy_b) e.copy_out = s.dzb;
  return mm_dx(m, s.dqkv, W(m, mod, o.wqkv), cur, true, T, 3 * d, d, e, st);          // cur = dx = dqkv Wqkv + dz1
}

// On entry s.curf holds the gradient with respect to the stack's output (fp32; for a stack of
// attention-only layers s.dzb holds its operand-typed copy as well).  With top_attention_only the rows part of
// the top layer has been done by the caller: s.dctx and s.othf hold what layer_rest_backward leaves, and the
// top layer runs its attention part only.  On return *d_in points at the fp32 gradient with respect to the input
// stream.
gram_status stack_backward(Model* m, Module& mod, Stack& s, const void* x_in_b, int64_t n_seq, int S, cudaStream_t st,
                           float** d_in, bool top_attention_only = false) {
  const int64_t T = s.packed_rows ? s.packed_rows : n_seq * S;
  float* cur = s.curf;
  float* oth = s.othf;
  for (int l = s.n_layers - 1; l >= 0; --l) {
    const void* xb_l = (l == 0) ? x_in_b : s.acts[l - 1].out;
    if (!(top_attention_only && l == s.n_layers - 1))
      GRAM_TRY(layer_rest_backward(m, mod, s.off[l], s, s.acts[l], T, &cur, &oth, st));
    GRAM_TRY(layer_attention_backward(m, mod, s, l, xb_l, n_seq, S, cur, oth, s.attn_only && l > 0, st));
  }
  *d_in = cur;
  return GRAM_OK;
}

gram_status read_i32(Model* m, const int32_t* d_ptr, int32_t* out, cudaStream_t st);

// encoder forward over n items (d_items, or first_item.. when null): H_out [n, d] fp32
gram_status encoder_forward_chunk(Model* m, const int32_t* d_item_tokens, const int32_t* d_items, int32_t first_item,
                                  int32_t n, float* H_out, cudaStream_t st) {
  const gram_config& c = m->cfg;
  gram_ctx* ctx = m->ctx;
  if (n > m->mb) return gram_set_error(ctx, "encoder pass over %d items exceeds the micro-batch of %d", n, m->mb), GRAM_ERR_WORKSPACE;
  GRAM_TRY(refresh_bf16(m, m->ce, st));
  // texts of different lengths: rows are packed, item u owns rows seq_off[u] .. + seq_len[u] and padding has no rows
  const int32_t* seq_len = nullptr;
  const int32_t* seq_off = nullptr;
  int64_t T = (int64_t)n * c.l_t;
  if (m->item_len) {
    GRAM_TRY(sequence_layout(ctx, m->item_len, d_items, first_item, n, c.n_items, c.l_t, m->seq_len, m->seq_off,
                             m->seq_groups, m->seq_info, st));
    GRAM_CUDA(ctx, cudaMemcpyAsync(m->h_pinned + 4, m->seq_info, 5 * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    GRAM_CUDA(ctx, cudaStreamSynchronize(st));
    const int32_t rows = m->h_pinned[8];
    int32_t in_groups = 0;
    for (int gi = 0; gi < 4; ++gi) {
      m->enc.groups.count[gi] = m->h_pinned[4 + gi];
      in_groups += m->h_pinned[4 + gi];
    }
    if (rows < n || rows > T || in_groups != n)
      return gram_set_error(ctx, "encoder pass: %d token rows, %d grouped sequences for %d items", rows, in_groups, n), GRAM_ERR_ID_RANGE;
    m->enc.groups.list = m->seq_groups;
    T = rows;
    seq_len = m->seq_len;
    seq_off = m->seq_off;
  }
  m->enc.seq_len = seq_len;
  m->enc.seq_off = seq_off;
  m->enc.packed_rows = seq_off ? T : 0;
  m->enc.grouped = seq_off != nullptr;
  m->saved_rows = T;
  GRAM_TRY(embed_forward(ctx, d_item_tokens ? d_item_tokens : m->item_tokens, d_items, first_item, n, c.n_items, c.l_t,
                         c.vocab, c.d, m->ce.w + m->o_tok, m->ce.w + m->o_pos, m->z0, m->tok_ids, seq_len, seq_off, st));
  GRAM_TRY(layernorm_forward(ctx, m->dtype, m->z0, m->ce.w + m->o_elng, m->ce.w + m->o_elnb, m->x0, m->mean0, m->rstd0, T,
                             c.d, st));
  StreamRef x0;
  x0.z = m->z0; x0.mean = m->mean0; x0.rstd = m->rstd0; x0.gamma = m->ce.w + m->o_elng; x0.beta = m->ce.w + m->o_elnb;
  StreamRef out;
  const void* out_b = nullptr;
  if (!m->cls_tail) {
    GRAM_TRY(stack_forward(m, m->ce, m->enc, x0, m->x0, n, c.l_t, st, &out, &out_b));
    if (c.pooling == GRAM_POOL_ADDITIVE) {
      GemmEpilogue e;
      e.bias = m->ce.w + m->o_pba;
      GRAM_TRY(mm_fwd(m, out_b, W(m, m->ce, m->o_pwa), m->pool_pre, false, T, c.d_a, c.d, e, st));     // pre = x Wa^T + ba
      GRAM_TRY(pool_additive_forward(ctx, m->dtype, out, m->pool_pre, m->ce.w + m->o_pqa, H_out, m->pool_alpha, n, c.l_t, c.d,
                                     c.d_a, seq_len, seq_off, st));
      m->pool_x = out;
      m->pool_xb = out_b;
    } else {
      GRAM_TRY(pool_forward(ctx, out, H_out, n, c.l_t, c.d, c.pooling, seq_len, seq_off, st));
    }
  } else {
    // all layers but the last, and the last layer's attention over whole sequences
    const int last = c.n_layers - 1;
    StreamRef x;
    const void* xb = nullptr;
    GRAM_TRY(stack_forward(m, m->ce, m->enc, x0, m->x0, n, c.l_t, st, &x, &xb, last));
    // row 0 of every item: the attention output and the last layer's input stream (values and LayerNorm statistics)
    LayerActs& ta = m->tail.acts[0];
    GRAM_TRY(take_strided_rows(ctx, m->enc.acts[last].ctx, n, c.l_t, seq_off, c.d, (int)m->esz, ta.ctx, st));
    GRAM_TRY(take_strided_rows(ctx, x.z, n, c.l_t, seq_off, c.d, 4, m->tail_z, st));
    GRAM_TRY(take_strided_rows(ctx, x.mean, n, c.l_t, seq_off, 1, 4, m->tail_mean, st));
    GRAM_TRY(take_strided_rows(ctx, x.rstd, n, c.l_t, seq_off, 1, 4, m->tail_rstd, st));
    StreamRef xr = x;
    xr.z = m->tail_z; xr.mean = m->tail_mean; xr.rstd = m->tail_rstd;
    GRAM_TRY(layer_rest_forward(m, m->ce, m->tail.off[0], ta, c.d, c.d_ff, 0, xr, ta.ctx, n, st, &out, &out_b));
    GRAM_TRY(pool_forward(ctx, out, H_out, n, 1, c.d, c.pooling, nullptr, nullptr, st));       // one row per item: the pooled row itself
  }
  m->saved_n = n;
  return GRAM_OK;
}

// encoder parameter gradients += VJP of the last encoder_forward_chunk with cotangent G [n, d] (fp32)
gram_status encoder_backward_chunk(Model* m, const float* G, int32_t n, cudaStream_t st) {
  const gram_config& c = m->cfg;
  gram_ctx* ctx = m->ctx;
  if (n != m->saved_n) return gram_set_error(ctx, "encoder backward over %d items, but activations of %d are saved", n, m->saved_n), GRAM_ERR_ARG;
  const int64_t T = m->saved_rows;
  const int32_t* seq_len = m->enc.seq_len;
  const int32_t* seq_off = m->enc.seq_off;
  float* dx0 = nullptr;
  if (!m->cls_tail) {
    if (c.pooling == GRAM_POOL_ADDITIVE) {
      GRAM_TRY(pool_additive_backward(ctx, m->dtype, m->pool_x, m->pool_pre, m->ce.w + m->o_pqa, m->pool_alpha, G, m->enc.curf,
                                      m->pool_dpre, m->ce.g + m->o_pqa, m->red, n, c.l_t, c.d, c.d_a, seq_len, seq_off, st));
      GRAM_TRY(colsum_accumulate(ctx, m->dtype, m->pool_dpre, T, c.d_a, m->ce.g + m->o_pba, m->red, st));
      GRAM_TRY(mm_dw(m, m->pool_dpre, m->pool_xb, m->ce.g + m->o_pwa, T, c.d_a, c.d, st));
      GemmEpilogue e;
      e.accumulate = 1;                  // the stream gradient already holds alpha_s G
      GRAM_TRY(mm_dx(m, m->pool_dpre, W(m, m->ce, m->o_pwa), m->enc.curf, true, T, c.d_a, c.d, e, st));
    } else {
      GRAM_TRY(pool_backward(ctx, G, m->enc.curf, n, c.l_t, c.d, c.pooling, seq_len, seq_off, st));
    }
    GRAM_TRY(stack_backward(m, m->ce, m->enc, m->x0, n, c.l_t, st, &dx0));
  } else {
    // the row-wise part of the last layer on one row per item
    Stack& tl = m->tail;
    GRAM_TRY(pool_backward(ctx, G, tl.curf, n, 1, c.d, c.pooling, nullptr, nullptr, st));
    float* cur = tl.curf;
    float* oth = tl.othf;
    GRAM_TRY(layer_rest_backward(m, m->ce, tl.off[0], tl, tl.acts[0], n, &cur, &oth, st));
    // back into whole sequences: every other row of the two gradients is zero
    GRAM_CUDA(ctx, cudaMemsetAsync(m->enc.dctx, 0, (size_t)T * c.d * m->esz, st));
    GRAM_CUDA(ctx, cudaMemsetAsync(m->enc.othf, 0, (size_t)T * c.d * 4, st));
    GRAM_TRY(put_strided_rows(ctx, tl.dctx, n, c.l_t, seq_off, c.d, (int)m->esz, m->enc.dctx, st));
    GRAM_TRY(put_strided_rows(ctx, oth, n, c.l_t, seq_off, c.d, 4, m->enc.othf, st));
    GRAM_TRY(stack_backward(m, m->ce, m->enc, m->x0, n, c.l_t, st, &dx0, true));
  }
  float* dz0 = (dx0 == m->enc.curf) ? m->enc.othf : m->enc.curf;
  GRAM_TRY(layernorm_backward(ctx, m->dtype, dx0, m->z0, m->mean0, m->rstd0, m->ce.w + m->o_elng, dz0, nullptr,
                              m->ce.g + m->o_elng, m->ce.g + m->o_elnb, nullptr, m->red, T, c.d, st));
  GRAM_TRY(periodic_rowsum_accumulate(ctx, dz0, n, c.l_t, c.d, m->ce.g + m->o_pos, m->red, seq_len, seq_off, st));
  // token-embedding gradient: sum dz0 over the occurrences of each token (same index kernels as stage 1 / 4)
  IndexWorkspace* iws = gram_index_ws(ctx);
  GRAM_TRY(dedup_launch(ctx, iws, m->tok_ids, T, c.vocab, m->tok_unique, m->tok_inverse, m->tok_perm, m->tok_seg, m->tok_nu, st));
  GRAM_TRY(accumulate_launch(ctx, iws, dz0, 0, m->tok_perm, m->tok_seg, T, 0, m->tok_nu, c.d, m->tok_unique, 1,
                             m->ce.g + m->o_tok, st));
  return GRAM_OK;
}

// Where the task module finds the encoding of position p: row p of `rows` (index == null, rows is fp32 [B*L, d]), or
// row index[p] of `rows` (n_rows rows of fp32, or of bf16 when rows_bf16: the Multi-step cache), i.e. stage 3 left to
// the task module's first load.
struct EncodingSource {
  const void* rows = nullptr;
  int rows_bf16 = 0;
  const int32_t* index = nullptr;
  int64_t n_rows = 0;
};

// Task module forward and backward.  dE (may be null for the KT task): receives dL/dE, fp32 [B*L, d].  *dE_at is set to
// where dL/dE can be read after the call: dE when given, else the task module's own input-gradient buffer (the KT input
// is a sum, so its gradient is the gradient of the encodings, row for row).
gram_status task_forward_backward(Model* m, const EncodingSource& src, const int32_t* labels, int32_t B, float* dE, float* loss,
                                  const float** dE_at, cudaStream_t st) {
  const gram_config& c = m->cfg;
  gram_ctx* ctx = m->ctx;
  const int64_t P = (int64_t)B * c.L;
  GRAM_TRY(refresh_bf16(m, m->task, st));
  GRAM_CUDA(ctx, cudaMemsetAsync(m->task.g, 0, m->task.n * 4, st));
  if (dE_at) *dE_at = dE;
  if (c.task == GRAM_TASK_KT) {
    GRAM_TRY(kt_input_forward(ctx, m->dtype, src.rows, src.rows_bf16, src.index, src.n_rows, m->task.w + m->t_pos,
                              m->task.w + m->t_resp, labels, m->tx, m->txb, B, c.L, c.d, st));
    StreamRef x;
    x.z = m->tx;
    StreamRef y;
    const void* y_b = nullptr;
    GRAM_TRY(stack_forward(m, m->task, m->tk, x, m->txb, B, c.L, st, &y, &y_b));
    void* dy_b = (m->tk.attn_only && m->tk.n_layers > 0) ? m->tk.dzb : nullptr;
    GRAM_TRY(kt_head(ctx, m->dtype, y, m->task.w + m->t_headw, m->task.w + m->t_headb, labels, m->tk.curf, dy_b,
                     m->task.g + m->t_headw, m->task.g + m->t_headb, loss, m->red, m->n_real, P, c.d, st));
    float* dx = nullptr;
    GRAM_TRY(stack_backward(m, m->task, m->tk, m->txb, B, c.L, st, &dx));
    GRAM_TRY(kt_input_backward(ctx, dx, labels, dE, m->task.g + m->t_pos, m->task.g + m->t_resp, m->red, B, c.L, c.d, st));
    if (!dE && dE_at) *dE_at = dx;
    return GRAM_OK;
  }
  if (c.task == GRAM_TASK_NR) {
    if (src.index || src.rows_bf16 || !dE) return gram_set_error(ctx, "the news task reads materialised fp32 encodings"), GRAM_ERR_ARG;
    const float* E = (const float*)src.rows;
    const float* E_in = E;
    float* dE_out = dE;
    const int n_hist = c.L - c.n_cand;
    const int64_t Th = (int64_t)B * n_hist;
    if (c.task_layers > 0) {
      // the clicked items of every user pass through the self-attention layers as one packed sequence per user; the rows
      // after the last clicked item are zero rows that no sequence owns, so the layers run on B * n_hist rows whatever
      // the number of clicks, and nothing has to be read back
      GRAM_TRY(nr_layout(ctx, labels, B, c.L, n_hist, m->nr_len, m->nr_off, m->nr_rows, m->nr_pos2row, st));
      GRAM_TRY(nr_pack(ctx, m->dtype, E_in, m->nr_rows, Th, c.d, m->tx, m->txb, st));
      m->tk.seq_len = m->nr_len; m->tk.seq_off = m->nr_off; m->tk.packed_rows = Th; m->tk.grouped = false;
      StreamRef x;
      x.z = m->tx;
      StreamRef y;
      const void* y_b = nullptr;
      GRAM_TRY(stack_forward(m, m->task, m->tk, x, m->txb, B, n_hist, st, &y, &y_b));
      GRAM_TRY(nr_select(ctx, y, m->nr_pos2row, E_in, P, c.d, m->nr_E2, st));
      E = m->nr_E2;
      dE = m->nr_dE2;
    }
    const void* Eb = E;                  // fp32 contexts: the stream is its own operand
    if (m->dtype == GRAM_BF16) {
      GRAM_TRY(convert_f32_to_bf16(ctx, E, (bf16*)m->Eb, (size_t)P * c.d, st));
      Eb = m->Eb;
    }
    GemmEpilogue e;
    e.bias = m->task.w + m->t_ba;
    GRAM_TRY(mm_fwd(m, Eb, W(m, m->task, m->t_wa), m->pre, false, P, c.d_a, c.d, e, st));
    GRAM_TRY(nr_user(ctx, m->dtype, E, m->pre, m->task.w + m->t_qa, dE, m->dpre, m->task.g + m->t_qa, loss, m->red, labels, B, c.L,
                     c.n_cand, c.d, c.d_a, st));
    GRAM_TRY(colsum_accumulate(ctx, m->dtype, m->dpre, P, c.d_a, m->task.g + m->t_ba, m->red, st));
    GRAM_TRY(mm_dw(m, m->dpre, Eb, m->task.g + m->t_wa, P, c.d_a, c.d, st));
    e = GemmEpilogue();
    e.accumulate = 1;                    // dE already holds the direct part
    GRAM_TRY(mm_dx(m, m->dpre, W(m, m->task, m->t_wa), dE, true, P, c.d_a, c.d, e, st));
    if (c.task_layers > 0) {
      // back through the layers: the gradient rows of the clicked items, packed; then every position takes the layers'
      // input gradient where it has a packed row and the direct gradient (candidates; zeros at empty slots) elsewhere
      void* dy_b = m->tk.attn_only ? m->tk.dzb : nullptr;
      GRAM_TRY(nr_pack(ctx, m->dtype, dE, m->nr_rows, Th, c.d, m->tk.curf, dy_b, st));
      float* dx = nullptr;
      GRAM_TRY(stack_backward(m, m->task, m->tk, m->txb, B, n_hist, st, &dx));
      StreamRef dxr;
      dxr.z = dx;
      GRAM_TRY(nr_select(ctx, dxr, m->nr_pos2row, dE, P, c.d, dE_out, st));
    }
    return GRAM_OK;
  }
  return gram_set_error(ctx, "the context has no task module"), GRAM_ERR_ARG;
}

gram_status read_i32(Model* m, const int32_t* d_ptr, int32_t* out, cudaStream_t st) {
  GRAM_CUDA(m->ctx, cudaMemcpyAsync(m->h_pinned, d_ptr, 4, cudaMemcpyDeviceToHost, st));
  GRAM_CUDA(m->ctx, cudaStreamSynchronize(st));
  *out = m->h_pinned[0];
  return GRAM_OK;
}

// the configured update of one module from its gradients: lr is the SGD step or Adam's peak rate
// gated: the kernel leaves the parameters alone when the context's status word holds an error (the caller then takes
// the update count back)
gram_status apply_sgd(Model* m, Module& mod, float lr, cudaStream_t st, bool gated = false) {
  if (lr == 0.f || mod.n == 0) return GRAM_OK;
  const int32_t* gate = gated ? gram_status_word(m->ctx) : nullptr;
  const gram_config& c = m->cfg;
  ++mod.updates;
  if (c.optimizer == GRAM_OPT_ADAM) {
    const float b1 = c.adam_beta1 > 0.f ? c.adam_beta1 : 0.9f, b2 = c.adam_beta2 > 0.f ? c.adam_beta2 : 0.999f;
    const float eps = c.adam_eps > 0.f ? c.adam_eps : 1e-8f;
    const float rate = (float)noam_rate(mod.updates, lr, c.noam_warmup);
    GRAM_TRY(adam_update(m->ctx, mod.w, mod.g, mod.am, mod.av, m->dtype == GRAM_BF16 ? mod.wb : nullptr, mod.n, mod.updates, rate,
                         b1, b2, eps, st, gate));
    mod.wb_stale = false;                       // the kernel wrote the bf16 copy as well
    return GRAM_OK;
  }
  GRAM_TRY(sgd_update(m->ctx, mod.w, mod.g, lr, mod.n, st, gate));
  mod.wb_stale = true;
  return GRAM_OK;
}

// encoder forward + backward over `n_total` items listed in d_items, in micro-batches; G_of(u0, n)
// must leave the cotangent rows of items [u0, u0+n) in m->G
template <typename GFn>
gram_status encoder_pass(Model* m, const int32_t* d_items, int32_t n_total, bool update_cache, GFn G_of, cudaStream_t st) {
  for (int32_t u0 = 0; u0 < n_total; u0 += m->mb) {
    const int32_t n = (n_total - u0 < m->mb) ? n_total - u0 : m->mb;
    GRAM_TRY(encoder_forward_chunk(m, nullptr, d_items + u0, 0, n, m->H, st));
    const float* G = nullptr;
    GRAM_TRY(G_of(u0, n, &G));                 // may read the cache rows of these items: before they are replaced
    if (update_cache) GRAM_TRY(scatter_rows(m->ctx, m->cache_dtype, m->H, d_items + u0, n, m->cfg.d, m->cfg.n_items, m->cache, st));
    GRAM_TRY(encoder_backward_chunk(m, G, n, st));
  }
  return GRAM_OK;
}

}  // namespace

gram_status model_optimizer_step(Model* m, int module, cudaStream_t st) {
  Module* mod = module == GRAM_MODULE_CE ? &m->ce : module == GRAM_MODULE_TASK ? &m->task : nullptr;
  if (!mod) return gram_set_error(m->ctx, "unknown module %d", module), GRAM_ERR_ARG;
  return apply_sgd(m, *mod, module == GRAM_MODULE_CE ? m->cfg.lr_ce : m->cfg.lr_task, st);
}

gram_status model_optimizer_reset(Model* m, cudaStream_t st) {
  for (Module* mod : {&m->ce, &m->task}) {
    mod->updates = 0;
    if (mod->am && mod->n) {
      GRAM_CUDA(m->ctx, cudaMemsetAsync(mod->am, 0, mod->n * 4, st));
      GRAM_CUDA(m->ctx, cudaMemsetAsync(mod->av, 0, mod->n * 4, st));
    }
  }
  return GRAM_OK;
}


// ===========================================================================================
gram_status model_create(gram_ctx* ctx, const gram_config* cfg, Model** out) {
  *out = nullptr;
  Model* m = new (std::nothrow) Model();
  if (!m) return GRAM_ERR_CUDA;
  *out = m;                             // destroyed by the caller on failure
  m->ctx = ctx;
  m->cfg = *cfg;
  const gram_config& c = m->cfg;
  m->dtype = c.dtype;
  if (c.dtype != GRAM_F32 && c.dtype != GRAM_BF16) return gram_set_error(ctx, "unknown dtype %d", c.dtype), GRAM_ERR_ARG;
  m->esz = c.dtype == GRAM_BF16 ? 2 : 4;
  if (c.d <= 0 || (c.d & 1)) return gram_set_error(ctx, "d must be positive and even"), GRAM_ERR_ARG;
  if (c.dtype == GRAM_BF16 && (c.d % 8 || c.d_ff % 8 || c.task_d_ff % 8 || c.d_a % 8))
    return gram_set_error(ctx, "bf16 contexts need widths that are multiples of 8"), GRAM_ERR_UNSUPPORTED;
  if (c.B_max <= 0 || c.L <= 0) return gram_set_error(ctx, "B_max and L must be positive"), GRAM_ERR_ARG;
  if (c.optimizer != GRAM_OPT_SGD && c.optimizer != GRAM_OPT_ADAM) return gram_set_error(ctx, "unknown optimizer %d", c.optimizer), GRAM_ERR_ARG;
  if (c.adam_beta1 >= 1.f || c.adam_beta2 >= 1.f) return gram_set_error(ctx, "Adam: beta1 and beta2 must be below 1"), GRAM_ERR_ARG;
  if (c.multistep_variant != GRAM_MULTI_TABLE && c.multistep_variant != GRAM_MULTI_PSEUDO_TARGET)
    return gram_set_error(ctx, "unknown multistep_variant %d", c.multistep_variant), GRAM_ERR_ARG;
  if (c.defer_update && c.refresh_after_update)
    return gram_set_error(ctx, "defer_update cannot be combined with refresh_after_update"), GRAM_ERR_UNSUPPORTED;
  m->pseudo = c.K > 1 && c.multistep_variant == GRAM_MULTI_PSEUDO_TARGET;
  m->cache_dtype = m->pseudo ? GRAM_F32 : c.dtype;
  // ---- parameter layouts (the order include/gram.h documents) ----
  size_t at = 0;
  if (c.n_layers > 0) {
    if (c.n_heads <= 0 || c.d % c.n_heads || c.l_t <= 0 || c.vocab <= 0 || c.d_ff <= 0)
      return gram_set_error(ctx, "bad encoder shape"), GRAM_ERR_ARG;
    m->o_tok = at; at += (size_t)c.vocab * c.d;
    m->o_pos = at; at += (size_t)c.l_t * c.d;
    m->o_elng = at; at += c.d;
    m->o_elnb = at; at += c.d;
    m->enc.d = c.d; m->enc.heads = c.n_heads; m->enc.d_ff = c.d_ff; m->enc.n_layers = c.n_layers;
    m->enc.attn_only = 0; m->enc.causal = 0;
    m->enc.off.resize(c.n_layers);
    for (int l = 0; l < c.n_layers; ++l) at = layer_layout(&m->enc.off[l], at, c.d, c.d_ff, 0);
    if (c.pooling == GRAM_POOL_ADDITIVE) {
      if (c.d_a <= 0) return gram_set_error(ctx, "additive pooling needs d_a > 0"), GRAM_ERR_ARG;
      m->o_pwa = at; at += (size_t)c.d_a * c.d;
      m->o_pba = at; at += c.d_a;
      m->o_pqa = at; at += c.d_a;
    } else if (c.pooling != GRAM_POOL_MEAN && c.pooling != GRAM_POOL_CLS) {
      return gram_set_error(ctx, "unknown pooling %d", c.pooling), GRAM_ERR_ARG;
    }
  }
  GRAM_TRY(module_alloc(ctx, &m->ce, at, c.dtype == GRAM_BF16, c.optimizer == GRAM_OPT_ADAM));
  at = 0;
  if (c.task == GRAM_TASK_KT) {
    if (c.task_layers > 0 && (c.task_heads <= 0 || c.d % c.task_heads)) return gram_set_error(ctx, "bad task shape"), GRAM_ERR_ARG;
    m->t_pos = at; at += (size_t)c.L * c.d;
    m->t_resp = at; at += (size_t)3 * c.d;
    m->tk.d = c.d; m->tk.heads = c.task_heads; m->tk.d_ff = c.task_d_ff; m->tk.n_layers = c.task_layers;
    m->tk.attn_only = c.task_attn_only ? 1 : 0; m->tk.causal = 1;
    m->tk.off.resize(c.task_layers);
    for (int l = 0; l < c.task_layers; ++l) at = layer_layout(&m->tk.off[l], at, c.d, c.task_d_ff, m->tk.attn_only);
    m->t_headw = at; at += c.d;
    m->t_headb = at; at += 1;
  } else if (c.task == GRAM_TASK_NR) {
    if (c.d_a <= 0 || c.n_cand <= 0 || c.n_cand >= c.L) return gram_set_error(ctx, "bad task shape"), GRAM_ERR_ARG;
    if (c.task_layers > 0) {             // self-attention layers over the clicked items, ahead of the additive attention
      if (c.task_heads <= 0 || c.d % c.task_heads) return gram_set_error(ctx, "bad task shape"), GRAM_ERR_ARG;
      m->tk.d = c.d; m->tk.heads = c.task_heads; m->tk.d_ff = c.task_d_ff; m->tk.n_layers = c.task_layers;
      m->tk.attn_only = c.task_attn_only ? 1 : 0; m->tk.causal = 0;
      m->tk.off.resize(c.task_layers);
      for (int l = 0; l < c.task_layers; ++l) at = layer_layout(&m->tk.off[l], at, c.d, c.task_d_ff, m->tk.attn_only);
    }
    m->t_wa = at; at += (size_t)c.d_a * c.d;
    m->t_ba = at; at += c.d_a;
    m->t_qa = at; at += c.d_a;
  }
  GRAM_TRY(module_alloc(ctx, &m->task, at, c.dtype == GRAM_BF16, c.optimizer == GRAM_OPT_ADAM));
  // ---- sizes ----
  const int64_t P = (int64_t)c.B_max * c.L;
  m->u_cap = (int32_t)(P < c.n_items ? P : c.n_items);
  int64_t mb = c.ce_micro_batch > 0 ? c.ce_micro_batch : (c.K > 1 ? c.n_items : m->u_cap);
  if (mb > c.n_items) mb = c.n_items;
  m->mb = (int32_t)mb;
  m->enc.cap = (int64_t)m->mb * c.l_t;
  m->tk.cap = c.task == GRAM_TASK_NR ? (int64_t)c.B_max * (c.L - c.n_cand) : P;
  m->cls_tail = c.n_layers > 0 && c.pooling == GRAM_POOL_CLS && c.l_t > 1;
  if (m->cls_tail) {
    m->tail.d = c.d; m->tail.heads = c.n_heads; m->tail.d_ff = c.d_ff; m->tail.n_layers = 1;
    m->tail.attn_only = 0; m->tail.causal = 0;
    m->tail.cap = m->mb;
    m->tail.off.assign(1, m->enc.off.back());
  }
  Arena dry;
  layout_buffers(m, dry);
  m->arena_bytes = dry.off + 256;
  GRAM_CUDA(ctx, cudaMalloc(&m->arena, m->arena_bytes));
  GRAM_CUDA(ctx, cudaMemset(m->arena, 0, m->arena_bytes));
  Arena real;
  real.base = m->arena;
  layout_buffers(m, real);
  for (int i = 0; i < 8; ++i) GRAM_CUDA(ctx, cudaEventCreate(&m->ev[i]));
  GRAM_CUDA(ctx, cudaMallocHost(&m->h_pinned, 16 * sizeof(int32_t)));
  return GRAM_OK;
}

void model_destroy(Model* m) {
  if (!m) return;
  cudaFree(m->ce.w); cudaFree(m->ce.g); cudaFree(m->ce.wb); cudaFree(m->ce.am); cudaFree(m->ce.av);
  cudaFree(m->task.w); cudaFree(m->task.g); cudaFree(m->task.wb); cudaFree(m->task.am); cudaFree(m->task.av);
  cudaFree(m->arena);
  for (int i = 0; i < 8; ++i) if (m->ev[i]) cudaEventDestroy(m->ev[i]);
  if (m->h_pinned) cudaFreeHost(m->h_pinned);
  delete m;
}

static Module* pick(Model* m, int module) {
  return module == GRAM_MODULE_CE ? &m->ce : (module == GRAM_MODULE_TASK ? &m->task : nullptr);
}

gram_status model_param_count(const Model* m, int module, size_t* n) {
  const Module* mod = pick(const_cast<Model*>(m), module);
  if (!mod) return GRAM_ERR_ARG;
  *n = mod->n;
  return GRAM_OK;
}

gram_status model_set_params(Model* m, int module, const float* h, size_t n) {
  Module* mod = pick(m, module);
  if (!mod || !h || n != mod->n) return gram_set_error(m->ctx, "gram_set_params: module or count mismatch (%zu given)", n), GRAM_ERR_ARG;
  GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
  GRAM_CUDA(m->ctx, cudaMemcpy(mod->w, h, n * 4, cudaMemcpyHostToDevice));
  mod->wb_stale = true;
  m->saved_n = -1;
  return GRAM_OK;
}

gram_status model_get_params(Model* m, int module, float* h, size_t n, int grads) {
  Module* mod = pick(m, module);
  if (!mod || !h || n != mod->n) return gram_set_error(m->ctx, "gram_get_params/grads: module or count mismatch"), GRAM_ERR_ARG;
  GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
  GRAM_CUDA(m->ctx, cudaMemcpy(h, grads ? mod->g : mod->w, n * 4, cudaMemcpyDeviceToHost));
  return GRAM_OK;
}

gram_status model_zero_grads(Model* m, int module, cudaStream_t st) {
  Module* mod = pick(m, module);
  if (!mod) return GRAM_ERR_ARG;
  if (mod->n) GRAM_CUDA(m->ctx, cudaMemsetAsync(mod->g, 0, mod->n * 4, st));
  return GRAM_OK;
}

gram_status model_grads_device(Model* m, int module, float** d_grads, size_t* n) {
  Module* mod = pick(m, module);
  if (!mod) return gram_set_error(m->ctx, "unknown module %d", module), GRAM_ERR_ARG;
  *d_grads = mod->g;
  *n = mod->n;
  return GRAM_OK;
}

gram_status model_set_item_tokens(Model* m, const int32_t* h_tokens) {
  if (!h_tokens || !m->item_tokens) return gram_set_error(m->ctx, "gram_set_item_tokens: no encoder or null tokens"), GRAM_ERR_ARG;
  GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
  GRAM_CUDA(m->ctx, cudaMemcpy(m->item_tokens, h_tokens, (size_t)m->cfg.n_items * m->cfg.l_t * 4, cudaMemcpyHostToDevice));
  return GRAM_OK;
}

gram_status model_set_item_lengths(Model* m, const int32_t* h_len) {
  if (!m->item_len_buf) return gram_set_error(m->ctx, "gram_set_item_lengths: the context has no encoder"), GRAM_ERR_ARG;
  GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
  m->saved_n = -1;
  if (!h_len) {                         // back to texts of exactly l_t tokens
    m->item_len = nullptr;
    return GRAM_OK;
  }
  for (int32_t i = 0; i < m->cfg.n_items; ++i)
    if (h_len[i] < 1 || h_len[i] > m->cfg.l_t)
      return gram_set_error(m->ctx, "gram_set_item_lengths: item %d has length %d outside 1..%d", i, h_len[i], m->cfg.l_t), GRAM_ERR_ARG;
  GRAM_CUDA(m->ctx, cudaMemcpy(m->item_len_buf, h_len, (size_t)m->cfg.n_items * 4, cudaMemcpyHostToDevice));
  m->item_len = m->item_len_buf;
  return GRAM_OK;
}

gram_status model_encode(Model* m, const int32_t* d_item_tokens, const int32_t* d_items, int32_t U, float* d_H, int save,
                         cudaStream_t st) {
  if (m->cfg.n_layers <= 0) return gram_set_error(m->ctx, "the context has no encoder"), GRAM_ERR_ARG;
  if (U < 0 || (U > 0 && (!d_items || !d_H))) return gram_set_error(m->ctx, "gram_encode_unique: bad argument"), GRAM_ERR_ARG;
  if (save && U > m->mb)
    return gram_set_error(m->ctx, "gram_encode_unique: %d items do not fit the micro-batch of %d when activations are kept", U, m->mb), GRAM_ERR_WORKSPACE;
  for (int32_t u0 = 0; u0 < U; u0 += m->mb) {
    const int32_t n = (U - u0 < m->mb) ? U - u0 : m->mb;
    GRAM_TRY(encoder_forward_chunk(m, d_item_tokens, d_items + u0, 0, n, d_H + (size_t)u0 * m->cfg.d, st));
  }
  if (!save || U == 0) m->saved_n = save ? 0 : -1;
  return GRAM_OK;
}

gram_status model_task(Model* m, const float* d_E, const int32_t* d_labels, int32_t B, float* d_dE, float* d_loss,
                       cudaStream_t st) {
  if (B < 0 || B > m->cfg.B_max) return gram_set_error(m->ctx, "gram_task: B=%d exceeds B_max=%d", B, m->cfg.B_max), GRAM_ERR_WORKSPACE;
  if (B == 0) return GRAM_OK;
  if (!d_E || !d_labels || !d_dE || !d_loss) return gram_set_error(m->ctx, "gram_task: null buffer"), GRAM_ERR_ARG;
  EncodingSource src;
  src.rows = d_E;
  return task_forward_backward(m, src, d_labels, B, d_dE, d_loss, nullptr, st);
}

gram_status model_encoder_backward(Model* m, const float* d_G, const int32_t* d_items, int32_t U, cudaStream_t st) {
  (void)d_items;
  if (m->cfg.n_layers <= 0) return gram_set_error(m->ctx, "the context has no encoder"), GRAM_ERR_ARG;
  if (U == 0) return GRAM_OK;
  if (!d_G) return gram_set_error(m->ctx, "gram_encoder_backward: null buffer"), GRAM_ERR_ARG;
  return encoder_backward_chunk(m, d_G, U, st);
}

float* model_table(Model* m) { return m->table; }
uint32_t* model_touched(Model* m) { return m->touched; }

gram_status model_window_reset(Model* m, cudaStream_t st) {
  if (!m->table) return gram_set_error(m->ctx, "the context was created with K <= 1"), GRAM_ERR_ARG;
  GRAM_CUDA(m->ctx, cudaMemsetAsync(m->table, 0, (size_t)m->cfg.n_items * m->cfg.d * 4, st));
  GRAM_CUDA(m->ctx, cudaMemsetAsync(m->touched, 0, (size_t)((m->cfg.n_items + 31) / 32) * 4, st));
  GRAM_CUDA(m->ctx, cudaMemsetAsync(m->tcount, 0, sizeof(int32_t), st));
  m->step_in_window = 0;
  return GRAM_OK;
}

gram_status model_cache_fill(Model* m, cudaStream_t st) {
  if (!m->cache) return gram_set_error(m->ctx, "the context was created with K <= 1"), GRAM_ERR_ARG;
  const gram_config& c = m->cfg;
  for (int32_t u0 = 0; u0 < c.n_items; u0 += m->mb) {
    const int32_t n = (c.n_items - u0 < m->mb) ? c.n_items - u0 : m->mb;
    GRAM_TRY(encoder_forward_chunk(m, nullptr, nullptr, u0, n, m->H, st));
    if (m->cache_dtype == GRAM_BF16) GRAM_TRY(convert_f32_to_bf16(m->ctx, m->H, (bf16*)m->cache + (size_t)u0 * c.d, (size_t)n * c.d, st));
    else GRAM_CUDA(m->ctx, cudaMemcpyAsync((float*)m->cache + (size_t)u0 * c.d, m->H, (size_t)n * c.d * 4, cudaMemcpyDeviceToDevice, st));
  }
  m->saved_n = -1;
  return GRAM_OK;
}

gram_status model_get_window(Model* m, float* h_table, uint32_t* h_touched, float* h_cache) {
  if (!m->table) return gram_set_error(m->ctx, "the context was created with K <= 1"), GRAM_ERR_ARG;
  const gram_config& c = m->cfg;
  GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
  if (h_table) GRAM_CUDA(m->ctx, cudaMemcpy(h_table, m->table, (size_t)c.n_items * c.d * 4, cudaMemcpyDeviceToHost));
  if (h_touched) GRAM_CUDA(m->ctx, cudaMemcpy(h_touched, m->touched, (size_t)((c.n_items + 31) / 32) * 4, cudaMemcpyDeviceToHost));
  if (h_cache) {
    // converted to fp32 on the device through the per-position gradient buffer, a batch's worth of rows at a time
    const size_t rows_per = (size_t)((int64_t)c.B_max * c.L);
    for (size_t r0 = 0; r0 < (size_t)c.n_items; r0 += rows_per) {
      const size_t nr = ((size_t)c.n_items - r0 < rows_per) ? (size_t)c.n_items - r0 : rows_per;
      GRAM_TRY(convert_to_f32(m->ctx, m->cache_dtype, (char*)m->cache + r0 * c.d * (m->cache_dtype == GRAM_BF16 ? 2 : 4), m->dE, nr * c.d, 0));
      GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
      GRAM_CUDA(m->ctx, cudaMemcpy(h_cache + r0 * c.d, m->dE, nr * c.d * 4, cudaMemcpyDeviceToHost));
    }
  }
  return GRAM_OK;
}

gram_status model_state_export(Model* m, float* h_table, uint32_t* h_touched, float* h_cache, int32_t* steps) {
  GRAM_TRY(model_get_window(m, h_table, h_touched, h_cache));
  if (steps) *steps = m->step_in_window;
  return GRAM_OK;
}

gram_status model_state_import(Model* m, const float* h_table, const uint32_t* h_touched, const float* h_cache, int32_t steps) {
  if (!m->table) return gram_set_error(m->ctx, "the context was created with K <= 1"), GRAM_ERR_ARG;
  const gram_config& c = m->cfg;
  if (steps < 0 || steps >= c.K) return gram_set_error(m->ctx, "gram_state_import: %d steps in a window of %d", steps, c.K), GRAM_ERR_ARG;
  GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
  if (h_table) GRAM_CUDA(m->ctx, cudaMemcpy(m->table, h_table, (size_t)c.n_items * c.d * 4, cudaMemcpyHostToDevice));
  if (h_touched) {
    GRAM_CUDA(m->ctx, cudaMemcpy(m->touched, h_touched, (size_t)((c.n_items + 31) / 32) * 4, cudaMemcpyHostToDevice));
    GRAM_TRY(touched_list_launch(m->ctx, m->touched, c.n_items, m->tlist, m->tcount, 0));     // recount the set bits
    GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
  }
  if (h_cache) {
    if (m->cache_dtype == GRAM_F32) {
      GRAM_CUDA(m->ctx, cudaMemcpy(m->cache, h_cache, (size_t)c.n_items * c.d * 4, cudaMemcpyHostToDevice));
    } else {      // through the fp32 gradient buffer, a batch's worth of rows at a time
      const size_t rows_per = (size_t)((int64_t)c.B_max * c.L);
      for (size_t r0 = 0; r0 < (size_t)c.n_items; r0 += rows_per) {
        const size_t nr = ((size_t)c.n_items - r0 < rows_per) ? (size_t)c.n_items - r0 : rows_per;
        GRAM_CUDA(m->ctx, cudaMemcpy(m->dE, h_cache + r0 * c.d, nr * c.d * 4, cudaMemcpyHostToDevice));
        GRAM_TRY(convert_f32_to_bf16(m->ctx, m->dE, (bf16*)m->cache + r0 * c.d, nr * c.d, 0));
        GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
      }
    }
  }
  m->step_in_window = steps;
  return GRAM_OK;
}

gram_status model_optimizer_export(Model* m, int module, float* h_m, float* h_v, int64_t* updates) {
  Module* mod = module == GRAM_MODULE_CE ? &m->ce : module == GRAM_MODULE_TASK ? &m->task : nullptr;
  if (!mod) return gram_set_error(m->ctx, "unknown module %d", module), GRAM_ERR_ARG;
  GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
  if (updates) *updates = mod->updates;
  if (mod->am && mod->n) {
    if (!h_m || !h_v) return gram_set_error(m->ctx, "gram_optimizer_export: Adam state needs both moment buffers"), GRAM_ERR_ARG;
    GRAM_CUDA(m->ctx, cudaMemcpy(h_m, mod->am, mod->n * 4, cudaMemcpyDeviceToHost));
    GRAM_CUDA(m->ctx, cudaMemcpy(h_v, mod->av, mod->n * 4, cudaMemcpyDeviceToHost));
  }
  return GRAM_OK;
}

gram_status model_optimizer_import(Model* m, int module, const float* h_m, const float* h_v, int64_t updates) {
  Module* mod = module == GRAM_MODULE_CE ? &m->ce : module == GRAM_MODULE_TASK ? &m->task : nullptr;
  if (!mod || updates < 0) return gram_set_error(m->ctx, "gram_optimizer_import: bad module or update count"), GRAM_ERR_ARG;
  GRAM_CUDA(m->ctx, cudaDeviceSynchronize());
  if (mod->am && mod->n) {
    if (!h_m || !h_v) return gram_set_error(m->ctx, "gram_optimizer_import: Adam state needs both moment buffers"), GRAM_ERR_ARG;
    GRAM_CUDA(m->ctx, cudaMemcpy(mod->am, h_m, mod->n * 4, cudaMemcpyHostToDevice));
    GRAM_CUDA(m->ctx, cudaMemcpy(mod->av, h_v, mod->n * 4, cudaMemcpyHostToDevice));
  }
  mod->updates = updates;
  return GRAM_OK;
}

// reads a few device words with one wait: out[k] = *d_ptr[k]
static gram_status read_words(Model* m, const int32_t* const* d_ptr, int n, int32_t* out, cudaStream_t st) {
  for (int k = 0; k < n; ++k)
    GRAM_CUDA(m->ctx, cudaMemcpyAsync(m->h_pinned + k, d_ptr[k], 4, cudaMemcpyDeviceToHost, st));
  GRAM_CUDA(m->ctx, cudaStreamSynchronize(st));
  for (int k = 0; k < n; ++k) out[k] = m->h_pinned[k];
  return GRAM_OK;
}

// an error word read back from the device: clears it and names it
static gram_status device_error(Model* m, int32_t code, cudaStream_t st) {
  GRAM_CUDA(m->ctx, cudaMemsetAsync(gram_status_word(m->ctx), 0, sizeof(int32_t), st));
  GRAM_CUDA(m->ctx, cudaStreamSynchronize(st));
  gram_set_error(m->ctx, code == GRAM_ERR_ID_RANGE ? "gram_step: an ID outside its range was met on the device; the step changed no state"
                                                   : (code == GRAM_ERR_TIMEOUT ? "gram_step: a bounded device-side wait ran out" : "gram_step: device-side error"));
  return (gram_status)code;
}

// Host synchronisation points: Single-step waits once after the dedup (it needs U to size the encoder pass, and reads the
// status word in the same wait, so a batch with an ID out of range is rejected before anything else runs) and once at the
// end.  A Multi-step step without encoder pass waits once, at the end: U stays on the device, and every kernel that
// changes state that outlives the step (table, touched bits, task parameters) is gated on the status word, so a rejected
// batch still changes nothing.  The K-th step of a window waits once more to read the number of touched items.
gram_status model_step(Model* m, const int32_t* ids_in, const int32_t* labels_in, int32_t B, int on_host,
                       gram_step_report* rep, cudaStream_t st) {
  const gram_config& c = m->cfg;
  gram_ctx* ctx = m->ctx;
  if (c.n_layers <= 0 || c.task == GRAM_TASK_NONE) return gram_set_error(ctx, "gram_step needs both modules"), GRAM_ERR_ARG;
  if (B <= 0 || B > c.B_max) return gram_set_error(ctx, "gram_step: B=%d outside 1..B_max=%d", B, c.B_max), GRAM_ERR_WORKSPACE;
  if (!ids_in || !labels_in) return gram_set_error(ctx, "gram_step: null buffer"), GRAM_ERR_ARG;
  const int64_t P = (int64_t)B * c.L;
  const bool multi = c.K > 1;
  const bool kt = c.task == GRAM_TASK_KT;
  cudaEvent_t* ev = m->ev;
  int32_t* status = gram_status_word(ctx);
  GRAM_CUDA(ctx, cudaEventRecord(ev[0], st));
  const int32_t* ids = ids_in;
  const int32_t* labels = labels_in;
  if (on_host) {
    GRAM_CUDA(ctx, cudaMemcpyAsync(m->ids, ids_in, (size_t)P * 4, cudaMemcpyHostToDevice, st));
    GRAM_CUDA(ctx, cudaMemcpyAsync(m->labels, labels_in, (size_t)P * 4, cudaMemcpyHostToDevice, st));
    ids = m->ids;
    labels = m->labels;
  }
  // stage 1
  IndexWorkspace* iws = gram_index_ws(ctx);
  GRAM_TRY(dedup_launch(ctx, iws, ids, P, c.n_items, m->unique, m->inverse, m->perm, m->seg_off, m->n_unique, st));
  int32_t U = 0, n_encoded = 0, n_touched = 0, encoder_ran = 0;
  const float* dE_at = nullptr;
  if (!multi) {
    const int32_t* words[2] = {m->n_unique, status};
    int32_t got[2] = {0, 0};
    GRAM_TRY(read_words(m, words, 2, got, st));
    if (got[1] != 0) return device_error(m, got[1], st);
    U = got[0];
    if (U <= 0 || U > m->u_cap) return gram_set_error(ctx, "gram_step: dedup returned U=%d", U), GRAM_ERR_ID_RANGE;
    GRAM_CUDA(ctx, cudaEventRecord(ev[1], st));
    // stage 2: one encoding per unique item (Eq. 4)
    for (int32_t u0 = 0; u0 < U; u0 += m->mb) {
      const int32_t n = (U - u0 < m->mb) ? U - u0 : m->mb;
      GRAM_TRY(encoder_forward_chunk(m, nullptr, m->unique + u0, 0, n, m->H + (size_t)u0 * c.d, st));
    }
    GRAM_CUDA(ctx, cudaEventRecord(ev[2], st));
    // stage 3: the KT task module gathers H[inverse[p]] in its first load; the NR module reads a materialised E
    EncodingSource src;
    if (kt) {
      src.rows = m->H; src.index = m->inverse; src.n_rows = U;
    } else {
      GRAM_TRY(gather_launch(ctx, m->H, U, m->inverse, P, c.d, 4, m->E, st));
      src.rows = m->E;
    }
    GRAM_CUDA(ctx, cudaEventRecord(ev[3], st));
    // task module forward / backward (Eq. 5) and dL/dE
    GRAM_TRY(task_forward_backward(m, src, labels, B, kt ? nullptr : m->dE, m->loss, &dE_at, st));
    GRAM_CUDA(ctx, cudaEventRecord(ev[4], st));
    // stage 4 (Eq. 6)
    GRAM_TRY(accumulate_launch(ctx, iws, dE_at, 0, m->perm, m->seg_off, P, U, nullptr, c.d, nullptr, 0, m->G, st));
    GRAM_CUDA(ctx, cudaEventRecord(ev[5], st));
    // stage 5 (Eq. 7)
    GRAM_CUDA(ctx, cudaMemsetAsync(m->ce.g, 0, m->ce.n * 4, st));
    if (U <= m->mb) {
      GRAM_TRY(encoder_backward_chunk(m, m->G, U, st));
    } else {
      // activations of one micro-batch at a time: run the forward again, then its backward
      float* Gbase = m->G;
      GRAM_TRY(encoder_pass(m, m->unique, U, false,
                            [&](int32_t u0, int32_t, const float** G) { *G = Gbase + (size_t)u0 * c.d; return GRAM_OK; }, st));
    }
    n_encoded = U;
    n_touched = U;
    encoder_ran = 1;
    if (!c.defer_update) {
      GRAM_TRY(apply_sgd(m, m->task, c.lr_task, st));
      GRAM_TRY(apply_sgd(m, m->ce, c.lr_ce, st));
    }
  } else {
    GRAM_CUDA(ctx, cudaEventRecord(ev[1], st));
    GRAM_CUDA(ctx, cudaEventRecord(ev[2], st));
    // stage 3 from the cache (Section 4.2): fused into the KT module's first load, materialised otherwise
    EncodingSource src;
    if (m->pseudo) {                   // the pseudo-targets h~ = cache - table of the items at every position (Eq. 6)
      GRAM_TRY(gather_diff_launch(ctx, (const float*)m->cache, m->table, c.n_items, ids, P, c.d, nullptr, m->E, st));
      src.rows = m->E;
    } else if (kt) {
      src.rows = m->cache; src.rows_bf16 = m->cache_dtype == GRAM_BF16; src.index = ids; src.n_rows = c.n_items;
    } else if (m->cache_dtype == GRAM_BF16) {       // rows of the bf16 cache, widened on the way
      GRAM_TRY(gather_widen_launch(ctx, m->cache, c.n_items, ids, P, c.d, m->E, st));
      src.rows = m->E;
    } else {
      GRAM_TRY(gather_launch(ctx, m->cache, c.n_items, ids, P, c.d, 4, m->E, st));
      src.rows = m->E;
    }
    GRAM_CUDA(ctx, cudaEventRecord(ev[3], st));
    GRAM_TRY(task_forward_backward(m, src, labels, B, kt ? nullptr : m->dE, m->loss, &dE_at, st));
    GRAM_CUDA(ctx, cudaEventRecord(ev[4], st));
    // stage 4 (Eq. 6) into the table; U is read on the device
    GRAM_TRY(accumulate_launch(ctx, iws, dE_at, 0, m->perm, m->seg_off, P, 0, m->n_unique, c.d, m->unique, 1, m->table, st, 1));
    GRAM_TRY(touched_mark_launch(ctx, m->unique, 0, m->n_unique, c.n_items, m->touched, m->tcount, 1, st));
    GRAM_CUDA(ctx, cudaEventRecord(ev[5], st));
    const int64_t task_updates = m->task.updates;
    if (!c.defer_update) GRAM_TRY(apply_sgd(m, m->task, c.lr_task, st, true));
    if (m->step_in_window + 1 >= c.K) {
      // last step of the window: the list of touched items and its length are needed on the host now
      GRAM_TRY(touched_list_launch(ctx, m->touched, c.n_items, m->tlist, m->tcount, st));
      const int32_t* words[3] = {m->tcount, m->n_unique, status};
      int32_t got[3] = {0, 0, 0};
      GRAM_TRY(read_words(m, words, 3, got, st));
      if (got[2] != 0) {
        m->task.updates = task_updates;
        m->task.wb_stale = true;
        return device_error(m, got[2], st);
      }
      n_touched = got[0];
      U = got[1];
      GRAM_CUDA(ctx, cudaMemsetAsync(m->ce.g, 0, m->ce.n * 4, st));
      GRAM_TRY(encoder_pass(m, m->tlist, n_touched, true,
                            [&](int32_t u0, int32_t n, const float** G) {
                              *G = m->G;
                              if (m->pseudo)       // Eq. 9: CE(c_i) - h~_i, with the forward values of this pass in H
                                return gather_diff_launch(ctx, (const float*)m->cache, m->table, c.n_items, m->tlist + u0, n, c.d,
                                                          m->H, m->G, st);
                              return gather_launch(ctx, m->table, c.n_items, m->tlist + u0, n, c.d, 4, m->G, st);
                            }, st));
      if (!c.defer_update) GRAM_TRY(apply_sgd(m, m->ce, c.lr_ce, st));
      if (c.refresh_after_update) {      // Eq. 4 with the updated parameters: the next window reads fresh encodings
        for (int32_t u0 = 0; u0 < n_touched; u0 += m->mb) {
          const int32_t n = (n_touched - u0 < m->mb) ? n_touched - u0 : m->mb;
          GRAM_TRY(encoder_forward_chunk(m, nullptr, m->tlist + u0, 0, n, m->H, st));
          GRAM_TRY(scatter_rows(ctx, m->cache_dtype, m->H, m->tlist + u0, n, c.d, c.n_items, m->cache, st));
        }
        m->saved_n = -1;
      }
      GRAM_TRY(model_window_reset(m, st));
      n_encoded = n_touched;
      encoder_ran = 1;
      GRAM_CUDA(ctx, cudaEventRecord(ev[6], st));
      GRAM_CUDA(ctx, cudaMemcpyAsync(m->h_pinned + 12, m->loss, 4, cudaMemcpyDeviceToHost, st));
      GRAM_CUDA(ctx, cudaStreamSynchronize(st));
    } else {
      GRAM_CUDA(ctx, cudaEventRecord(ev[6], st));
      GRAM_CUDA(ctx, cudaMemcpyAsync(m->h_pinned + 12, m->loss, 4, cudaMemcpyDeviceToHost, st));
      const int32_t* words[3] = {m->tcount, m->n_unique, status};
      int32_t got[3] = {0, 0, 0};
      GRAM_TRY(read_words(m, words, 3, got, st));           // the step's only wait
      if (got[2] != 0) {
        m->task.updates = task_updates;
        m->task.wb_stale = true;
        return device_error(m, got[2], st);
      }
      n_touched = got[0];
      U = got[1];
      ++m->step_in_window;
    }
  }
  if (!multi) {
    GRAM_CUDA(ctx, cudaEventRecord(ev[6], st));
    GRAM_CUDA(ctx, cudaMemcpyAsync(m->h_pinned + 12, m->loss, 4, cudaMemcpyDeviceToHost, st));
    GRAM_CUDA(ctx, cudaStreamSynchronize(st));
  }
  if (rep) {
    memset(rep, 0, sizeof(*rep));
    memcpy(&rep->loss, m->h_pinned + 12, 4);
    rep->n_positions = (int32_t)P;
    rep->n_unique = U;
    rep->boost_ratio = U > 0 ? (float)P / (float)U : 0.f;
    rep->n_touched = n_touched;
    rep->encoder_pass = encoder_ran;
    rep->n_encoded = n_encoded;
    float* ms[6] = {&rep->ms_dedup, &rep->ms_encode, &rep->ms_gather, &rep->ms_task, &rep->ms_accumulate, &rep->ms_backward};
    for (int i = 0; i < 6; ++i) cudaEventElapsedTime(ms[i], ev[i], ev[i + 1]);
    cudaEventElapsedTime(&rep->ms_total, ev[0], ev[6]);
  }
  return GRAM_OK;
}
