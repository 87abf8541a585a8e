// The C ABI of libgram: context life cycle, argument checks, and the calls of include/gram.h.
#include <stdarg.h>

#include <new>

#include "gemm.h"
#include "gram_internal.h"
#include "model.h"
#include "layers.h"

constexpr int kProfSlots = 16384;
struct ProfRec {
  int kind;
  const char* tag;
  double work;
  int launches;
};
constexpr int kProfTags = 64;
struct ProfTag {
  const char* tag;
  int kind;
  double ms, work;
  int64_t launches;
};

struct gram_ctx {
  gram_config cfg;
  // measurement
  int64_t launch_count = 0;
  bool prof_on = false;
  cudaEvent_t* prof_ev = nullptr;       // [2 * kProfSlots], created on first enable
  ProfRec* prof_rec = nullptr;
  int prof_used = 0;
  double prof_ms[GRAM_K_COUNT] = {}, prof_work[GRAM_K_COUNT] = {};
  int64_t prof_launches[GRAM_K_COUNT] = {};
  ProfTag prof_tags[kProfTags] = {};
  int prof_ntags = 0;
  char err[512];
  int32_t* d_status = nullptr;      // device status word (first device-side error)
  IndexWorkspace iws;
  GemmWorkspace gws;
  Model* model = nullptr;           // encoder + task module state (null for an index-only context)
};

void gram_set_error(gram_ctx* ctx, const char* fmt, ...) {
  if (!ctx) return;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
  va_end(ap);
}

int32_t* gram_status_word(gram_ctx* ctx) { return ctx->d_status; }

void gram_prof_open(gram_ctx* ctx, int kind, const char* tag, double work, int launches, cudaStream_t st, int* slot) {
  *slot = -1;
  if (!ctx) return;
  ctx->launch_count += launches;
  if (!ctx->prof_on || ctx->prof_used >= kProfSlots) return;
  const int k = ctx->prof_used++;
  ctx->prof_rec[k] = ProfRec{kind, tag, work, launches};
  cudaEventRecord(ctx->prof_ev[2 * k], st);
  *slot = k;
}
void gram_prof_close(gram_ctx* ctx, int slot, cudaStream_t st) { cudaEventRecord(ctx->prof_ev[2 * slot + 1], st); }

// folds the recorded event pairs into the per-kind totals (the device must be idle)
static void prof_fold(gram_ctx* ctx) {
  for (int k = 0; k < ctx->prof_used; ++k) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->prof_ev[2 * k], ctx->prof_ev[2 * k + 1]) == cudaSuccess) {
      const ProfRec& r = ctx->prof_rec[k];
      ctx->prof_ms[r.kind] += ms;
      ctx->prof_work[r.kind] += r.work;
      ctx->prof_launches[r.kind] += r.launches;
      if (r.tag) {
        int t = 0;
        while (t < ctx->prof_ntags && ctx->prof_tags[t].tag != r.tag && strcmp(ctx->prof_tags[t].tag, r.tag) != 0) ++t;
        if (t == ctx->prof_ntags && t < kProfTags) ctx->prof_tags[ctx->prof_ntags++] = ProfTag{r.tag, r.kind, 0, 0, 0};
        if (t < kProfTags) {
          ctx->prof_tags[t].ms += ms;
          ctx->prof_tags[t].work += r.work;
          ctx->prof_tags[t].launches += r.launches;
        }
      }
    }
  }
  ctx->prof_used = 0;
}
IndexWorkspace* gram_index_ws(gram_ctx* ctx) { return &ctx->iws; }
GemmWorkspace* gram_gemm_ws(gram_ctx* ctx) { return &ctx->gws; }
const gram_config* gram_cfg(const gram_ctx* ctx) { return &ctx->cfg; }

static cudaStream_t S(gram_stream s) { return reinterpret_cast<cudaStream_t>(s); }

static gram_status check_device_status(gram_ctx* ctx) {
  int32_t h = 0;
  GRAM_CUDA(ctx, cudaMemcpy(&h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost));
  if (h != 0) {
    GRAM_CUDA(ctx, cudaMemset(ctx->d_status, 0, sizeof(int32_t)));
    gram_set_error(ctx, h == GRAM_ERR_ID_RANGE ? "an ID outside its range was met on the device"
                                               : (h == GRAM_ERR_TIMEOUT ? "a bounded device-side wait ran out" : "device-side error"));
    return (gram_status)h;
  }
  return GRAM_OK;
}

extern "C" {

gram_status gram_create(const gram_config* cfg, gram_ctx** out) {
  if (out) *out = nullptr;
  if (!cfg || !out) return GRAM_ERR_ARG;
  if (cfg->n_items <= 0 || cfg->B_max < 0 || cfg->L < 0 || cfg->P_max < 0 || cfg->K < 0 || cfg->n_layers < 0) return GRAM_ERR_ARG;
  gram_ctx* ctx = new (std::nothrow) gram_ctx();
  if (!ctx) return GRAM_ERR_CUDA;
  ctx->cfg = *cfg;
  ctx->err[0] = 0;
  if (ctx->cfg.K == 0) ctx->cfg.K = 1;
  int64_t P_max = cfg->P_max > 0 ? cfg->P_max : (int64_t)cfg->B_max * cfg->L;
  if (ctx->cfg.n_layers > 0) {       // the token-embedding gradient reuses the index kernels over token positions
    const int64_t u_cap = P_max < cfg->n_items ? P_max : cfg->n_items;
    int64_t mb = cfg->ce_micro_batch > 0 ? cfg->ce_micro_batch : (ctx->cfg.K > 1 ? cfg->n_items : u_cap);
    if (mb > cfg->n_items) mb = cfg->n_items;
    const int64_t tok = mb * cfg->l_t;
    if (tok > P_max) P_max = tok;
  }
  ctx->cfg.P_max = P_max;
  int32_t d_max = cfg->d_max > 0 ? cfg->d_max : cfg->d;
  if (d_max < cfg->d) d_max = cfg->d;
  ctx->cfg.d_max = d_max;
  gram_status s = GRAM_OK;
  do {
    if (cudaMalloc(&ctx->d_status, sizeof(int32_t)) != cudaSuccess || cudaMemset(ctx->d_status, 0, sizeof(int32_t)) != cudaSuccess) {
      s = GRAM_ERR_CUDA;
      break;
    }
    int32_t n_keys = cfg->n_items > cfg->vocab ? cfg->n_items : cfg->vocab;
    s = index_ws_alloc(ctx, &ctx->iws, P_max, n_keys, d_max);
    if (s != GRAM_OK) break;
    {  // split-K partial products: up to 16 parts of the largest weight matrix, within 32..256 MB
      size_t w = (size_t)(cfg->d_ff > cfg->task_d_ff ? cfg->d_ff : cfg->task_d_ff) * (size_t)cfg->d * sizeof(float) * 16;
      if (w < ((size_t)32 << 20)) w = (size_t)32 << 20;
      if (w > ((size_t)256 << 20)) w = (size_t)256 << 20;
      s = gemm_ws_alloc(ctx, &ctx->gws, w);
      if (s != GRAM_OK) break;
    }
    if (ctx->cfg.n_layers > 0 || ctx->cfg.task != GRAM_TASK_NONE) {
      s = model_create(ctx, &ctx->cfg, &ctx->model);
      if (s != GRAM_OK) break;
    }
  } while (0);
  if (s != GRAM_OK) {
    fprintf(stderr, "gram_create failed: %s\n", ctx->err);
    gram_destroy(ctx);
    return s;
  }
  *out = ctx;
  return GRAM_OK;
}

gram_status gram_destroy(gram_ctx* ctx) {
  if (!ctx) return GRAM_OK;
  cudaDeviceSynchronize();
  if (ctx->model) model_destroy(ctx->model);
  if (ctx->prof_ev) {
    for (int i = 0; i < 2 * kProfSlots; ++i) cudaEventDestroy(ctx->prof_ev[i]);
    delete[] ctx->prof_ev;
    delete[] ctx->prof_rec;
  }
  index_ws_free(&ctx->iws);
  gemm_ws_free(&ctx->gws);
  cudaFree(ctx->d_status);
  delete ctx;
  return GRAM_OK;
}

gram_status gram_sync(gram_ctx* ctx, gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  GRAM_CUDA(ctx, cudaStreamSynchronize(S(stream)));
  return check_device_status(ctx);
}

const char* gram_last_error(const gram_ctx* ctx) { return ctx ? ctx->err : "null context"; }

gram_status gram_profile(gram_ctx* ctx, int enable) {
  if (!ctx) return GRAM_ERR_ARG;
  GRAM_CUDA(ctx, cudaDeviceSynchronize());
  if (enable && !ctx->prof_ev) {
    ctx->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfSlots];
    ctx->prof_rec = new (std::nothrow) ProfRec[kProfSlots];
    if (!ctx->prof_ev || !ctx->prof_rec) return gram_set_error(ctx, "out of host memory"), GRAM_ERR_CUDA;
    for (int i = 0; i < 2 * kProfSlots; ++i) GRAM_CUDA(ctx, cudaEventCreate(&ctx->prof_ev[i]));
  }
  ctx->prof_on = enable != 0;
  ctx->prof_used = 0;
  ctx->prof_ntags = 0;
  for (int k = 0; k < GRAM_K_COUNT; ++k) {
    ctx->prof_ms[k] = 0;
    ctx->prof_work[k] = 0;
    ctx->prof_launches[k] = 0;
  }
  return GRAM_OK;
}

gram_status gram_profile_read(gram_ctx* ctx, int kind, double* ms, double* work, int64_t* launches) {
  if (!ctx || kind < 0 || kind >= GRAM_K_COUNT) return GRAM_ERR_ARG;
  GRAM_CUDA(ctx, cudaDeviceSynchronize());
  prof_fold(ctx);
  if (ms) *ms = ctx->prof_ms[kind];
  if (work) *work = ctx->prof_work[kind];
  if (launches) *launches = ctx->prof_launches[kind];
  return GRAM_OK;
}

gram_status gram_profile_dump(gram_ctx* ctx, char* h_text, size_t n) {
  if (!ctx || !h_text || n == 0) return GRAM_ERR_ARG;
  GRAM_CUDA(ctx, cudaDeviceSynchronize());
  prof_fold(ctx);
  size_t o = 0;
  h_text[0] = 0;
  for (int t = 0; t < ctx->prof_ntags && o + 128 < n; ++t) {
    const ProfTag& g = ctx->prof_tags[t];
    o += (size_t)snprintf(h_text + o, n - o, "%s %d %.6f %.6e %lld\n", g.tag, g.kind, g.ms, g.work, (long long)g.launches);
  }
  return GRAM_OK;
}

gram_status gram_launch_count(const gram_ctx* ctx, int64_t* launches) {
  if (!ctx || !launches) return GRAM_ERR_ARG;
  *launches = ctx->launch_count;
  return GRAM_OK;
}

gram_status gram_dedup(gram_ctx* ctx, const int32_t* d_ids, int64_t P, int32_t n_items, int32_t* d_unique,
                       int32_t* d_inverse, int32_t* d_perm, int32_t* d_seg_off, int32_t* d_n_unique,
                       gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  return dedup_launch(ctx, &ctx->iws, d_ids, P, n_items, d_unique, d_inverse, d_perm, d_seg_off, d_n_unique, S(stream));
}

gram_status gram_selftest_bounded_wait(gram_ctx* ctx, gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  return dedup_wait_selftest(ctx, &ctx->iws, S(stream));
}
gram_status gram_gather(gram_ctx* ctx, const void* d_src, int64_t n_src_rows, const int32_t* d_index, int64_t P,
                        int32_t d, int dtype, void* d_E, gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  if (dtype != GRAM_F32 && dtype != GRAM_BF16) return gram_set_error(ctx, "gram_gather: unknown dtype"), GRAM_ERR_ARG;
  return gather_launch(ctx, d_src, n_src_rows, d_index, P, d, dtype == GRAM_F32 ? 4 : 2, d_E, S(stream));
}

gram_status gram_accumulate(gram_ctx* ctx, const float* d_dE, const int32_t* d_perm, const int32_t* d_seg_off,
                            int64_t P, int32_t U, int32_t d, float* d_G, gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  return accumulate_launch(ctx, &ctx->iws, d_dE, 0, d_perm, d_seg_off, P, U, nullptr, d, nullptr, 0, d_G, S(stream));
}

gram_status gram_accumulate_multistep(gram_ctx* ctx, const float* d_dE, const int32_t* d_perm,
                                      const int32_t* d_seg_off, const int32_t* d_unique, int64_t P, int32_t U,
                                      int32_t d, int32_t n_items, float* d_table, uint32_t* d_touched_bits,
                                      gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  if (!d_unique && U > 0) return gram_set_error(ctx, "gram_accumulate_multistep: null d_unique"), GRAM_ERR_ARG;
  if (!d_table || !d_touched_bits) {
    if (!ctx->model || !model_table(ctx->model) || n_items != ctx->cfg.n_items || d != ctx->cfg.d)
      return gram_set_error(ctx, "gram_accumulate_multistep: no table given and the context holds none of this shape"), GRAM_ERR_ARG;
    if (!d_table) d_table = model_table(ctx->model);
    if (!d_touched_bits) d_touched_bits = model_touched(ctx->model);
  }
  GRAM_TRY(accumulate_launch(ctx, &ctx->iws, d_dE, 0, d_perm, d_seg_off, P, U, nullptr, d, d_unique, 1, d_table, S(stream)));
  return touched_mark_launch(ctx, d_unique, U, nullptr, n_items, d_touched_bits, nullptr, 0, S(stream));
}

gram_status gram_touched_list(gram_ctx* ctx, const uint32_t* d_touched_bits, int32_t n_items, int32_t* d_list,
                              int32_t* d_count, gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  return touched_list_launch(ctx, d_touched_bits, n_items, d_list, d_count, S(stream));
}

// ---- calls that need the modules -----------------------------------------------------------
#define NEED_MODEL(name)                                                                                  \
  if (!ctx) return GRAM_ERR_ARG;                                                                          \
  if (!ctx->model) return gram_set_error(ctx, name ": the context was created without modules"), GRAM_ERR_ARG;

gram_status gram_param_count(const gram_ctx* ctx, int module, size_t* n) {
  if (!ctx || !n || !ctx->model) return GRAM_ERR_ARG;
  return model_param_count(ctx->model, module, n);
}
gram_status gram_set_params(gram_ctx* ctx, int module, const float* h, size_t n) {
  NEED_MODEL("gram_set_params");
  return model_set_params(ctx->model, module, h, n);
}
gram_status gram_get_params(gram_ctx* ctx, int module, float* h, size_t n) {
  NEED_MODEL("gram_get_params");
  return model_get_params(ctx->model, module, h, n, 0);
}
gram_status gram_get_grads(gram_ctx* ctx, int module, float* h, size_t n) {
  NEED_MODEL("gram_get_grads");
  return model_get_params(ctx->model, module, h, n, 1);
}
gram_status gram_zero_grads(gram_ctx* ctx, int module, gram_stream stream) {
  NEED_MODEL("gram_zero_grads");
  return model_zero_grads(ctx->model, module, S(stream));
}
gram_status gram_grads_device(gram_ctx* ctx, int module, float** d_grads, size_t* n) {
  NEED_MODEL("gram_grads_device");
  if (!d_grads || !n) return gram_set_error(ctx, "gram_grads_device: null output"), GRAM_ERR_ARG;
  return model_grads_device(ctx->model, module, d_grads, n);
}
gram_status gram_optimizer_step(gram_ctx* ctx, int module, gram_stream stream) {
  NEED_MODEL("gram_optimizer_step");
  return model_optimizer_step(ctx->model, module, S(stream));
}
gram_status gram_optimizer_reset(gram_ctx* ctx, gram_stream stream) {
  NEED_MODEL("gram_optimizer_reset");
  return model_optimizer_reset(ctx->model, S(stream));
}
gram_status gram_noam_rate(int64_t t, float peak, int32_t warmup, float* h_rate) {
  if (!h_rate || t < 1) return GRAM_ERR_ARG;
  *h_rate = (float)noam_rate(t, (double)peak, warmup);
  return GRAM_OK;
}
gram_status gram_adam_update(gram_ctx* ctx, float* d_w, const float* d_g, float* d_m, float* d_v, size_t n, int64_t t,
                             float rate, float beta1, float beta2, float eps, void* d_w_bf16, gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  if (n && (!d_w || !d_g || !d_m || !d_v)) return gram_set_error(ctx, "gram_adam_update: null buffer"), GRAM_ERR_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f && beta2 >= 0.f && beta2 < 1.f))
    return gram_set_error(ctx, "gram_adam_update: beta1 and beta2 must lie in [0, 1)"), GRAM_ERR_ARG;
  return adam_update(ctx, d_w, d_g, d_m, d_v, d_w_bf16, n, t, rate, beta1, beta2, eps, S(stream));
}
gram_status gram_set_item_tokens(gram_ctx* ctx, const int32_t* h_tokens) {
  NEED_MODEL("gram_set_item_tokens");
  return model_set_item_tokens(ctx->model, h_tokens);
}
gram_status gram_set_item_lengths(gram_ctx* ctx, const int32_t* h_lengths) {
  NEED_MODEL("gram_set_item_lengths");
  return model_set_item_lengths(ctx->model, h_lengths);
}
gram_status gram_encode_unique(gram_ctx* ctx, const int32_t* d_item_tokens, const int32_t* d_items, int32_t U,
                               float* d_H, int save_activations, gram_stream stream) {
  NEED_MODEL("gram_encode_unique");
  return model_encode(ctx->model, d_item_tokens, d_items, U, d_H, save_activations, S(stream));
}
gram_status gram_task(gram_ctx* ctx, const float* d_E, const int32_t* d_labels, int32_t B, float* d_dE, float* d_loss,
                      gram_stream stream) {
  NEED_MODEL("gram_task");
  return model_task(ctx->model, d_E, d_labels, B, d_dE, d_loss, S(stream));
}
gram_status gram_encoder_backward(gram_ctx* ctx, const float* d_G, const int32_t* d_items, int32_t U,
                                  gram_stream stream) {
  NEED_MODEL("gram_encoder_backward");
  return model_encoder_backward(ctx->model, d_G, d_items, U, S(stream));
}
gram_status gram_step(gram_ctx* ctx, const int32_t* d_ids, const int32_t* d_labels, int32_t B,
                      gram_step_report* report, gram_stream stream) {
  NEED_MODEL("gram_step");
  GRAM_TRY(model_step(ctx->model, d_ids, d_labels, B, 0, report, S(stream)));
  return check_device_status(ctx);
}
gram_status gram_step_host(gram_ctx* ctx, const int32_t* h_ids, const int32_t* h_labels, int32_t B,
                           gram_step_report* report, gram_stream stream) {
  NEED_MODEL("gram_step_host");
  GRAM_TRY(model_step(ctx->model, h_ids, h_labels, B, 1, report, S(stream)));
  return check_device_status(ctx);
}
gram_status gram_cache_fill(gram_ctx* ctx, gram_stream stream) {
  NEED_MODEL("gram_cache_fill");
  return model_cache_fill(ctx->model, S(stream));
}
gram_status gram_window_reset(gram_ctx* ctx, gram_stream stream) {
  NEED_MODEL("gram_window_reset");
  return model_window_reset(ctx->model, S(stream));
}
gram_status gram_get_window(gram_ctx* ctx, float* h_table, uint32_t* h_touched, float* h_cache) {
  NEED_MODEL("gram_get_window");
  return model_get_window(ctx->model, h_table, h_touched, h_cache);
}
gram_status gram_state_export(gram_ctx* ctx, float* h_table, uint32_t* h_touched, float* h_cache, int32_t* steps_in_window) {
  NEED_MODEL("gram_state_export");
  return model_state_export(ctx->model, h_table, h_touched, h_cache, steps_in_window);
}
gram_status gram_state_import(gram_ctx* ctx, const float* h_table, const uint32_t* h_touched, const float* h_cache,
                              int32_t steps_in_window) {
  NEED_MODEL("gram_state_import");
  return model_state_import(ctx->model, h_table, h_touched, h_cache, steps_in_window);
}
gram_status gram_optimizer_export(gram_ctx* ctx, int module, float* h_m, float* h_v, int64_t* updates) {
  NEED_MODEL("gram_optimizer_export");
  return model_optimizer_export(ctx->model, module, h_m, h_v, updates);
}
gram_status gram_optimizer_import(gram_ctx* ctx, int module, const float* h_m, const float* h_v, int64_t updates) {
  NEED_MODEL("gram_optimizer_import");
  return model_optimizer_import(ctx->model, module, h_m, h_v, updates);
}
gram_status gram_gemm_bf16(gram_ctx* ctx, const void* d_A, int a_kmajor, const void* d_B, int b_kmajor, void* d_C,
                           int c_f32, const float* d_bias, int accumulate, int64_t M, int32_t N, int64_t K,
                           gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  if (M < 0 || N < 0 || K <= 0 || (M % 8) || (N % 8) || (K % 8))
    return gram_set_error(ctx, "gram_gemm_bf16: M, N, K must be positive multiples of 8"), GRAM_ERR_ARG;
  GemmEpilogue e;
  e.bias = d_bias;
  e.accumulate = accumulate;
  return gemm_launch(ctx, &ctx->gws, GRAM_BF16, d_A, a_kmajor, a_kmajor ? K : M, d_B, b_kmajor, b_kmajor ? K : N, d_C,
                     c_f32, N, M, N, K, e, 1, S(stream));
}

gram_status gram_gemm_bf16_epilogue(gram_ctx* ctx, const void* d_A, int a_kmajor, const void* d_B, int b_kmajor, void* d_C,
                                    int c_f32, const gram_gemm_epilogue* ep, int64_t M, int32_t N, int64_t K,
                                    gram_stream stream) {
  if (!ctx) return GRAM_ERR_ARG;
  if (M < 0 || N < 0 || K <= 0 || (M % 8) || (N % 8) || (K % 8))
    return gram_set_error(ctx, "gram_gemm_bf16_epilogue: M, N, K must be positive multiples of 8"), GRAM_ERR_ARG;
  GemmEpilogue e;
  if (ep) {
    if (ep->d_res_mean && !(ep->d_res && ep->d_res_rstd && ep->d_res_gamma && ep->d_res_beta))
      return gram_set_error(ctx, "gram_gemm_bf16_epilogue: LayerNorm on the residual needs all of res, mean, rstd, gamma, beta"), GRAM_ERR_ARG;
    e.bias = ep->d_bias;
    e.res = ep->d_res; e.res_mean = ep->d_res_mean; e.res_rstd = ep->d_res_rstd; e.res_gamma = ep->d_res_gamma; e.res_beta = ep->d_res_beta;
    e.pre = ep->d_gelu_grad_out;
    e.dgelu_pre = ep->d_gelu_grad_in;
    e.copy_out = ep->d_copy_bf16;
    e.gelu = ep->gelu;
    e.accumulate = ep->accumulate;
    e.tag = "gemm_epilogue";
  }
  return gemm_launch(ctx, &ctx->gws, GRAM_BF16, d_A, a_kmajor, a_kmajor ? K : M, d_B, b_kmajor, b_kmajor ? K : N, d_C,
                     c_f32, N, M, N, K, e, 0, S(stream));
}

}  // extern "C"
