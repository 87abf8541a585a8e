// Encoder (CE) and task module (CF) state and the calls api.cu forwards to.
#pragma once
#include "gram_internal.h"

struct Model;

IndexWorkspace* gram_index_ws(gram_ctx* ctx);
const gram_config* gram_cfg(const gram_ctx* ctx);

gram_status model_create(gram_ctx* ctx, const gram_config* cfg, Model** out);
void model_destroy(Model* m);
gram_status model_param_count(const Model* m, int module, size_t* n);
gram_status model_set_params(Model* m, int module, const float* h, size_t n);
gram_status model_get_params(Model* m, int module, float* h, size_t n, int grads);
gram_status model_zero_grads(Model* m, int module, cudaStream_t st);
gram_status model_grads_device(Model* m, int module, float** d_grads, size_t* n);
gram_status model_optimizer_step(Model* m, int module, cudaStream_t st);
gram_status model_optimizer_reset(Model* m, cudaStream_t st);
double noam_rate(int64_t t, double peak, int warmup);
gram_status model_set_item_tokens(Model* m, const int32_t* h_tokens);
gram_status model_set_item_lengths(Model* m, const int32_t* h_len);
gram_status model_encode(Model* m, const int32_t* d_item_tokens, const int32_t* d_items, int32_t U, float* d_H,
                         int save, cudaStream_t st);
gram_status model_task(Model* m, const float* d_E, const int32_t* d_labels, int32_t B, float* d_dE, float* d_loss,
                       cudaStream_t st);
gram_status model_encoder_backward(Model* m, const float* d_G, const int32_t* d_items, int32_t U, cudaStream_t st);
gram_status model_step(Model* m, const int32_t* ids, const int32_t* labels, int32_t B, int on_host,
                       gram_step_report* report, cudaStream_t st);
gram_status model_cache_fill(Model* m, cudaStream_t st);
gram_status model_window_reset(Model* m, cudaStream_t st);
gram_status model_get_window(Model* m, float* h_table, uint32_t* h_touched, float* h_cache);
gram_status model_state_export(Model* m, float* h_table, uint32_t* h_touched, float* h_cache, int32_t* steps);
gram_status model_state_import(Model* m, const float* h_table, const uint32_t* h_touched, const float* h_cache, int32_t steps);
gram_status model_optimizer_export(Model* m, int module, float* h_m, float* h_v, int64_t* updates);
gram_status model_optimizer_import(Model* m, int module, const float* h_m, const float* h_v, int64_t updates);
float* model_table(Model* m);
uint32_t* model_touched(Model* m);

struct GemmWorkspace;
GemmWorkspace* gram_gemm_ws(gram_ctx* ctx);
