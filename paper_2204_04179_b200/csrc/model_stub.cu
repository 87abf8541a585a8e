#include "model.h"
struct Model { int x; };
gram_status model_create(gram_ctx* ctx, const gram_config*, Model**) { gram_set_error(ctx, "stub"); return GRAM_ERR_UNSUPPORTED; }
void model_destroy(Model*) {}
gram_status model_param_count(const Model*, int, size_t*) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_set_params(Model*, int, const float*, size_t) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_get_params(Model*, int, float*, size_t, int) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_zero_grads(Model*, int, cudaStream_t) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_set_item_tokens(Model*, const int32_t*) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_encode(Model*, const int32_t*, const int32_t*, int32_t, void*, int, cudaStream_t) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_task(Model*, const void*, const int32_t*, int32_t, float*, float*, cudaStream_t) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_encoder_backward(Model*, const float*, const int32_t*, int32_t, cudaStream_t) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_step(Model*, const int32_t*, const int32_t*, int32_t, int, gram_step_report*, cudaStream_t) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_cache_fill(Model*, cudaStream_t) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_window_reset(Model*, cudaStream_t) { return GRAM_ERR_UNSUPPORTED; }
gram_status model_get_window(Model*, float*, uint32_t*, float*) { return GRAM_ERR_UNSUPPORTED; }
float* model_table(Model*) { return nullptr; }
uint32_t* model_touched(Model*) { return nullptr; }
