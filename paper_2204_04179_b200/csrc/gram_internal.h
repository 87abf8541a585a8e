// Internal declarations shared by the CUDA translation units of libgram.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "gram.h"

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------------------
// error plumbing
// ---------------------------------------------------------------------------
struct gram_ctx;
void gram_set_error(gram_ctx* ctx, const char* fmt, ...);

#define GRAM_CUDA(ctx, expr)                                                              \
  do {                                                                                    \
    cudaError_t e__ = (expr);                                                             \
    if (e__ != cudaSuccess) {                                                             \
      gram_set_error((ctx), "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), __FILE__, __LINE__); \
      return GRAM_ERR_CUDA;                                                               \
    }                                                                                     \
  } while (0)

#define GRAM_TRY(expr)                        \
  do {                                        \
    gram_status s__ = (expr);                 \
    if (s__ != GRAM_OK) return s__;           \
  } while (0)

#define GRAM_LAUNCH_CHECK(ctx) GRAM_CUDA(ctx, cudaGetLastError())

static inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// ---------------------------------------------------------------------------
// index / accumulation workspaces (dedup.cu, gather_accum.cu)
// ---------------------------------------------------------------------------
constexpr int kAccMaxChunks = 148 * 16;   // work units of the segmented sum
constexpr int kNumSMs = 148;

struct IndexWorkspace {
  int64_t P_max = 0;
  int32_t n_items_max = 0;
  int32_t d_max = 0;
  int32_t *keys0 = nullptr, *keys1 = nullptr, *vals0 = nullptr, *vals1 = nullptr;  // [P_max] radix ping-pong
  uint32_t* sort_ctl = nullptr;   // tile tickets, digit totals and per-tile status words of the sort (cleared per call)
  int32_t* rank_table = nullptr;  // [n_items_max] item ID -> index in unique
  float* partial = nullptr;       // [kAccMaxChunks * 2 * d_max] chunk-boundary partial sums, then kAccMaxChunks (item, last chunk) pairs
};

gram_status index_ws_alloc(gram_ctx* ctx, IndexWorkspace* ws, int64_t P_max, int32_t n_items_max, int32_t d_max);
void index_ws_free(IndexWorkspace* ws);

gram_status dedup_launch(gram_ctx* ctx, IndexWorkspace* ws, const int32_t* d_ids, int64_t P, int32_t n_items,
                         int32_t* d_unique, int32_t* d_inverse, int32_t* d_perm, int32_t* d_seg_off,
                         int32_t* d_n_unique, cudaStream_t st);

gram_status dedup_wait_selftest(gram_ctx* ctx, IndexWorkspace* ws, cudaStream_t st);

gram_status gather_launch(gram_ctx* ctx, const void* d_src, int64_t n_src_rows, const int32_t* d_index, int64_t P,
                          int32_t d, int elem_bytes, void* d_E, cudaStream_t st);

// out[r, :] = a[index[r], :] - b[index[r], :] (d_x == NULL), or d_x[r, :] - (a[index[r], :] - b[index[r], :]); fp32 rows.
// Multi-step with pseudo-targets: the first form is h~ = cache - table gathered into the positions (Eq. 6), the
// second the cotangent CE(c) - h~ of the pseudo-loss (Eq. 9).
gram_status gather_diff_launch(gram_ctx* ctx, const float* d_a, const float* d_b, int64_t n_src_rows, const int32_t* d_index,
                               int64_t n, int32_t d, const float* d_x, float* d_out, cudaStream_t st);

// d_E[p, :] (fp32) = d_src_bf16[d_index[p], :] (bf16 rows of d elements, d a multiple of 8): gather and widen in one pass
gram_status gather_widen_launch(gram_ctx* ctx, const void* d_src_bf16, int64_t n_src_rows, const int32_t* d_index, int64_t P,
                                int32_t d, float* d_E, cudaStream_t st);

// in_bf16: rows of d_in are bf16 instead of fp32.  d_U (may be NULL): the number of segments is read
// from the device instead of U.  d_rows (may be NULL): output row of segment u is d_rows[u] instead
// of u.  add != 0: out[row] += sum instead of out[row] = sum.  gated != 0: the kernels leave d_out alone
// when the context's status word already holds an error (a step that must not change state after a bad input).
gram_status accumulate_launch(gram_ctx* ctx, IndexWorkspace* ws, const void* d_in, int in_bf16, const int32_t* d_perm,
                              const int32_t* d_seg_off, int64_t P, int32_t U, const int32_t* d_U, int32_t d,
                              const int32_t* d_rows, int add, float* d_out, cudaStream_t st, int gated = 0);

// sets bit d_unique[u] for u < U (U read from d_U when that is not NULL); d_count (may be NULL) counts the bits that
// were not set before; gated as above
gram_status touched_mark_launch(gram_ctx* ctx, const int32_t* d_unique, int32_t U, const int32_t* d_U, int32_t n_items,
                                uint32_t* d_bits, int32_t* d_count, int gated, cudaStream_t st);
gram_status touched_list_launch(gram_ctx* ctx, const uint32_t* d_bits, int32_t n_items, int32_t* d_list,
                                int32_t* d_count, cudaStream_t st);

// ---------------------------------------------------------------------------
// measurement: every launch wrapper opens a ProfScope.  It always counts the launches; when
// profiling is on it also brackets them with CUDA events on the launching stream and files the
// elapsed time and the algorithmic work (flops or bytes) under the kernel kind.
// ---------------------------------------------------------------------------
void gram_prof_open(gram_ctx* ctx, int kind, const char* tag, double work, int launches, cudaStream_t st, int* slot);
void gram_prof_close(gram_ctx* ctx, int slot, cudaStream_t st);
struct ProfScope {
  gram_ctx* ctx;
  cudaStream_t st;
  int slot = -1;
  // tag: a string literal naming the call site (shown by gram_profile_dump)
  ProfScope(gram_ctx* c, int kind, double work, int launches, cudaStream_t s, const char* tag = nullptr) : ctx(c), st(s) {
    gram_prof_open(c, kind, tag, work, launches, s, &slot);
  }
  ~ProfScope() { if (slot >= 0) gram_prof_close(ctx, slot, st); }
};

// the device status word: kernels record the first error kind they meet
__device__ __forceinline__ void gram_device_fail(int32_t* status, int32_t code) { atomicCAS(status, 0, code); }
int32_t* gram_status_word(gram_ctx* ctx);
