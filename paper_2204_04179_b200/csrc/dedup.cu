// Stage 1 of the GRAM step: the unique-item set B_I of a mini-batch (Table 1) and the
// occurrence -> item map of Fig. 1, as a stable LSD radix sort of (item ID, position) over
// the low ceil(log2 n_items) key bits followed by a run-length pass.
//
// Per radix pass (8 bits): block histograms -> exclusive scan (digit-major) -> stable scatter.
// Traffic per pass: 4P (histogram read) + 8P read + 8P write; the first pass generates the
// position payload instead of reading it.
#include "gram_internal.h"

namespace {

constexpr int RS_THREADS = 256;
constexpr int RS_ITEMS = 16;
constexpr int RS_TILE = RS_THREADS * RS_ITEMS;   // keys per block
constexpr int RS_WARPS = RS_THREADS / 32;
constexpr int SCAN_THREADS = 1024;

// ---- histogram of one digit over a block's tile -----------------------------------------
__global__ void __launch_bounds__(RS_THREADS) radix_hist_kernel(const int32_t* __restrict__ keys, int64_t P, int shift,
                                                                int32_t n_items, int check_range, int nblocks,
                                                                int32_t* __restrict__ hist, int32_t* status) {
  __shared__ int32_t sh[256];
  sh[threadIdx.x] = 0;
  __syncthreads();
  const int64_t base = (int64_t)blockIdx.x * RS_TILE;
  bool bad = false;
#pragma unroll 4
  for (int i = 0; i < RS_ITEMS; ++i) {
    int64_t j = base + (int64_t)i * RS_THREADS + threadIdx.x;
    if (j < P) {
      int32_t k = keys[j];
      if (check_range && (k < 0 || k >= n_items)) { bad = true; k = 0; }
      atomicAdd(&sh[(k >> shift) & 255], 1);
    }
  }
  if (bad) gram_device_fail(status, GRAM_ERR_ID_RANGE);
  __syncthreads();
  hist[(int64_t)threadIdx.x * nblocks + blockIdx.x] = sh[threadIdx.x];
}

// ---- device-wide exclusive scan of int32 (three launches) --------------------------------
// tile sums
__global__ void __launch_bounds__(SCAN_THREADS) scan_reduce_kernel(const int32_t* __restrict__ in, int64_t n,
                                                                   int32_t* __restrict__ sums) {
  __shared__ int32_t sw[32];
  const int64_t base = (int64_t)blockIdx.x * (SCAN_THREADS * 4);
  int32_t v = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int64_t j = base + (int64_t)threadIdx.x * 4 + i;
    if (j < n) v += in[j];
  }
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) sw[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x < 32) {
    v = sw[threadIdx.x];
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    if (threadIdx.x == 0) sums[blockIdx.x] = v;
  }
}

// exclusive scan of one block's worth of values held as 4 per thread; returns the thread's base
__device__ __forceinline__ int32_t block_exclusive_scan(int32_t thread_total, int32_t* sw /*[33]*/, int32_t* block_total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int32_t incl = thread_total;
  for (int o = 1; o < 32; o <<= 1) {
    int32_t t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) sw[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int32_t w = (lane < (int)(blockDim.x >> 5)) ? sw[lane] : 0;
    int32_t wi = w;
    for (int o = 1; o < 32; o <<= 1) {
      int32_t t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    sw[lane] = wi - w;
    if (lane == 31) sw[32] = wi;
  }
  __syncthreads();
  int32_t r = sw[warp] + incl - thread_total;
  if (block_total) *block_total = sw[32];
  __syncthreads();
  return r;
}

// in-place exclusive scan of the tile sums by ONE block (n up to a few million); total -> *total_out
__global__ void __launch_bounds__(SCAN_THREADS) scan_sums_kernel(int32_t* __restrict__ sums, int64_t n,
                                                                 int32_t* __restrict__ total_out) {
  __shared__ int32_t sw[33];
  int32_t carry = 0;
  for (int64_t base = 0; base < n; base += SCAN_THREADS * 4) {
    int32_t v[4], tot = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int64_t j = base + (int64_t)threadIdx.x * 4 + i;
      v[i] = (j < n) ? sums[j] : 0;
      tot += v[i];
    }
    int32_t btot;
    int32_t ex = block_exclusive_scan(tot, sw, &btot) + carry;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int64_t j = base + (int64_t)threadIdx.x * 4 + i;
      if (j < n) sums[j] = ex;
      ex += v[i];
    }
    carry += btot;
  }
  if (threadIdx.x == 0 && total_out) *total_out = carry;
}

// in and out may be the same array: a thread reads its four values before it writes them
__global__ void __launch_bounds__(SCAN_THREADS) scan_apply_kernel(const int32_t* in, int64_t n,
                                                                  const int32_t* __restrict__ sums, int32_t* out) {
  __shared__ int32_t sw[33];
  const int64_t base = (int64_t)blockIdx.x * (SCAN_THREADS * 4);
  int32_t v[4], tot = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int64_t j = base + (int64_t)threadIdx.x * 4 + i;
    v[i] = (j < n) ? in[j] : 0;
    tot += v[i];
  }
  int32_t ex = block_exclusive_scan(tot, sw, nullptr) + sums[blockIdx.x];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int64_t j = base + (int64_t)threadIdx.x * 4 + i;
    if (j < n) out[j] = ex;
    ex += v[i];
  }
}

// ---- stable scatter of one digit --------------------------------------------------------
// Warp w of a block owns 32*RS_ITEMS consecutive keys and visits them 32 at a time, so that
// (block, warp, round, lane) order is position order.  The rank of a key among equal digits:
// global offset of (digit, block) + keys of that digit in earlier warps + earlier rounds of
// this warp + earlier lanes of this round.
__global__ void __launch_bounds__(RS_THREADS) radix_scatter_kernel(const int32_t* __restrict__ keys_in,
                                                                   const int32_t* __restrict__ vals_in, int64_t P,
                                                                   int shift, int32_t n_items, int check_range,
                                                                   int nblocks,
                                                                   const int32_t* __restrict__ offsets,
                                                                   int32_t* __restrict__ keys_out,
                                                                   int32_t* __restrict__ vals_out) {
  __shared__ int32_t cnt[RS_WARPS][256];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int i = threadIdx.x; i < RS_WARPS * 256; i += RS_THREADS) (&cnt[0][0])[i] = 0;
  __syncthreads();
  const int64_t wbase = (int64_t)blockIdx.x * RS_TILE + (int64_t)warp * (32 * RS_ITEMS);
  int32_t key[RS_ITEMS];
  int32_t rank[RS_ITEMS];
  const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
  for (int r = 0; r < RS_ITEMS; ++r) {
    int64_t j = wbase + r * 32 + lane;
    bool valid = j < P;
    key[r] = valid ? keys_in[j] : 0;
    if (check_range && (key[r] < 0 || key[r] >= n_items)) key[r] = 0;   // counted as 0 by the histogram too
    int dig = valid ? ((key[r] >> shift) & 255) : 256;          // 256: past the end, never counted
    uint32_t peers = __match_any_sync(0xffffffffu, dig);
    int32_t before = 0;
    if (valid) before = cnt[warp][dig];
    __syncwarp();
    rank[r] = before + __popc(peers & lt);
    if (valid && (peers & lt) == 0) cnt[warp][dig] = before + __popc(peers);
    __syncwarp();
  }
  __syncthreads();
  {  // per digit: exclusive scan over the warps, seeded with the global offset of (digit, block)
    const int dig = threadIdx.x;
    int32_t run = offsets[(int64_t)dig * nblocks + blockIdx.x];
#pragma unroll
    for (int w = 0; w < RS_WARPS; ++w) {
      int32_t c = cnt[w][dig];
      cnt[w][dig] = run;
      run += c;
    }
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < RS_ITEMS; ++r) {
    int64_t j = wbase + r * 32 + lane;
    if (j < P) {
      int dig = (key[r] >> shift) & 255;
      int32_t dst = cnt[warp][dig] + rank[r];
      keys_out[dst] = key[r];
      vals_out[dst] = vals_in ? vals_in[j] : (int32_t)j;
    }
  }
}

// ---- run-length pass over the sorted keys -------------------------------------------------
__global__ void __launch_bounds__(SCAN_THREADS) rle_count_kernel(const int32_t* __restrict__ sk, int64_t P,
                                                                 int32_t* __restrict__ sums) {
  __shared__ int32_t sw[32];
  const int64_t base = (int64_t)blockIdx.x * (SCAN_THREADS * 4);
  int32_t v = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int64_t j = base + (int64_t)threadIdx.x * 4 + i;
    if (j < P) v += (j == 0 || sk[j] != sk[j - 1]) ? 1 : 0;
  }
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) sw[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x < 32) {
    v = sw[threadIdx.x];
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    if (threadIdx.x == 0) sums[blockIdx.x] = v;
  }
}

__global__ void __launch_bounds__(SCAN_THREADS) rle_write_kernel(const int32_t* __restrict__ sk, int64_t P,
                                                                 const int32_t* __restrict__ sums,
                                                                 const int32_t* __restrict__ n_unique,
                                                                 int32_t* __restrict__ unique,
                                                                 int32_t* __restrict__ seg_off,
                                                                 int32_t* __restrict__ rank_table) {
  __shared__ int32_t sw[33];
  const int64_t base = (int64_t)blockIdx.x * (SCAN_THREADS * 4);
  int32_t h[4], k[4], tot = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int64_t j = base + (int64_t)threadIdx.x * 4 + i;
    h[i] = 0;
    k[i] = 0;
    if (j < P) {
      k[i] = sk[j];
      h[i] = (j == 0 || k[i] != sk[j - 1]) ? 1 : 0;
    }
    tot += h[i];
  }
  int32_t ex = block_exclusive_scan(tot, sw, nullptr) + sums[blockIdx.x];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int64_t j = base + (int64_t)threadIdx.x * 4 + i;
    if (h[i]) {
      unique[ex] = k[i];
      seg_off[ex] = (int32_t)j;
      rank_table[k[i]] = ex;
      ++ex;
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) seg_off[*n_unique] = (int32_t)P;
}

__global__ void inverse_kernel(const int32_t* __restrict__ ids, int64_t P, int32_t n_items,
                               const int32_t* __restrict__ rank_table, int32_t* __restrict__ inverse) {
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < P; p += (int64_t)gridDim.x * blockDim.x) {
    int32_t id = ids[p];
    inverse[p] = (id >= 0 && id < n_items) ? rank_table[id] : -1;      // out of range: already recorded
  }
}

__global__ void dedup_empty_kernel(int32_t* seg_off, int32_t* n_unique) {
  seg_off[0] = 0;
  *n_unique = 0;
}

}  // namespace

gram_status index_ws_alloc(gram_ctx* ctx, IndexWorkspace* ws, int64_t P_max, int32_t n_items_max, int32_t d_max) {
  ws->P_max = P_max;
  ws->n_items_max = n_items_max;
  ws->d_max = d_max;
  ws->n_sort_blocks = (int32_t)ceil_div64(P_max > 0 ? P_max : 1, RS_TILE);
  const size_t pb = (size_t)(P_max > 0 ? P_max : 1) * sizeof(int32_t);
  GRAM_CUDA(ctx, cudaMalloc(&ws->keys0, pb));
  GRAM_CUDA(ctx, cudaMalloc(&ws->keys1, pb));
  GRAM_CUDA(ctx, cudaMalloc(&ws->vals0, pb));
  GRAM_CUDA(ctx, cudaMalloc(&ws->vals1, pb));
  GRAM_CUDA(ctx, cudaMalloc(&ws->hist, (size_t)256 * ws->n_sort_blocks * sizeof(int32_t)));
  size_t nsums = (size_t)ceil_div64((int64_t)256 * ws->n_sort_blocks, SCAN_THREADS * 4) +
                 (size_t)ceil_div64(P_max > 0 ? P_max : 1, SCAN_THREADS * 4) + 8;
  GRAM_CUDA(ctx, cudaMalloc(&ws->block_sums, nsums * sizeof(int32_t)));
  GRAM_CUDA(ctx, cudaMalloc(&ws->rank_table, (size_t)(n_items_max > 0 ? n_items_max : 1) * sizeof(int32_t)));
  GRAM_CUDA(ctx, cudaMalloc(&ws->partial, ((size_t)kAccMaxChunks * 2 * (d_max > 0 ? d_max : 1) + 2 * kAccMaxChunks) * sizeof(float)));
  return GRAM_OK;
}

void index_ws_free(IndexWorkspace* ws) {
  cudaFree(ws->keys0); cudaFree(ws->keys1); cudaFree(ws->vals0); cudaFree(ws->vals1);
  cudaFree(ws->hist); cudaFree(ws->block_sums); cudaFree(ws->rank_table); cudaFree(ws->partial);
  *ws = IndexWorkspace();
}

gram_status dedup_launch(gram_ctx* ctx, IndexWorkspace* ws, const int32_t* d_ids, int64_t P, int32_t n_items,
                         int32_t* d_unique, int32_t* d_inverse, int32_t* d_perm, int32_t* d_seg_off,
                         int32_t* d_n_unique, cudaStream_t st) {
  if (P < 0 || n_items <= 0 || !d_unique || !d_inverse || !d_perm || !d_seg_off || !d_n_unique || (P > 0 && !d_ids))
    return gram_set_error(ctx, "gram_dedup: bad argument"), GRAM_ERR_ARG;
  if (P > ws->P_max || n_items > ws->n_items_max || P > INT32_MAX)
    return gram_set_error(ctx, "gram_dedup: P=%lld n_items=%d exceed the context's P_max=%lld n_items=%d",
                          (long long)P, n_items, (long long)ws->P_max, ws->n_items_max), GRAM_ERR_WORKSPACE;
  if (P == 0) {
    dedup_empty_kernel<<<1, 1, 0, st>>>(d_seg_off, d_n_unique);
    GRAM_LAUNCH_CHECK(ctx);
    return GRAM_OK;
  }
  int bits = 0;
  while (((int64_t)1 << bits) < (int64_t)n_items) ++bits;
  const int passes = bits == 0 ? 1 : (bits + 7) / 8;
  const int nblocks = (int)ceil_div64(P, RS_TILE);
  const int64_t nh = (int64_t)256 * nblocks;
  const int nh_tiles = (int)ceil_div64(nh, SCAN_THREADS * 4);
  int32_t* status = gram_status_word(ctx);
  ProfScope prof(ctx, GRAM_K_DEDUP, (16.0 * passes + 20.0) * (double)P, 5 * passes + 4, st);

  const int32_t* kin = d_ids;

  const int32_t* vin = nullptr;
  int32_t* kbuf[2] = {ws->keys0, ws->keys1};
  int32_t* vbuf[2] = {ws->vals0, ws->vals1};
  for (int p = 0; p < passes; ++p) {
    int32_t* kout = kbuf[p & 1];
    int32_t* vout = (p == passes - 1) ? d_perm : vbuf[p & 1];
    radix_hist_kernel<<<nblocks, RS_THREADS, 0, st>>>(kin, P, 8 * p, n_items, p == 0, nblocks, ws->hist, status);
    scan_reduce_kernel<<<nh_tiles, SCAN_THREADS, 0, st>>>(ws->hist, nh, ws->block_sums);
    scan_sums_kernel<<<1, SCAN_THREADS, 0, st>>>(ws->block_sums, nh_tiles, nullptr);
    scan_apply_kernel<<<nh_tiles, SCAN_THREADS, 0, st>>>(ws->hist, nh, ws->block_sums, ws->hist);
    radix_scatter_kernel<<<nblocks, RS_THREADS, 0, st>>>(kin, vin, P, 8 * p, n_items, p == 0, nblocks, ws->hist, kout,
                                                         vout);
    kin = kout;
    vin = vout;
  }
  GRAM_LAUNCH_CHECK(ctx);
  const int ntiles = (int)ceil_div64(P, SCAN_THREADS * 4);
  rle_count_kernel<<<ntiles, SCAN_THREADS, 0, st>>>(kin, P, ws->block_sums);
  scan_sums_kernel<<<1, SCAN_THREADS, 0, st>>>(ws->block_sums, ntiles, d_n_unique);
  rle_write_kernel<<<ntiles, SCAN_THREADS, 0, st>>>(kin, P, ws->block_sums, d_n_unique, d_unique, d_seg_off,
                                                    ws->rank_table);
  int ib = (int)ceil_div64(P, 256);
  if (ib > kNumSMs * 16) ib = kNumSMs * 16;
  inverse_kernel<<<ib, 256, 0, st>>>(d_ids, P, n_items, ws->rank_table, d_inverse);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
