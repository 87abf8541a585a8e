// Stage 1 of the GRAM step: the unique-item set B_I of a mini-batch (Table 1) and the
// occurrence -> item map of Fig. 1, as a stable LSD radix sort of (item ID, position) over
// the low ceil(log2 n_items) key bits followed by a run-length pass.
//
// One launch per 8-bit radix pass: a block takes the next tile of 8192 keys (a ticket, so that
// every earlier tile is already running), ranks its keys within the tile, publishes the tile's
// digit counts and obtains the counts of all earlier tiles by looking back over their status
// words (the chained-scan idea of Merrill & Garland's decoupled look-back, as used by one-sweep
// radix sorts), then reorders the tile by digit in shared memory so that every digit leaves as
// one contiguous run.  Traffic per pass: 8P read + 8P written (the first pass generates the
// position payload instead of reading it); the digit totals of all passes come from one read of
// the keys before the first pass.  The run-length pass is one launch of the same kind.
//
// Every wait on another tile is bounded: a tile that gives up records GRAM_ERR_TIMEOUT, releases
// its successors and writes nothing; every scattered write is bounds-checked.
#include "gram_internal.h"

namespace {

constexpr int RADIX = 256;
constexpr int RS_THREADS = 512;
constexpr int RS_ITEMS = 16;
constexpr int RS_TILE = RS_THREADS * RS_ITEMS;   // keys per tile
constexpr int RS_WARPS = RS_THREADS / 32;
constexpr int kMaxPasses = 4;
constexpr int RLE_THREADS = 512;
constexpr int RLE_ITEMS = 16;
constexpr int RLE_TILE = RLE_THREADS * RLE_ITEMS;
constexpr int TOT_THREADS = 512;

// status word of a (tile, digit): two flag bits above a 30-bit count
constexpr uint32_t LB_AGG = 1u << 30;      // the tile's own count
constexpr uint32_t LB_INCL = 2u << 30;     // the count of this tile and all earlier ones
constexpr uint32_t LB_MASK = LB_AGG - 1u;
constexpr int kSpinLimit = 1 << 20;        // polls of one predecessor before giving up (about a second)

// control block (32-bit words), cleared by one memset per call:
// tickets of the radix passes, ticket of the run-length pass, digit totals [kMaxPasses][256],
// then the status words of every pass and of the run-length pass
constexpr int CTL_TICKET = 0, CTL_RLE_TICKET = 4, CTL_TOTALS = 8, CTL_WORDS = CTL_TOTALS + kMaxPasses * RADIX;

__device__ __forceinline__ uint32_t lb_load(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void lb_store(uint32_t* p, uint32_t v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Publishes `own` for (tile, slot) and returns in *excl the sum of `own` over all earlier tiles.
// A word carries its flag and its count together, so no ordering between two stores is needed.
// The words of LB_WINDOW predecessors are fetched at once (independent loads), so a look-back of
// depth n costs about n / LB_WINDOW round trips to L2.
// false: a predecessor never published within the limit (the caller must then write nothing).
constexpr int LB_WINDOW = 8;
__device__ __forceinline__ bool lookback_prefix(uint32_t* lb, int tile, int stride, int slot, uint32_t own, uint32_t* excl) {
  uint32_t* mine = lb + (size_t)tile * stride + slot;
  *excl = 0;
  if (tile == 0) {
    lb_store(mine, own | LB_INCL);
    return true;
  }
  lb_store(mine, own | LB_AGG);
  uint32_t sum = 0;
  int spins = 0;
  int t = tile - 1;
  while (true) {
    uint32_t w[LB_WINDOW];
#pragma unroll
    for (int i = 0; i < LB_WINDOW; ++i)
      w[i] = (t - i >= 0) ? lb_load(lb + (size_t)(t - i) * stride + slot) : LB_INCL;   // before tile 0: nothing
    int used = 0;
    bool done = false;
#pragma unroll
    for (int i = 0; i < LB_WINDOW; ++i) {
      if (!done && used == i && (w[i] & ~LB_MASK) != 0u) {
        sum += w[i] & LB_MASK;
        used = i + 1;
        done = (w[i] & LB_INCL) != 0u;
      }
    }
    if (done) break;
    t -= used;
    if (used < LB_WINDOW) {                 // tile t has not published yet
      if (++spins > kSpinLimit) {
        lb_store(mine, LB_INCL);            // let the tiles after this one finish (their output is void as well)
        return false;
      }
      __nanosleep(40);
    }
  }
  lb_store(mine, ((sum + own) & LB_MASK) | LB_INCL);
  *excl = sum;
  return true;
}

// The same for one word per tile, by a whole warp: lane l inspects tile - 1 - l of the current window.
__device__ __forceinline__ bool lookback_prefix_warp(uint32_t* lb, int tile, uint32_t own, uint32_t* excl) {
  const int lane = threadIdx.x & 31;
  uint32_t* mine = lb + tile;
  *excl = 0;
  if (tile == 0) {
    if (lane == 0) lb_store(mine, own | LB_INCL);
    return true;
  }
  if (lane == 0) lb_store(mine, own | LB_AGG);
  uint32_t sum = 0;
  int spins = 0;
  int t = tile - 1;
  while (true) {
    const uint32_t w = (t - lane >= 0) ? lb_load(lb + (t - lane)) : LB_INCL;
    const uint32_t ready = __ballot_sync(0xffffffffu, (w & ~LB_MASK) != 0u);
    const uint32_t incl = __ballot_sync(0xffffffffu, (w & LB_INCL) != 0u);
    const int n_ready = __ffs(~ready) - 1;                    // leading lanes that have published (-1: all 32)
    const int first_incl = __ffs(incl) - 1;                   // -1: none
    int take = n_ready < 0 ? 32 : n_ready;                    // lanes 0..take-1 are consumed
    bool done = false;
    if (first_incl >= 0 && first_incl < take) { take = first_incl + 1; done = true; }
    uint32_t v = lane < take ? (w & LB_MASK) : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    sum += v;
    if (done) break;
    t -= take;
    if (take < 32) {
      if (++spins > kSpinLimit) {
        if (lane == 0) lb_store(mine, LB_INCL);
        return false;
      }
      __nanosleep(40);
    }
  }
  if (lane == 0) lb_store(mine, ((sum + own) & LB_MASK) | LB_INCL);
  *excl = sum;
  return true;
}

// ---- digit totals of every pass from one read of the keys; range check of the IDs -----------
// Shared-memory histograms in TOT_COPIES interleaved copies (a lane adds to copy lane % TOT_COPIES):
// the occurrences of a hot item inside a warp spread over the copies, which sit in different banks.
constexpr int TOT_COPIES = 8;
__global__ void __launch_bounds__(TOT_THREADS) digit_totals_kernel(const int32_t* __restrict__ keys, int64_t P, int passes,
                                                                   int32_t n_items, uint32_t* __restrict__ totals,
                                                                   int32_t* status) {
  __shared__ uint32_t sh[kMaxPasses * RADIX * TOT_COPIES];
  for (int i = threadIdx.x; i < passes * RADIX * TOT_COPIES; i += TOT_THREADS) sh[i] = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int copy = lane & (TOT_COPIES - 1);
  constexpr int UNROLL = 4;
  const int64_t stride = (int64_t)gridDim.x * TOT_THREADS * UNROLL;
  bool bad = false;
  // a warp reads UNROLL runs of 32 consecutive keys per iteration (independent loads)
  for (int64_t j0 = ((int64_t)blockIdx.x * TOT_THREADS + (threadIdx.x & ~31)) * UNROLL; j0 < P; j0 += stride) {
    int32_t k[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int64_t j = j0 + u * 32 + lane;
      k[u] = (j < P) ? keys[j] : -1;
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      if (j0 + u * 32 + lane < P) {
        if (k[u] < 0 || k[u] >= n_items) { bad = true; k[u] = 0; }
        for (int p = 0; p < passes; ++p) atomicAdd(&sh[(p * RADIX + ((k[u] >> (8 * p)) & 255)) * TOT_COPIES + copy], 1u);
      }
    }
  }
  if (bad) gram_device_fail(status, GRAM_ERR_ID_RANGE);
  __syncthreads();
  for (int i = threadIdx.x; i < passes * RADIX; i += TOT_THREADS) {
    uint32_t c = 0;
#pragma unroll
    for (int q = 0; q < TOT_COPIES; ++q) c += sh[i * TOT_COPIES + q];
    if (c) atomicAdd(&totals[i], c);
  }
}

// exclusive scan over threads 0..255 of two values at once (threads 256.. pass zeros); all threads call
__device__ __forceinline__ int2 scan256_pair(int a, int b, int32_t (*sw)[8]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int ta = __shfl_up_sync(0xffffffffu, ia, o), tb = __shfl_up_sync(0xffffffffu, ib, o);
    if (lane >= o) { ia += ta; ib += tb; }
  }
  if (warp < 8 && lane == 31) { sw[0][warp] = ia; sw[1][warp] = ib; }
  __syncthreads();
  int pa = 0, pb = 0;
  for (int w = 0; w < 8; ++w)
    if (w < warp) { pa += sw[0][w]; pb += sw[1][w]; }
  return make_int2(pa + ia - a, pb + ib - b);
}

struct PassSmem {
  uint16_t cnt[RS_WARPS][RADIX];   // keys of (warp, digit); later the warp's base inside the tile's digit run
  int32_t tile_excl[RADIX];        // start of a digit's run inside the reordered tile
  int32_t gbase[RADIX];            // global position of reordered element i of digit g is gbase[g] + i
  int32_t scan_w[2][8];
  int32_t tile, abort;
  int32_t keys[RS_TILE];
  int32_t vals[RS_TILE];
};

// ---- one stable radix pass ------------------------------------------------------------------
// Warp w of a tile owns 32*RS_ITEMS consecutive keys and visits them 32 at a time, so that
// (tile, warp, round, lane) order is position order.  The rank of a key among equal digits:
// all earlier tiles + earlier warps of this tile + earlier rounds of this warp + earlier lanes.
template <int NBITS>
__global__ void __launch_bounds__(RS_THREADS, 2) radix_pass_kernel(const int32_t* __restrict__ keys_in,
                                                                   const int32_t* __restrict__ vals_in, int64_t P, int shift,
                                                                   int32_t n_items, int check_range,
                                                                   const uint32_t* __restrict__ totals, uint32_t* lb,
                                                                   int32_t* ticket, int32_t* __restrict__ keys_out,
                                                                   int32_t* __restrict__ vals_out, int32_t* status) {
  extern __shared__ __align__(16) unsigned char pass_smem_raw[];
  PassSmem& s = *reinterpret_cast<PassSmem*>(pass_smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s.tile = atomicAdd(ticket, 1);
    s.abort = 0;
  }
  for (int i = tid; i < RS_WARPS * RADIX / 2; i += RS_THREADS) reinterpret_cast<uint32_t*>(&s.cnt[0][0])[i] = 0u;
  __syncthreads();
  const int tile = s.tile;
  const int64_t tbase = (int64_t)tile * RS_TILE;
  const int64_t left = P - tbase;
  const int n_valid = left < RS_TILE ? (int)left : RS_TILE;      // keys of this tile
  const int lbase = warp * (32 * RS_ITEMS) + lane;               // this lane's first key inside the tile
  const int32_t* kin = keys_in + tbase;
  int32_t key[RS_ITEMS];
  int32_t pos[RS_ITEMS];
#pragma unroll
  for (int r = 0; r < RS_ITEMS; ++r) {
    key[r] = (lbase + r * 32 < n_valid) ? kin[lbase + r * 32] : 0;
    if (check_range && (key[r] < 0 || key[r] >= n_items)) key[r] = 0;   // counted as 0 by the totals too
  }
  const uint32_t lt = (1u << lane) - 1u;
  uint16_t* my_cnt = s.cnt[warp];
#pragma unroll
  for (int r = 0; r < RS_ITEMS; ++r) {
    const bool valid = lbase + r * 32 < n_valid;
    const int dig = (key[r] >> shift) & 255;
    // lanes of this round with the same digit: one vote per digit bit that can be set in this pass (a fixed cost,
    // unlike a hardware match, whose latency grows with the number of distinct values)
    uint32_t peers = __ballot_sync(0xffffffffu, valid);
#pragma unroll
    for (int b = 0; b < NBITS; ++b) {
      const bool bit = (dig >> b) & 1;
      const uint32_t vote = __ballot_sync(0xffffffffu, bit);
      peers &= bit ? vote : ~vote;
    }
    int32_t before = 0;
    if (valid) before = my_cnt[dig];
    __syncwarp();
    pos[r] = before + __popc(peers & lt);
    if (valid && (peers & lt) == 0u) my_cnt[dig] = (uint16_t)(before + __popc(peers));
    __syncwarp();
  }
  __syncthreads();
  int32_t count = 0, tot = 0;
  if (tid < RADIX) {
    int32_t run = 0;
#pragma unroll
    for (int w = 0; w < RS_WARPS; ++w) {
      const int32_t c = s.cnt[w][tid];
      s.cnt[w][tid] = (uint16_t)run;
      run += c;
    }
    count = run;
    tot = (int32_t)totals[tid];
  }
  const int2 ex = scan256_pair(count, tot, s.scan_w);
  if (tid < RADIX) {
    s.tile_excl[tid] = ex.x;
    uint32_t before_tiles;
    if (!lookback_prefix(lb, tile, RADIX, tid, (uint32_t)count, &before_tiles)) {
      s.abort = 1;
      gram_device_fail(status, GRAM_ERR_TIMEOUT);
    }
    s.gbase[tid] = ex.y + (int32_t)before_tiles - ex.x;
  }
  __syncthreads();
  if (s.abort) return;
  // reorder the tile by digit in shared memory
#pragma unroll
  for (int r = 0; r < RS_ITEMS; ++r) {
    if (lbase + r * 32 < n_valid) {
      const int dig = (key[r] >> shift) & 255;
      pos[r] += s.tile_excl[dig] + my_cnt[dig];
      s.keys[pos[r]] = key[r];
    }
  }
  int32_t val[RS_ITEMS];
  const int32_t* vin = vals_in ? vals_in + tbase : nullptr;
#pragma unroll
  for (int r = 0; r < RS_ITEMS; ++r)
    val[r] = (vin && lbase + r * 32 < n_valid) ? vin[lbase + r * 32] : (int32_t)tbase + lbase + r * 32;
#pragma unroll
  for (int r = 0; r < RS_ITEMS; ++r)
    if (lbase + r * 32 < n_valid) s.vals[pos[r]] = val[r];
  __syncthreads();
  for (int i = tid; i < n_valid; i += RS_THREADS) {
    const int32_t k = s.keys[i];
    const uint32_t dst = (uint32_t)(s.gbase[(k >> shift) & 255] + i);
    if (dst < (uint32_t)P) {                 // always true unless an earlier tile gave up
      keys_out[dst] = k;
      vals_out[dst] = s.vals[i];
    }
  }
}

typedef void (*RadixPassFn)(const int32_t*, const int32_t*, int64_t, int, int32_t, int, const uint32_t*, uint32_t*, int32_t*,
                            int32_t*, int32_t*, int32_t*);
// the instantiation for a pass whose digits have `nbits` bits that can be set
RadixPassFn radix_pass_fn(int nbits) {
  switch (nbits) {
    case 1: return radix_pass_kernel<1>;
    case 2: return radix_pass_kernel<2>;
    case 3: return radix_pass_kernel<3>;
    case 4: return radix_pass_kernel<4>;
    case 5: return radix_pass_kernel<5>;
    case 6: return radix_pass_kernel<6>;
    case 7: return radix_pass_kernel<7>;
    default: return radix_pass_kernel<8>;
  }
}

// exclusive scan of one value per thread over the block; returns the thread's base
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

// ---- run-length pass over the sorted keys: unique, seg_off, item -> rank table, U -------------
__global__ void __launch_bounds__(RLE_THREADS) rle_kernel(const int32_t* __restrict__ sk, int64_t P, int ntiles, int32_t cap, int32_t n_items,
                                                          uint32_t* lb, int32_t* ticket, int32_t* __restrict__ unique,
                                                          int32_t* __restrict__ seg_off, int32_t* __restrict__ rank_table,
                                                          int32_t* __restrict__ n_unique, int32_t* status) {
  __shared__ int32_t sw[33];
  __shared__ int32_t s_tile, s_excl, s_abort;
  if (threadIdx.x == 0) {
    s_tile = atomicAdd(ticket, 1);
    s_abort = 0;
  }
  __syncthreads();
  const int tile = s_tile;
  const int64_t base = (int64_t)tile * RLE_TILE + (int64_t)threadIdx.x * RLE_ITEMS;
  int32_t k[RLE_ITEMS], tot = 0;
  uint32_t heads = 0;
  int32_t prev = (base > 0 && base <= P) ? sk[base - 1] : -1;           // IDs are non-negative
#pragma unroll
  for (int i = 0; i < RLE_ITEMS; ++i) {
    const int64_t j = base + i;
    k[i] = (j < P) ? sk[j] : prev;
    if (j < P && k[i] != prev) { heads |= 1u << i; ++tot; }
    prev = k[i];
  }
  int32_t btot;
  int32_t ex = block_exclusive_scan(tot, sw, &btot);
  if (threadIdx.x < 32) {
    uint32_t before_tiles;
    const bool ok = lookback_prefix_warp(lb, tile, (uint32_t)btot, &before_tiles);
    if (threadIdx.x == 0) {
      if (!ok) {
        s_abort = 1;
        gram_device_fail(status, GRAM_ERR_TIMEOUT);
      }
      s_excl = (int32_t)before_tiles;
    }
  }
  __syncthreads();
  if (s_abort) return;
  ex += s_excl;
#pragma unroll
  for (int i = 0; i < RLE_ITEMS; ++i) {
    if (heads & (1u << i)) {
      if (ex < cap && (uint32_t)k[i] < (uint32_t)n_items) {   // always true unless an earlier tile or pass gave up
        unique[ex] = k[i];
        seg_off[ex] = (int32_t)(base + i);
        rank_table[k[i]] = ex;
      }
      ++ex;
    }
  }
  if (tile == ntiles - 1 && threadIdx.x == 0) {
    const int32_t U = s_excl + btot;
    *n_unique = U;
    if (U <= cap) seg_off[U] = (int32_t)P;
  }
}

__global__ void __launch_bounds__(256) inverse_kernel(const int32_t* __restrict__ ids, int64_t P, int32_t n_items,
                                                      const int32_t* __restrict__ rank_table, int32_t* __restrict__ inverse) {
  constexpr int UNROLL = 4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x * UNROLL;
  for (int64_t p0 = (int64_t)blockIdx.x * blockDim.x * UNROLL + threadIdx.x; p0 < P; p0 += stride) {
    int32_t id[UNROLL], r[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int64_t p = p0 + (int64_t)u * blockDim.x;
      id[u] = (p < P) ? ids[p] : -1;
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) r[u] = (id[u] >= 0 && id[u] < n_items) ? rank_table[id[u]] : -1;   // out of range: already recorded
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int64_t p = p0 + (int64_t)u * blockDim.x;
      if (p < P) inverse[p] = r[u];
    }
  }
}

__global__ void dedup_empty_kernel(int32_t* seg_off, int32_t* n_unique) {
  seg_off[0] = 0;
  *n_unique = 0;
}

int radix_passes(int32_t n_items) {
  int bits = 0;
  while (((int64_t)1 << bits) < (int64_t)n_items) ++bits;
  return bits == 0 ? 1 : (bits + 7) / 8;
}

size_t ctl_words(int64_t P, int passes) {
  const int64_t p = P > 0 ? P : 1;
  return (size_t)CTL_WORDS + (size_t)passes * (size_t)ceil_div64(p, RS_TILE) * RADIX + (size_t)ceil_div64(p, RLE_TILE);
}

}  // namespace

gram_status index_ws_alloc(gram_ctx* ctx, IndexWorkspace* ws, int64_t P_max, int32_t n_items_max, int32_t d_max) {
  ws->P_max = P_max;
  ws->n_items_max = n_items_max;
  ws->d_max = d_max;
  const size_t pb = (size_t)(P_max > 0 ? P_max : 1) * sizeof(int32_t);
  GRAM_CUDA(ctx, cudaMalloc(&ws->keys0, pb));
  GRAM_CUDA(ctx, cudaMalloc(&ws->keys1, pb));
  GRAM_CUDA(ctx, cudaMalloc(&ws->vals0, pb));
  GRAM_CUDA(ctx, cudaMalloc(&ws->vals1, pb));
  GRAM_CUDA(ctx, cudaMalloc(&ws->sort_ctl, ctl_words(P_max, radix_passes(n_items_max > 0 ? n_items_max : 1)) * sizeof(uint32_t)));
  GRAM_CUDA(ctx, cudaMalloc(&ws->rank_table, (size_t)(n_items_max > 0 ? n_items_max : 1) * sizeof(int32_t)));
  GRAM_CUDA(ctx, cudaMalloc(&ws->partial, ((size_t)kAccMaxChunks * 2 * (d_max > 0 ? d_max : 1) + 2 * kAccMaxChunks) * sizeof(float)));
  for (int b = 1; b <= 8; ++b)
    GRAM_CUDA(ctx, cudaFuncSetAttribute(radix_pass_fn(b), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(PassSmem)));
  return GRAM_OK;
}

void index_ws_free(IndexWorkspace* ws) {
  cudaFree(ws->keys0); cudaFree(ws->keys1); cudaFree(ws->vals0); cudaFree(ws->vals1);
  cudaFree(ws->sort_ctl); cudaFree(ws->rank_table); cudaFree(ws->partial);
  *ws = IndexWorkspace();
}

// A wait that nothing satisfies, to show that it ends: the run-length kernel is launched as tile 1 of a
// one-key input whose tile 0 never runs, so its look-back finds no status word, gives up after kSpinLimit
// polls (about a second), records GRAM_ERR_TIMEOUT and writes nothing.
gram_status dedup_wait_selftest(gram_ctx* ctx, IndexWorkspace* ws, cudaStream_t st) {
  if (ws->P_max < 2) return gram_set_error(ctx, "the bounded-wait self-test needs a context with P_max >= 2"), GRAM_ERR_WORKSPACE;
  uint32_t* ctl = ws->sort_ctl;
  GRAM_CUDA(ctx, cudaMemsetAsync(ctl, 0, (size_t)(CTL_WORDS + 2) * sizeof(uint32_t), st));
  static const int32_t one = 1;
  GRAM_CUDA(ctx, cudaMemcpyAsync(reinterpret_cast<int32_t*>(ctl) + CTL_RLE_TICKET, &one, sizeof(one), cudaMemcpyHostToDevice, st));
  GRAM_CUDA(ctx, cudaMemsetAsync(ws->keys0, 0, sizeof(int32_t), st));
  rle_kernel<<<1, RLE_THREADS, 0, st>>>(ws->keys0, 1, 2, 1, 1, ctl + CTL_WORDS, reinterpret_cast<int32_t*>(ctl) + CTL_RLE_TICKET,
                                        ws->keys1, ws->vals0, ws->rank_table, ws->vals1, gram_status_word(ctx));
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status dedup_launch(gram_ctx* ctx, IndexWorkspace* ws, const int32_t* d_ids, int64_t P, int32_t n_items,
                         int32_t* d_unique, int32_t* d_inverse, int32_t* d_perm, int32_t* d_seg_off,
                         int32_t* d_n_unique, cudaStream_t st) {
  if (P < 0 || n_items <= 0 || !d_unique || !d_inverse || !d_perm || !d_seg_off || !d_n_unique || (P > 0 && !d_ids))
    return gram_set_error(ctx, "gram_dedup: bad argument"), GRAM_ERR_ARG;
  if (P > ws->P_max || n_items > ws->n_items_max)
    return gram_set_error(ctx, "gram_dedup: P=%lld n_items=%d exceed the context's P_max=%lld n_items=%d",
                          (long long)P, n_items, (long long)ws->P_max, ws->n_items_max), GRAM_ERR_WORKSPACE;
  if (P > (int64_t)LB_MASK)
    return gram_set_error(ctx, "gram_dedup: P=%lld is above the limit of 2^30 - 1 positions per call", (long long)P), GRAM_ERR_UNSUPPORTED;
  if (P == 0) {
    dedup_empty_kernel<<<1, 1, 0, st>>>(d_seg_off, d_n_unique);
    GRAM_LAUNCH_CHECK(ctx);
    return GRAM_OK;
  }
  const int passes = radix_passes(n_items);
  int key_bits = 0;
  while (((int64_t)1 << key_bits) < (int64_t)n_items) ++key_bits;
  const int ntiles = (int)ceil_div64(P, RS_TILE);
  const int rtiles = (int)ceil_div64(P, RLE_TILE);
  int32_t* status = gram_status_word(ctx);
  ProfScope prof(ctx, GRAM_K_DEDUP, (16.0 * passes + 20.0) * (double)P, passes + 3, st);

  uint32_t* ctl = ws->sort_ctl;
  GRAM_CUDA(ctx, cudaMemsetAsync(ctl, 0, ctl_words(P, passes) * sizeof(uint32_t), st));
  uint32_t* totals = ctl + CTL_TOTALS;
  uint32_t* lb = ctl + CTL_WORDS;
  int tb = (int)ceil_div64(P, (int64_t)TOT_THREADS * 16);
  if (tb > kNumSMs * 4) tb = kNumSMs * 4;
  digit_totals_kernel<<<tb, TOT_THREADS, 0, st>>>(d_ids, P, passes, n_items, totals, status);

  const int32_t* kin = d_ids;
  const int32_t* vin = nullptr;
  int32_t* kbuf[2] = {ws->keys0, ws->keys1};
  int32_t* vbuf[2] = {ws->vals0, ws->vals1};
  for (int p = 0; p < passes; ++p) {
    int32_t* kout = kbuf[p & 1];
    int32_t* vout = (p == passes - 1) ? d_perm : vbuf[p & 1];
    const int pass_bits = (key_bits - 8 * p) < 8 ? (key_bits - 8 * p < 1 ? 1 : key_bits - 8 * p) : 8;   // digit bits that can be set
    radix_pass_fn(pass_bits)<<<ntiles, RS_THREADS, sizeof(PassSmem), st>>>(kin, vin, P, 8 * p, n_items, p == 0, totals + p * RADIX,
                                                                          lb + (size_t)p * ntiles * RADIX,
                                                                          reinterpret_cast<int32_t*>(ctl) + CTL_TICKET + p,
                                                                          kout, vout, status);
    kin = kout;
    vin = vout;
  }
  GRAM_LAUNCH_CHECK(ctx);
  const int32_t cap = (int32_t)(P < (int64_t)n_items ? P : (int64_t)n_items);
  rle_kernel<<<rtiles, RLE_THREADS, 0, st>>>(kin, P, rtiles, cap, n_items, lb + (size_t)passes * ntiles * RADIX,
                                             reinterpret_cast<int32_t*>(ctl) + CTL_RLE_TICKET, d_unique, d_seg_off,
                                             ws->rank_table, d_n_unique, status);
  int ib = (int)ceil_div64(P, 256 * 4);
  if (ib > kNumSMs * 16) ib = kNumSMs * 16;
  inverse_kernel<<<ib, 256, 0, st>>>(d_ids, P, n_items, ws->rank_table, d_inverse);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
