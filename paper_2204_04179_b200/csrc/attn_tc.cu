// Attention on the 5th-generation tensor cores (bf16 operands, head width 64): softmax(Q K^T / sqrt(dh)) V per
// (sequence, head), forward and backward.  HBM-bound by design: every tile of Q, K, V (and dO) is read once and every
// result written once, in whole 128-byte rows.
//
// Tiling.  All products run on 128-row tiles.  Sequences of up to 128 rows are packed into a tile in SLOTS of 8, 16,
// 32, 64 or 128 rows (the smallest power of two that holds the launch's longest sequence): slot k of a tile holds one
// sequence in tile rows k * slot .., fetched by its own bulk tensor copy from wherever that sequence's rows are
// (packed rows have no alignment; the rows a slot fetches beyond its sequence belong to the next sequence or are the
// zero fill past the matrix, and are masked).  The score tile S = Q K^T is then block diagonal: row r only looks at
// the columns of its own slot, the others are never read from tensor memory and their probabilities are written as
// zeros.  Sequences longer than 128 rows take one tile per 128 queries and loop over 128-row key tiles with a running
// maximum and sum (forward), resp. one pass per key tile and one per query tile (backward).
//
// Roles of a block (persistent, one per SM): warp 0 issues the bulk tensor copies, warp 1 issues the MMAs, warps 2-5
// and 6-9 are two softmax groups of 128 threads (thread = tile row = tensor-memory lane).  The groups take the block's
// work items alternately, each with its own score / output accumulators in tensor memory and its own probability
// tile in shared memory, so that one group's softmax overlaps the other's products and stores.  Every wait is an
// mbarrier wait with a time limit; a wait that runs out records GRAM_ERR_TIMEOUT, raises the block's abort flag, and
// every role leaves through the common exit that frees tensor memory.
#include <stdlib.h>

#include "layers.h"
#include "tc_common.cuh"

namespace {
using namespace tc;

constexpr int TQ = 128;                       // rows of a tile
constexpr int DH = 64;                        // head width
constexpr int TILE_BYTES = TQ * DH * 2;       // one 128 x 64 bf16 tile: 128-byte rows, 128-byte swizzle
constexpr int FWD_STAGES = 3;
constexpr int FWD_STAGE_BYTES = 3 * TILE_BYTES;               // Q, K, V
constexpr int P_BYTES = 2 * TILE_BYTES;                       // a 128 x 128 bf16 tile as two 64-column halves
constexpr int FWD_SMEM = FWD_STAGES * FWD_STAGE_BYTES + 2 * P_BYTES + 1024 /*alignment*/ + 256 /*barriers*/;
constexpr int ATT_THREADS = 64 + 256;

struct AttnArgs {
  bf16* out;                 // forward: ctx [T, d]
  float* lse;                // [H, T]: log2 of the softmax denominator plus the scaled maximum, per row and head
  int64_t T;                 // token rows in use
  int32_t n_seq, S, d, H, causal;
  int32_t slot;              // rows per slot (power of two), 128 in long mode
  int32_t box_rows;          // rows per bulk tensor copy (slot, or 128 when whole tiles are contiguous)
  int32_t long_mode;         // sequences of more than 128 rows
  int32_t nq_max;            // long mode: query tiles per sequence
  int64_t n_items;
  const int32_t* seq_len;
  const int32_t* seq_off;
  const int32_t* seq_list;
  float c;                   // scale * log2(e)
  int32_t* status;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
      "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
      "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tc_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// first row and length of the sequence with running number q of a launch (q >= n_seq: an empty slot)
__device__ __forceinline__ void seq_rows(const AttnArgs& a, int64_t q, int64_t& row0, int32_t& len) {
  if (q >= a.n_seq) { row0 = 0; len = 0; return; }
  const int64_t s = a.seq_list ? a.seq_list[q] : q;
  row0 = a.seq_off ? (int64_t)a.seq_off[s] : s * a.S;
  len = a.seq_len ? a.seq_len[s] : a.S;
}

// A work item: one 128-row query tile of one head.  Short mode: tile t holds sequences t*ns .. t*ns + ns - 1 in its
// slots and is its own (only) key tile.  Long mode: query tile qt of one sequence, key tiles 0 .. nk-1.
struct Item {
  int64_t tile;      // short: tile number; long: sequence number of the launch
  int32_t h, qt, nk;
};
__device__ __forceinline__ Item item_of(const AttnArgs& a, int64_t it) {
  Item x;
  x.h = (int32_t)(it % a.H);
  const int64_t r = it / a.H;
  if (!a.long_mode) {
    x.tile = r; x.qt = 0; x.nk = 1;
    return x;
  }
  x.qt = (int32_t)(r % a.nq_max);
  x.tile = r / a.nq_max;
  int64_t row0; int32_t len;
  seq_rows(a, x.tile, row0, len);
  if (x.qt * TQ >= len) x.nk = 0;                          // this sequence has no such query tile
  else x.nk = a.causal ? x.qt + 1 : (len + TQ - 1) / TQ;
  return x;
}

// Visible key columns [lo, hi) of key tile j for tile row r of an item; grow: the row's place in the token matrix,
// valid: the row belongs to a sequence.
struct RowInfo {
  int64_t grow;
  int32_t lo, limit;   // short: lo = first column of the row's slot, limit = visible keys counted from lo (all key tiles: j = 0)
                       // long: lo = 0, limit = visible keys counted from the sequence's first row
  bool valid;
};
__device__ __forceinline__ RowInfo row_info(const AttnArgs& a, const Item& x, int r) {
  RowInfo ri;
  int64_t row0; int32_t len;
  if (!a.long_mode) {
    const int ns = TQ / a.slot;
    const int k = r / a.slot, rl = r - k * a.slot;
    seq_rows(a, x.tile * ns + k, row0, len);
    ri.valid = rl < len;
    ri.grow = row0 + rl;
    ri.lo = k * a.slot;
    ri.limit = ri.valid ? (a.causal ? min(rl + 1, len) : len) : 0;
  } else {
    seq_rows(a, x.tile, row0, len);
    const int rl = x.qt * TQ + r;
    ri.valid = rl < len;
    ri.grow = row0 + rl;
    ri.lo = 0;
    ri.limit = ri.valid ? (a.causal ? min(rl + 1, len) : len) : 0;
  }
  return ri;
}
__device__ __forceinline__ void key_range(const AttnArgs& a, const RowInfo& ri, int j, int& lo, int& hi) {
  lo = ri.lo;
  hi = a.long_mode ? max(0, min(TQ, ri.limit - j * TQ)) : ri.lo + ri.limit;
}

// the bulk tensor copies that fill one 128 x 64 tile of matrix `which` (0 Q, 1 K, 2 V of qkv; 0 of a [T, d] matrix):
// tile rows come from token rows row0 .. in long mode, from the slots' sequences in short mode
__device__ __forceinline__ void load_tile(const AttnArgs& a, const CUtensorMap* map, uint32_t dst, int col, const Item& x,
                                          int tile_row_block /*long: 128-row block of the sequence*/, uint32_t bar) {
  if (a.long_mode) {
    int64_t row0; int32_t len;
    seq_rows(a, x.tile, row0, len);
    tma_load_2d(dst, map, col, (int32_t)(row0 + (int64_t)tile_row_block * TQ), bar);
    return;
  }
  const int ns = TQ / a.slot, spb = a.box_rows / a.slot;
  for (int b = 0; b * a.box_rows < TQ; ++b) {
    int64_t row0; int32_t len;
    seq_rows(a, x.tile * ns + b * spb, row0, len);
    tma_load_2d(dst + (uint32_t)(b * a.box_rows * 128), map, col, (int32_t)row0, bar);
  }
}

// 16 bytes of bf16 at tile row r, 16-byte piece `piece` (0..7) of a 128-byte row, as the 128-byte swizzle places it
__device__ __forceinline__ uint32_t swz(uint32_t base, int r, int piece) {
  return base + (uint32_t)r * 128u + ((uint32_t)(piece ^ (r & 7)) << 4);
}

constexpr uint32_t idesc(int M, int N, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
// D[128, N] (+)= A[128, K] B[N, K]^T over K = 16 * ksteps, A and B K-major 128 x 64 tiles (64 = one 128-byte row)
__device__ __forceinline__ void mma_kk(uint32_t tmem_d, uint32_t sa, uint32_t sb, int N, int ksteps, bool accumulate) {
  const uint32_t id = (N == 128) ? idesc(128, 128, false, false) : idesc(128, 64, false, false);
  for (int k = 0; k < ksteps; ++k)
    tc_mma(tmem_d, make_desc(sa + (uint32_t)((k >> 2) * TILE_BYTES + (k & 3) * 32), 16, 1024),
           make_desc(sb + (uint32_t)((k >> 2) * TILE_BYTES + (k & 3) * 32), 16, 1024), id, (accumulate || k > 0) ? 1u : 0u);
}
// D[128, 64] (+)= A[128, 128] B[128, 64]: A K-major (two 64-column halves), B a 128 x 64 tile read along its rows
__device__ __forceinline__ void mma_k_mn(uint32_t tmem_d, uint32_t sa, uint32_t sb, bool accumulate) {
  constexpr uint32_t id = idesc(128, 64, false, true);
  for (int k = 0; k < 8; ++k)
    tc_mma(tmem_d, make_desc(sa + (uint32_t)((k >> 2) * TILE_BYTES + (k & 3) * 32), 16, 1024),
           make_desc(sb + (uint32_t)(k * 2048), 8192, 1024), id, (accumulate || k > 0) ? 1u : 0u);
}
// D[128, 64] (+)= A^T B with A stored [128 k][128 m] (two 64-column halves, read along its rows) and B a 128 x 64 tile
// read along its rows
__device__ __forceinline__ void mma_mn_mn(uint32_t tmem_d, uint32_t sa, uint32_t sb, bool accumulate) {
  constexpr uint32_t id = idesc(128, 64, true, true);
  for (int k = 0; k < 8; ++k)
    tc_mma(tmem_d, make_desc(sa + (uint32_t)(k * 2048), TILE_BYTES, 1024), make_desc(sb + (uint32_t)(k * 2048), 8192, 1024), id,
           (accumulate || k > 0) ? 1u : 0u);
}

// ---- register-resident softmax blocks for tiles whose rows look at no more than W = 32 or 64 score columns ----
// (slots of up to 64 rows: a warp's 32 rows then share one window of W columns starting at cb)

// 16 bytes of zeros into every 16-byte piece of row r of a 128 x 128 bf16 tile (two halves) outside columns [cb, cb + W)
template <int W>
__device__ __forceinline__ void zero_outside(uint32_t buf, int r, int cb) {
#pragma unroll
  for (int piece = 0; piece < 16; ++piece) {
    const int col = piece * 8;
    if (col < cb || col >= cb + W) sts128(swz(buf + (uint32_t)(piece >> 3) * TILE_BYTES, r, piece & 7), 0u, 0u, 0u, 0u);
  }
}
// the 16 words pk (32 bf16 columns from column c0) into row r of such a tile
__device__ __forceinline__ void store_block32(uint32_t buf, int r, int c0, const uint32_t (&pk)[16]) {
  const int piece0 = c0 >> 3;
#pragma unroll
  for (int c4 = 0; c4 < 4; ++c4) {
    const int piece = piece0 + c4;
    sts128(swz(buf + (uint32_t)(piece >> 3) * TILE_BYTES, r, piece & 7), pk[4 * c4], pk[4 * c4 + 1], pk[4 * c4 + 2], pk[4 * c4 + 3]);
  }
}

// Forward: the scores of this thread's row in columns [cb, cb + W) of S (tensor memory) -> probabilities exp2(c s - c max)
// in the probability tile (zeros outside [lo, hi) and outside the window); returns the row maximum and the sum.
template <int W, bool full>
__device__ __forceinline__ void fwd_block_m(uint32_t s_addr, uint32_t pb, int r, int cb, int l0, int h0, float c, float& mx_out,
                                            float& sum_out) {
  constexpr int NB = W / 32;
  uint32_t v[NB][32];
#pragma unroll
  for (int i = 0; i < NB; ++i) tc_ld32_issue(s_addr + (uint32_t)(cb + 32 * i), v[i]);
#pragma unroll
  for (int i = 0; i < NB; ++i) tc_ld32_wait(v[i]);
  float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};          // four chains: the reductions are latency-bound otherwise
#pragma unroll
  for (int i = 0; i < NB; ++i)
#pragma unroll
    for (int e = 0; e < 32; ++e)
      if (full || (32 * i + e >= l0 && 32 * i + e < h0)) m4[e & 3] = fmaxf(m4[e & 3], __uint_as_float(v[i][e]));
  const float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
  const float mc = (mx == -INFINITY) ? 0.f : mx * c;
  float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int i = 0; i < NB; ++i) {
    uint32_t pk[16];
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
      const int k0 = 32 * i + e;
      const float p0 = (full || (k0 >= l0 && k0 < h0)) ? ex2(fmaf(__uint_as_float(v[i][e]), c, -mc)) : 0.f;
      const float p1 = (full || (k0 + 1 >= l0 && k0 + 1 < h0)) ? ex2(fmaf(__uint_as_float(v[i][e + 1]), c, -mc)) : 0.f;
      s4[(e >> 1) & 3] += p0 + p1;
      pk[e >> 1] = pack_bf16x2(p0, p1);
    }
    store_block32(pb, r, cb + 32 * i, pk);
  }
  zero_outside<W>(pb, r, cb);
  mx_out = mx;
  sum_out = (s4[0] + s4[1]) + (s4[2] + s4[3]);
}
// the unmasked variant when every row of the warp sees the whole window (equal-length sequences that fill their slots,
// no causal mask): the per-element range tests are then not even fetched
template <int W>
__device__ __forceinline__ void fwd_block(uint32_t s_addr, uint32_t pb, int r, int cb, int lo, int hi, float c, float& mx_out,
                                          float& sum_out) {
  const int l0 = lo - cb, h0 = hi - cb;
  if (__all_sync(0xffffffffu, l0 == 0 && h0 == W)) fwd_block_m<W, true>(s_addr, pb, r, cb, l0, h0, c, mx_out, sum_out);
  else fwd_block_m<W, false>(s_addr, pb, r, cb, l0, h0, c, mx_out, sum_out);
}

// Backward: S and dP of this thread's row in columns [cb, cb + W) -> P = exp2(c S - lse) and dS = P (dP - delta) scale, bf16,
// into the two tiles (zeros outside).  own_delta: delta is the row's sum of P dP (single key tile), else delta_in.
template <int W, bool full>
__device__ __forceinline__ void bwd_block_m(uint32_t lane_base, uint32_t pbuf, uint32_t dsbuf, int r, int cb, int l0, int h0, float c,
                                            float lse2, float scale, bool own_delta, float delta_in) {
  constexpr int NB = W / 32;
  uint32_t v[NB][32], w[NB][32];
#pragma unroll
  for (int i = 0; i < NB; ++i) {
    tc_ld32_issue(lane_base + (uint32_t)(cb + 32 * i), v[i]);
    tc_ld32_issue(lane_base + 128u + (uint32_t)(cb + 32 * i), w[i]);
  }
#pragma unroll
  for (int i = 0; i < NB; ++i) { tc_ld32_wait(v[i]); tc_ld32_wait(w[i]); }
  float d4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int i = 0; i < NB; ++i)
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      const int k0 = 32 * i + e;
      const float p = (full || (k0 >= l0 && k0 < h0)) ? ex2(fmaf(__uint_as_float(v[i][e]), c, -lse2)) : 0.f;
      v[i][e] = __float_as_uint(p);
      d4[e & 3] = fmaf(p, __uint_as_float(w[i][e]), d4[e & 3]);
    }
  const float delta = own_delta ? (d4[0] + d4[1]) + (d4[2] + d4[3]) : delta_in;
#pragma unroll
  for (int i = 0; i < NB; ++i) {
    uint32_t pk[16], dk[16];
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
      const float p0 = __uint_as_float(v[i][e]), p1 = __uint_as_float(v[i][e + 1]);
      pk[e >> 1] = pack_bf16x2(p0, p1);
      dk[e >> 1] = pack_bf16x2(p0 * scale * (__uint_as_float(w[i][e]) - delta), p1 * scale * (__uint_as_float(w[i][e + 1]) - delta));
    }
    store_block32(pbuf, r, cb + 32 * i, pk);
    store_block32(dsbuf, r, cb + 32 * i, dk);
  }
  zero_outside<W>(pbuf, r, cb);
  zero_outside<W>(dsbuf, r, cb);
}
template <int W>
__device__ __forceinline__ void bwd_block(uint32_t lane_base, uint32_t pbuf, uint32_t dsbuf, int r, int cb, int lo, int hi, float c,
                                          float lse2, float scale, bool own_delta, float delta_in) {
  const int l0 = lo - cb, h0 = hi - cb;
  if (__all_sync(0xffffffffu, l0 == 0 && h0 == W)) bwd_block_m<W, true>(lane_base, pbuf, dsbuf, r, cb, l0, h0, c, lse2, scale, own_delta, delta_in);
  else bwd_block_m<W, false>(lane_base, pbuf, dsbuf, r, cb, l0, h0, c, lse2, scale, own_delta, delta_in);
}

// ---- pieces of the general softmax path (windows of up to 128 columns, several key tiles): 32 columns at a time ----
// FULL: every row of the warp sees all 32 columns (no range tests)
template <bool FULL>
__device__ __forceinline__ void chunk_max(const uint32_t (&v)[32], int c0, int lo, int hi, float (&m4)[4]) {
#pragma unroll
  for (int e = 0; e < 32; ++e)
    if (FULL || (c0 + e >= lo && c0 + e < hi)) m4[e & 3] = fmaxf(m4[e & 3], __uint_as_float(v[e]));
}
// probabilities exp2(c s - off) of 32 columns, packed to bf16 in pk; their sum goes to s4
template <bool FULL>
__device__ __forceinline__ void chunk_exp(const uint32_t (&v)[32], int c0, int lo, int hi, float c, float off, uint32_t (&pk)[16],
                                          float (&s4)[4]) {
#pragma unroll
  for (int e = 0; e < 32; e += 2) {
    const float p0 = (FULL || (c0 + e >= lo && c0 + e < hi)) ? ex2(fmaf(__uint_as_float(v[e]), c, -off)) : 0.f;
    const float p1 = (FULL || (c0 + e + 1 >= lo && c0 + e + 1 < hi)) ? ex2(fmaf(__uint_as_float(v[e + 1]), c, -off)) : 0.f;
    s4[(e >> 1) & 3] += p0 + p1;
    pk[e >> 1] = pack_bf16x2(p0, p1);
  }
}

// ============================================================================================
// forward
// barriers: full[s], empty[s] per stage; per softmax group g: s_full[g] (scores in tensor memory),
// p_full[g] (probabilities in shared memory, one arrival per warp), pv_done[g] (output accumulator complete)
// tensor memory: S_g at columns 128 g, O_g at columns 256 + 64 g
// ============================================================================================
// WM: 32 or 64: short mode with slots of up to 32 / 64 rows (a row's scores fit a register-resident window); 128: the rest
template <int WM>
__global__ void __launch_bounds__(ATT_THREADS, 1) attn_tc_fwd_kernel(const __grid_constant__ CUtensorMap tm_qkv, AttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  const uint32_t pbuf = tiles + FWD_STAGES * FWD_STAGE_BYTES;
  const uint32_t bar0 = pbuf + 2 * P_BYTES;
  uint8_t* gen0 = smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen0 + FWD_STAGES * FWD_STAGE_BYTES + 2 * P_BYTES);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (FWD_STAGES + s); };
  auto sfull_bar = [&](int g) { return bar0 + 8u * (2 * FWD_STAGES + g); };
  auto pfull_bar = [&](int g) { return bar0 + 8u * (2 * FWD_STAGES + 2 + g); };
  auto pvdone_bar = [&](int g) { return bar0 + 8u * (2 * FWD_STAGES + 4 + g); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * FWD_STAGES + 6);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < FWD_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int g = 0; g < 2; ++g) { mbar_init(sfull_bar(g), 1); mbar_init(pfull_bar(g), 4); mbar_init(pvdone_bar(g), 1); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool failed = false;

  if (warp == 0) {
    // ------------------------------ bulk tensor copies ------------------------------
    if (lane == 0) {
      int64_t n = 0;
      for (int64_t it = blockIdx.x; it < a.n_items && !failed; it += gridDim.x) {
        const Item x = item_of(a, it);
        for (int j = 0; j < x.nk; ++j, ++n) {
          const int s = (int)(n % FWD_STAGES);
          if (!mbar_wait(empty_bar(s), (uint32_t)((n / FWD_STAGES) & 1) ^ 1u, abort_flag)) { failed = true; break; }
          mbar_expect_tx(full_bar(s), FWD_STAGE_BYTES);
          const uint32_t st = tiles + s * FWD_STAGE_BYTES;
          load_tile(a, &tm_qkv, st, x.h * DH, x, x.qt, full_bar(s));
          load_tile(a, &tm_qkv, st + TILE_BYTES, a.d + x.h * DH, x, j, full_bar(s));
          load_tile(a, &tm_qkv, st + 2 * TILE_BYTES, 2 * a.d + x.h * DH, x, j, full_bar(s));
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issue ------------------------------
    if (lane == 0) {
      int64_t n = 0, ord = 0;
      int pend_stage[2] = {-1, -1};
      bool pend_acc[2] = {false, false};
      uint32_t pcount[2] = {0, 0};
      auto issue_pv = [&](int g) -> bool {
        if (!mbar_wait(pfull_bar(g), pcount[g] & 1u, abort_flag)) return false;
        ++pcount[g];
        tc_fence_after();
        const uint32_t st = tiles + pend_stage[g] * FWD_STAGE_BYTES;
        mma_k_mn(tmem_base + 256u + 64u * g, pbuf + g * P_BYTES, st + 2 * TILE_BYTES, pend_acc[g]);
        tc_commit(pvdone_bar(g));
        tc_commit(empty_bar(pend_stage[g]));
        pend_stage[g] = -1;
        return true;
      };
      for (int64_t it = blockIdx.x; it < a.n_items && !failed; it += gridDim.x) {
        const Item x = item_of(a, it);
        if (x.nk == 0) continue;
        const int g = (int)(ord & 1);
        ++ord;
        for (int j = 0; j < x.nk; ++j, ++n) {
          if (pend_stage[g] >= 0 && !issue_pv(g)) { failed = true; break; }
          const int s = (int)(n % FWD_STAGES);
          if (!mbar_wait(full_bar(s), (uint32_t)((n / FWD_STAGES) & 1), abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t st = tiles + s * FWD_STAGE_BYTES;
          mma_kk(tmem_base + 128u * g, st, st + TILE_BYTES, 128, 4, false);          // S = Q K^T
          tc_commit(sfull_bar(g));
          pend_stage[g] = s;
          pend_acc[g] = j > 0;
        }
      }
      for (int g = 0; g < 2 && !failed; ++g)
        if (pend_stage[g] >= 0 && !issue_pv(g)) failed = true;
    }
  } else {
    // ------------------------------ softmax groups ------------------------------
    const int g = (warp - 2) >> 2;                 // group 0: warps 2-5, group 1: warps 6-9
    const int quarter = warp & 3;                  // the tensor-memory lanes this warp may touch
    const int r = quarter * 32 + lane;             // tile row of this thread
    const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t s_addr = lane_base + 128u * g, o_addr = lane_base + 256u + 64u * g;
    const uint32_t pb = pbuf + g * P_BYTES;
    int64_t ord = 0;
    uint32_t k = 0;                                // steps this group has taken (barrier phases)
    for (int64_t it = blockIdx.x; it < a.n_items && !failed; it += gridDim.x) {
      const Item x = item_of(a, it);
      if (x.nk == 0) continue;
      const bool mine = (ord & 1) == g;
      ++ord;
      if (!mine) continue;
      const RowInfo ri = row_info(a, x, r);
      float m_run = -INFINITY, l_run = 0.f;
      for (int j = 0; j < x.nk && !failed; ++j, ++k) {
        int lo, hi;
        key_range(a, ri, j, lo, hi);
        if (!mbar_wait(sfull_bar(g), k & 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        if constexpr (WM <= 64) {
          // one key tile and a window of at most 64 columns per row: everything stays in registers
          float mx, sum;
          fwd_block<WM>(s_addr, pb, r, WM * ((quarter * 32) / WM), lo, hi, a.c, mx, sum);
          m_run = mx;
          l_run = sum;
        } else {
        // the 32-column blocks some row of this warp needs
        const int wlo = __reduce_min_sync(0xffffffffu, hi > lo ? lo : TQ), whi = __reduce_max_sync(0xffffffffu, hi > lo ? hi : 0);
        const int q0 = wlo >> 5, q1 = (whi + 31) >> 5;     // blocks [q0, q1)
        // the whole window visible to every row of the warp (inner key tiles of long sequences): no per-element tests
        const bool full = __all_sync(0xffffffffu, lo == 0 && hi == TQ);
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        for (int q = q0; q < q1; ++q) {
          uint32_t v[32];
          tc_ld32_issue(s_addr + 32u * q, v);
          tc_ld32_wait(v);
          if (full) chunk_max<true>(v, 32 * q, lo, hi, m4);
          else chunk_max<false>(v, 32 * q, lo, hi, m4);
        }
        const float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        const float m_new = fmaxf(m_run, mx);
        const float mc = (m_new == -INFINITY) ? 0.f : m_new * a.c;
        const float alpha = (m_run == -INFINITY) ? 0.f : ex2(m_run * a.c - mc);
        if (j > 0) {
          // the previous key tile's product must be complete before its accumulator is rescaled and before the
          // probability tile it reads is overwritten
          if (!mbar_wait(pvdone_bar(g), (k - 1) & 1u, abort_flag)) { failed = true; break; }
          tc_fence_after();
#pragma unroll 1
          for (int hblk = 0; hblk < 2; ++hblk) {
            uint32_t v[32];
            tc_ld32_issue(o_addr + 32u * hblk, v);
            tc_ld32_wait(v);
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * alpha);
            tc_st32(o_addr + 32u * hblk, v);
          }
          tc_st_wait();
        }
        float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
        for (int q = 0; q < 4; ++q) {
          uint32_t pk[16];
          if (q >= q0 && q < q1) {
            uint32_t v[32];
            tc_ld32_issue(s_addr + 32u * q, v);
            tc_ld32_wait(v);
            if (full) chunk_exp<true>(v, 32 * q, lo, hi, a.c, mc, pk, s4);
            else chunk_exp<false>(v, 32 * q, lo, hi, a.c, mc, pk, s4);
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) pk[e] = 0u;
          }
          const uint32_t half = pb + (uint32_t)(q >> 1) * TILE_BYTES;
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4)
            sts128(swz(half, r, (q & 1) * 4 + c4), pk[4 * c4], pk[4 * c4 + 1], pk[4 * c4 + 2], pk[4 * c4 + 3]);
        }
        const float sum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
        l_run = l_run * alpha + sum;
        m_run = m_new;
        }
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(pfull_bar(g));      // one arrival per warp: 128 would serialise on the barrier word
      }
      if (failed) break;
      // ---- the item's output: O / l, bf16, through this warp's rows of the probability tile, in whole rows ----
      if (!mbar_wait(pvdone_bar(g), (k - 1) & 1u, abort_flag)) { failed = true; break; }
      tc_fence_after();
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      {
        uint32_t o[2][32];
        tc_ld32_issue(o_addr, o[0]);
        tc_ld32_issue(o_addr + 32u, o[1]);
        tc_ld32_wait(o[0]);
        tc_ld32_wait(o[1]);
#pragma unroll
        for (int hblk = 0; hblk < 2; ++hblk)
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4)
            sts128(swz(pb, r, hblk * 4 + c4),
                   pack_bf16x2(__uint_as_float(o[hblk][8 * c4]) * inv, __uint_as_float(o[hblk][8 * c4 + 1]) * inv),
                   pack_bf16x2(__uint_as_float(o[hblk][8 * c4 + 2]) * inv, __uint_as_float(o[hblk][8 * c4 + 3]) * inv),
                   pack_bf16x2(__uint_as_float(o[hblk][8 * c4 + 4]) * inv, __uint_as_float(o[hblk][8 * c4 + 5]) * inv),
                   pack_bf16x2(__uint_as_float(o[hblk][8 * c4 + 6]) * inv, __uint_as_float(o[hblk][8 * c4 + 7]) * inv));
      }
      tc_fence_before();
      if (a.lse && ri.valid) a.lse[(int64_t)x.h * a.T + ri.grow] = m_run * a.c + lg2(l_run);
      __syncwarp();
      // eight lanes per row, four rows per instruction
      const int piece = lane & 7, sub = lane >> 3;
#pragma unroll
      for (int rr = 0; rr < 8; ++rr) {
        const int row_l = rr * 4 + sub;                      // row within this warp's 32
        const int64_t grow = __shfl_sync(0xffffffffu, ri.grow, row_l);
        const int ok = __shfl_sync(0xffffffffu, (int)ri.valid, row_l);
        const uint4 val = lds128(swz(pb, quarter * 32 + row_l, piece));
        if (ok) *reinterpret_cast<uint4*>(a.out + grow * a.d + x.h * DH + piece * 8) = val;
      }
      __syncwarp();
    }
    if (failed && lane == 0) {
      *abort_flag = 1;
      gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
    }
  }
  if (failed && warp < 2 && lane == 0) {
    *abort_flag = 1;
    gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
  }

  // ------------------------------ exit ------------------------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // a wait gave up: let copies and MMAs already issued drain (bounded) before shared and tensor memory go
    if (threadIdx.x == 0) {
      const uint64_t t0 = clock64();
      while (clock64() - t0 < WAIT_LIMIT_CYCLES / 64) {}
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ============================================================================================
// backward
// One pair step = one 128-row query tile i against one 128-row key tile j of a head: S = Q_i K_j^T and
// dP = dO_i V_j^T into tensor memory; the softmax group turns them into P = exp2(c S - lse) and
// dS = P (dP - delta) / sqrt(dh), bf16, in shared memory; then dV_j += P^T dO_i, dK_j += dS^T Q_i, dQ_i += dS K_j.
//   mode 0 (sequences of up to 128 rows): one pair step per item, all three results; delta = sum_j P dP of the row.
//   mode 1 (longer sequences): an item is a key tile and walks the query tiles that see it: dK, dV.
//   mode 2: an item is a query tile and walks its key tiles: dQ.  Modes 1 and 2 read delta = dO . O per row from memory.
// barriers: full[s], empty[s] (four arrivals: the MMA thread's commits for a step inside an item, the group's four warps
// after the item's last step, because the results leave through the stage's own tiles); per group g: sdp_full, pds_full
// (one arrival per warp), out_full, out_free, csum (one per warp).
// tensor memory: S 0..127, dP 128..255, dV 256..319, dK 320..383, dQ 384..447
// ============================================================================================
constexpr int BWD_STAGES = 2;
constexpr int BWD_STAGE_BYTES = 4 * TILE_BYTES;               // Q, K, V, dO
constexpr int BWD_PART_BYTES = 2 * 3 * 4 * 64 * 4;            // per group, matrix and warp: 64 partial column sums
constexpr int BWD_SMEM = BWD_STAGES * BWD_STAGE_BYTES + 2 * P_BYTES + BWD_PART_BYTES + 1024 + 256;

struct AttnBwdArgs {
  AttnArgs f;                // geometry shared with the forward pass (out and lse: the saved row statistics)
  bf16* dqkv;                // [T, 3d]
  const float* delta;        // [H, T], modes 1 and 2
  float* colpart;            // [tiles, 3d] partial column sums of dqkv, or null
  int64_t colpart_row0;      // first row of this launch's tiles in colpart
  int32_t mode;
  float scale;               // 1 / sqrt(dh)
};

// pair steps of an item: query tile qi(t) and key tile kj(t) for t = 0 .. n-1; out_tile: the tile whose rows the item writes
struct BwdItem {
  Item x;
  int32_t n, first;          // number of pair steps; first walking index
};
__device__ __forceinline__ BwdItem bwd_item_of(const AttnBwdArgs& b, int64_t it) {
  BwdItem y;
  y.x = item_of(b.f, it);
  y.first = 0;
  if (b.mode == 0) { y.n = 1; return y; }
  if (y.x.nk == 0) { y.n = 0; return y; }     // no such tile in this sequence
  int64_t row0; int32_t len;
  seq_rows(b.f, y.x.tile, row0, len);
  const int nt = (len + TQ - 1) / TQ;
  if (b.mode == 1) {                           // x.qt is the key tile; query tiles first .. nt-1
    y.first = b.f.causal ? y.x.qt : 0;
    y.n = nt - y.first;
  } else {                                     // x.qt is the query tile; key tiles 0 .. nk-1
    y.n = y.x.nk;
  }
  return y;
}

template <int WM>
__global__ void __launch_bounds__(ATT_THREADS, 1) attn_tc_bwd_kernel(const __grid_constant__ CUtensorMap tm_qkv,
                                                                     const __grid_constant__ CUtensorMap tm_do, AttnBwdArgs b) {
  const AttnArgs& a = b.f;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  const uint32_t pbuf = tiles + BWD_STAGES * BWD_STAGE_BYTES, dsbuf = pbuf + P_BYTES;
  const uint32_t part0 = dsbuf + P_BYTES;
  const uint32_t bar0 = part0 + BWD_PART_BYTES;
  uint8_t* gen0 = smem_raw + (tiles - raw);
  float* part = reinterpret_cast<float*>(gen0 + BWD_STAGES * BWD_STAGE_BYTES + 2 * P_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen0 + BWD_STAGES * BWD_STAGE_BYTES + 2 * P_BYTES + BWD_PART_BYTES);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (BWD_STAGES + s); };
  auto sdp_bar = [&](int g) { return bar0 + 8u * (2 * BWD_STAGES + g); };
  auto pds_bar = [&](int g) { return bar0 + 8u * (2 * BWD_STAGES + 2 + g); };
  auto outfull_bar = [&](int g) { return bar0 + 8u * (2 * BWD_STAGES + 4 + g); };
  auto outfree_bar = [&](int g) { return bar0 + 8u * (2 * BWD_STAGES + 6 + g); };
  auto csum_bar = [&](int g) { return bar0 + 8u * (2 * BWD_STAGES + 8 + g); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * BWD_STAGES + 10);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < BWD_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 4); }
    for (int g = 0; g < 2; ++g) {
      mbar_init(sdp_bar(g), 1); mbar_init(pds_bar(g), 4); mbar_init(outfull_bar(g), 1); mbar_init(outfree_bar(g), 4);
      mbar_init(csum_bar(g), 4);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool failed = false;
  const bool want_kv = b.mode != 2, want_q = b.mode != 1;

  if (warp == 0) {
    // ------------------------------ bulk tensor copies ------------------------------
    if (lane == 0) {
      int64_t n = 0;
      for (int64_t it = blockIdx.x; it < a.n_items && !failed; it += gridDim.x) {
        const BwdItem y = bwd_item_of(b, it);
        for (int t = 0; t < y.n; ++t, ++n) {
          const int qi = b.mode == 1 ? y.first + t : y.x.qt, kj = b.mode == 2 ? t : y.x.qt;
          const int s = (int)(n % BWD_STAGES);
          if (!mbar_wait(empty_bar(s), (uint32_t)((n / BWD_STAGES) & 1) ^ 1u, abort_flag)) { failed = true; break; }
          mbar_expect_tx(full_bar(s), BWD_STAGE_BYTES);
          const uint32_t st = tiles + s * BWD_STAGE_BYTES;
          load_tile(a, &tm_qkv, st, y.x.h * DH, y.x, qi, full_bar(s));
          load_tile(a, &tm_qkv, st + TILE_BYTES, a.d + y.x.h * DH, y.x, kj, full_bar(s));
          load_tile(a, &tm_qkv, st + 2 * TILE_BYTES, 2 * a.d + y.x.h * DH, y.x, kj, full_bar(s));
          load_tile(a, &tm_do, st + 3 * TILE_BYTES, y.x.h * DH, y.x, qi, full_bar(s));
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issue ------------------------------
    if (lane == 0) {
      int64_t n = 0, ord = 0;
      uint32_t steps[2] = {0, 0}, items[2] = {0, 0};
      int prev_g = -1;
      for (int64_t it = blockIdx.x; it < a.n_items && !failed; it += gridDim.x) {
        const BwdItem y = bwd_item_of(b, it);
        if (y.n == 0) continue;
        const int g = (int)(ord & 1);
        ++ord;
        for (int t = 0; t < y.n; ++t, ++n) {
          const int s = (int)(n % BWD_STAGES);
          if (!mbar_wait(full_bar(s), (uint32_t)((n / BWD_STAGES) & 1), abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t st = tiles + s * BWD_STAGE_BYTES;
          mma_kk(tmem_base, st, st + TILE_BYTES, 128, 4, false);                                   // S = Q K^T
          mma_kk(tmem_base + 128u, st + 3 * TILE_BYTES, st + 2 * TILE_BYTES, 128, 4, false);      // dP = dO V^T
          tc_commit(sdp_bar(g));
          if (!mbar_wait(pds_bar(g), steps[g] & 1u, abort_flag)) { failed = true; break; }
          ++steps[g];
          if (t == 0 && prev_g >= 0) {             // the previous item's results have been read out of tensor memory
            if (!mbar_wait(outfree_bar(prev_g), (items[prev_g] - 1) & 1u, abort_flag)) { failed = true; break; }
          }
          tc_fence_after();
          if (want_kv) {
            mma_mn_mn(tmem_base + 256u, pbuf, st + 3 * TILE_BYTES, t > 0);                        // dV += P^T dO
            mma_mn_mn(tmem_base + 320u, dsbuf, st, t > 0);                                        // dK += dS^T Q
          }
          if (want_q) mma_k_mn(tmem_base + 384u, dsbuf, st + TILE_BYTES, t > 0);                  // dQ += dS K
          if (t + 1 < y.n) {
            for (int k4 = 0; k4 < 4; ++k4) tc_commit(empty_bar(s));   // the stage is free once these products are done
          } else {
            tc_commit(outfull_bar(g));
            ++items[g];
            prev_g = g;
          }
        }
      }
    }
  } else {
    // ------------------------------ softmax groups ------------------------------
    const int g = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
    float* mypart = part + g * (3 * 4 * 64);
    int64_t ord = 0, n = 0;
    uint32_t k = 0, ki = 0;                         // pair steps and items this group has taken
    for (int64_t it = blockIdx.x; it < a.n_items && !failed; it += gridDim.x) {
      const BwdItem y = bwd_item_of(b, it);
      if (y.n == 0) continue;
      const bool mine = (ord & 1) == g;
      ++ord;
      if (!mine) { n += y.n; continue; }
      int last_stage = 0;
      for (int t = 0; t < y.n && !failed; ++t, ++k, ++n) {
        last_stage = (int)(n % BWD_STAGES);
        Item xq = y.x;                               // the query tile of this pair step
        xq.qt = b.mode == 1 ? y.first + t : y.x.qt;
        const int kj = b.mode == 2 ? t : y.x.qt;
        const RowInfo ri = row_info(a, xq, r);
        int lo, hi;
        key_range(a, ri, kj, lo, hi);
        const int wlo = __reduce_min_sync(0xffffffffu, hi > lo ? lo : TQ), whi = __reduce_max_sync(0xffffffffu, hi > lo ? hi : 0);
        const int q0 = wlo >> 5, q1 = (whi + 31) >> 5;
        const float lse2 = ri.valid ? a.lse[(int64_t)y.x.h * a.T + ri.grow] : 0.f;
        float delta = (b.mode != 0 && ri.valid) ? b.delta[(int64_t)y.x.h * a.T + ri.grow] : 0.f;
        if (!mbar_wait(sdp_bar(g), k & 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        if constexpr (WM <= 64) {
          bwd_block<WM>(lane_base, pbuf, dsbuf, r, WM * ((quarter * 32) / WM), lo, hi, a.c, lse2, b.scale, true, 0.f);
        } else {
        // pass 1: P (bf16, to shared memory) and, in mode 0, delta = sum_j P dP
        float dsum = 0.f;
#pragma unroll 1
        for (int q = 0; q < 4; ++q) {
          uint32_t pk[16];
          if (q >= q0 && q < q1) {
            uint32_t v[32], w[32];
            tc_ld32_issue(lane_base + 32u * q, v);
            tc_ld32_issue(lane_base + 128u + 32u * q, w);
            tc_ld32_wait(v);
            tc_ld32_wait(w);
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const int cidx = 32 * q + e;
              const float p0 = (cidx >= lo && cidx < hi) ? ex2(fmaf(__uint_as_float(v[e]), a.c, -lse2)) : 0.f;
              const float p1 = (cidx + 1 >= lo && cidx + 1 < hi) ? ex2(fmaf(__uint_as_float(v[e + 1]), a.c, -lse2)) : 0.f;
              dsum = fmaf(p0, __uint_as_float(w[e]), dsum);
              dsum = fmaf(p1, __uint_as_float(w[e + 1]), dsum);
              pk[e >> 1] = pack_bf16x2(p0, p1);
            }
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) pk[e] = 0u;
          }
          const uint32_t half = pbuf + (uint32_t)(q >> 1) * TILE_BYTES;
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4)
            sts128(swz(half, r, (q & 1) * 4 + c4), pk[4 * c4], pk[4 * c4 + 1], pk[4 * c4 + 2], pk[4 * c4 + 3]);
        }
        if (b.mode == 0) delta = dsum;
        // pass 2: dS = P (dP - delta) / sqrt(dh), with P as it was rounded
#pragma unroll 1
        for (int q = 0; q < 4; ++q) {
          uint32_t pk[16];
          if (q >= q0 && q < q1) {
            uint32_t w[32];
            tc_ld32_issue(lane_base + 128u + 32u * q, w);
            const uint32_t half = pbuf + (uint32_t)(q >> 1) * TILE_BYTES;
            uint4 pp[4];
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) pp[c4] = lds128(swz(half, r, (q & 1) * 4 + c4));
            tc_ld32_wait(w);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
              const uint32_t pw[4] = {pp[c4].x, pp[c4].y, pp[c4].z, pp[c4].w};
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float2 p2 = unpack_bf16x2(pw[i]);
                const int e = 8 * c4 + 2 * i;
                pk[4 * c4 + i] = pack_bf16x2(p2.x * (__uint_as_float(w[e]) - delta) * b.scale,
                                            p2.y * (__uint_as_float(w[e + 1]) - delta) * b.scale);
              }
            }
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) pk[e] = 0u;
          }
          const uint32_t half = dsbuf + (uint32_t)(q >> 1) * TILE_BYTES;
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4)
            sts128(swz(half, r, (q & 1) * 4 + c4), pk[4 * c4], pk[4 * c4 + 1], pk[4 * c4 + 2], pk[4 * c4 + 3]);
        }
        }
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(pds_bar(g));
      }
      if (failed) break;
      // ---- the item's results: bf16, through the (no longer read) tiles of the item's last stage, in whole rows ----
      if (!mbar_wait(outfull_bar(g), ki & 1u, abort_flag)) { failed = true; break; }
      ++ki;
      tc_fence_after();
      const RowInfo ro = row_info(a, y.x, r);          // the rows this item writes (its query tile, resp. key tile)
      const uint32_t st = tiles + last_stage * BWD_STAGE_BYTES;
      // which: 0 dQ (over the Q tile), 1 dK (over K), 2 dV (over V); tensor-memory columns 384, 320, 256
#pragma unroll 1
      for (int which = 0; which < 3; ++which) {
        if ((which == 0 && !want_q) || (which > 0 && !want_kv)) continue;
        const uint32_t tcol = which == 0 ? 384u : (which == 1 ? 320u : 256u);
        const uint32_t dst = st + (uint32_t)which * TILE_BYTES;
        uint32_t o[2][32];
        tc_ld32_issue(lane_base + tcol, o[0]);
        tc_ld32_issue(lane_base + tcol + 32u, o[1]);
        tc_ld32_wait(o[0]);
        tc_ld32_wait(o[1]);
#pragma unroll
        for (int hblk = 0; hblk < 2; ++hblk) {
          if (!ro.valid) {
#pragma unroll
            for (int e = 0; e < 32; ++e) o[hblk][e] = 0u;
          }
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4)
            sts128(swz(dst, r, hblk * 4 + c4),
                   pack_bf16x2(__uint_as_float(o[hblk][8 * c4]), __uint_as_float(o[hblk][8 * c4 + 1])),
                   pack_bf16x2(__uint_as_float(o[hblk][8 * c4 + 2]), __uint_as_float(o[hblk][8 * c4 + 3])),
                   pack_bf16x2(__uint_as_float(o[hblk][8 * c4 + 4]), __uint_as_float(o[hblk][8 * c4 + 5])),
                   pack_bf16x2(__uint_as_float(o[hblk][8 * c4 + 6]), __uint_as_float(o[hblk][8 * c4 + 7])));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(outfree_bar(g));      // tensor memory may take the next item's results
      const int piece = lane & 7, sub = lane >> 3;
#pragma unroll 1
      for (int which = 0; which < 3; ++which) {
        if ((which == 0 && !want_q) || (which > 0 && !want_kv)) continue;
        const uint32_t src = st + (uint32_t)which * TILE_BYTES;
#pragma unroll
        for (int rr = 0; rr < 8; ++rr) {
          const int row_l = rr * 4 + sub;
          const int64_t grow = __shfl_sync(0xffffffffu, ro.grow, row_l);
          const int ok = __shfl_sync(0xffffffffu, (int)ro.valid, row_l);
          const uint4 val = lds128(swz(src, quarter * 32 + row_l, piece));
          if (ok) *reinterpret_cast<uint4*>(b.dqkv + grow * 3 * (int64_t)a.d + (int64_t)which * a.d + y.x.h * DH + piece * 8) = val;
        }
        if (b.colpart) {
          // this warp's 32 rows (rows outside a sequence hold zeros), columns 2 lane and 2 lane + 1, rows ascending
          float s0 = 0.f, s1 = 0.f;
          const int pc = lane >> 2, wd = (lane & 3) * 4;
#pragma unroll 8
          for (int rr = 0; rr < 32; ++rr) {
            const int row = quarter * 32 + rr;
            uint32_t w;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(swz(src, row, pc) + (uint32_t)wd) : "memory");
            const float2 f = unpack_bf16x2(w);
            s0 += f.x;
            s1 += f.y;
          }
          *reinterpret_cast<float2*>(mypart + (which * 4 + quarter) * 64 + 2 * lane) = make_float2(s0, s1);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(last_stage));      // this warp no longer touches the stage's tiles
      if (b.colpart) {
        if (lane == 0) mbar_arrive(csum_bar(g));       // after the __syncwarp above: this warp's partial sums are written
        if (!mbar_wait(csum_bar(g), (ki - 1) & 1u, abort_flag)) { failed = true; break; }
        // the four warps' sums in warp order: 192 columns, two per thread
        const int t2 = threadIdx.x - 64 - g * 128;            // 0..127 within the group
        if (t2 < 96) {
          const int which = t2 >> 5, c2 = (t2 & 31) * 2;
          if (!((which == 0 && !want_q) || (which > 0 && !want_kv))) {
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int qq = 0; qq < 4; ++qq) {
              const float2 f = *reinterpret_cast<const float2*>(mypart + (which * 4 + qq) * 64 + c2);
              s0 += f.x;
              s1 += f.y;
            }
            const int64_t prow = b.colpart_row0 + (a.long_mode ? y.x.tile * a.nq_max + y.x.qt : y.x.tile);
            *reinterpret_cast<float2*>(b.colpart + prow * 3 * (int64_t)a.d + (int64_t)which * a.d + y.x.h * DH + c2) = make_float2(s0, s1);
          }
        }
      }
    }
    if (failed && lane == 0) {
      *abort_flag = 1;
      gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
    }
  }
  if (failed && warp < 2 && lane == 0) {
    *abort_flag = 1;
    gram_device_fail(a.status, GRAM_ERR_TIMEOUT);
  }

  // ------------------------------ exit ------------------------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      const uint64_t t0 = clock64();
      while (clock64() - t0 < WAIT_LIMIT_CYCLES / 64) {}
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// delta[h, row] = sum_c dO[row, h*64 + c] * O[row, h*64 + c]: the row term of the softmax derivative, for the passes over
// long sequences (one warp per row, two columns per lane and head)
__global__ void __launch_bounds__(256) attn_delta_kernel(const bf16* __restrict__ dO, const bf16* __restrict__ O, float* __restrict__ delta,
                                                         int64_t T, int d, int H) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5, nw = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t row = warp; row < T; row += nw) {
    for (int h = 0; h < H; ++h) {
      const float2 x = unpack_bf16x2(*reinterpret_cast<const uint32_t*>(dO + row * d + h * DH + 2 * lane));
      const float2 o = unpack_bf16x2(*reinterpret_cast<const uint32_t*>(O + row * d + h * DH + 2 * lane));
      float v = x.x * o.x + x.y * o.y;
      for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      if (lane == 0) delta[(int64_t)h * T + row] = v;
    }
  }
}

// slot size, box height and item count of a launch whose longest sequence has S rows
void plan_launch(AttnArgs& a, int64_t n_seq, int S, bool contiguous) {
  a.long_mode = S > TQ;
  if (a.long_mode) {
    a.slot = TQ;
    a.box_rows = TQ;
    a.nq_max = (S + TQ - 1) / TQ;
    a.n_items = n_seq * a.nq_max * a.H;
  } else {
    int slot = 8;
    while (slot < S) slot <<= 1;
    a.slot = slot;
    a.box_rows = (contiguous && slot == S) ? TQ : slot;      // whole tiles of equal-length sequences are one copy
    a.nq_max = 1;
    const int ns = TQ / slot;
    a.n_items = ((n_seq + ns - 1) / ns) * a.H;
  }
}

}  // namespace

// Which sequences take these kernels: GRAM_ATTN_TC=1 in the environment: all (head width 64); GRAM_ATTN_TC=0: none;
// unset: sequences of more than 64 rows.  Up to 64 rows the warp-level kernels keep several small blocks per SM resident
// and hide memory latency by occupancy, which one persistent block per SM does not (measured on the knowledge-tracing
// encoder: 5.9 + 16.2 ms per step against 6.9 + 19.0 ms); from 65 rows on their one-sequence tile fills an SM with a
// single block, and beyond 128 rows they cannot hold a sequence at all.
bool attention_tc_supported(int S, int d, int n_heads) {
  static const int mode = []() { const char* v = getenv("GRAM_ATTN_TC"); return !v ? 2 : (v[0] == '0' ? 0 : 1); }();
  if (mode == 0 || !(S >= 1 && n_heads > 0 && d == n_heads * DH && get_encode_fn() != nullptr)) return false;
  return mode == 1 || S > 64;
}

gram_status attention_forward_tc(gram_ctx* ctx, const void* qkv, void* out, float* lse, int64_t rows, int64_t n_seq, int S, int d,
                                 int n_heads, int causal, const int32_t* seq_len, const int32_t* seq_off, const int32_t* seq_list,
                                 cudaStream_t st) {
  if (n_seq == 0) return GRAM_OK;
  if (rows <= 0 || rows >= ((int64_t)1 << 31)) return gram_set_error(ctx, "attention: row count out of range"), GRAM_ERR_ARG;
  AttnArgs a = {};
  a.out = (bf16*)out; a.lse = lse; a.T = rows; a.n_seq = (int32_t)n_seq; a.S = S; a.d = d; a.H = n_heads; a.causal = causal;
  a.seq_len = seq_len; a.seq_off = seq_off; a.seq_list = seq_list;
  a.c = 1.4426950408889634f / sqrtf((float)DH);
  a.status = gram_status_word(ctx);
  plan_launch(a, n_seq, S, !seq_off && !seq_list);
  CUtensorMap tm;
  if (!make_map(&tm, qkv, (uint64_t)3 * d, (uint64_t)rows, (uint64_t)3 * d, DH, (uint32_t)a.box_rows))
    return gram_set_error(ctx, "attention: cuTensorMapEncodeTiled failed"), GRAM_ERR_CUDA;
  static bool attr_set = false;
  if (!attr_set) {
    GRAM_CUDA(ctx, cudaFuncSetAttribute(attn_tc_fwd_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM));
    GRAM_CUDA(ctx, cudaFuncSetAttribute(attn_tc_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM));
    GRAM_CUDA(ctx, cudaFuncSetAttribute(attn_tc_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM));
    attr_set = true;
  }
  const int grid = (int)(a.n_items < kNumSMs ? a.n_items : kNumSMs);
  if (!a.long_mode && a.slot <= 32) attn_tc_fwd_kernel<32><<<grid, ATT_THREADS, FWD_SMEM, st>>>(tm, a);
  else if (!a.long_mode && a.slot == 64) attn_tc_fwd_kernel<64><<<grid, ATT_THREADS, FWD_SMEM, st>>>(tm, a);
  else attn_tc_fwd_kernel<128><<<grid, ATT_THREADS, FWD_SMEM, st>>>(tm, a);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

// rows of the partial-sum matrix the backward pass of n_seq sequences of up to S rows fills (one per tile)
int64_t attention_tc_colpart_rows(int64_t n_seq, int S) {
  if (S > TQ) return n_seq * ((S + TQ - 1) / TQ);
  int slot = 8;
  while (slot < S) slot <<= 1;
  const int ns = TQ / slot;
  return (n_seq + ns - 1) / ns;
}

gram_status attention_backward_tc(gram_ctx* ctx, const void* qkv, const void* dctx, const void* octx, const float* lse, float* delta,
                                  void* dqkv, float* colpart, int64_t colpart_row0, int64_t rows, int64_t n_seq, int S, int d,
                                  int n_heads, int causal, const int32_t* seq_len, const int32_t* seq_off, const int32_t* seq_list,
                                  cudaStream_t st) {
  if (n_seq == 0) return GRAM_OK;
  if (rows <= 0 || rows >= ((int64_t)1 << 31)) return gram_set_error(ctx, "attention: row count out of range"), GRAM_ERR_ARG;
  if (!lse) return gram_set_error(ctx, "attention backward: the forward pass's row statistics are missing"), GRAM_ERR_ARG;
  AttnBwdArgs b = {};
  AttnArgs& a = b.f;
  a.out = nullptr; a.lse = const_cast<float*>(lse); a.T = rows; a.n_seq = (int32_t)n_seq; a.S = S; a.d = d; a.H = n_heads; a.causal = causal;
  a.seq_len = seq_len; a.seq_off = seq_off; a.seq_list = seq_list;
  a.c = 1.4426950408889634f / sqrtf((float)DH);
  a.status = gram_status_word(ctx);
  plan_launch(a, n_seq, S, !seq_off && !seq_list);
  b.dqkv = (bf16*)dqkv; b.delta = delta; b.colpart = colpart; b.colpart_row0 = colpart_row0; b.scale = 1.f / sqrtf((float)DH);
  CUtensorMap tq, td;
  if (!make_map(&tq, qkv, (uint64_t)3 * d, (uint64_t)rows, (uint64_t)3 * d, DH, (uint32_t)a.box_rows) ||
      !make_map(&td, dctx, (uint64_t)d, (uint64_t)rows, (uint64_t)d, DH, (uint32_t)a.box_rows))
    return gram_set_error(ctx, "attention: cuTensorMapEncodeTiled failed"), GRAM_ERR_CUDA;
  static bool attr_set = false;
  if (!attr_set) {
    GRAM_CUDA(ctx, cudaFuncSetAttribute(attn_tc_bwd_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, BWD_SMEM));
    GRAM_CUDA(ctx, cudaFuncSetAttribute(attn_tc_bwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BWD_SMEM));
    GRAM_CUDA(ctx, cudaFuncSetAttribute(attn_tc_bwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BWD_SMEM));
    attr_set = true;
  }
  const int grid = (int)(a.n_items < kNumSMs ? a.n_items : kNumSMs);
  if (!a.long_mode) {
    b.mode = 0;
    if (a.slot <= 32) attn_tc_bwd_kernel<32><<<grid, ATT_THREADS, BWD_SMEM, st>>>(tq, td, b);
    else if (a.slot == 64) attn_tc_bwd_kernel<64><<<grid, ATT_THREADS, BWD_SMEM, st>>>(tq, td, b);
    else attn_tc_bwd_kernel<128><<<grid, ATT_THREADS, BWD_SMEM, st>>>(tq, td, b);
  } else {
    if (!delta || !octx) return gram_set_error(ctx, "attention backward: long sequences need the forward output and a scratch row vector"), GRAM_ERR_ARG;
    int blocks = (int)((rows + 7) / 8);
    if (blocks > kNumSMs * 8) blocks = kNumSMs * 8;
    attn_delta_kernel<<<blocks, 256, 0, st>>>((const bf16*)dctx, (const bf16*)octx, delta, rows, d, n_heads);
    if (colpart)      // tiles a sequence does not have leave their rows unwritten
      GRAM_CUDA(ctx, cudaMemsetAsync(colpart + colpart_row0 * 3 * (int64_t)d, 0, (size_t)(n_seq * a.nq_max) * 3 * d * sizeof(float), st));
    b.mode = 1;
    attn_tc_bwd_kernel<128><<<grid, ATT_THREADS, BWD_SMEM, st>>>(tq, td, b);
    b.mode = 2;
    attn_tc_bwd_kernel<128><<<grid, ATT_THREADS, BWD_SMEM, st>>>(tq, td, b);
  }
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}
