// Stage 3 (gather encodings into sequence positions) and stage 4 (sum the per-position
// gradients of each item, Eq. 6; Multi-step: add them into the per-item table, Section 4.2).
// Both are HBM-bound: 128-bit accesses, a warp per row, several rows in flight per warp.
#include "gram_internal.h"

namespace {

// ---------------------------------------------------------------------------
// gather: E[p, :] = src[index[p], :]
// Algorithmic bytes: P*row written + (distinct rows)*row read + 4P index.
// ---------------------------------------------------------------------------
template <int ROWS>   // rows a warp keeps in flight
__global__ void __launch_bounds__(256) gather_rows_kernel(const uint4* __restrict__ src, int64_t n_src_rows,
                                                          const int32_t* __restrict__ index, int64_t P, int nvec,
                                                          uint4* __restrict__ dst, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t p0 = warp * ROWS; p0 < P; p0 += nwarps * ROWS) {
    int64_t row[ROWS];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      int64_t p = p0 + r;
      int32_t i = (p < P) ? index[p] : 0;
      if (i < 0 || i >= n_src_rows) {
        gram_device_fail(status, GRAM_ERR_ID_RANGE);
        i = 0;
      }
      row[r] = i;
    }
    for (int c = lane; c < nvec; c += 32) {
      uint4 v[ROWS];
#pragma unroll
      for (int r = 0; r < ROWS; ++r) v[r] = __ldg(src + row[r] * nvec + c);
#pragma unroll
      for (int r = 0; r < ROWS; ++r)
        if (p0 + r < P) __stcs(dst + (p0 + r) * nvec + c, v[r]);
    }
  }
}

// rows whose byte length is not a multiple of 16: element-wise copy of 2- or 4-byte elements
template <typename T>
__global__ void gather_scalar_kernel(const T* __restrict__ src, int64_t n_src_rows, const int32_t* __restrict__ index,
                                     int64_t P, int d, T* __restrict__ dst, int32_t* status) {
  const int64_t n = P * d;
  for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n; k += (int64_t)gridDim.x * blockDim.x) {
    int64_t p = k / d;
    int c = (int)(k - p * d);
    int32_t i = index[p];
    if (i < 0 || i >= n_src_rows) {
      gram_device_fail(status, GRAM_ERR_ID_RANGE);
      i = 0;
    }
    dst[k] = src[(int64_t)i * d + c];
  }
}

// dst[p, :] (fp32) = src[index[p], :] (bf16): the Multi-step gather from a bf16 encoding cache, widened on the way so
// that the task module's fp32 input is written once.  A warp per row, 8 elements (16 bytes in, 32 out) per lane and step.
template <int ROWS>
__global__ void __launch_bounds__(256) gather_widen_kernel(const uint4* __restrict__ src, int64_t n_src_rows,
                                                           const int32_t* __restrict__ index, int64_t P, int nvec,
                                                           float4* __restrict__ dst, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t p0 = warp * ROWS; p0 < P; p0 += nwarps * ROWS) {
    int64_t row[ROWS];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      int64_t p = p0 + r;
      int32_t i = (p < P) ? index[p] : 0;
      if (i < 0 || i >= n_src_rows) {
        gram_device_fail(status, GRAM_ERR_ID_RANGE);
        i = 0;
      }
      row[r] = i;
    }
    for (int c = lane; c < nvec; c += 32) {
      uint4 v[ROWS];
#pragma unroll
      for (int r = 0; r < ROWS; ++r) v[r] = __ldg(src + row[r] * nvec + c);
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        if (p0 + r < P) {
          const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v[r].x));
          const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v[r].y));
          const float2 e = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v[r].z));
          const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v[r].w));
          float4* q = dst + ((p0 + r) * nvec + c) * 2;
          __stcs(q, make_float4(a.x, a.y, b.x, b.y));
          __stcs(q + 1, make_float4(e.x, e.y, f.x, f.y));
        }
      }
    }
  }
}

// out[r, :] = a[index[r], :] - b[index[r], :], or x[r, :] - that; a warp per row, 4 floats per lane and step
__global__ void __launch_bounds__(256) gather_diff_kernel(const float* __restrict__ a, const float* __restrict__ b,
                                                          int64_t n_src_rows, const int32_t* __restrict__ index, int64_t n,
                                                          int d, const float* __restrict__ x, float* __restrict__ out,
                                                          int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const bool vec = (d & 3) == 0;
  for (int64_t r = warp; r < n; r += nwarps) {
    int32_t i = index[r];
    if (i < 0 || i >= n_src_rows) {
      gram_device_fail(status, GRAM_ERR_ID_RANGE);
      i = 0;
    }
    const float* pa = a + (int64_t)i * d;
    const float* pb = b + (int64_t)i * d;
    const float* px = x ? x + r * d : nullptr;
    float* po = out + r * d;
    if (vec) {
      for (int c = lane * 4; c < d; c += 128) {
        const float4 va = *reinterpret_cast<const float4*>(pa + c), vb = *reinterpret_cast<const float4*>(pb + c);
        float4 v = make_float4(va.x - vb.x, va.y - vb.y, va.z - vb.z, va.w - vb.w);
        if (px) {
          const float4 vx = *reinterpret_cast<const float4*>(px + c);
          v = make_float4(vx.x - v.x, vx.y - v.y, vx.z - v.z, vx.w - v.w);
        }
        *reinterpret_cast<float4*>(po + c) = v;
      }
    } else {
      for (int c = lane; c < d; c += 32) {
        const float v = pa[c] - pb[c];
        po[c] = px ? px[c] - v : v;
      }
    }
  }
}

// ---------------------------------------------------------------------------
// segmented sum.  The sorted order j in [0, P) is cut into nchunks equal chunks of R rows; the
// columns into slabs of VPL*128 floats.  One warp owns one (chunk, slab): it walks its rows in
// order, adding into registers, and closes a sum whenever the item changes.
//   - an item whose rows all lie inside the chunk is written to its output row directly;
//   - the item that entered the chunk from the left leaves its part in partial[chunk][0];
//   - the item that leaves the chunk to the right leaves its part in partial[chunk][1].
// A second launch adds, for every item that spans chunks, partial[first][1] and the following
// chunks' partial[c][0] in a fixed association (eight interleaved ascending runs, then their sum).  The order of additions depends only
// on (P, U, seg_off), never on scheduling: repeated runs are bit-identical.
// Algorithmic bytes: 4*P*d read + 4*U*d written + 4P (perm) + 4(U+1) (seg_off).
// ---------------------------------------------------------------------------
template <typename InT> struct Row4;
template <> struct Row4<float> {
  typedef float4 vec;
  static __device__ __forceinline__ float4 load(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
};
template <> struct Row4<bf16> {
  typedef uint2 vec;
  static __device__ __forceinline__ float4 load(const bf16* p) {
    uint2 u = __ldcs(reinterpret_cast<const uint2*>(p));
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x), b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
    float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
    return make_float4(fa.x, fa.y, fb.x, fb.y);
  }
};

// largest u in [0, U) with seg_off[u] <= j, found by the whole warp: every lane probes one of 32 evenly spaced
// entries per round, so U = 10^6 takes four dependent loads instead of twenty.  All 32 lanes must call it.
__device__ __forceinline__ int32_t find_segment(const int32_t* __restrict__ seg_off, int32_t U, int64_t j, int lane) {
  int32_t lo = 0, n = U;                       // the answer lies in [lo, lo + n) and seg_off[lo] <= j
  while (n > 1) {
    const int32_t step = (n + 31) >> 5;
    const int32_t idx = lo + lane * step;
    const bool ok = (lane * step < n) && (seg_off[idx] <= j);
    const unsigned m = __ballot_sync(0xffffffffu, ok) | 1u;
    const int k = 31 - __clz(m);
    n = min(step, n - k * step);
    lo += k * step;
  }
  return lo;
}

template <int VPL>
__device__ __forceinline__ void store_row(float* __restrict__ out, int64_t row, int d, int col0, int lane,
                                          const float4 (&acc)[VPL], bool add) {
#pragma unroll
  for (int v = 0; v < VPL; ++v) {
    int c = col0 + (v * 32 + lane) * 4;
    if (c < d) {
      float4* q = reinterpret_cast<float4*>(out + row * d + c);
      float4 a = acc[v];
      if (add) {
        float4 o = *q;
        a.x += o.x; a.y += o.y; a.z += o.z; a.w += o.w;
      }
      *q = a;
    }
  }
}

template <typename InT, int VPL, int UNROLL>
__global__ void __launch_bounds__(256) segsum_chunks_kernel(const InT* __restrict__ in, const int32_t* __restrict__ perm,
                                                            const int32_t* __restrict__ seg_off, int64_t P, int32_t U,
                                                            int d, int64_t R, int nchunks, int nslabs,
                                                            const int32_t* __restrict__ rows, int add,
                                                            float* __restrict__ out, float* __restrict__ partial,
                                                            int2* __restrict__ span, int32_t* status,
                                                            const int32_t* __restrict__ d_U,
                                                            const int32_t* __restrict__ gate) {
  if (d_U) U = *d_U;            // the number of items may live on the device
  if (U <= 0) return;
  if (gate && *gate) return;    // an earlier kernel of the step reported an error: leave the accumulated rows alone
  const int lane = threadIdx.x & 31;
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (w >= (int64_t)nchunks * nslabs) return;
  const int chunk = (int)(w / nslabs), slab = (int)(w - (int64_t)chunk * nslabs);
  const int col0 = slab * (VPL * 128);
  const int64_t c0 = (int64_t)chunk * R, c1 = min(c0 + R, P);
  if (c0 >= c1) return;

  int32_t u = find_segment(seg_off, U, c0, lane);
  int64_t seg_begin = seg_off[u], seg_end = seg_off[u + 1];
  float4 acc[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);

  for (int64_t j0 = c0; j0 < c1; j0 += 32) {
    const int nrow = (int)min((int64_t)32, c1 - j0);
    int32_t my = (lane < nrow) ? perm[j0 + lane] : 0;
    if ((uint32_t)my >= (uint32_t)P) {       // a position outside the batch: record it, read row 0 instead
      gram_device_fail(status, GRAM_ERR_ID_RANGE);
      my = 0;
    }
    for (int b = 0; b < nrow; b += UNROLL) {
      float4 x[UNROLL][VPL];
#pragma unroll
      for (int r = 0; r < UNROLL; ++r) {
        const int32_t p = __shfl_sync(0xffffffffu, my, (b + r) & 31);
        const bool live = (b + r) < nrow;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
          int c = col0 + (v * 32 + lane) * 4;
          x[r][v] = (live && c < d) ? Row4<InT>::load(in + (int64_t)p * d + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
#pragma unroll
      for (int r = 0; r < UNROLL; ++r) {
        const int64_t j = j0 + b + r;
        if (j < c1) {
          while (j == seg_end && u + 1 < U) {   // item u is complete (its end lies inside this chunk)
            if (seg_begin >= c0) store_row<VPL>(out, rows ? rows[u] : u, d, col0, lane, acc, add != 0);
            else store_row<VPL>(partial, (int64_t)chunk * 2 + 0, d, col0, lane, acc, false);
            ++u;
            seg_begin = seg_end;
            seg_end = seg_off[u + 1];
#pragma unroll
            for (int v = 0; v < VPL; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int v = 0; v < VPL; ++v) {
            acc[v].x += x[r][v].x; acc[v].y += x[r][v].y; acc[v].z += x[r][v].z; acc[v].w += x[r][v].w;
          }
        }
      }
    }
  }
  // the item still open at the end of the chunk
  int2 sp = make_int2(-1, 0);
  if (seg_end <= c1) {             // it ends exactly at the chunk end
    if (seg_begin >= c0) store_row<VPL>(out, rows ? rows[u] : u, d, col0, lane, acc, add != 0);
    else store_row<VPL>(partial, (int64_t)chunk * 2 + 0, d, col0, lane, acc, false);
  } else {                         // it continues to the right
    store_row<VPL>(partial, (int64_t)chunk * 2 + (seg_begin >= c0 ? 1 : 0), d, col0, lane, acc, false);
    if (seg_begin >= c0) sp = make_int2(u, (int)((seg_end - 1) / R));      // it starts here: the fix-up adds its parts
  }
  if (slab == 0 && lane == 0) span[chunk] = sp;   // (item, last chunk it reaches), or -1: nothing to fix up from here
}

// one block per (chunk, slab): if an item starts in this chunk and runs past its end, add its parts.  Warp w adds
// the following chunks' parts number w, w+8, ... (ascending), warp 0 starts from this chunk's own part, and the
// eight warp sums are added in ascending w: a fixed association, whatever the schedule.
template <int VPL>
__global__ void __launch_bounds__(256) segsum_fixup_kernel(const int32_t* __restrict__ seg_off, int64_t P, int32_t U,
                                                           int d, int64_t R, int nchunks, int nslabs,
                                                           const int32_t* __restrict__ rows, int add,
                                                           float* __restrict__ out, const float* __restrict__ partial,
                                                           const int2* __restrict__ span, const int32_t* __restrict__ d_U,
                                                           const int32_t* __restrict__ gate) {
  __shared__ float4 red[8][VPL][32];
  if (d_U) U = *d_U;
  if (U <= 0) return;
  if (gate && *gate) return;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int chunk = blockIdx.x / nslabs, slab = blockIdx.x - chunk * nslabs;
  const int col0 = slab * (VPL * 128);
  const int64_t c0 = (int64_t)chunk * R, c1 = min(c0 + R, P);
  if (c0 >= c1 || c1 >= P) return;
  const int2 sp = span[chunk];                       // left by the first launch
  if (sp.x < 0) return;                              // no item starts here and runs on (same for the whole block)
  const int32_t u = sp.x;
  const int last = min(sp.y, nchunks - 1);
  float4 acc[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) {
    const int c = col0 + (v * 32 + lane) * 4;
    acc[v] = (w == 0 && c < d) ? *reinterpret_cast<const float4*>(partial + ((int64_t)chunk * 2 + 1) * d + c)
                               : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int c = chunk + 1 + w; c <= last; c += 32) {   // four parts in flight per warp
    float4 x[4][VPL];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) {
        const int cc = col0 + (v * 32 + lane) * 4;
        x[k][v] = (c + 8 * k <= last && cc < d) ? *reinterpret_cast<const float4*>(partial + ((int64_t)(c + 8 * k) * 2 + 0) * d + cc)
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (c + 8 * k <= last) {
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
          acc[v].x += x[k][v].x; acc[v].y += x[k][v].y; acc[v].z += x[k][v].z; acc[v].w += x[k][v].w;
        }
      }
    }
  }
#pragma unroll
  for (int v = 0; v < VPL; ++v) red[w][v][lane] = acc[v];
  __syncthreads();
  if (w == 0) {
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      float4 t = red[0][v][lane];
#pragma unroll
      for (int k = 1; k < 8; ++k) {
        const float4 y = red[k][v][lane];
        t.x += y.x; t.y += y.y; t.z += y.z; t.w += y.w;
      }
      acc[v] = t;
    }
    store_row<VPL>(out, rows ? rows[u] : u, d, col0, lane, acc, add != 0);
  }
}

// d_U (may be null): the number of items lives on the device.  count (may be null): one word that counts the set
// bits (integer adds: the total does not depend on their order).  gated: nothing is marked once the status word is set.
__global__ void touched_mark_kernel(const int32_t* __restrict__ unique, int32_t U, const int32_t* __restrict__ d_U,
                                    int32_t n_items, uint32_t* __restrict__ bits, int32_t* __restrict__ count,
                                    int32_t* status, int gated) {
  if (d_U) U = *d_U;
  if (gated && *status) return;
  for (int32_t u = blockIdx.x * blockDim.x + threadIdx.x; u < U; u += gridDim.x * blockDim.x) {
    const int32_t i = unique[u];
    if (i < 0 || i >= n_items) {
      gram_device_fail(status, GRAM_ERR_ID_RANGE);
      continue;
    }
    const uint32_t bit = 1u << (i & 31);
    const uint32_t old = atomicOr(&bits[i >> 5], bit);
    if (count && !(old & bit)) atomicAdd(count, 1);
  }
}

// ascending list of set bits, one block
__global__ void __launch_bounds__(1024) touched_list_kernel(const uint32_t* __restrict__ bits, int32_t n_items,
                                                            int32_t* __restrict__ list, int32_t* __restrict__ count) {
  __shared__ int32_t sw[33];
  const int nwords = (n_items + 31) >> 5;
  const int per = (nwords + 1023) / 1024;
  const int w0 = threadIdx.x * per, w1 = min(w0 + per, nwords);
  int32_t c = 0;
  for (int w = w0; w < w1; ++w) {
    uint32_t b = bits[w];
    if (w == nwords - 1 && (n_items & 31)) b &= (1u << (n_items & 31)) - 1u;
    c += __popc(b);
  }
  // exclusive scan over the 1024 threads
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int32_t incl = c;
  for (int o = 1; o < 32; o <<= 1) {
    int32_t t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) sw[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int32_t x = sw[lane], xi = x;
    for (int o = 1; o < 32; o <<= 1) {
      int32_t t = __shfl_up_sync(0xffffffffu, xi, o);
      if (lane >= o) xi += t;
    }
    sw[lane] = xi - x;
    if (lane == 31) sw[32] = xi;
  }
  __syncthreads();
  int32_t pos = sw[warp] + incl - c;
  for (int w = w0; w < w1; ++w) {
    uint32_t b = bits[w];
    if (w == nwords - 1 && (n_items & 31)) b &= (1u << (n_items & 31)) - 1u;
    while (b) {
      int bit = __ffs(b) - 1;
      list[pos++] = w * 32 + bit;
      b &= b - 1;
    }
  }
  if (threadIdx.x == 0) *count = sw[32];
}

}  // namespace

gram_status gather_launch(gram_ctx* ctx, const void* d_src, int64_t n_src_rows, const int32_t* d_index, int64_t P,
                          int32_t d, int elem_bytes, void* d_E, cudaStream_t st) {
  if (P < 0 || d <= 0 || n_src_rows < 0 || (elem_bytes != 2 && elem_bytes != 4))
    return gram_set_error(ctx, "gram_gather: bad argument"), GRAM_ERR_ARG;
  if (P == 0) return GRAM_OK;
  if (!d_src || !d_index || !d_E || n_src_rows == 0)
    return gram_set_error(ctx, "gram_gather: null buffer"), GRAM_ERR_ARG;
  int32_t* status = gram_status_word(ctx);
  const int64_t row_bytes = (int64_t)d * elem_bytes;
  ProfScope prof(ctx, GRAM_K_GATHER, (double)row_bytes * (double)(P + (n_src_rows < P ? n_src_rows : P)) + 4.0 * P, 1, st);
  const bool vec_ok = (row_bytes % 16 == 0) && ((uintptr_t)d_src % 16 == 0) && ((uintptr_t)d_E % 16 == 0);
  if (vec_ok) {
    const int nvec = (int)(row_bytes / 16);
    constexpr int ROWS = 4;
    int64_t warps = ceil_div64(P, ROWS);
    int blocks = (int)ceil_div64(warps, 8);
    const int cap = kNumSMs * 8;
    if (blocks > cap) blocks = cap;
    gather_rows_kernel<ROWS><<<blocks, 256, 0, st>>>((const uint4*)d_src, n_src_rows, d_index, P, nvec, (uint4*)d_E,
                                                     status);
  } else {
    int64_t n = P * d;
    int blocks = (int)ceil_div64(n, 256);
    if (blocks > kNumSMs * 16) blocks = kNumSMs * 16;
    if (elem_bytes == 4)
      gather_scalar_kernel<float><<<blocks, 256, 0, st>>>((const float*)d_src, n_src_rows, d_index, P, d, (float*)d_E, status);
    else
      gather_scalar_kernel<bf16><<<blocks, 256, 0, st>>>((const bf16*)d_src, n_src_rows, d_index, P, d, (bf16*)d_E, status);
  }
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status gather_widen_launch(gram_ctx* ctx, const void* d_src_bf16, int64_t n_src_rows, const int32_t* d_index, int64_t P,
                                int32_t d, float* d_E, cudaStream_t st) {
  if (P < 0 || d <= 0 || n_src_rows <= 0 || (d % 8) || ((uintptr_t)d_src_bf16 % 16) || ((uintptr_t)d_E % 16))
    return gram_set_error(ctx, "widening gather: bad argument (rows of a multiple of 8 elements, 16-byte aligned)"), GRAM_ERR_ARG;
  if (P == 0) return GRAM_OK;
  if (!d_src_bf16 || !d_index || !d_E) return gram_set_error(ctx, "widening gather: null buffer"), GRAM_ERR_ARG;
  ProfScope prof(ctx, GRAM_K_GATHER, 4.0 * (double)d * (double)P + 2.0 * (double)d * (double)(n_src_rows < P ? n_src_rows : P) + 4.0 * P, 1, st);
  constexpr int ROWS = 4;
  int blocks = (int)ceil_div64(ceil_div64(P, ROWS), 8);
  if (blocks > kNumSMs * 8) blocks = kNumSMs * 8;
  gather_widen_kernel<ROWS><<<blocks, 256, 0, st>>>((const uint4*)d_src_bf16, n_src_rows, d_index, P, d / 8, (float4*)d_E,
                                                    gram_status_word(ctx));
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status gather_diff_launch(gram_ctx* ctx, const float* d_a, const float* d_b, int64_t n_src_rows, const int32_t* d_index,
                               int64_t n, int32_t d, const float* d_x, float* d_out, cudaStream_t st) {
  if (n < 0 || d <= 0 || n_src_rows <= 0 || (n > 0 && (!d_a || !d_b || !d_index || !d_out)))
    return gram_set_error(ctx, "gather of pseudo-targets: bad argument"), GRAM_ERR_ARG;
  if (n == 0) return GRAM_OK;
  ProfScope prof(ctx, GRAM_K_GATHER, (double)n * d * 4.0 * (d_x ? 4.0 : 3.0) + 4.0 * (double)n, 1, st);
  int blocks = (int)ceil_div64(n, 8);
  if (blocks > kNumSMs * 8) blocks = kNumSMs * 8;
  gather_diff_kernel<<<blocks, 256, 0, st>>>(d_a, d_b, n_src_rows, d_index, n, d, d_x, d_out, gram_status_word(ctx));
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

template <typename InT, int VPL>
static void segsum_run(const void* d_in, const int32_t* d_perm, const int32_t* d_seg_off, int64_t P, int32_t U, int32_t d,
                       int64_t R, int nchunks, const int32_t* d_rows, int add, float* d_out, float* partial, int2* span,
                       int32_t* status, const int32_t* d_U, cudaStream_t st, const int32_t* gate = nullptr) {
  const int nslabs = ceil_div(d, VPL * 128);
  const int64_t warps = (int64_t)nchunks * nslabs;
  const int blocks = (int)ceil_div64(warps, 8);
  segsum_chunks_kernel<InT, VPL, 8><<<blocks, 256, 0, st>>>((const InT*)d_in, d_perm, d_seg_off, P, U, d, R, nchunks, nslabs,
                                                            d_rows, add, d_out, partial, span, status, d_U, gate);
  if (nchunks > 1)
    segsum_fixup_kernel<VPL><<<(unsigned)warps, 256, 0, st>>>(d_seg_off, P, U, d, R, nchunks, nslabs, d_rows, add, d_out, partial, span, d_U, gate);
}

gram_status accumulate_launch(gram_ctx* ctx, IndexWorkspace* ws, const void* d_in, int in_bf16, const int32_t* d_perm,
                              const int32_t* d_seg_off, int64_t P, int32_t U, const int32_t* d_U, int32_t d,
                              const int32_t* d_rows, int add, float* d_out, cudaStream_t st, int gated) {
  if (P < 0 || U < 0 || d <= 0 || U > P) return gram_set_error(ctx, "gram_accumulate: bad argument"), GRAM_ERR_ARG;
  if (P == 0 || (U == 0 && !d_U)) return GRAM_OK;
  if (!d_in || !d_perm || !d_seg_off || !d_out) return gram_set_error(ctx, "gram_accumulate: null buffer"), GRAM_ERR_ARG;
  if (d % 4 != 0 || ((uintptr_t)d_in % (in_bf16 ? 8 : 16)) || ((uintptr_t)d_out % 16))
    return gram_set_error(ctx, "gram_accumulate: d must be a multiple of 4 and buffers 16-byte aligned"), GRAM_ERR_UNSUPPORTED;
  if (d > ws->d_max) return gram_set_error(ctx, "gram_accumulate: d=%d exceeds the context's d_max=%d", d, ws->d_max), GRAM_ERR_WORKSPACE;
  // chunks: at least 16 rows each, at most kAccMaxChunks
  int64_t nchunks = ceil_div64(P, 16);
  if (nchunks > kAccMaxChunks) nchunks = kAccMaxChunks;
  const int64_t R = ceil_div64(P, nchunks);
  nchunks = ceil_div64(P, R);
  int2* span = reinterpret_cast<int2*>(ws->partial + (size_t)kAccMaxChunks * 2 * (ws->d_max > 0 ? ws->d_max : 1));   // after the partial sums
  ProfScope prof(ctx, GRAM_K_ACCUMULATE, (in_bf16 ? 2.0 : 4.0) * (double)P * d + 4.0 * (double)U * d + 4.0 * P + 4.0 * (U + 1),
                 nchunks > 1 ? 2 : 1, st);
  int32_t* sw = gram_status_word(ctx);
  const int32_t* gate = gated ? sw : nullptr;
  if (d >= 256) {
    if (in_bf16) segsum_run<bf16, 2>(d_in, d_perm, d_seg_off, P, U, d, R, (int)nchunks, d_rows, add, d_out, ws->partial, span, sw, d_U, st, gate);
    else segsum_run<float, 2>(d_in, d_perm, d_seg_off, P, U, d, R, (int)nchunks, d_rows, add, d_out, ws->partial, span, sw, d_U, st, gate);
  } else {
    if (in_bf16) segsum_run<bf16, 1>(d_in, d_perm, d_seg_off, P, U, d, R, (int)nchunks, d_rows, add, d_out, ws->partial, span, sw, d_U, st, gate);
    else segsum_run<float, 1>(d_in, d_perm, d_seg_off, P, U, d, R, (int)nchunks, d_rows, add, d_out, ws->partial, span, sw, d_U, st, gate);
  }
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status touched_mark_launch(gram_ctx* ctx, const int32_t* d_unique, int32_t U, const int32_t* d_U, int32_t n_items,
                                uint32_t* d_bits, int32_t* d_count, int gated, cudaStream_t st) {
  if (U <= 0 && !d_U) return GRAM_OK;
  if (d_U) U = n_items;                              // upper bound for the launch shape
  ProfScope prof(ctx, GRAM_K_OTHER, 8.0 * U, 1, st);
  int blocks = ceil_div(U, 256);
  if (blocks > kNumSMs * 4) blocks = kNumSMs * 4;
  touched_mark_kernel<<<blocks, 256, 0, st>>>(d_unique, U, d_U, n_items, d_bits, d_count, gram_status_word(ctx), gated);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

gram_status touched_list_launch(gram_ctx* ctx, const uint32_t* d_bits, int32_t n_items, int32_t* d_list,
                                int32_t* d_count, cudaStream_t st) {
  if (n_items <= 0 || !d_bits || !d_list || !d_count) return gram_set_error(ctx, "gram_touched_list: bad argument"), GRAM_ERR_ARG;
  ProfScope prof(ctx, GRAM_K_OTHER, (double)n_items / 8.0, 1, st);
  touched_list_kernel<<<1, 1024, 0, st>>>(d_bits, n_items, d_list, d_count);
  GRAM_LAUNCH_CHECK(ctx);
  return GRAM_OK;
}

// ---------------------------------------------------------------------------------------------
// The segmented sum for callers that must not allocate.  Its chunk-boundary partial sums live in
// a fixed array that is part of the library image, so the call touches no allocator at all.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr int kStaticChunks = 592;            // work units (4 per SM)
constexpr int kStaticMaxD = 1024;             // widest row the fixed scratch can serve
constexpr size_t kStaticPartialFloats = (size_t)kStaticChunks * 2 * kStaticMaxD;
// [0, kStaticPartialFloats): partial sums; then 64 floats whose first word is the device status word; then one
// (item, last chunk) pair per work unit
static __device__ __align__(256) float g_static_scratch[kStaticPartialFloats + 64 + 2 * kStaticChunks];

constexpr int kMaxDevices = 64;
float* g_static_ptr[kMaxDevices] = {};        // device address of the array, looked up once per device

void static_fail(char* h_err, size_t n, const char* msg) {
  if (h_err && n) snprintf(h_err, n, "%s", msg);
}
}  // namespace

extern "C" gram_status gram_accumulate_static(const float* d_dE, const int32_t* d_perm, const int32_t* d_seg_off,
                                               int64_t P, int32_t U, int32_t d, float* d_G, gram_stream stream,
                                               char* h_err, size_t err_len) {
  if (h_err && err_len) h_err[0] = 0;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (P < 0 || U < 0 || d <= 0 || U > P) return static_fail(h_err, err_len, "gram_accumulate_static: bad size"), GRAM_ERR_ARG;
  if (d > kStaticMaxD) {
    if (h_err && err_len) snprintf(h_err, err_len, "gram_accumulate_static: d=%d exceeds the fixed scratch's maximum of %d columns", d, kStaticMaxD);
    return GRAM_ERR_WORKSPACE;
  }
  if (P > INT32_MAX) return static_fail(h_err, err_len, "gram_accumulate_static: P exceeds 2^31-1 positions"), GRAM_ERR_WORKSPACE;
  if (P == 0 || U == 0) return GRAM_OK;
  if (!d_dE || !d_perm || !d_seg_off || !d_G) return static_fail(h_err, err_len, "gram_accumulate_static: null buffer"), GRAM_ERR_ARG;
  if (d % 4 != 0 || ((uintptr_t)d_dE % 16) || ((uintptr_t)d_G % 16))
    return static_fail(h_err, err_len, "gram_accumulate_static: d must be a multiple of 4 and buffers 16-byte aligned"), GRAM_ERR_UNSUPPORTED;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return static_fail(h_err, err_len, "gram_accumulate_static: cannot identify the current device"), GRAM_ERR_CUDA;
  if (!g_static_ptr[dev]) {
    // in host code the array's name is only a handle: ask the runtime for its address on this device
    float* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr) {
      if (h_err && err_len) snprintf(h_err, err_len, "gram_accumulate_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
      return GRAM_ERR_CUDA;
    }
    g_static_ptr[dev] = ptr;
  }
  float* partial = g_static_ptr[dev];
  int32_t* status = reinterpret_cast<int32_t*>(partial + kStaticPartialFloats);
  int2* span = reinterpret_cast<int2*>(partial + kStaticPartialFloats + 64);
  // the status word must start at zero; the partial sums and the (item, last chunk) pairs need no clearing
  // (each slot that is read in a call has been written earlier in the same call)
  if (cudaMemsetAsync(status, 0, sizeof(int32_t), st) != cudaSuccess)
    return static_fail(h_err, err_len, "gram_accumulate_static: clearing the status word failed"), GRAM_ERR_CUDA;
  int64_t nchunks = ceil_div64(P, 16);
  if (nchunks > kStaticChunks) nchunks = kStaticChunks;
  const int64_t R = ceil_div64(P, nchunks);
  nchunks = ceil_div64(P, R);
  if (d >= 256) segsum_run<float, 2>(d_dE, d_perm, d_seg_off, P, U, d, R, (int)nchunks, nullptr, 0, d_G, partial, span, status, nullptr, st);
  else segsum_run<float, 1>(d_dE, d_perm, d_seg_off, P, U, d, R, (int)nchunks, nullptr, 0, d_G, partial, span, status, nullptr, st);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    if (h_err && err_len) snprintf(h_err, err_len, "gram_accumulate_static: launch failed: %s", cudaGetErrorString(e));
    return GRAM_ERR_CUDA;
  }
  return GRAM_OK;
}
