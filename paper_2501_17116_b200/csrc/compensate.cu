// Outlier compensation (Section 3.2: the sparse residual times a dense high-precision matrix):
// forward fused with the final store, weight gradient (Eq. 6) as compact rows for the GEMM's epilogue.
//
//   forward   Y[m, :]  = store( Y1[m, :] + sum_{(m,k) in dA} dA[m,k] * W[k, :] )
//   wgrad     C[slot(k), :] = sum_{(m,k) in dA} dA[m,k] * dY[m, :]   for the columns k that hold entries;
//             the weight-gradient GEMM adds C and applies the DGE factor in its epilogue
//
// Both are "sparse row times dense BF16 matrix" with fp32 accumulation on the plain ALUs: a warp
// owns one output row and 256 of its columns (8 per lane); the sparse entries of that row (CSR
// for the forward, CSC for the weight gradient) are walked in order, so the result is
// deterministic.  The FP4 branch and the compensation meet in fp32 and are rounded once.
#include <cuda_fp16.h>

#include "common.cuh"

namespace {

constexpr int COMP_THREADS = 256;          // 8 warps = 8 output rows per block
constexpr int COMP_COLS = 256;             // columns per block (8 per lane)

__device__ __forceinline__ void fma8(float (&acc)[8], float v, const uint4& d) {
  const uint32_t w[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    acc[2 * q] = fmaf(v, __uint_as_float(w[q] << 16), acc[2 * q]);
    acc[2 * q + 1] = fmaf(v, __uint_as_float(w[q] & 0xFFFF0000u), acc[2 * q + 1]);
  }
}

__device__ __forceinline__ void store8(void* out, int out_f32, long long off, const float (&y)[8]) {
  if (out_f32) {
    float4* dst = reinterpret_cast<float4*>(static_cast<float*>(out) + off);
    dst[0] = make_float4(y[0], y[1], y[2], y[3]);
    dst[1] = make_float4(y[4], y[5], y[6], y[7]);
  } else {
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      __nv_bfloat162 h = __floats2bfloat162_rn(y[2 * q], y[2 * q + 1]);
      w[q] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(out) + off) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// acc[0..7] += sum over the entries [e0, e1) of val[e] * dense[idx[e], col .. col+7]
__device__ __forceinline__ void sparse_row_times_dense(float (&acc)[8], const int* __restrict__ idx,
                                                       const float* __restrict__ val, int e0, int e1,
                                                       const uint4* __restrict__ dense, int vec_per_row, int vcol) {
  int e = e0;
  for (; e + 4 <= e1; e += 4) {                 // four independent loads in flight
    int r[4];
    float v[4];
    uint4 d[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      r[u] = __ldg(&idx[e + u]);
      v[u] = __ldg(&val[e + u]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) d[u] = __ldg(&dense[(long long)r[u] * vec_per_row + vcol]);
#pragma unroll
    for (int u = 0; u < 4; ++u) fma8(acc, v[u], d[u]);
  }
  for (; e < e1; ++e) {
    const uint4 d = __ldg(&dense[(long long)__ldg(&idx[e]) * vec_per_row + vcol]);
    fma8(acc, __ldg(&val[e]), d);
  }
}

__global__ void __launch_bounds__(COMP_THREADS)
comp_fwd_kernel(const float* __restrict__ y1, const int* __restrict__ rowptr, const int* __restrict__ col,
                const float* __restrict__ val, const uint4* __restrict__ w, int M, int N, void* y, int out_f32) {
  // blocks that follow one another share the 256 output columns, i.e. the same slab of the weight
  // rows (K x 512 bytes): it stays in L2 while the tokens stream past
  const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int n0 = blockIdx.y * COMP_COLS + 8 * (threadIdx.x & 31);
  if (m >= M || n0 >= N) return;
  // Y1 is requested first: its latency runs under the dependent chain row pointer -> entry -> weight row
  const long long off = (long long)m * N + n0;
  const float4 a = __ldg(reinterpret_cast<const float4*>(y1 + off));
  const float4 b = __ldg(reinterpret_cast<const float4*>(y1 + off + 4));
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  sparse_row_times_dense(acc, col, val, __ldg(&rowptr[m]), __ldg(&rowptr[m + 1]), w, N >> 3, n0 >> 3);
  const float y8[8] = {a.x + acc[0], a.y + acc[1], a.z + acc[2], a.w + acc[3],
                       b.x + acc[4], b.y + acc[5], b.z + acc[6], b.w + acc[7]};
  store8(y, out_f32, off, y8);
}

// The same with the entries of the hot columns left out (the GEMM's dense tail has added them):
// slot_of_col[k] in [0, *tail_count) marks a hot column.  The lanes of a warp share the token, so
// they read 32 entries at a time, drop the hot ones and hand the others round by shuffle, four
// weight-row loads in flight as above; the order of the additions stays ascending.
__global__ void __launch_bounds__(COMP_THREADS)
comp_fwd_skip_kernel(const float* __restrict__ y1, const int* __restrict__ rowptr, const int* __restrict__ col,
                     const float* __restrict__ val, const uint4* __restrict__ w, int M, int N, void* y, int out_f32,
                     const int* __restrict__ slot_of_col, const int* __restrict__ tail_count) {
  const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int n0 = blockIdx.y * COMP_COLS + 8 * lane;
  if (m >= M) return;                                   // whole warps only: the shuffles below need every lane
  const bool live = n0 < N;
  const long long off = (long long)m * N + (live ? n0 : 0);
  float4 a = make_float4(0, 0, 0, 0), b = a;
  if (live) {
    a = __ldg(reinterpret_cast<const float4*>(y1 + off));
    b = __ldg(reinterpret_cast<const float4*>(y1 + off + 4));
  }
  const unsigned hot = unsigned(__ldg(tail_count));
  const int vec_per_row = N >> 3, vcol = (live ? n0 : 0) >> 3;
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  const int e1 = __ldg(&rowptr[m + 1]);
  for (int base = __ldg(&rowptr[m]); base < e1; base += 32) {
    const int e = base + lane;
    int k = 0;
    float v = 0.0f;
    bool keep = false;
    if (e < e1) {
      k = __ldg(&col[e]);
      v = __ldg(&val[e]);
      keep = unsigned(__ldg(&slot_of_col[k])) >= hot;   // -1 (no slot) compares as a large number
    }
    unsigned mask = __ballot_sync(0xFFFFFFFFu, keep);
    while (mask) {
      int r[4];
      float vv[4];
      uint4 d[4];
      int cnt = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int src = mask ? __ffs(mask) - 1 : 0;
        r[u] = __shfl_sync(0xFFFFFFFFu, k, src);
        vv[u] = __shfl_sync(0xFFFFFFFFu, v, src);
        if (mask) { ++cnt; mask &= mask - 1; } else vv[u] = 0.0f;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (u < cnt) d[u] = __ldg(&w[(long long)r[u] * vec_per_row + vcol]);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (u < cnt) fma8(acc, vv[u], d[u]);
    }
  }
  if (!live) return;
  const float y8[8] = {a.x + acc[0], a.y + acc[1], a.z + acc[2], a.w + acc[3],
                       b.x + acc[4], b.y + acc[5], b.z + acc[6], b.w + acc[7]};
  store8(y, out_f32, off, y8);
}

// The forward compensation when the dense tail is in use: tail_a has listed, per token, the entries
// the tail does not cover (`kept`: column and value bits, at the token's own range of the CSR, ending
// at kept_end[m]), so this kernel walks a plain list: one 8-byte broadcast load per entry, eight
// weight-row gathers in flight per lane at four blocks per SM (measured on the 13B layer: four in
// flight 9.3 ms per step, eight 7.7 ms, twelve at three blocks 8.0 ms, sixteen at two blocks 10.2 ms).  If the tail was switched off on the device (*tail_count == 0: a value
// FP16 cannot hold) the list is not valid and the whole CSR row is added instead.
constexpr int FWD_FLY = 8;                 // weight-row gathers a lane keeps in flight
__global__ void __launch_bounds__(COMP_THREADS, 4)
comp_fwd_kept_kernel(const float* __restrict__ y1, const int* __restrict__ rowptr, const int* __restrict__ col,
                     const float* __restrict__ val, const uint2* __restrict__ kept, const int* __restrict__ kept_end,
                     const uint4* __restrict__ w, int M, int N, void* y, int out_f32,
                     const int* __restrict__ tail_count) {
  const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int n0 = blockIdx.y * COMP_COLS + 8 * (threadIdx.x & 31);
  if (m >= M || n0 >= N) return;
  const long long off = (long long)m * N + n0;
  const float4 a = __ldg(reinterpret_cast<const float4*>(y1 + off));
  const float4 b = __ldg(reinterpret_cast<const float4*>(y1 + off + 4));
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  const int vec_per_row = N >> 3, vcol = n0 >> 3;
  if (__ldg(tail_count) > 0) {
    int e = __ldg(&rowptr[m]);
    const int e1 = __ldg(&kept_end[m]);
    for (; e + FWD_FLY <= e1; e += FWD_FLY) {
      uint2 t[FWD_FLY];
      uint4 d[FWD_FLY];
#pragma unroll
      for (int u = 0; u < FWD_FLY; ++u) t[u] = __ldg(&kept[e + u]);
#pragma unroll
      for (int u = 0; u < FWD_FLY; ++u) d[u] = __ldg(&w[(long long)t[u].x * vec_per_row + vcol]);
#pragma unroll
      for (int u = 0; u < FWD_FLY; ++u) fma8(acc, __uint_as_float(t[u].y), d[u]);
    }
    for (; e + 4 <= e1; e += 4) {
      uint2 t[4];
      uint4 d[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) t[u] = __ldg(&kept[e + u]);
#pragma unroll
      for (int u = 0; u < 4; ++u) d[u] = __ldg(&w[(long long)t[u].x * vec_per_row + vcol]);
#pragma unroll
      for (int u = 0; u < 4; ++u) fma8(acc, __uint_as_float(t[u].y), d[u]);
    }
    for (; e < e1; ++e) {
      const uint2 t = __ldg(&kept[e]);
      fma8(acc, __uint_as_float(t.y), __ldg(&w[(long long)t.x * vec_per_row + vcol]));
    }
  } else {
    sparse_row_times_dense(acc, col, val, __ldg(&rowptr[m]), __ldg(&rowptr[m + 1]), w, vec_per_row, vcol);
  }
  const float y8[8] = {a.x + acc[0], a.y + acc[1], a.z + acc[2], a.w + acc[3],
                       b.x + acc[4], b.y + acc[5], b.z + acc[6], b.w + acc[7]};
  store8(y, out_f32, off, y8);
}

constexpr int LONG_COLUMN = 512;           // entries from which a column gets a whole 1024-thread block
constexpr int LONG_THREADS = 1024;

// Exclusive scan of one int per thread over a 1024-thread block; the block's total goes to *total.
__device__ __forceinline__ int block_exclusive_scan_1024(int c, int* warp_tot, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = c;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
    if (lane >= off) incl += up;
  }
  __syncthreads();                                   // warp_tot may still be read from the previous scan
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int v = warp_tot[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, v, off);
      if (lane >= off) v += up;
    }
    warp_tot[lane] = v;
  }
  __syncthreads();
  *total = warp_tot[31];
  return incl - c + (warp ? warp_tot[warp - 1] : 0);
}

// Hot columns of the residual for the forward GEMM's dense tail: the first TAIL_MAX_COLS columns, in
// ascending order, that hold at least `hot_from` entries.  slot_of_col[k] is column k's position
// among them or -1, list_hot the inverse, *count their number.
__global__ void __launch_bounds__(1024, 1)
hot_columns_kernel(const int* __restrict__ colptr, int K, int hot_from, int* __restrict__ list_hot,
                   int* __restrict__ slot_of_col, int* __restrict__ count) {
  __shared__ int warp_tot[32];
  const int t = threadIdx.x;
  const int per = (K + 1023) / 1024;
  const int b = min(K, t * per), e = min(K, b + per);
  int c = 0;
  for (int k = b; k < e; ++k) c += (colptr[k + 1] - colptr[k] >= hot_from) ? 1 : 0;
  int total;
  int rank = block_exclusive_scan_1024(c, warp_tot, &total);
  for (int k = b; k < e; ++k) {
    int slot = -1;
    if (colptr[k + 1] - colptr[k] >= hot_from) {
      if (rank < TAIL_MAX_COLS) { slot = rank; list_hot[rank] = k; }
      ++rank;
    }
    slot_of_col[k] = slot;
  }
  if (t == 0) *count = min(total, TAIL_MAX_COLS);
}

// Two-term FP16 split of x: hi = RN16(x), lo = RN16(x - hi), stored for the cross products as
// hi_small = hi / TAIL_BALANCE and lo_big = TAIL_BALANCE * lo (exact powers of two: see GemmTail).
__device__ __forceinline__ void split_half(float x, __half& hi, __half& hi_small, __half& lo_big) {
  hi = __float2half_rn(x);
  const float h = __half2float(hi);
  hi_small = __float2half_rn(h * (1.0f / TAIL_BALANCE));
  lo_big = __float2half_rn((x - h) * TAIL_BALANCE);
}

// A operand of the dense tail: row m holds, for hot column s = 64 j + c, the value
// x = residual[m, k_s] / (d_A[m] * TAIL_SCALE) as x_hi at column 192 j + c, x_hi / TAIL_BALANCE at
// 192 j + 64 + c and TAIL_BALANCE x_lo at 192 j + 128 + c; zero elsewhere.  One warp per token walks the token's CSR row.  A value
// that FP16 cannot hold (or a token whose de-scale is zero) switches the tail off for this call:
// *count becomes 0 and the per-entry kernel keeps every entry.
__global__ void __launch_bounds__(COMP_THREADS)
tail_a_kernel(const int* __restrict__ rowptr, const int* __restrict__ col, const float* __restrict__ val,
              const int* __restrict__ slot_of_col, int* __restrict__ count, const float* __restrict__ amax_row,
              float row_div, __half* __restrict__ ta, int M, uint2* __restrict__ kept, int* __restrict__ kept_end) {
  const int hot = *count;
  if (hot == 0) return;
  const int lane = threadIdx.x & 31;
  const int m = blockIdx.x * (COMP_THREADS / 32) + (threadIdx.x >> 5);
  if (m >= M) return;
  uint32_t* row32 = reinterpret_cast<uint32_t*>(ta + size_t(m) * TAIL_WIDTH);
  for (int i = lane; i < TAIL_WIDTH / 2; i += 32) row32[i] = 0u;
  __syncwarp();
  const float scale = __fdiv_rn(__ldg(&amax_row[m]), row_div) * TAIL_SCALE;
  __half* row = ta + size_t(m) * TAIL_WIDTH;
  bool bad = false;
  const int e0 = rowptr[m], e1 = rowptr[m + 1];
  int n_kept = e0;                                       // the kept entries go to this token's own range
  for (int base = e0; base < e1; base += 32) {
    const int e = base + lane;
    int k = 0, slot = -1;
    float v = 0.0f;
    if (e < e1) {
      k = col[e];
      v = val[e];
      slot = slot_of_col[k];
    }
    const bool is_hot = e < e1 && unsigned(slot) < unsigned(hot);
    const bool keep = e < e1 && !is_hot;
    if (kept) {                                          // entries the tail does not cover, in column order
      const unsigned km = __ballot_sync(0xFFFFFFFFu, keep);
      if (keep) kept[n_kept + __popc(km & ((1u << lane) - 1u))] = make_uint2(uint32_t(k), __float_as_uint(v));
      n_kept += __popc(km);
    }
    if (!is_hot) continue;
    const float x = __fdiv_rn(v, scale);
    if (!(fabsf(x) <= 65504.0f)) { bad = true; continue; }         // also catches NaN (0 / 0)
    __half hi, hi_small, lo_big;
    split_half(x, hi, hi_small, lo_big);
    const int at = 192 * (slot >> 6) + (slot & 63);
    row[at] = hi;
    row[at + 64] = hi_small;
    row[at + 128] = lo_big;
  }
  if (kept && lane == 0) kept_end[m] = n_kept;
  if (bad) atomicExch(count, 0);
}

// B operand of the dense tail: row n holds, for hot column s = 64 j + c, the value
// x = TAIL_SCALE * W[k_s, n] / d_W[n] as x_hi at 192 j + c, TAIL_BALANCE x_lo at 192 j + 64 + c and
// x_hi / TAIL_BALANCE at 192 j + 128 + c (|x| <= 6 * 4, or 448 * 4 for an FP8 weight: the weight is at
// most amax in magnitude).  The buffer
// was cleared before.  One thread per (n, group of hot columns).
__global__ void __launch_bounds__(256)
tail_b_kernel(const __nv_bfloat16* __restrict__ w, const int* __restrict__ list_hot, const int* __restrict__ count,
              const float* __restrict__ amax_col, float col_div, __half* __restrict__ tb, int N) {
  const int hot = *count;
  const int n = blockIdx.x * 256 + threadIdx.x;
  if (n >= N) return;
  const float d = __fdiv_rn(__ldg(&amax_col[n]), col_div);
  const float inv_ok = d > 0.0f ? 1.0f : 0.0f;
  __half* row = tb + size_t(n) * TAIL_WIDTH;
  for (int s = blockIdx.y; s < hot; s += gridDim.y) {
    const float wv = __bfloat162float(w[size_t(list_hot[s]) * N + n]);
    const float x = inv_ok != 0.0f ? __fdiv_rn(wv * TAIL_SCALE, d) : 0.0f;
    __half hi, hi_small, lo_big;
    split_half(x, hi, hi_small, lo_big);
    const int at = 192 * (s >> 6) + (s & 63);
    row[at] = hi;
    row[at + 64] = lo_big;
    row[at + 128] = hi_small;
  }
}

// The columns of the residual that hold entries, by how full they are: "dense" (at least
// `dense_from` entries, the first DENSE_TC_MAX of them: outlier channels that most tokens hit,
// Appendix D), "long" (at least LONG_COLUMN entries) and "short".  The long and the short ones
// are listed in ascending order; counts[0..2] are the three sizes.  Rows of the compact buffer:
// dense columns first, then the long, then the short ones, each in ascending column order;
// slot_of_col[k] is column k's row or -1.  dense_from = INT_MAX switches the dense class off.
__global__ void __launch_bounds__(1024, 1)
nonempty_columns_kernel(const int* __restrict__ colptr, int K, int dense_from, int* __restrict__ list_long,
                        int* __restrict__ list_short, int* __restrict__ counts, int* __restrict__ slot_of_col) {
  __shared__ int warp_tot[32];
  const int t = threadIdx.x;
  const int per = (K + 1023) / 1024;
  const int b = min(K, t * per), e = min(K, b + per);
  int c_cand = 0;
  for (int k = b; k < e; ++k) c_cand += (colptr[k + 1] - colptr[k] >= dense_from) ? 1 : 0;
  int n_cand;
  int rank = block_exclusive_scan_1024(c_cand, warp_tot, &n_cand);     // dense candidates before this thread
  const int n_dense = min(n_cand, DENSE_TC_MAX);
  int c_long = 0, c_short = 0;
  {
    int r = rank;
    for (int k = b; k < e; ++k) {
      const int n = colptr[k + 1] - colptr[k];
      if (n >= dense_from && r++ < DENSE_TC_MAX) continue;
      if (n >= LONG_COLUMN) ++c_long;
      else if (n > 0) ++c_short;
    }
  }
  int n_long, n_short;
  int pos_long = block_exclusive_scan_1024(c_long, warp_tot, &n_long);
  int pos_short = block_exclusive_scan_1024(c_short, warp_tot, &n_short);
  for (int k = b; k < e; ++k) {
    const int n = colptr[k + 1] - colptr[k];
    int slot = -1;
    if (n >= dense_from && rank < DENSE_TC_MAX) slot = rank;
    else if (n >= LONG_COLUMN) { slot = n_dense + pos_long; list_long[pos_long++] = k; }
    else if (n > 0) { slot = n_dense + n_long + pos_short; list_short[pos_short++] = k; }
    if (n >= dense_from) ++rank;
    slot_of_col[k] = slot;
  }
  if (t == 0) {
    counts[0] = n_dense;
    counts[1] = n_long;
    counts[2] = n_short;
  }
}

// Dense columns (their partial sums come from the tensor-core kernel, one set per range of tokens):
// C[slot, n] = sum over the ranges, in order.
__global__ void __launch_bounds__(256)
dense_reduce_kernel(float* __restrict__ comp, const float* __restrict__ partial, const int* __restrict__ counts, int N,
                    int chunks, long long chunk_stride) {
  const long long total = (long long)counts[0] * N;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    float t = 0.0f;
    for (int c0 = 0; c0 < chunks; c0 += 8) {            // eight loads in flight, added in chunk order
      float p[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) p[u] = c0 + u < chunks ? __ldg(&partial[(long long)(c0 + u) * chunk_stride + i]) : 0.0f;
#pragma unroll
      for (int u = 0; u < 8; ++u) t += p[u];
    }
    comp[i] = t;
  }
}

// acc[0..7] += sum of val[e] * dense[idx[e], vcol] over e = first, first + step, ... < e1, eight
// gathers in flight and the indices of the next round fetched under them.
__device__ __forceinline__ void strided_entries_times_dense(float (&acc)[8], const int* __restrict__ idx,
                                                            const float* __restrict__ val, int first, int e1,
                                                            int step, const uint4* __restrict__ dense,
                                                            int vec_per_row, int vcol) {
  int r[8];
  float v[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const bool live = first + step * u < e1;          // past the end: value 0 times row 0
    r[u] = live ? __ldg(&idx[first + step * u]) : 0;
    v[u] = live ? __ldg(&val[first + step * u]) : 0.0f;
  }
  for (int e = first; e < e1; e += 8 * step) {
    uint4 d[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) d[u] = __ldg(&dense[(long long)r[u] * vec_per_row + vcol]);
    int rn[8];
    float vn[8];
    const int nxt = e + 8 * step;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const bool live = nxt + step * u < e1;
      rn[u] = live ? __ldg(&idx[nxt + step * u]) : 0;
      vn[u] = live ? __ldg(&val[nxt + step * u]) : 0.0f;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) fma8(acc, v[u], d[u]);
#pragma unroll
    for (int u = 0; u < 8; ++u) { r[u] = rn[u]; v[u] = vn[u]; }
  }
}

__device__ __forceinline__ void store8_f32(float* dst, const float (&t)[8]) {
  *reinterpret_cast<float4*>(dst) = make_float4(t[0], t[1], t[2], t[3]);
  *reinterpret_cast<float4*>(dst + 4) = make_float4(t[4], t[5], t[6], t[7]);
}

// Weight-gradient compensation, step 1: S[k, n-block] += sum over the entries of column k of
// dA[m,k] * dY[m, n-block].  Outliers sit in a few channels (Appendix D): a handful of columns
// hold thousands of entries, a few hundred hold one or two, most hold none.
// Long columns: one 1024-thread block per (column, 256 outputs); its 32 warps take the entries
// round-robin and their partial sums are added in warp order (independent of scheduling).
__global__ void __launch_bounds__(LONG_THREADS, 1)
comp_wgrad_long_kernel(float* __restrict__ comp, const int* __restrict__ colptr, const int* __restrict__ row,
                       const float* __restrict__ val, const uint4* __restrict__ dy, const int* __restrict__ list,
                       const int* __restrict__ count, int N) {
  __shared__ float part[32][32][9];                 // [warp][lane][8 (+1 pad)]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * COMP_COLS + 8 * lane;
  const bool in_cols = n0 < N;
  const int n_dense = count[0], n_cols = count[1];
  for (int slot = blockIdx.y; slot < n_cols; slot += gridDim.y) {
    const int k = list[slot];
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (in_cols)
      strided_entries_times_dense(acc, row, val, colptr[k] + warp, colptr[k + 1], 32, dy, N >> 3, n0 >> 3);
    __syncthreads();                                // the previous column's partials have been read
#pragma unroll
    for (int c = 0; c < 8; ++c) part[warp][lane][c] = acc[c];
    __syncthreads();
    if (warp == 0 && in_cols) {
      float t[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      for (int w = 0; w < 32; ++w) {
#pragma unroll
        for (int c = 0; c < 8; ++c) t[c] += part[w][lane][c];
      }
      store8_f32(comp + (long long)(n_dense + slot) * N + n0, t);
    }
  }
}

// Short columns: one warp per (column, 256 outputs), entries in order.  The work items (block of 256
// outputs, group of 8 columns) are numbered with the block of outputs as the slow index and taken
// in that order, so that the blocks in flight at any time read one or two 512-byte-wide slabs of dY
// (tokens x 512 bytes: a few MB, which stay in L2) instead of all of it: every token's piece of a
// slab is gathered by about 1 % of the columns, and those re-reads then hit L2.
__global__ void __launch_bounds__(COMP_THREADS, 4)
comp_wgrad_short_kernel(float* __restrict__ comp, const int* __restrict__ colptr, const int* __restrict__ row,
                        const float* __restrict__ val, const uint4* __restrict__ dy, const int* __restrict__ list,
                        const int* __restrict__ counts, int N) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_before = counts[0] + counts[1], n_cols = counts[2];
  const int groups = (n_cols + 7) >> 3;
  const int n_blocks = (N + COMP_COLS - 1) / COMP_COLS;
  const long long items = (long long)groups * n_blocks;
  for (long long it = blockIdx.x; it < items; it += gridDim.x) {
    const int nb = int(it / groups);
    const int slot = int(it - (long long)nb * groups) * 8 + warp;
    const int n0 = nb * COMP_COLS + 8 * lane;
    if (slot >= n_cols || n0 >= N) continue;
    const int k = list[slot];
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    {
      const int vec_per_row = N >> 3, vcol = n0 >> 3;
      int e = colptr[k];
      const int e1 = colptr[k + 1];
      for (; e + 8 <= e1; e += 8) {                 // eight gathers in flight, entries in order
        int r[8];
        float v[8];
        uint4 d[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) { r[u] = __ldg(&row[e + u]); v[u] = __ldg(&val[e + u]); }
#pragma unroll
        for (int u = 0; u < 8; ++u) d[u] = __ldg(&dy[(long long)r[u] * vec_per_row + vcol]);
#pragma unroll
        for (int u = 0; u < 8; ++u) fma8(acc, v[u], d[u]);
      }
      for (; e < e1; ++e) fma8(acc, __ldg(&val[e]), __ldg(&dy[(long long)__ldg(&row[e]) * vec_per_row + vcol]));
    }
    store8_f32(comp + (long long)(n_before + slot) * N + n0, acc);
  }
}

// Measurement support: every block reads the whole buffer once per repeat with 16-byte loads that
// bypass L1, starting at its own offset, so that a buffer smaller than L2 is served by L2 alone.
__global__ void __launch_bounds__(256)
l2_read_probe_kernel(const uint4* __restrict__ buf, long long n_vec, int repeats, unsigned* __restrict__ sink) {
  unsigned acc = 0;
  const long long start = ((long long)blockIdx.x * 9973 * 256) % n_vec;
  for (int r = 0; r < repeats; ++r) {
    for (long long i0 = 0; i0 < n_vec; i0 += 8 * 256) {
      uint4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        long long i = start + i0 + u * 256 + threadIdx.x;
        if (i >= n_vec) i -= n_vec;
        if (i >= n_vec) i -= n_vec;
        asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(v[u].x), "=r"(v[u].y), "=r"(v[u].z), "=r"(v[u].w)
                     : "l"(buf + i));
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
  }
  if (acc == 0x9E3779B9u) *sink = acc;               // keeps the loads alive
}

}  // namespace

extern "C" int fp4_l2_read_probe(void* stream, const void* buf, size_t bytes, int repeats, int blocks, unsigned* sink) {
  if (!buf || !sink) return FP4_ERR_NULL;
  if (bytes < 4096 * 16 || (bytes % (8 * 256 * 16)) || repeats <= 0 || blocks <= 0 ||
      (reinterpret_cast<uintptr_t>(buf) & 15))
    return FP4_ERR_ARG;
  l2_read_probe_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(buf), (long long)(bytes / 16), repeats, sink);
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}

int launch_comp_fwd(fp4_ctx* ctx, cudaStream_t stream, const float* y1, const int32_t* rowptr, const int32_t* col,
                    const float* val, const void* w_bf16, int64_t M, int64_t, int64_t N, void* y, int out_f32,
                    const int* slot_of_col, const int* tail_count, const void* kept, const int* kept_end) {
  const dim3 grid(unsigned((M + 7) / 8), unsigned((N + COMP_COLS - 1) / COMP_COLS));
  KernelScope scope(ctx, stream, KC_COMP_FWD, 1);
  if (kept && kept_end && tail_count)
    comp_fwd_kept_kernel<<<grid, COMP_THREADS, 0, stream>>>(y1, rowptr, col, val, static_cast<const uint2*>(kept),
                                                            kept_end, static_cast<const uint4*>(w_bf16), int(M), int(N),
                                                            y, out_f32, tail_count);
  else if (slot_of_col && tail_count)
    comp_fwd_skip_kernel<<<grid, COMP_THREADS, 0, stream>>>(y1, rowptr, col, val, static_cast<const uint4*>(w_bf16),
                                                            int(M), int(N), y, out_f32, slot_of_col, tail_count);
  else
    comp_fwd_kernel<<<grid, COMP_THREADS, 0, stream>>>(y1, rowptr, col, val, static_cast<const uint4*>(w_bf16), int(M),
                                                       int(N), y, out_f32);
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}

size_t comp_wgrad_scratch_bytes(int64_t M, int64_t K, int64_t N) {
  auto r256 = [](size_t b) { return (b + 255) & ~size_t(255); };
  size_t b = r256((2 * size_t(K) + 4) * 4) + r256(size_t(K) * 4);                     // lists + counters, slots
  b += dense_tc_scratch_bytes(M, N);                                                  // BF16 terms, partial sums
  return b;
}

// Residual entries up to which the forward lists the entries its dense tail does not cover
// (4 % of the activation: alpha >= 0.98); heavier residuals filter inside the per-entry kernel.
static int64_t kept_list_capacity(int64_t M, int64_t K) { return M * K / 25; }

size_t fwd_tail_scratch_bytes(int64_t M, int64_t K, int64_t N) {
  auto r256 = [](size_t b) { return (b + 255) & ~size_t(255); };
  return r256(size_t(M) * TAIL_WIDTH * 2) + r256(size_t(N) * TAIL_WIDTH * 2) + r256(size_t(K) * 4) +
         r256(TAIL_MAX_COLS * 4) + 256 + r256(size_t(kept_list_capacity(M, K)) * 8) + r256(size_t(M) * 4);
}

// Prepares the dense tail of the forward GEMM from the saved activation `a` (CSR, CSC column
// pointers, row amax) and the weights; fills `tail` and hands back the slot vector and the count
// for the per-entry kernel.  Buffers come from `scratch` (fwd_tail_scratch_bytes).
int launch_fwd_tail(fp4_ctx* ctx, cudaStream_t stream, const fp4_qtensor* a, const void* w_bf16, const float* w_amax,
                    float w_div, Arena& scratch, int64_t M, int64_t K, int64_t N, GemmTail* tail,
                    const int** slot_of_col_out, const void** kept_out, const int** kept_end_out) {
  __half* ta = scratch.take<__half>(size_t(M) * TAIL_WIDTH);
  __half* tb = scratch.take<__half>(size_t(N) * TAIL_WIDTH);
  int* slot_of_col = scratch.take<int>(size_t(K));
  int* list_hot = scratch.take<int>(TAIL_MAX_COLS);
  int* count = scratch.take<int>(1);
  const bool list_kept = a->sparse_cap <= kept_list_capacity(M, K);
  uint2* kept = list_kept ? scratch.take<uint2>(size_t(kept_list_capacity(M, K))) : nullptr;
  int* kept_end = list_kept ? scratch.take<int>(size_t(M)) : nullptr;
  if (!scratch.ok) return FP4_ERR_WORKSPACE;
  *kept_out = kept;
  *kept_end_out = kept_end;
  const int hot_from = int(M / 4 > LONG_COLUMN ? M / 4 : LONG_COLUMN);
  KernelScope scope(ctx, stream, KC_COMP_FWD, 3);
  hot_columns_kernel<<<1, 1024, 0, stream>>>(a->csc_colptr, int(K), hot_from, list_hot, slot_of_col, count);
  FP4_CUDA_TRY(cudaMemsetAsync(tb, 0, size_t(N) * TAIL_WIDTH * 2, stream));
  tail_a_kernel<<<unsigned((M + 7) / 8), COMP_THREADS, 0, stream>>>(a->csr_rowptr, a->csr_col, a->csr_val, slot_of_col,
                                                                   count, a->amax, 6.0f, ta, int(M), kept, kept_end);
  tail_b_kernel<<<dim3(unsigned((N + 255) / 256), 16), 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(w_bf16),
                                                                        list_hot, count, w_amax, w_div, tb, int(N));
  FP4_CUDA_TRY(cudaGetLastError());
  tail->a = ta;
  tail->b = tb;
  tail->count = count;
  *slot_of_col_out = slot_of_col;
  return FP4_OK;
}

int launch_comp_wgrad(fp4_ctx* ctx, cudaStream_t stream, const fp4_qtensor* a, const void* dy_bf16, Arena& scratch,
                      int** slot_of_col_out, float* comp, int64_t M, int64_t K, int64_t N, int32_t* status) {
  // lists: [K] long columns, [K] short columns, three counters
  int* lists = scratch.take<int>(2 * size_t(K) + 4);
  int* slot_of_col = scratch.take<int>(size_t(K));
  const int splits = dense_tc_splits(ctx, M, N);
  void* vt = scratch.take<uint16_t>(size_t(3) * DENSE_TC_MAX * size_t(M));
  float* partial = scratch.take<float>(size_t(splits) * DENSE_TC_MAX * size_t(N));
  if (!scratch.ok) return FP4_ERR_WORKSPACE;
  *slot_of_col_out = slot_of_col;
  int* list_long = lists;
  int* list_short = lists + K;
  int* counts = lists + 2 * K;
  // Columns that at least a quarter of the tokens hit (the outlier channels) form the dense class,
  // whose product runs on the tensor cores; it needs the CSR.  It costs three launches, which pay
  // when the residual is heavy: when it may hold at least 1 % of the activation (alpha <= 0.995).
  // (No column can reach LONG_COLUMN entries with fewer tokens than that.)
  const bool dense = a->csr_rowptr != nullptr && a->sparse_cap * 100 >= M * K && M >= LONG_COLUMN;
  const int dense_from = dense ? int(M / 4 > LONG_COLUMN ? M / 4 : LONG_COLUMN) : INT_MAX;
  const unsigned n_blocks = unsigned((N + COMP_COLS - 1) / COMP_COLS);
  KernelScope scope(ctx, stream, KC_COMP_WGRAD, 3 + (dense ? (splits > 1 ? 3 : 2) : 0));
  nonempty_columns_kernel<<<1, 1024, 0, stream>>>(a->csc_colptr, int(K), dense_from, list_long, list_short, counts,
                                                  slot_of_col);
  const uint4* dy = static_cast<const uint4*>(dy_bf16);
  if (dense) {
    const int rc = launch_comp_wgrad_dense_tc(ctx, stream, a, slot_of_col, counts, dy_bf16, vt,
                                              splits > 1 ? partial : comp, splits, M, N, status);
    if (rc != FP4_OK) return rc;
    if (splits > 1)
      dense_reduce_kernel<<<unsigned(2 * ctx->num_sms), 256, 0, stream>>>(comp, partial, counts, int(N), splits,
                                                                         (long long)DENSE_TC_MAX * N);
  }
  unsigned gy = unsigned(4 * ctx->num_sms) / n_blocks;          // long columns: 2 resident blocks per SM
  gy = gy < 1 ? 1 : (gy > unsigned(K) ? unsigned(K) : gy);
  comp_wgrad_long_kernel<<<dim3(n_blocks, gy), LONG_THREADS, 0, stream>>>(comp, a->csc_colptr, a->csc_row, a->csc_val,
                                                                         dy, list_long, counts, int(N));
  {
    // short columns: 8 per block; about 32 blocks per SM in all, each taking work items in order
    const long long max_items = (long long)((K + 7) / 8) * n_blocks;
    long long g = 32LL * ctx->num_sms;
    g = g > max_items ? max_items : g;
    comp_wgrad_short_kernel<<<unsigned(g), COMP_THREADS, 0, stream>>>(comp, a->csc_colptr, a->csc_row, a->csc_val, dy,
                                                                      list_short, counts, int(N));
  }
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}
