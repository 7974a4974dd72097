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
  const int m = blockIdx.y * 8 + (threadIdx.x >> 5);
  const int n0 = blockIdx.x * COMP_COLS + 8 * (threadIdx.x & 31);
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

constexpr int LONG_COLUMN = 64;            // entries from which a column gets a whole 1024-thread block
constexpr int LONG_THREADS = 1024;

// Two ascending lists of the columns that hold residual entries: "long" columns (at least
// LONG_COLUMN entries: the outlier channels) and "short" ones; counts[0], counts[1] their sizes.
__global__ void __launch_bounds__(1024, 1)
nonempty_columns_kernel(const int* __restrict__ colptr, int K, int* __restrict__ list_long,
                        int* __restrict__ list_short, int* __restrict__ counts, int* __restrict__ slot_of_col) {
  __shared__ unsigned long long warp_tot[32];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int per = (K + 1023) / 1024;
  const int b = min(K, t * per), e = min(K, b + per);
  unsigned long long c = 0;                          // low word: long columns, high word: short columns
  for (int k = b; k < e; ++k) {
    const int n = colptr[k + 1] - colptr[k];
    if (n >= LONG_COLUMN) c += 1ull;
    else if (n > 0) c += 1ull << 32;
  }
  unsigned long long incl = c;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
    if (lane >= off) incl += up;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    unsigned long long v = warp_tot[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, v, off);
      if (lane >= off) v += up;
    }
    warp_tot[lane] = v;
  }
  __syncthreads();
  const unsigned long long before = incl - c + (warp ? warp_tot[warp - 1] : 0ull);
  // rows of the compact buffer: long columns first (in list order), then the short ones
  const int n_long = int(warp_tot[31] & 0xFFFFFFFFull);
  int pos_long = int(before & 0xFFFFFFFFull), pos_short = int(before >> 32);
  for (int k = b; k < e; ++k) {
    const int n = colptr[k + 1] - colptr[k];
    int slot = -1;
    if (n >= LONG_COLUMN) { slot = pos_long; list_long[pos_long++] = k; }
    else if (n > 0) { slot = n_long + pos_short; list_short[pos_short++] = k; }
    slot_of_col[k] = slot;
  }
  if (t == 1023) {
    counts[0] = int(warp_tot[31] & 0xFFFFFFFFull);
    counts[1] = int(warp_tot[31] >> 32);
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
  const int n_cols = *count;
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
      store8_f32(comp + (long long)slot * N + n0, t);
    }
  }
}

// Short columns: one warp per (column, 256 outputs), entries in order.
__global__ void __launch_bounds__(COMP_THREADS)
comp_wgrad_short_kernel(float* __restrict__ comp, const int* __restrict__ colptr, const int* __restrict__ row,
                        const float* __restrict__ val, const uint4* __restrict__ dy, const int* __restrict__ list,
                        const int* __restrict__ counts, int N) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * COMP_COLS + 8 * lane;
  if (n0 >= N) return;
  const int n_long = counts[0], n_cols = counts[1];
  for (int slot = blockIdx.y * 8 + warp; slot < n_cols; slot += gridDim.y * 8) {
    const int k = list[slot];
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    strided_entries_times_dense(acc, row, val, colptr[k], colptr[k + 1], 1, dy, N >> 3, n0 >> 3);
    store8_f32(comp + (long long)(n_long + slot) * N + n0, acc);
  }
}

}  // namespace

int launch_comp_fwd(fp4_ctx* ctx, cudaStream_t stream, const float* y1, const int32_t* rowptr, const int32_t* col,
                    const float* val, const void* w_bf16, int64_t M, int64_t, int64_t N, void* y, int out_f32) {
  const dim3 grid(unsigned((N + COMP_COLS - 1) / COMP_COLS), unsigned((M + 7) / 8));
  KernelScope scope(ctx, stream, KC_COMP_FWD, 1);
  comp_fwd_kernel<<<grid, COMP_THREADS, 0, stream>>>(y1, rowptr, col, val, static_cast<const uint4*>(w_bf16), int(M),
                                                     int(N), y, out_f32);
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}

int launch_comp_wgrad(fp4_ctx* ctx, cudaStream_t stream, const int32_t* colptr, const int32_t* row, const float* val,
                      const void* dy_bf16, int* lists, int* slot_of_col, float* comp, int64_t K, int64_t N) {
  KernelScope scope(ctx, stream, KC_COMP_WGRAD, 3);
  // lists: [K] long columns, [K] short columns, two counters
  int* list_long = lists;
  int* list_short = lists + K;
  int* counts = lists + 2 * K;
  nonempty_columns_kernel<<<1, 1024, 0, stream>>>(colptr, int(K), list_long, list_short, counts, slot_of_col);
  const unsigned n_blocks = unsigned((N + COMP_COLS - 1) / COMP_COLS);
  const uint4* dy = static_cast<const uint4*>(dy_bf16);
  unsigned gy = unsigned(4 * ctx->num_sms) / n_blocks;          // long columns: 2 resident blocks per SM
  gy = gy < 1 ? 1 : (gy > unsigned(K) ? unsigned(K) : gy);
  comp_wgrad_long_kernel<<<dim3(n_blocks, gy), LONG_THREADS, 0, stream>>>(comp, colptr, row, val, dy, list_long,
                                                                         counts, int(N));
  gy = unsigned(32 * ctx->num_sms) / n_blocks;                   // short columns: 8 per block
  gy = gy < 1 ? 1 : (gy > unsigned((K + 7) / 8) ? unsigned((K + 7) / 8) : gy);
  comp_wgrad_short_kernel<<<dim3(n_blocks, gy), COMP_THREADS, 0, stream>>>(comp, colptr, row, val, dy, list_short,
                                                                           counts, int(N));
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}
