// Quantiser kernels: exact quantile selection, clamp, vector-wise absmax, E2M1 encoding in both
// packed layouts, and extraction of the sparse residual (Eq. 1, Appendix A, Section 3.2).
//
// Passes over a [rows x cols] BF16 tensor:
//   with outlier clamping (activations)
//     1. hist_rowminmax   one read: 65536-bin histogram of the BF16 bit patterns (exact, in shared
//                         memory) + signed max / min of every row
//     2. select           cumulative counts -> the two order statistics lo, hi (bit exact)
//     3. encode           one read: clamp, per-row scale from the clamped row extremes, Q, both
//                         nibble layouts, and a 1-bit-per-element mask of the clamped entries
//     4. mask -> CSR/CSC  counts, prefix sums and ordered fills driven by the mask (1/16 of the
//                         tensor); values are gathered from the few marked entries
//   without clamping (weights, output gradients)
//     1. absmax           one read: max |x| per row or per column (after the optional prescale)
//     2. encode           one read
#include "common.cuh"

namespace {

constexpr int HIST_THREADS = 1024;
constexpr int HIST_WORDS = 32768;                 // two 16-bit counters per word
constexpr int ENC_TM = 64;                        // tile rows of the encoder
constexpr int ENC_TK = 256;                       // tile columns
constexpr int ENC_THREADS = 256;
constexpr int MAX_SPLITS = 64;

__device__ __forceinline__ int float_to_ordered(float f) {
  const int b = __float_as_int(f);
  return b ^ ((b >> 31) & 0x7FFFFFFF);            // signed integer order == float order
}
__device__ __forceinline__ float ordered_to_float(int k) {
  return __int_as_float(k ^ ((k >> 31) & 0x7FFFFFFF));
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// ------------------------------------------------------------------------------------------
// 1. histogram of bit patterns + row extremes
// ------------------------------------------------------------------------------------------
__global__ void init_row_extremes_kernel(int* row_max, int* row_min, int rows) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < rows) {
    row_max[i] = INT_MIN;
    row_min[i] = INT_MAX;
  }
}

// Shared-memory counters are 16-bit pairs.  A counter that reaches 0x8000 is moved to the global
// histogram by the thread that made it so.  Between two block barriers the block adds at most
// 8192 elements, so a counter stays below 0xC000 and never carries into its neighbour.
__device__ __forceinline__ void bump(uint32_t* h, uint32_t* ghist, uint32_t bits) {
  const uint32_t sh = (bits & 1u) << 4;
  const uint32_t old = atomicAdd(&h[bits >> 1], 1u << sh);
  if (((old >> sh) & 0xFFFFu) == 0x7FFFu) {
    atomicSub(&h[bits >> 1], 0x8000u << sh);
    atomicAdd(&ghist[bits], 0x8000u);
  }
}

__global__ void __launch_bounds__(HIST_THREADS, 1)
hist_rowminmax_kernel(const uint4* __restrict__ x, long long n_vec, int vec_per_row, uint32_t* __restrict__ ghist,
                      int* __restrict__ row_max, int* __restrict__ row_min) {
  extern __shared__ uint32_t h[];
  for (int i = threadIdx.x; i < HIST_WORDS; i += HIST_THREADS) h[i] = 0;
  __syncthreads();
  const long long stride = (long long)gridDim.x * HIST_THREADS;
  long long i = (long long)blockIdx.x * HIST_THREADS + threadIdx.x;
  uint4 nxt = make_uint4(0, 0, 0, 0);
  if (i < n_vec) nxt = __ldg(&x[i]);
  for (long long base = (long long)blockIdx.x * HIST_THREADS; base < n_vec; base += stride, i += stride) {
    const uint4 v = nxt;
    const bool valid = i < n_vec;
    if (i + stride < n_vec) nxt = __ldg(&x[i + stride]);
    if (valid) {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        bump(h, ghist, w[q] & 0xFFFFu);
        bump(h, ghist, w[q] >> 16);
      }
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(w);
      const __nv_bfloat162 mx = __hmax2(__hmax2(p[0], p[1]), __hmax2(p[2], p[3]));
      const __nv_bfloat162 mn = __hmin2(__hmin2(p[0], p[1]), __hmin2(p[2], p[3]));
      int kmax = float_to_ordered(fmaxf(__low2float(mx), __high2float(mx)));
      int kmin = float_to_ordered(fminf(__low2float(mn), __high2float(mn)));
      // 16 consecutive vectors (128 elements) never straddle a row: cols is a multiple of 128
      const unsigned group = (threadIdx.x & 16) ? 0xFFFF0000u : 0x0000FFFFu;
      kmax = __reduce_max_sync(group, kmax);
      kmin = __reduce_min_sync(group, kmin);
      if ((threadIdx.x & 15) == 0) {
        const int row = int(i / vec_per_row);
        atomicMax(&row_max[row], kmax);
        atomicMin(&row_min[row], kmin);
      }
    }
    __syncthreads();
  }
  for (int idx = threadIdx.x; idx < HIST_WORDS; idx += HIST_THREADS) {
    const uint32_t w = h[idx];
    if (w & 0xFFFFu) atomicAdd(&ghist[2 * idx], w & 0xFFFFu);
    if (w >> 16) atomicAdd(&ghist[2 * idx + 1], w >> 16);
  }
}

// ------------------------------------------------------------------------------------------
// 2. order statistics from the histogram
// ------------------------------------------------------------------------------------------
// Position p in ascending real order: p < 32768 are the negative patterns from 0xFFFF down to
// 0x8000 (-0), p >= 32768 the non-negative patterns from 0x0000 up.
__device__ __forceinline__ uint32_t pos_to_bits(int p) { return p < 32768 ? uint32_t(0xFFFF - p) : uint32_t(p - 32768); }

__global__ void __launch_bounds__(1024, 1)
select_thresholds_kernel(const uint32_t* __restrict__ ghist, long long n, long long n_tail, float* thresholds) {
  __shared__ long long part[1024];
  __shared__ int found[2];
  const int t = threadIdx.x;
  long long s = 0;
  for (int p = 64 * t; p < 64 * t + 64; ++p) s += ghist[pos_to_bits(p)];
  part[t] = s;
  __syncthreads();
  // inclusive scan over the 1024 partial sums (Hillis-Steele; runs once per call)
  for (int off = 1; off < 1024; off <<= 1) {
    const long long add = t >= off ? part[t - off] : 0;
    __syncthreads();
    part[t] += add;
    __syncthreads();
  }
  const long long before = part[t] - s;            // entries in positions below 64 t
  const long long rank[2] = {n_tail, n - 1 - n_tail};
  for (int q = 0; q < 2; ++q) {
    if (rank[q] >= before && rank[q] < before + s) {
      long long cum = before;
      for (int p = 64 * t; p < 64 * t + 64; ++p) {
        cum += ghist[pos_to_bits(p)];
        if (cum > rank[q]) { found[q] = p; break; }
      }
    }
  }
  __syncthreads();
  if (t < 2) {
    uint32_t bits = pos_to_bits(found[t]);
    if (bits == 0x8000u) bits = 0;                 // thresholds are real numbers: -0 is +0
    thresholds[t] = __uint_as_float(bits << 16);
  }
}

// ------------------------------------------------------------------------------------------
// absmax without clamping
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float prescale_value(const float* p, int idx) { return __ldg(&p[idx]); }

// d[i] = amax[i] / 6 rounded once: the de-scale vector of a quantised operand, used as a prescale
__global__ void descale_kernel(const float* __restrict__ amax, int n, float* __restrict__ d) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) d[i] = __fdiv_rn(amax[i], 6.0f);
}

// one scale per row: flat sweep, 16-lane groups cover 128 consecutive elements of one row
template <bool PRESCALE>
__global__ void __launch_bounds__(256)
absmax_rows_kernel(const uint4* __restrict__ x, long long n_vec, int vec_per_row, const float* __restrict__ prescale,
                   uint32_t* __restrict__ vec_amax) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
    const uint4 v = __ldg(&x[i]);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    const int row = int(i / vec_per_row);
    const int c0 = int(i - (long long)row * vec_per_row) * 8;
    float m = 0.0f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float a = bf16_lo(w[q]), b = bf16_hi(w[q]);
      if (PRESCALE) {
        a = __fmul_rn(a, prescale_value(prescale, c0 + 2 * q));
        b = __fmul_rn(b, prescale_value(prescale, c0 + 2 * q + 1));
      }
      m = fmaxf(m, fmaxf(fabsf(a), fabsf(b)));
    }
    const unsigned group = (threadIdx.x & 16) ? 0xFFFF0000u : 0x0000FFFFu;
    const uint32_t gm = __reduce_max_sync(group, __float_as_uint(m));   // non-negative floats order as integers
    if ((threadIdx.x & 15) == 0) atomicMax(&vec_amax[row], gm);
  }
}

// one scale per column: each thread owns 8 adjacent columns over a strip of rows
template <bool PRESCALE>
__global__ void __launch_bounds__(256)
absmax_cols_kernel(const uint4* __restrict__ x, int rows, int vec_per_row, int rows_per_strip,
                   const float* __restrict__ prescale, uint32_t* __restrict__ vec_amax) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= vec_per_row) return;
  const int r0 = blockIdx.y * rows_per_strip;
  const int r1 = min(rows, r0 + rows_per_strip);
  float m[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll 4
  for (int r = r0; r < r1; ++r) {
    const uint4 v = __ldg(&x[(long long)r * vec_per_row + j]);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    const float p = PRESCALE ? prescale_value(prescale, r) : 1.0f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float a = bf16_lo(w[q]), b = bf16_hi(w[q]);
      if (PRESCALE) { a = __fmul_rn(a, p); b = __fmul_rn(b, p); }
      m[2 * q] = fmaxf(m[2 * q], fabsf(a));
      m[2 * q + 1] = fmaxf(m[2 * q + 1], fabsf(b));
    }
  }
#pragma unroll
  for (int c = 0; c < 8; ++c) atomicMax(&vec_amax[8 * j + c], __float_as_uint(m[c]));
}

// ------------------------------------------------------------------------------------------
// 3. encoder
// ------------------------------------------------------------------------------------------
// Q of Appendix A for eight float32 values -> eight nibbles (element 0 in bits 3:0).
// The chain sends a value that equals a threshold to the larger neighbour, i.e. it rounds to the
// nearest grid value with ties toward +infinity.  The hardware conversion rounds ties to even, so
// each input is first moved off the tie: its magnitude bits become (bits - sign) | 1.  Thresholds
// have a zero last bit, so no other value crosses one.  The conversion's "-0" nibble is cleared.
__device__ __forceinline__ float nudge(float v) {
  const uint32_t u = __float_as_uint(v);
  return __uint_as_float((u - (u >> 31)) | 1u);
}
__device__ __forceinline__ uint32_t encode8(const float (&v)[8]) {
  uint32_t w;
  asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
      "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
      : "=r"(w)
      : "f"(nudge(v[0])), "f"(nudge(v[1])), "f"(nudge(v[2])), "f"(nudge(v[3])), "f"(nudge(v[4])),
        "f"(nudge(v[5])), "f"(nudge(v[6])), "f"(nudge(v[7])));
  const uint32_t m = w & 0x77777777u;
  const uint32_t nz = (m | (m >> 1) | (m >> 2)) & 0x11111111u;   // 1 where the magnitude is not zero
  return w & ((nz << 3) | 0x77777777u);
}

// 8 x 8 nibble transpose: in[r] nibble c  ->  out[c] nibble r
__device__ __forceinline__ void transpose8x8_nibbles(uint32_t (&r)[8]) {
  uint32_t t[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {                       // swap the off-diagonal 4x4 blocks
    t[i] = __byte_perm(r[i], r[i + 4], 0x5410);
    t[i + 4] = __byte_perm(r[i], r[i + 4], 0x7632);
  }
#pragma unroll
  for (int g = 0; g < 8; g += 4) {                    // 2x2 blocks inside each 4x4 block
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      r[g + i] = __byte_perm(t[g + i], t[g + i + 2], 0x6240);
      r[g + i + 2] = __byte_perm(t[g + i], t[g + i + 2], 0x7351);
    }
  }
#pragma unroll
  for (int i = 0; i < 8; i += 2) {                    // single nibbles inside each 2x2 block
    const uint32_t a = r[i], b = r[i + 1];
    r[i] = (a & 0x0F0F0F0Fu) | ((b << 4) & 0xF0F0F0F0u);
    r[i + 1] = ((a >> 4) & 0x0F0F0F0Fu) | (b & 0xF0F0F0F0u);
  }
}

struct EncodeArgs {
  const uint4* x;
  int rows, cols;
  const float* prescale;
  const uint32_t* vec_amax;     // no clamp: max |x| per scaled vector (float bits)
  const int* row_max;           // clamp: ordered-int row extremes
  const int* row_min;
  const float* thresholds;      // clamp: lo, hi
  uint32_t* codes;              // [rows x cols/8] words or null
  uint32_t* codes_t;            // [cols x rows/8] words or null
  float* amax_out;
  uint8_t* mask;                // clamp: [rows x cols/8] bytes
};

// AXIS 0: one scale per row; AXIS 1: one per column.  OCC implies AXIS 0 and no prescale.
template <int AXIS, bool OCC, bool PRESCALE>
__global__ void __launch_bounds__(ENC_THREADS)
encode_kernel(const EncodeArgs a) {
  __shared__ float s_gamma[ENC_TK];
  __shared__ float s_pre[ENC_TM];
  __shared__ uint32_t tile_t[8 * 8 * 32];
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int row0 = blockIdx.y * ENC_TM;
  const int col0 = blockIdx.x * ENC_TK;
  const int vec_per_row = a.cols >> 3;
  float lo = 0.f, hi = 0.f;
  if (OCC) { lo = a.thresholds[0]; hi = a.thresholds[1]; }

  if (AXIS == 0) {
    if (tid < ENC_TM) {
      const int r = row0 + tid;
      float amax;
      if (OCC) {
        const float mx = fminf(fmaxf(ordered_to_float(a.row_max[r]), lo), hi);
        const float mn = fminf(fmaxf(ordered_to_float(a.row_min[r]), lo), hi);
        amax = fmaxf(fabsf(mx), fabsf(mn));
      } else {
        amax = __uint_as_float(a.vec_amax[r]);
      }
      s_gamma[tid] = amax > 0.0f ? __fdiv_rn(6.0f, amax) : 0.0f;
      if (blockIdx.x == 0) a.amax_out[r] = amax;
    }
  } else {
    const int c = col0 + tid;
    if (c < a.cols) {
      const float amax = __uint_as_float(a.vec_amax[c]);
      s_gamma[tid] = amax > 0.0f ? __fdiv_rn(6.0f, amax) : 0.0f;
      if (blockIdx.y == 0) a.amax_out[c] = amax;
    }
    if (PRESCALE && tid < ENC_TM) s_pre[tid] = prescale_value(a.prescale, row0 + tid);
  }
  __syncthreads();

  const int col = col0 + 8 * lane;                   // first of this thread's 8 columns
  const bool in_cols = col < a.cols;                 // ragged last tile in the column direction
  uint4 v[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    v[r] = make_uint4(0, 0, 0, 0);
    if (in_cols) v[r] = __ldg(&a.x[(long long)(row0 + 8 * warp + r) * vec_per_row + (col >> 3)]);
  }
  float g[8], p[8];
  if (AXIS == 1) {
#pragma unroll
    for (int c = 0; c < 8; ++c) g[c] = s_gamma[8 * lane + c];
  }
  if (AXIS == 0 && PRESCALE && in_cols) {
#pragma unroll
    for (int c = 0; c < 8; ++c) p[c] = prescale_value(a.prescale, col + c);
  }

  uint32_t word[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const uint32_t w[4] = {v[r].x, v[r].y, v[r].z, v[r].w};
    float f[8];
    uint32_t obits = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      f[2 * q] = bf16_lo(w[q]);
      f[2 * q + 1] = bf16_hi(w[q]);
    }
    const float grow = AXIS == 0 ? s_gamma[8 * warp + r] : 0.0f;
    const float prow = (AXIS == 1 && PRESCALE) ? s_pre[8 * warp + r] : 1.0f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      float xv = f[c];
      if (PRESCALE) xv = __fmul_rn(xv, AXIS == 0 ? p[c] : prow);
      if (OCC) {
        const float xc = fminf(fmaxf(xv, lo), hi);
        obits |= (xc != xv ? 1u : 0u) << c;
        xv = xc;
      }
      // + 0.0f turns a -0 product into +0 (the nudge below needs a non-negative zero)
      f[c] = __fmaf_rn(xv, AXIS == 0 ? grow : g[c], 0.0f);
    }
    word[r] = encode8(f);
    if (in_cols) {
      const long long o = (long long)(row0 + 8 * warp + r) * vec_per_row + (col >> 3);
      if (a.codes) a.codes[o] = word[r];
      if (OCC) a.mask[o] = uint8_t(obits);
    }
  }

  if (a.codes_t) {
    transpose8x8_nibbles(word);
#pragma unroll
    for (int c = 0; c < 8; ++c) tile_t[(c * 8 + warp) * 32 + lane] = word[c];
    __syncthreads();
    // thread (c = warp, j = lane) owns column col0 + 8 j + c: 64 rows = 8 words = 32 bytes
    const int k = col0 + 8 * lane + warp;
    if (k < a.cols) {
      uint32_t o[8];
#pragma unroll
      for (int w8 = 0; w8 < 8; ++w8) o[w8] = tile_t[(warp * 8 + w8) * 32 + lane];
      uint4* dst = reinterpret_cast<uint4*>(a.codes_t + (long long)k * (a.rows >> 3) + (row0 >> 3));
      dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
      dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
  }
}

// ------------------------------------------------------------------------------------------
// 4. mask -> CSR / CSC
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
csr_count_kernel(const uint32_t* __restrict__ mask, int rows, int words_per_row, int* __restrict__ row_cnt) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  int c = 0;
  for (int w = lane; w < words_per_row; w += 32) c += __popc(mask[(long long)row * words_per_row + w]);
  c = __reduce_add_sync(0xFFFFFFFFu, c);
  if (lane == 0) row_cnt[row] = c;
}

// Exclusive prefix sum of n counts by one block; ptr[n] = total.  Also publishes nnz and raises
// the overflow flag when the total exceeds the caller's capacity.
__global__ void __launch_bounds__(1024, 1)
scan_counts_kernel(const int* __restrict__ cnt, int n, int* __restrict__ ptr, int* nnz_out, long long cap,
                   int32_t* status) {
  __shared__ int part[1024];
  const int t = threadIdx.x;
  const int per = (n + 1023) / 1024;
  const int b = min(n, t * per), e = min(n, b + per);
  int s = 0;
  for (int i = b; i < e; ++i) s += cnt[i];
  part[t] = s;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {
    const int add = t >= off ? part[t - off] : 0;
    __syncthreads();
    part[t] += add;
    __syncthreads();
  }
  int run = part[t] - s;
  for (int i = b; i < e; ++i) {
    ptr[i] = run;
    run += cnt[i];
  }
  if (t == 1023) {
    ptr[n] = part[1023];
    if (nnz_out) *nnz_out = part[1023];
    if (status && (long long)part[1023] > cap) atomicOr(status, FP4_DEV_SPARSE_OVERFLOW);
  }
}

__device__ __forceinline__ float residual_of(const __nv_bfloat16* x, long long idx, float lo, float hi) {
  const float v = __bfloat162float(x[idx]);
  return __fsub_rn(v, v > hi ? hi : lo);
}

__global__ void __launch_bounds__(256)
csr_fill_kernel(const uint32_t* __restrict__ mask, const __nv_bfloat16* __restrict__ x, int rows, int cols,
                const float* __restrict__ thresholds, const int* __restrict__ rowptr, long long cap,
                int* __restrict__ csr_col, float* __restrict__ csr_val) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const int words_per_row = cols >> 5;
  const float lo = thresholds[0], hi = thresholds[1];
  int base = rowptr[row];
  for (int w0 = 0; w0 < words_per_row; w0 += 32) {
    const int w = w0 + lane;
    uint32_t m = w < words_per_row ? mask[(long long)row * words_per_row + w] : 0u;
    const int c = __popc(m);
    int incl = c;                                     // inclusive warp scan of the counts
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
      if (lane >= off) incl += up;
    }
    int pos = base + incl - c;
    while (m) {
      const int b = __ffs(m) - 1;
      m &= m - 1;
      const int col = 32 * w + b;
      if (pos < cap) {
        csr_col[pos] = col;
        csr_val[pos] = residual_of(x, (long long)row * cols + col, lo, hi);
      }
      ++pos;
    }
    base += __shfl_sync(0xFFFFFFFFu, incl, 31);
  }
}

// Column direction: warp <-> one 32-column word of the mask, lane <-> one column, a strip of rows.
__global__ void __launch_bounds__(256)
csc_count_kernel(const uint32_t* __restrict__ mask, int rows, int cols, int rows_per_split,
                 int* __restrict__ split_cnt) {
  const int q = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int words_per_row = cols >> 5;
  if (q >= words_per_row) return;
  const int r0 = blockIdx.y * rows_per_split, r1 = min(rows, r0 + rows_per_split);
  int c = 0;
  for (int r = r0; r < r1; ++r) c += (mask[(long long)r * words_per_row + q] >> lane) & 1u;
  split_cnt[(long long)blockIdx.y * cols + 32 * q + lane] = c;
}

// Per column: turn the per-strip counts into running offsets inside the column, total -> col_cnt.
__global__ void __launch_bounds__(256)
csc_split_prefix_kernel(int* __restrict__ split_cnt, int cols, int splits, int* __restrict__ col_cnt) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= cols) return;
  int run = 0;
  for (int s = 0; s < splits; ++s) {
    const int c = split_cnt[(long long)s * cols + k];
    split_cnt[(long long)s * cols + k] = run;
    run += c;
  }
  col_cnt[k] = run;
}

__global__ void __launch_bounds__(256)
csc_fill_kernel(const uint32_t* __restrict__ mask, const __nv_bfloat16* __restrict__ x, int rows, int cols,
                int rows_per_split, const float* __restrict__ thresholds, const int* __restrict__ colptr,
                const int* __restrict__ split_off, long long cap, int* __restrict__ csc_row,
                float* __restrict__ csc_val) {
  const int q = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int words_per_row = cols >> 5;
  if (q >= words_per_row) return;
  const int col = 32 * q + lane;
  const int r0 = blockIdx.y * rows_per_split, r1 = min(rows, r0 + rows_per_split);
  const float lo = thresholds[0], hi = thresholds[1];
  int pos = colptr[col] + split_off[(long long)blockIdx.y * cols + col];
  for (int r = r0; r < r1; ++r) {
    if ((mask[(long long)r * words_per_row + q] >> lane) & 1u) {
      if (pos < cap) {
        csc_row[pos] = r;
        csc_val[pos] = residual_of(x, (long long)r * cols + col, lo, hi);
      }
      ++pos;
    }
  }
}

int pick_splits(int rows, int cols, int num_sms) {
  // enough (column-block x strip) CTAs to fill the machine, strips of at least 64 rows
  const int col_blocks = (cols / 32 + 7) / 8;
  int splits = (4 * num_sms + col_blocks - 1) / col_blocks;
  if (splits > rows / 64) splits = rows / 64;
  if (splits > MAX_SPLITS) splits = MAX_SPLITS;
  if (splits < 1) splits = 1;
  return splits;
}

size_t r256(size_t b) { return (b + 255) & ~size_t(255); }

}  // namespace

size_t quantize_scratch_bytes(int64_t rows, int64_t cols) {
  size_t b = 0;
  b += r256(65536 * 4);                                        // histogram
  b += 2 * r256(size_t(rows) * 4);                             // row extremes
  b += r256(size_t(rows > cols ? rows : cols) * 4);            // absmax per vector
  b += r256(size_t(rows) * size_t(cols) / 8);                  // outlier mask
  b += r256(size_t(rows) * 4) + r256(size_t(cols) * 4);        // counts
  b += r256(size_t(MAX_SPLITS) * size_t(cols) * 4);            // per-strip column counts
  b += r256(size_t(rows > cols ? rows : cols) * 4);            // de-scale vector used as prescale
  return b;
}

int launch_quantize(fp4_ctx* ctx, cudaStream_t stream, Arena& arena, const void* x_bf16, int64_t rows64,
                    int64_t cols64, int scale_axis, double alpha, const float* prescale, int prescale_is_amax,
                    fp4_qtensor* out, int32_t* status) {
  const int rows = int(rows64), cols = int(cols64);
  const long long n = (long long)rows * cols;
  const long long n_vec = n / 8;
  const int vec_per_row = cols / 8;
  const bool occ = alpha < 1.0;
  const uint4* x = static_cast<const uint4*>(x_bf16);

  uint32_t* hist = arena.take<uint32_t>(65536);
  int* row_max = arena.take<int>(rows);
  int* row_min = arena.take<int>(rows);
  uint32_t* vec_amax = arena.take<uint32_t>(rows > cols ? rows : cols);
  uint8_t* mask = arena.take<uint8_t>(size_t(n / 8));
  int* row_cnt = arena.take<int>(rows);
  int* col_cnt = arena.take<int>(cols);
  int* split_cnt = arena.take<int>(size_t(MAX_SPLITS) * cols);
  float* pre_d = arena.take<float>(rows > cols ? rows : cols);
  if (!arena.ok) return FP4_ERR_WORKSPACE;
  if (prescale && prescale_is_amax) {
    const int np = scale_axis == 0 ? cols : rows;
    KernelScope scope(ctx, stream, KC_ABSMAX, 1);
    descale_kernel<<<(np + 255) / 256, 256, 0, stream>>>(prescale, np, pre_d);
    prescale = pre_d;
  }

  EncodeArgs ea = {};
  ea.x = x;
  ea.rows = rows;
  ea.cols = cols;
  ea.prescale = prescale;
  ea.vec_amax = vec_amax;
  ea.row_max = row_max;
  ea.row_min = row_min;
  ea.thresholds = out->thresholds;
  ea.codes = reinterpret_cast<uint32_t*>(out->codes);
  ea.codes_t = reinterpret_cast<uint32_t*>(out->codes_t);
  ea.amax_out = out->amax;
  ea.mask = mask;
  const dim3 enc_grid((cols + ENC_TK - 1) / ENC_TK, rows / ENC_TM);

  if (occ) {
    const long long n_tail = llround((1.0 - alpha) * double(n));
    {
    KernelScope scope(ctx, stream, KC_SELECT, 3);
    FP4_CUDA_TRY(cudaMemsetAsync(hist, 0, 65536 * 4, stream));
    init_row_extremes_kernel<<<(rows + 255) / 256, 256, 0, stream>>>(row_max, row_min, rows);
    FP4_CUDA_TRY(cudaFuncSetAttribute(hist_rowminmax_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      HIST_WORDS * 4));
    long long blocks = (n_vec + HIST_THREADS - 1) / HIST_THREADS;
    if (blocks > ctx->num_sms) blocks = ctx->num_sms;
    hist_rowminmax_kernel<<<int(blocks), HIST_THREADS, HIST_WORDS * 4, stream>>>(x, n_vec, vec_per_row, hist, row_max,
                                                                                row_min);
    select_thresholds_kernel<<<1, 1024, 0, stream>>>(hist, n, n_tail, out->thresholds);
    }
    {
      KernelScope scope(ctx, stream, KC_ENCODE, 1);
      encode_kernel<0, true, false><<<enc_grid, ENC_THREADS, 0, stream>>>(ea);
    }
    KernelScope scope(ctx, stream, KC_SPARSE, 7);

    const uint32_t* mask32 = reinterpret_cast<const uint32_t*>(mask);
    const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x_bf16);
    csr_count_kernel<<<(rows + 7) / 8, 256, 0, stream>>>(mask32, rows, cols / 32, row_cnt);
    scan_counts_kernel<<<1, 1024, 0, stream>>>(row_cnt, rows, out->csr_rowptr, out->nnz, out->sparse_cap, status);
    csr_fill_kernel<<<(rows + 7) / 8, 256, 0, stream>>>(mask32, xb, rows, cols, out->thresholds, out->csr_rowptr,
                                                        out->sparse_cap, out->csr_col, out->csr_val);
    const int splits = pick_splits(rows, cols, ctx->num_sms);
    const int rows_per_split = (rows + splits - 1) / splits;
    const dim3 cgrid((cols / 32 + 7) / 8, splits);
    csc_count_kernel<<<cgrid, 256, 0, stream>>>(mask32, rows, cols, rows_per_split, split_cnt);
    csc_split_prefix_kernel<<<(cols + 255) / 256, 256, 0, stream>>>(split_cnt, cols, splits, col_cnt);
    scan_counts_kernel<<<1, 1024, 0, stream>>>(col_cnt, cols, out->csc_colptr, nullptr, out->sparse_cap, nullptr);
    csc_fill_kernel<<<cgrid, 256, 0, stream>>>(mask32, xb, rows, cols, rows_per_split, out->thresholds,
                                               out->csc_colptr, split_cnt, out->sparse_cap, out->csc_row,
                                               out->csc_val);
  } else {
    const int n_amax = scale_axis == 0 ? rows : cols;
    FP4_CUDA_TRY(cudaMemsetAsync(vec_amax, 0, size_t(n_amax) * 4, stream));
    if (scale_axis == 0) {
      long long blocks = (n_vec + 255) / 256;
      if (blocks > 8LL * ctx->num_sms) blocks = 8LL * ctx->num_sms;
      {
        KernelScope scope(ctx, stream, KC_ABSMAX, 1);
        if (prescale)
          absmax_rows_kernel<true><<<int(blocks), 256, 0, stream>>>(x, n_vec, vec_per_row, prescale, vec_amax);
        else
          absmax_rows_kernel<false><<<int(blocks), 256, 0, stream>>>(x, n_vec, vec_per_row, nullptr, vec_amax);
      }
      KernelScope scope(ctx, stream, KC_ENCODE, 1);
      if (prescale)
        encode_kernel<0, false, true><<<enc_grid, ENC_THREADS, 0, stream>>>(ea);
      else
        encode_kernel<0, false, false><<<enc_grid, ENC_THREADS, 0, stream>>>(ea);
    } else {
      const int col_blocks = (vec_per_row + 255) / 256;
      int strips = (8 * ctx->num_sms + col_blocks - 1) / col_blocks;
      if (strips > rows / 16) strips = rows / 16;
      if (strips < 1) strips = 1;
      const int rows_per_strip = (rows + strips - 1) / strips;
      const dim3 agrid(col_blocks, (rows + rows_per_strip - 1) / rows_per_strip);
      {
        KernelScope scope(ctx, stream, KC_ABSMAX, 1);
        if (prescale)
          absmax_cols_kernel<true><<<agrid, 256, 0, stream>>>(x, rows, vec_per_row, rows_per_strip, prescale,
                                                              vec_amax);
        else
          absmax_cols_kernel<false><<<agrid, 256, 0, stream>>>(x, rows, vec_per_row, rows_per_strip, nullptr,
                                                               vec_amax);
      }
      KernelScope scope(ctx, stream, KC_ENCODE, 1);
      if (prescale)
        encode_kernel<1, false, true><<<enc_grid, ENC_THREADS, 0, stream>>>(ea);
      else
        encode_kernel<1, false, false><<<enc_grid, ENC_THREADS, 0, stream>>>(ea);
    }
  }
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}

// ------------------------------------------------------------------------------------------
// Quantile thresholds without any allocation
// ------------------------------------------------------------------------------------------
// Scratch of fp4_quantile_thresholds_static: the 65536-bin histogram followed by the row
// extremes of up to FP4_STATIC_MAX_ROWS rows.  It lives in the library image: every GPU that
// loads the library holds these 768 KB until the process exits.
namespace {
constexpr size_t STATIC_HIST_BYTES = 65536 * sizeof(uint32_t);
constexpr size_t STATIC_SCRATCH_BYTES = STATIC_HIST_BYTES + 2 * size_t(FP4_STATIC_MAX_ROWS) * sizeof(int);
constexpr int STATIC_MAX_DEVICES = 64;
}  // namespace
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

extern "C" int fp4_quantile_thresholds_static(void* stream, const void* x_bf16, int64_t rows, int64_t cols,
                                              double alpha, float* thresholds) {
  // In host code `g_static_scratch` is only a handle; the device address of this device's copy
  // is looked up once per device and cached.
  static void* scratch_of_device[STATIC_MAX_DEVICES] = {};
  static int sms_of_device[STATIC_MAX_DEVICES] = {};
  if (!x_bf16 || !thresholds) return FP4_ERR_NULL;
  if (rows <= 0 || cols <= 0 || (rows % 128) || (cols % 128) || rows * cols >= (int64_t(1) << 31))
    return FP4_ERR_SHAPE;
  if (rows > FP4_STATIC_MAX_ROWS) return FP4_ERR_STATIC_LIMIT;
  if (!(alpha > 0.5 && alpha < 1.0)) return FP4_ERR_ALPHA;
  if (reinterpret_cast<uintptr_t>(x_bf16) & 15) return FP4_ERR_ALIGN;
  const long long n = (long long)rows * cols;
  const long long n_tail = llround((1.0 - alpha) * double(n));
  if (2 * n_tail >= n) return FP4_ERR_ALPHA;

  int device = -1;
  FP4_CUDA_TRY(cudaGetDevice(&device));
  if (device < 0 || device >= STATIC_MAX_DEVICES) return FP4_ERR_ARG;
  if (!scratch_of_device[device]) {
    void* ptr = nullptr;
    FP4_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
    int sms = 0;
    FP4_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    FP4_CUDA_TRY(cudaFuncSetAttribute(hist_rowminmax_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      HIST_WORDS * 4));
    sms_of_device[device] = sms;
    scratch_of_device[device] = ptr;
  }
  unsigned char* base = static_cast<unsigned char*>(scratch_of_device[device]);
  uint32_t* hist = reinterpret_cast<uint32_t*>(base);
  int* row_max = reinterpret_cast<int*>(base + STATIC_HIST_BYTES);
  int* row_min = row_max + FP4_STATIC_MAX_ROWS;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array keeps what the previous call left: the histogram must start from zero and the
  // row extremes from their identities.
  FP4_CUDA_TRY(cudaMemsetAsync(hist, 0, STATIC_HIST_BYTES, st));
  init_row_extremes_kernel<<<int((rows + 255) / 256), 256, 0, st>>>(row_max, row_min, int(rows));
  const long long n_vec = n / 8;
  long long blocks = (n_vec + HIST_THREADS - 1) / HIST_THREADS;
  if (blocks > sms_of_device[device]) blocks = sms_of_device[device];
  hist_rowminmax_kernel<<<int(blocks), HIST_THREADS, HIST_WORDS * 4, st>>>(static_cast<const uint4*>(x_bf16), n_vec,
                                                                          int(cols / 8), hist, row_max, row_min);
  select_thresholds_kernel<<<1, 1024, 0, st>>>(hist, n, n_tail, thresholds);
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}
