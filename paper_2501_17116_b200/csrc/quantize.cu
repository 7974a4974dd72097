// Quantiser kernels: exact quantile selection, clamp, vector-wise absmax, E2M1 encoding in both
// packed layouts, and extraction of the sparse residual (Eq. 1, Appendix A, Section 3.2).
//
// Passes over a [rows x cols] BF16 tensor:
//   with outlier clamping (activations)
//     1. hist_select      one read: 65536-bin histogram of the BF16 bit patterns (exact, in shared
//                         memory) + signed max / min of every row; the block that finishes last
//     2.                  turns the cumulative counts into the two order statistics lo, hi
//     3. encode           one read: clamp, per-row scale from the clamped row extremes, Q, both
//                         nibble layouts, a 1-bit-per-element mask of the clamped entries, and
//                         the number of clamped entries per row and per (64-row strip, column)
//     4. mask -> CSR/CSC  prefix sums of those counts and ordered fills driven by the mask (1/16
//                         of the tensor); values are gathered from the few marked entries
//   without clamping (weights, output gradients)
//     1. absmax           one read: max |x| per row and / or per column (after the prescale)
//     2. encode           one read
// The "dual" mode serves the backward pass: one read of dY yields the token-wise codes of
// dY (.) d_W[n] and the channel-wise codes of dY (.) d_A[m].
#include <mutex>

#include "common.cuh"

namespace {

constexpr int HIST_THREADS = 1024;
constexpr int ENC_TM = 64;                        // tile rows of the encoder (= one strip)
constexpr int ENC_TK = 256;                       // tile columns
constexpr int ENC_THREADS = 256;

enum Mode { MODE_ROWS = 0, MODE_COLS = 1, MODE_DUAL = 2 };

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
// 1. + 2. histogram of bit patterns, row extremes, order statistics -- one kernel
// ------------------------------------------------------------------------------------------
// Exact histogram with 32-bit shared-memory counters over a window of HIST_EXPS binary exponents
// (both signs, all 128 mantissas): real tensors spread over far fewer exponents than BF16 offers.
// Each block places its window HIST_HEADROOM binades above the largest magnitude of its first 8192
// elements.  A vector of eight elements is tested against the window as a whole (four packed BF16
// comparisons); if all eight are inside, each costs one extraction, one address and one increment.
// Patterns outside the window (tiny values, later giants) go straight to the global histogram and
// exact zeros are counted in registers, so every element is counted exactly once.  The window is
// replicated HIST_COPIES times (one copy per group of warps) to thin out same-address conflicts;
// the increments return no value and need no overflow handling.  What bounds the loop is the
// shared-memory pipe: the increments of a warp fall into random banks.
//
// A block owns whole rows (a contiguous range of them), so the signed max / min of a row are
// reduced in shared memory and written with plain stores, as is the zero that starts the row's
// count of clamped entries: nothing the kernel writes per row needs initialising.
//
// Every count also goes into one of 32 coarse counters (2048 consecutive positions of the
// ascending real order each).  The block that finishes last (a ticket, no waiting) finds the
// coarse range of each of the two ranks and reads only those 2048 fine counters: lo and hi.
// The context keeps two sets of counters and a device-side parity: a call counts into set p,
// clears set 1 - p at its start (every block a slice, plain stores) and flips the parity at its
// end, so the set a call counts into is always zero and no separate clearing pass exists.  With
// `parity` null (the allocation-free entry point, which clears its one set itself) set 0 is used.
constexpr int HIST_EXPS = 24;
constexpr int HIST_WINDOW = HIST_EXPS * 128;       // 3072 magnitudes in the window, per sign
constexpr int HIST_COPIES = 4;
constexpr int HIST_HEADROOM = 1;                   // binades between the sample's maximum and the window's top
constexpr int HIST_FLY = 4;                        // vectors a lane loads per unit
constexpr int HIST_CHUNK = 32 * HIST_FLY;          // vectors of one row a warp takes at a time
// Counter of pattern b in copy c: word c * HIST_WINDOW + (b - base).  The sign bit of b is left in
// place, so the negative half of every copy lies 0x8000 words (128 KB) above its positive half and
// the index of an element is its pattern minus a constant; the words between the halves are unused.
constexpr int HIST_NEG_WORD = 0x8000;
constexpr int HIST_SMEM_BYTES = (HIST_NEG_WORD + HIST_COPIES * HIST_WINDOW) * 4;
constexpr int HIST_ROW_SLOTS = 512;                // rows whose extremes a block reduces at a time
constexpr int HIST_COARSE = 32;                    // coarse counters: 2048 positions each
constexpr int HIST_SET_WORDS = 65536 + HIST_COARSE; // one set: fine counters, then coarse counters

// Inclusive scan of one value per thread over a block of 1024 threads.
__device__ __forceinline__ long long block_scan_1024(long long v, long long* warp_tot /*[32] shared*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const long long up = __shfl_up_sync(0xFFFFFFFFu, v, off);
    if (lane >= off) v += up;
  }
  if (lane == 31) warp_tot[warp] = v;
  __syncthreads();
  if (warp == 0) {
    long long t = warp_tot[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const long long up = __shfl_up_sync(0xFFFFFFFFu, t, off);
      if (lane >= off) t += up;
    }
    warp_tot[lane] = t;
  }
  __syncthreads();
  if (warp > 0) v += warp_tot[warp - 1];
  return v;
}

// Position p in ascending real order: p < 32768 are the negative patterns from 0xFFFF down to
// 0x8000 (-0), p >= 32768 the non-negative patterns from 0x0000 up.
__device__ __forceinline__ uint32_t pos_to_bits(int p) { return p < 32768 ? uint32_t(0xFFFF - p) : uint32_t(p - 32768); }
__device__ __forceinline__ int bits_to_pos(uint32_t bits) { return (bits & 0x8000u) ? int(0xFFFFu - bits) : int(bits) + 32768; }

__global__ void __launch_bounds__(HIST_THREADS, 1)
hist_select_kernel(const uint4* __restrict__ x, int rows, int vec_per_row, uint32_t* sets, unsigned* parity,
                   int* __restrict__ row_max, int* __restrict__ row_min, int* __restrict__ row_cnt, long long n,
                   long long n_tail, float* __restrict__ thresholds, unsigned* ticket, int32_t* status, int abs_mode) {
  extern __shared__ uint32_t h[];
  __shared__ uint32_t s_top;
  __shared__ int s_rmax[HIST_ROW_SLOTS], s_rmin[HIST_ROW_SLOTS];
  __shared__ uint32_t s_coarse[HIST_COARSE];
  __shared__ int s_last;
  const int tid = threadIdx.x;
  const int r_begin = int((long long)rows * blockIdx.x / gridDim.x);
  const int r_end = int((long long)rows * (blockIdx.x + 1) / gridDim.x);
  const int lane = tid & 31;
  // sample for the window's top, issued first: its latency hides behind the clearing below
  uint4 sample = make_uint4(0, 0, 0, 0);
  {
    const long long i0 = (long long)r_begin * vec_per_row + tid;
    if (i0 < (long long)r_end * vec_per_row) sample = __ldg(&x[i0]);
  }
  const unsigned par = parity ? (*reinterpret_cast<volatile unsigned*>(parity) & 1u) : 0u;
  uint32_t* ghist = sets + size_t(par) * HIST_SET_WORDS;
  uint32_t* gcoarse = ghist + 65536;
  if (parity) {
    // this block's slice of the other set, for the next call
    uint32_t* other = sets + size_t(par ^ 1u) * HIST_SET_WORDS;
    const int per = (HIST_SET_WORDS + gridDim.x - 1) / gridDim.x;
    const int w0 = blockIdx.x * per, w1 = min(HIST_SET_WORDS, w0 + per);
    for (int i = w0 + tid; i < w1; i += HIST_THREADS) other[i] = 0;
  }
  {
    uint4* pos4 = reinterpret_cast<uint4*>(h);
    uint4* neg4 = reinterpret_cast<uint4*>(h + HIST_NEG_WORD);
    for (int i = tid; i < HIST_WINDOW * HIST_COPIES / 4; i += HIST_THREADS)
      pos4[i] = neg4[i] = make_uint4(0, 0, 0, 0);
  }
  if (tid < HIST_COARSE) s_coarse[tid] = 0;
  if (tid == 0) s_top = 0;
  __syncthreads();
  {
    // window top: largest exponent-and-mantissa field among this block's first vectors
    const uint32_t w[4] = {sample.x, sample.y, sample.z, sample.w};
    uint32_t m = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) m = max(m, max(w[q] & 0x7FFFu, (w[q] >> 16) & 0x7FFFu));
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if ((tid & 31) == 0 && m) atomicMax(&s_top, m);
  }
  __syncthreads();
  // window = exponents [e_top - HIST_EXPS + 1, e_top] with e_top HIST_HEADROOM binades above the sample's
  // maximum (what lies above the window is counted in global memory like what lies below it)
  const int e_top = min(254, int(s_top >> 7) + HIST_HEADROOM);
  const uint32_t base = uint32_t(max(0, e_top - HIST_EXPS + 1)) << 7;
  // The window's bounds as BF16 numbers (magnitudes order like their patterns; the upper bound is at
  // most the pattern of infinity, and a NaN fails every comparison)
  const __nv_bfloat162 lo_bf = __halves2bfloat162(__ushort_as_bfloat16((unsigned short)base),
                                                  __ushort_as_bfloat16((unsigned short)base));
  const __nv_bfloat162 hi_bf = __halves2bfloat162(__ushort_as_bfloat16((unsigned short)(base + HIST_WINDOW)),
                                                  __ushort_as_bfloat16((unsigned short)(base + HIST_WINDOW)));
  // this warp's copy: counter of pattern b at word b + my_off
  const int my_off = ((tid >> 5) & (HIST_COPIES - 1)) * HIST_WINDOW - int(base);
  uint32_t zeros_pos = 0, zeros_neg = 0;
  bool nonfinite = false;
  for (int r0 = r_begin; r0 < r_end; r0 += HIST_ROW_SLOTS) {
    const int r1 = min(r_end, r0 + HIST_ROW_SLOTS);
    for (int r = tid; r < r1 - r0; r += HIST_THREADS) {
      s_rmax[r] = INT_MIN;
      s_rmin[r] = INT_MAX;
    }
    __syncthreads();
    // A unit is a stretch of up to HIST_CHUNK consecutive vectors of one row; warp w takes units
    // w, w + 32, ...  A lane loads its HIST_FLY vectors of the unit (vectors lane, lane + 32, ... of
    // the stretch) before it counts any of them, keeps the unit's extremes packed in two registers,
    // and the warp reduces them once per unit.
    const int chunks_per_row = (vec_per_row + HIST_CHUNK - 1) / HIST_CHUNK;
    const int units = (r1 - r0) * chunks_per_row;
    for (int u = tid >> 5; u < units; u += HIST_THREADS / 32) {
      const int row = u / chunks_per_row;
      const int v0 = (u - row * chunks_per_row) * HIST_CHUNK;
      const int mine = min(HIST_CHUNK, vec_per_row - v0) - lane;       // vectors lane, lane + 32, ... below this
      const uint4* px = x + ((long long)(r0 + row) * vec_per_row + v0 + lane);
      uint4 vv[HIST_FLY];
#pragma unroll
      for (int k = 0; k < HIST_FLY; ++k)
        if (32 * k < mine) vv[k] = __ldg(px + 32 * k);
      __nv_bfloat162 umax = __float2bfloat162_rn(-INFINITY), umin = __float2bfloat162_rn(INFINITY);
#pragma unroll
      for (int k = 0; k < HIST_FLY; ++k) {
        if (32 * k >= mine) break;
        const uint32_t w[4] = {vv[k].x, vv[k].y, vv[k].z, vv[k].w};
        const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(w);
        // all eight magnitudes inside the window?  (half-precision comparisons: they leave the
        // integer pipe to the index arithmetic)
        bool inside = true;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const __nv_bfloat162 mag = __habs2(p[q]);
          inside = inside && __hbge2(mag, lo_bf) && __hblt2(mag, hi_bf);
        }
        if (inside) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            atomicAdd(&h[int(w[q] & 0xFFFFu) + my_off], 1u);
            atomicAdd(&h[int(w[q] >> 16) + my_off], 1u);
          }
        } else {
#pragma unroll 1
          for (int e = 0; e < 8; ++e) {
            const uint32_t word = (e & 4) ? ((e & 2) ? w[3] : w[2]) : ((e & 2) ? w[1] : w[0]);
            const uint32_t bits = (e & 1) ? (word >> 16) : (word & 0xFFFFu);
            const uint32_t m15 = bits & 0x7FFFu;
            if (m15 - base < uint32_t(HIST_WINDOW)) {
              atomicAdd(&h[int(bits) + my_off], 1u);
            } else if (m15 == 0) {
              if (bits) ++zeros_neg; else ++zeros_pos;
            } else {
              atomicAdd(&ghist[bits], 1u);
              atomicAdd(&s_coarse[bits_to_pos(bits) >> 11], 1u);
              if (m15 >= 0x7F80u) nonfinite = true;       // infinity or NaN: always outside the window
            }
          }
        }
        umax = __hmax2(umax, __hmax2(__hmax2(p[0], p[1]), __hmax2(p[2], p[3])));
        umin = __hmin2(umin, __hmin2(__hmin2(p[0], p[1]), __hmin2(p[2], p[3])));
      }
      int kmax = float_to_ordered(fmaxf(__low2float(umax), __high2float(umax)));
      int kmin = float_to_ordered(fminf(__low2float(umin), __high2float(umin)));
      kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
      kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
      if (lane == 0) {
        atomicMax(&s_rmax[row], kmax);
        atomicMin(&s_rmin[row], kmin);
      }
    }
    __syncthreads();
    for (int r = tid; r < r1 - r0; r += HIST_THREADS) {
      row_max[r0 + r] = s_rmax[r];
      row_min[r0 + r] = s_rmin[r];
      if (row_cnt) row_cnt[r0 + r] = 0;
    }
    __syncthreads();
  }
  if (__any_sync(0xFFFFFFFFu, nonfinite) && (tid & 31) == 0 && status) atomicOr(status, FP4_DEV_NONFINITE);
  zeros_pos = __reduce_add_sync(0xFFFFFFFFu, zeros_pos);
  zeros_neg = __reduce_add_sync(0xFFFFFFFFu, zeros_neg);
  if ((tid & 31) == 0) {
    if (zeros_pos) { atomicAdd(&ghist[0x0000], zeros_pos); atomicAdd(&s_coarse[bits_to_pos(0x0000u) >> 11], zeros_pos); }
    if (zeros_neg) { atomicAdd(&ghist[0x8000], zeros_neg); atomicAdd(&s_coarse[bits_to_pos(0x8000u) >> 11], zeros_neg); }
  }
  // Two neighbouring counters (an even pattern and the next one: same sign, same coarse range) leave
  // with one 64-bit add; no 32-bit half can overflow into the other (n < 2^31).
  for (int idx = tid; idx < HIST_WINDOW; idx += HIST_THREADS) {
    const int neg = idx >= HIST_WINDOW / 2, off = 2 * (idx - neg * (HIST_WINDOW / 2));
    uint32_t c0 = 0, c1 = 0;
#pragma unroll
    for (int r = 0; r < HIST_COPIES; ++r) {
      const uint2 c = *reinterpret_cast<const uint2*>(&h[neg * HIST_NEG_WORD + r * HIST_WINDOW + off]);
      c0 += c.x;
      c1 += c.y;
    }
    if (c0 | c1) {
      const uint32_t bits = (uint32_t(neg) << 15) | (base + uint32_t(off));
      atomicAdd(reinterpret_cast<unsigned long long*>(&ghist[bits]), (unsigned long long)c0 | ((unsigned long long)c1 << 32));
      atomicAdd(&s_coarse[bits_to_pos(bits) >> 11], c0 + c1);
    }
  }
  __syncthreads();
  if (tid < HIST_COARSE && s_coarse[tid]) atomicAdd(&gcoarse[tid], s_coarse[tid]);
  // ---- the last block to get here selects -------------------------------------------------
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  {
    // Rank q (0: lower, 1: upper) is served by warps 16 q .. 16 q + 15.  Every warp finds the rank's
    // coarse range (one coarse counter per lane), then warp st of the 16 reads step st of the range's
    // 2048 fine counters: 128 consecutive positions, 4 per lane.  The step totals meet in shared
    // memory; the warp whose step holds the rank writes the threshold.
    static_assert(HIST_THREADS == 1024, "two ranks x sixteen steps, one warp each");
    __shared__ long long s_step[2][16];
    const int warp = tid >> 5, lane = tid & 31, q = warp >> 4, st = warp & 15;
    // abs_mode: one rank in the order of the magnitudes (both warp groups find it, the first writes
    // -t and t): magnitude range c holds the positive range 16 + c and the negative range 15 - c.
    const long long rank = abs_mode ? n - 1 - 2 * n_tail : (q == 0 ? n_tail : n - 1 - n_tail);
    const long long cc = !abs_mode ? (long long)__ldcg(&gcoarse[lane])
                         : (lane < 16 ? (long long)__ldcg(&gcoarse[16 + lane]) + __ldcg(&gcoarse[15 - lane]) : 0ll);
    long long sc = cc;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const long long up = __shfl_up_sync(0xFFFFFFFFu, sc, off);
      if (lane >= off) sc += up;
    }
    const unsigned holds = __ballot_sync(0xFFFFFFFFu, rank >= sc - cc && rank < sc);   // exactly one lane
    const int region = holds ? __ffs(holds) - 1 : 0;
    long long run = __shfl_sync(0xFFFFFFFFu, sc - cc, region);                          // counts before the range
    // positions of the range in ascending order; in memory they ascend (region >= 16) or descend
    const bool desc = !abs_mode && region < 16;
    const uint32_t* first = abs_mode ? ghist + 2048 * region
                                     : ghist + (desc ? (0xFFFF - 2048 * region - 2047) : 2048 * (region - 16));
    const int word = desc ? (2048 - 128 * st - 4 * lane - 4) : (128 * st + 4 * lane);
    uint4 c = __ldcg(reinterpret_cast<const uint4*>(first + word));
    if (abs_mode) {                                   // the same magnitudes with the sign bit set
      const uint4 cn = __ldcg(reinterpret_cast<const uint4*>(first + 0x8000 + word));
      c = make_uint4(c.x + cn.x, c.y + cn.y, c.z + cn.z, c.w + cn.w);
    }
    // in ascending position order
    const long long v0 = desc ? c.w : c.x, v1 = desc ? c.z : c.y;
    const long long v2 = desc ? c.y : c.z, v3 = desc ? c.x : c.w;
    const long long mine = v0 + v1 + v2 + v3;
    long long incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const long long up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
      if (lane >= off) incl += up;
    }
    if (lane == 31) s_step[q][st] = incl;
    __syncthreads();
    for (int j = 0; j < st; ++j) run += s_step[q][j];
    const long long before = run + incl - mine;
    if (holds && rank >= before && rank < before + mine) {
      const int p0 = 2048 * region + 128 * st + 4 * lane;
      const int k = rank < before + v0 ? 0 : (rank < before + v0 + v1 ? 1 : (rank < before + v0 + v1 + v2 ? 2 : 3));
      if (abs_mode) {
        const uint32_t m15 = uint32_t(p0 + k);          // p0 counts magnitudes here
        if (q == 0) {
          thresholds[1] = __uint_as_float(m15 << 16);
          thresholds[0] = __uint_as_float(m15 ? (m15 | 0x8000u) << 16 : 0u);
        }
      } else {
        const uint32_t bits = pos_to_bits(p0 + k);
        thresholds[q] = __uint_as_float((bits == 0x8000u ? 0u : bits) << 16);   // thresholds are real numbers: -0 is +0
      }
    }
  }
  __syncthreads();
  if (tid == 0) {
    if (parity) *parity = par ^ 1u;
    *ticket = 0;
  }
}

// ------------------------------------------------------------------------------------------
// 1c. thresholds per token (a variant outside the paper, which clamps at tensor-wide quantiles)
// ------------------------------------------------------------------------------------------
// One block per row: exact order statistics of the row's 16-bit patterns by a two-pass radix
// select in shared memory (high byte of the position in ascending real order, then the low byte
// inside the bin that holds the rank), both ranks at once; also the row's extremes, the zero that
// starts its count of clamped entries, and the non-finite flag, like the tensor-wide kernel.
// thresholds[2 m] = lo of row m, thresholds[2 m + 1] = hi (a -0 threshold is written as +0).
__global__ void __launch_bounds__(256)
row_select_kernel(const uint4* __restrict__ x, int vec_per_row, int n_tail, int* __restrict__ row_max,
                  int* __restrict__ row_min, int* __restrict__ row_cnt, float* __restrict__ thresholds,
                  int32_t* status) {
  __shared__ uint32_t hist[3][256];          // pass 1; pass 2 for the lower rank; pass 2 for the upper rank
  __shared__ int s_bin[2], s_rank[2], s_max[8], s_min[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int m = blockIdx.x;
  const uint4* row = x + (long long)m * vec_per_row;
  const int cols = 8 * vec_per_row;
  for (int i = tid; i < 3 * 256; i += 256) (&hist[0][0])[i] = 0;
  __syncthreads();
  int kmax = INT_MIN, kmin = INT_MAX;
  bool nonfinite = false;
  for (int v = tid; v < vec_per_row; v += 256) {
    const uint4 q = __ldg(&row[v]);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const uint32_t bits = (e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu);
      atomicAdd(&hist[0][bits_to_pos(bits) >> 8], 1u);
      if ((bits & 0x7FFFu) >= 0x7F80u) nonfinite = true;
      const int key = float_to_ordered(__uint_as_float(bits << 16));
      kmax = max(kmax, key);
      kmin = min(kmin, key);
    }
  }
  kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
  kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
  if (lane == 0) { s_max[warp] = kmax; s_min[warp] = kmin; }
  if (__any_sync(0xFFFFFFFFu, nonfinite) && lane == 0 && status) atomicOr(status, FP4_DEV_NONFINITE);
  __syncthreads();
  if (tid == 0) {
    int a = s_max[0], b = s_min[0];
    for (int i = 1; i < 8; ++i) { a = max(a, s_max[i]); b = min(b, s_min[i]); }
    row_max[m] = a;
    row_min[m] = b;
    if (row_cnt) row_cnt[m] = 0;
  }
  // the bin of each rank: warp q scans the 256 counts for rank q (8 per lane)
  if (warp < 2) {
    const int rank = warp == 0 ? n_tail : cols - 1 - n_tail;
    int c[8], mine = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { c[i] = int(hist[0][8 * lane + i]); mine += c[i]; }
    int incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
      if (lane >= off) incl += up;
    }
    int before = incl - mine;
    if (rank >= before && rank < incl) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (rank >= before && rank < before + c[i]) { s_bin[warp] = 8 * lane + i; s_rank[warp] = rank - before; }
        before += c[i];
      }
    }
  }
  __syncthreads();
  const int bin_lo = s_bin[0], bin_hi = s_bin[1];
  for (int v = tid; v < vec_per_row; v += 256) {      // second pass: the row is in L1 / L2 now
    const uint4 q = __ldg(&row[v]);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const uint32_t bits = (e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu);
      const int pos = bits_to_pos(bits);
      if ((pos >> 8) == bin_lo) atomicAdd(&hist[1][pos & 255], 1u);
      if ((pos >> 8) == bin_hi) atomicAdd(&hist[2][pos & 255], 1u);
    }
  }
  __syncthreads();
  if (warp < 2) {
    const int rank = s_rank[warp];
    int c[8], mine = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { c[i] = int(hist[1 + warp][8 * lane + i]); mine += c[i]; }
    int incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
      if (lane >= off) incl += up;
    }
    int before = incl - mine;
    if (rank >= before && rank < incl) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (rank >= before && rank < before + c[i]) {
          const uint32_t bits = pos_to_bits(256 * s_bin[warp] + 8 * lane + i);
          thresholds[2 * m + warp] = __uint_as_float((bits == 0x8000u ? 0u : bits) << 16);
        }
        before += c[i];
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// absmax without clamping
// ------------------------------------------------------------------------------------------
// d[i] = amax[i] / MAX rounded once (MAX = 6 for E2M1, 448 for E4M3): the de-scale vector of a
// quantised operand, used as a prescale
__global__ void descale_kernel(const float* __restrict__ amax, int n, float div, float* __restrict__ d) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) d[i] = __fdiv_rn(amax[i], div);
}

struct AbsmaxArgs {
  const uint4* x;
  int rows, cols;
  const float* pre_col;         // multiplies along columns before the row-wise maximum (or null)
  const float* pre_row;         // multiplies along rows before the column-wise maximum (or null)
  float pre_col_div, pre_row_div;   // > 0: the vector holds amax values: use amax / div (6 or 448) and store it
  float* d_col_out;             // dual mode: the de-scale vectors actually used, for the encoder
  float* d_row_out;
  uint32_t* amax_rows;          // float bits, zero-initialised (non-negative floats order as integers)
  uint32_t* amax_cols;
  int32_t* status;              // FP4_DEV_NONFINITE is raised when a maximum is infinite or NaN
};

// Tile of 64 rows x 256 columns per block, same thread mapping as the encoder: warp w owns rows
// 8w..8w+7, lane l the 8 columns 8l..8l+7.
template <int MODE>
__global__ void __launch_bounds__(ENC_THREADS)
absmax_tile_kernel(const AbsmaxArgs a) {
  __shared__ float s_pcol[ENC_TK];
  __shared__ float s_prow[ENC_TM];
  __shared__ uint32_t s_cmax[8][ENC_TK];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row0 = blockIdx.y * ENC_TM, col0 = blockIdx.x * ENC_TK;
  const int vec_per_row = a.cols >> 3;
  constexpr bool want_rows = MODE != MODE_COLS, want_cols = MODE != MODE_ROWS;
  if (want_rows && a.pre_col) {
    const int c = col0 + tid;
    if (c < a.cols) {
      const float v = __ldg(&a.pre_col[c]);
      s_pcol[tid] = a.pre_col_div > 0.0f ? __fdiv_rn(v, a.pre_col_div) : v;
      if (a.d_col_out && blockIdx.y == 0) a.d_col_out[c] = s_pcol[tid];
    }
  }
  if (want_cols && a.pre_row && tid < ENC_TM) {
    const float v = __ldg(&a.pre_row[row0 + tid]);
    s_prow[tid] = a.pre_row_div > 0.0f ? __fdiv_rn(v, a.pre_row_div) : v;
    if (a.d_row_out && blockIdx.x == 0) a.d_row_out[row0 + tid] = s_prow[tid];
  }
  __syncthreads();
  const int col = col0 + 8 * lane;
  const bool in_cols = col < a.cols;
  uint4 v[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    v[r] = make_uint4(0, 0, 0, 0);
    if (in_cols) v[r] = __ldg(&a.x[(long long)(row0 + 8 * warp + r) * vec_per_row + (col >> 3)]);
  }
  float pc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) pc[c] = (want_rows && a.pre_col && in_cols) ? s_pcol[8 * lane + c] : 1.0f;
  // maxima as unsigned bit patterns of |x|: they order like the numbers, and a NaN (which fmaxf
  // would drop) ends up above infinity and is seen
  uint32_t cm[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const uint32_t w[4] = {v[r].x, v[r].y, v[r].z, v[r].w};
    const float pr = (want_cols && a.pre_row) ? s_prow[8 * warp + r] : 1.0f;
    uint32_t rm = 0;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const float f = (c & 1) ? bf16_hi(w[c >> 1]) : bf16_lo(w[c >> 1]);
      if (want_rows) rm = max(rm, __float_as_uint(fabsf(a.pre_col ? __fmul_rn(f, pc[c]) : f)));
      if (want_cols) cm[c] = max(cm[c], __float_as_uint(fabsf(a.pre_row ? __fmul_rn(f, pr) : f)));
    }
    if (want_rows) {
      const uint32_t g = __reduce_max_sync(0xFFFFFFFFu, rm);
      if (lane == 0) {
        atomicMax(&a.amax_rows[row0 + 8 * warp + r], g);
        if (g >= 0x7F800000u && a.status) atomicOr(a.status, FP4_DEV_NONFINITE);
      }
    }
  }
  if (want_cols) {
#pragma unroll
    for (int c = 0; c < 8; ++c) s_cmax[warp][8 * lane + c] = cm[c];
    __syncthreads();
    uint32_t m = 0;
#pragma unroll
    for (int w8 = 0; w8 < 8; ++w8) m = max(m, s_cmax[w8][tid]);
    if (col0 + tid < a.cols) {
      atomicMax(&a.amax_cols[col0 + tid], m);
      if (m >= 0x7F800000u && a.status) atomicOr(a.status, FP4_DEV_NONFINITE);
    }
  }
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
  const float* pre_col;         // prescale along columns (row-scaled output) or null
  const float* pre_row;         // prescale along rows (column-scaled output) or null
  const uint32_t* amax_rows;    // no clamp: max |x| per row (float bits)
  const uint32_t* amax_cols;    // max |x| per column
  const int* row_max;           // clamp: ordered-int row extremes
  const int* row_min;
  const float* thresholds;      // clamp: lo, hi
  uint32_t* codes;              // [rows x cols/8] words or null   (row-scaled in dual mode)
  uint32_t* codes_t;            // [cols x rows/8] words or null   (column-scaled in dual mode)
  float* amax_out_rows;
  float* amax_out_cols;
  uint8_t* mask;                // clamp: [rows x cols/8] bytes
  int* row_cnt;                 // clamp: clamped entries per row (zero-initialised)
  uint8_t* strip_cnt;           // clamp: [rows/64 x cols] clamped entries per (strip, column)
  int* col_cnt;                 // clamp: clamped entries per column (zero-initialised)
  float fmax;                   // FP8 encoder: the format's largest value (448 or 57344)
  int e5m2;                     // FP8 encoder: E5M2 bytes instead of E4M3 bytes
};

// MODE_ROWS: one scale per row -> codes and / or codes_t.  MODE_COLS: one scale per column.
// MODE_DUAL: codes hold the row-scaled tensor x (.) pre_col, codes_t the column-scaled tensor
// x (.) pre_row.  OCC (clamping) implies MODE_ROWS without prescale.
template <int MODE, bool OCC, bool PRESCALE, bool PER_TOKEN = false>
__global__ void __launch_bounds__(ENC_THREADS, 4)
encode_kernel(const EncodeArgs a) {
  __shared__ float s_gcol[ENC_TK];
  __shared__ float s_grow[ENC_TM];
  __shared__ float s_prow[ENC_TM];
  __shared__ uint32_t tile_t[8 * 8 * 32];
  __shared__ int s_colcnt[OCC ? ENC_TK : 1];
  __shared__ float s_thr[PER_TOKEN ? 2 * ENC_TM : 1];      // per-token clamp: lo, hi of the tile's rows
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int row0 = blockIdx.y * ENC_TM;
  const int col0 = blockIdx.x * ENC_TK;
  const int vec_per_row = a.cols >> 3;
  constexpr bool ROW_SCALED = MODE != MODE_COLS;      // a row-scaled output exists
  constexpr bool COL_SCALED = MODE != MODE_ROWS;
  float lo = 0.f, hi = 0.f;
  if (OCC) {
    if constexpr (!PER_TOKEN) {
      lo = a.thresholds[0];
      hi = a.thresholds[1];
    }
    s_colcnt[tid] = 0;
  }

  if (ROW_SCALED && tid < ENC_TM) {
    const int r = row0 + tid;
    float amax;
    if (OCC) {
      if constexpr (PER_TOKEN) {
        lo = s_thr[2 * tid] = a.thresholds[2 * r];
        hi = s_thr[2 * tid + 1] = a.thresholds[2 * r + 1];
      }
      const float mx = fminf(fmaxf(ordered_to_float(a.row_max[r]), lo), hi);
      const float mn = fminf(fmaxf(ordered_to_float(a.row_min[r]), lo), hi);
      amax = fmaxf(fabsf(mx), fabsf(mn));
    } else {
      amax = __uint_as_float(a.amax_rows[r]);
    }
    s_grow[tid] = amax > 0.0f ? __fdiv_rn(6.0f, amax) : 0.0f;
    if (blockIdx.x == 0) a.amax_out_rows[r] = amax;
  }
  if (COL_SCALED) {
    const int c = col0 + tid;
    if (c < a.cols) {
      const float amax = __uint_as_float(a.amax_cols[c]);
      s_gcol[tid] = amax > 0.0f ? __fdiv_rn(6.0f, amax) : 0.0f;
      if (blockIdx.y == 0) a.amax_out_cols[c] = amax;
    }
    if (PRESCALE && tid < ENC_TM) s_prow[tid] = __ldg(&a.pre_row[row0 + tid]);
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
  float gc[8], pc[8];
  if (COL_SCALED) {
#pragma unroll
    for (int c = 0; c < 8; ++c) gc[c] = in_cols ? s_gcol[8 * lane + c] : 0.0f;
  }
  if (ROW_SCALED && PRESCALE) {
#pragma unroll
    for (int c = 0; c < 8; ++c) pc[c] = in_cols ? __ldg(&a.pre_col[col + c]) : 0.0f;
  }

  uint32_t word[8];                                   // codes of the row-major output
  uint32_t word_t[MODE == MODE_DUAL ? 8 : 1];         // dual: codes of the column-scaled tensor
  uint32_t any_bits = 0, lo4 = 0, hi4 = 0;            // clamp: mask bytes of rows 0..3 / 4..7
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const uint32_t w[4] = {v[r].x, v[r].y, v[r].z, v[r].w};
    float f[8], f2[8];
    uint32_t obits = 0;
    const float grow = ROW_SCALED ? s_grow[8 * warp + r] : 0.0f;
    const float prow = (COL_SCALED && PRESCALE) ? s_prow[8 * warp + r] : 1.0f;
    if constexpr (PER_TOKEN) {
      lo = s_thr[2 * (8 * warp + r)];
      hi = s_thr[2 * (8 * warp + r) + 1];
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      float xv = (c & 1) ? bf16_hi(w[c >> 1]) : bf16_lo(w[c >> 1]);
      if (OCC) {
        const float xc = fminf(fmaxf(xv, lo), hi);
        obits |= (xc != xv ? 1u : 0u) << c;
        xv = xc;
      }
      // "+ 0.0f" turns a -0 product into +0 (the nudge needs a non-negative zero)
      if constexpr (MODE == MODE_ROWS) {
        f[c] = __fmaf_rn(PRESCALE ? __fmul_rn(xv, pc[c]) : xv, grow, 0.0f);
      } else if constexpr (MODE == MODE_COLS) {
        f[c] = __fmaf_rn(PRESCALE ? __fmul_rn(xv, prow) : xv, gc[c], 0.0f);
      } else {
        f[c] = __fmaf_rn(__fmul_rn(xv, pc[c]), grow, 0.0f);
        f2[c] = __fmaf_rn(__fmul_rn(xv, prow), gc[c], 0.0f);
      }
    }
    word[r] = encode8(f);
    if constexpr (MODE == MODE_DUAL) word_t[r] = encode8(f2);
    if (in_cols) {
      const long long o = (long long)(row0 + 8 * warp + r) * vec_per_row + (col >> 3);
      if (a.codes) a.codes[o] = word[r];
      if (OCC) a.mask[o] = uint8_t(obits);
    }
    if (OCC) {
      any_bits |= obits;
      if (r < 4) lo4 |= obits << (8 * r); else hi4 |= obits << (8 * (r - 4));
      const int cnt = __reduce_add_sync(0xFFFFFFFFu, __popc(obits));
      if (lane == 0 && cnt) atomicAdd(&a.row_cnt[row0 + 8 * warp + r], cnt);
    }
  }
  if (OCC) {
    // per-column counts of this 64-row strip: only threads that saw a clamped entry take part
    while (any_bits) {
      const int c = __ffs(any_bits) - 1;
      any_bits &= any_bits - 1;
      const uint32_t sel = 0x01010101u << c;
      atomicAdd(&s_colcnt[8 * lane + c], __popc(lo4 & sel) + __popc(hi4 & sel));
    }
  }

  if (a.codes_t) {
    if constexpr (MODE == MODE_DUAL) {
#pragma unroll
      for (int r = 0; r < 8; ++r) word[r] = word_t[r];
    }
    transpose8x8_nibbles(word);
#pragma unroll
    for (int c = 0; c < 8; ++c) tile_t[(c * 8 + warp) * 32 + lane] = word[c];
  }
  __syncthreads();
  if (OCC && col0 + tid < a.cols) {
    a.strip_cnt[(long long)blockIdx.y * a.cols + col0 + tid] = uint8_t(s_colcnt[tid]);
    if (s_colcnt[tid]) atomicAdd(&a.col_cnt[col0 + tid], s_colcnt[tid]);     // integer sums: order-independent
  }
  if (a.codes_t) {
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
// 3b. FP8 encoder (FP8 operands of the W4A8 / W8A4 settings and of the FP8 reading of dY)
// ------------------------------------------------------------------------------------------
// Two floats -> two FP8 bytes (first value in the low byte), E4M3 or E5M2: nearest even, saturating
// at the format's largest finite value (448 / 57344), the sign kept also on zero.
__device__ __forceinline__ uint32_t fp8x2(float lo, float hi, int e5m2) {
  uint16_t r;
  if (e5m2)
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  else
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
// 4 x 4 byte transpose: in[r] byte c -> out[c] byte r
__device__ __forceinline__ void transpose4x4_bytes(uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t (&c)[4]) {
  const uint32_t t0 = __byte_perm(a0, a1, 0x5140), t1 = __byte_perm(a2, a3, 0x5140);
  const uint32_t t2 = __byte_perm(a0, a1, 0x7362), t3 = __byte_perm(a2, a3, 0x7362);
  c[0] = __byte_perm(t0, t1, 0x5410);
  c[1] = __byte_perm(t0, t1, 0x7632);
  c[2] = __byte_perm(t2, t3, 0x5410);
  c[3] = __byte_perm(t2, t3, 0x7632);
}

// Same tile and thread mapping as encode_kernel, one byte per element: `codes` [rows x cols] bytes
// (row-scaled in dual mode), `codes_t` [cols x rows] bytes (column-scaled in dual mode).  No
// clamping: outlier clamping belongs to 4-bit activations.
template <int MODE, bool PRESCALE>
__global__ void __launch_bounds__(ENC_THREADS)
encode_fp8_kernel(const EncodeArgs a) {
  __shared__ float s_gcol[ENC_TK];
  __shared__ float s_grow[ENC_TM];
  __shared__ float s_prow[ENC_TM];
  __shared__ uint2 tile_t[8 * 8 * 32];
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int row0 = blockIdx.y * ENC_TM;
  const int col0 = blockIdx.x * ENC_TK;
  const int vec_per_row = a.cols >> 3;
  constexpr bool ROW_SCALED = MODE != MODE_COLS;
  constexpr bool COL_SCALED = MODE != MODE_ROWS;
  if (ROW_SCALED && tid < ENC_TM) {
    const int r = row0 + tid;
    const float amax = __uint_as_float(a.amax_rows[r]);
    s_grow[tid] = amax > 0.0f ? __fdiv_rn(a.fmax, amax) : 0.0f;
    if (blockIdx.x == 0) a.amax_out_rows[r] = amax;
  }
  if (COL_SCALED) {
    const int c = col0 + tid;
    if (c < a.cols) {
      const float amax = __uint_as_float(a.amax_cols[c]);
      s_gcol[tid] = amax > 0.0f ? __fdiv_rn(a.fmax, amax) : 0.0f;
      if (blockIdx.y == 0) a.amax_out_cols[c] = amax;
    }
    if (PRESCALE && tid < ENC_TM) s_prow[tid] = __ldg(&a.pre_row[row0 + tid]);
  }
  __syncthreads();

  const int col = col0 + 8 * lane;
  const bool in_cols = col < a.cols;
  uint4 v[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    v[r] = make_uint4(0, 0, 0, 0);
    if (in_cols) v[r] = __ldg(&a.x[(long long)(row0 + 8 * warp + r) * vec_per_row + (col >> 3)]);
  }
  float gc[8], pc[8];
  if (COL_SCALED) {
#pragma unroll
    for (int c = 0; c < 8; ++c) gc[c] = in_cols ? s_gcol[8 * lane + c] : 0.0f;
  }
  if (ROW_SCALED && PRESCALE) {
#pragma unroll
    for (int c = 0; c < 8; ++c) pc[c] = in_cols ? __ldg(&a.pre_col[col + c]) : 0.0f;
  }
  uint32_t lo4[8], hi4[8];                            // bytes of columns 0..3 / 4..7 of each row (output for codes_t)
  uint8_t* codes8 = reinterpret_cast<uint8_t*>(a.codes);
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const uint32_t w[4] = {v[r].x, v[r].y, v[r].z, v[r].w};
    float f[8], f2[8];
    const float grow = ROW_SCALED ? s_grow[8 * warp + r] : 0.0f;
    const float prow = (COL_SCALED && PRESCALE) ? s_prow[8 * warp + r] : 1.0f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const float xv = (c & 1) ? bf16_hi(w[c >> 1]) : bf16_lo(w[c >> 1]);
      if constexpr (MODE == MODE_ROWS) {
        f[c] = __fmul_rn(PRESCALE ? __fmul_rn(xv, pc[c]) : xv, grow);
      } else if constexpr (MODE == MODE_COLS) {
        f[c] = __fmul_rn(PRESCALE ? __fmul_rn(xv, prow) : xv, gc[c]);
      } else {
        f[c] = __fmul_rn(__fmul_rn(xv, pc[c]), grow);
        f2[c] = __fmul_rn(__fmul_rn(xv, prow), gc[c]);
      }
    }
    const uint32_t b_lo = fp8x2(f[0], f[1], a.e5m2) | (fp8x2(f[2], f[3], a.e5m2) << 16);
    const uint32_t b_hi = fp8x2(f[4], f[5], a.e5m2) | (fp8x2(f[6], f[7], a.e5m2) << 16);
    if (in_cols && codes8)
      *reinterpret_cast<uint2*>(codes8 + (long long)(row0 + 8 * warp + r) * a.cols + col) = make_uint2(b_lo, b_hi);
    if constexpr (MODE == MODE_DUAL) {
      lo4[r] = fp8x2(f2[0], f2[1], a.e5m2) | (fp8x2(f2[2], f2[3], a.e5m2) << 16);
      hi4[r] = fp8x2(f2[4], f2[5], a.e5m2) | (fp8x2(f2[6], f2[7], a.e5m2) << 16);
    } else {
      lo4[r] = b_lo;
      hi4[r] = b_hi;
    }
  }
  if (a.codes_t) {
    // 8 x 8 byte transpose in registers: column c of this thread's block as the bytes of rows 0..7
    uint32_t q00[4], q01[4], q10[4], q11[4];
    transpose4x4_bytes(lo4[0], lo4[1], lo4[2], lo4[3], q00);     // columns 0..3, rows 0..3
    transpose4x4_bytes(lo4[4], lo4[5], lo4[6], lo4[7], q01);     // columns 0..3, rows 4..7
    transpose4x4_bytes(hi4[0], hi4[1], hi4[2], hi4[3], q10);     // columns 4..7, rows 0..3
    transpose4x4_bytes(hi4[4], hi4[5], hi4[6], hi4[7], q11);     // columns 4..7, rows 4..7
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      tile_t[(c * 8 + warp) * 32 + lane] = make_uint2(q00[c], q01[c]);
      tile_t[((c + 4) * 8 + warp) * 32 + lane] = make_uint2(q10[c], q11[c]);
    }
  }
  __syncthreads();
  if (a.codes_t) {
    // thread (c = warp, j = lane) owns column col0 + 8 j + c: 64 rows = 64 bytes
    const int k = col0 + 8 * lane + warp;
    if (k < a.cols) {
      uint2 o[8];
#pragma unroll
      for (int w8 = 0; w8 < 8; ++w8) o[w8] = tile_t[(warp * 8 + w8) * 32 + lane];
      uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(a.codes_t) + (long long)k * a.rows + row0);
#pragma unroll
      for (int h = 0; h < 4; ++h) dst[h] = make_uint4(o[2 * h].x, o[2 * h].y, o[2 * h + 1].x, o[2 * h + 1].y);
    }
  }
}

// ------------------------------------------------------------------------------------------
// 4. mask -> CSR / CSC
// ------------------------------------------------------------------------------------------
// The CSR and the CSC of the residual are built from the encoder's mask and counts in three launches
// (formerly five, two of them single-block scans).
//
// Launch 1, sparse_prefix_kernel: block 0 turns the row counts into csr_rowptr (and nnz); every
// other block owns 1024 columns: their column pointers -- the counts of all earlier columns are
// summed by the block itself, so no block waits for another -- and, per column, the running offsets
// of the 64-row strips (strip_off), from which the fill kernel places a strip's entries.
// (A total cannot exceed the caller's capacity: the host refuses capacities below 2 n_tail, and at
// most n_tail entries lie beyond either threshold.  The fill kernel still guards every write.)
__global__ void __launch_bounds__(1024, 1)
sparse_prefix_kernel(const int* __restrict__ row_cnt, int rows, int* __restrict__ rowptr, int* __restrict__ nnz_out,
                     const int* __restrict__ col_cnt, const uint8_t* __restrict__ strip_cnt, int cols, int strips,
                     int* __restrict__ colptr, int* __restrict__ strip_off) {
  __shared__ long long warp_tot[32];
  const int t = threadIdx.x;
  if (blockIdx.x == 0) {
    const int per = (rows + 1023) / 1024;
    const int b = min(rows, t * per), e = min(rows, b + per);
    int s = 0;
    for (int i = b; i < e; ++i) s += row_cnt[i];
    const long long incl = block_scan_1024(s, warp_tot);
    int run = int(incl) - s;
    for (int i = b; i < e; ++i) {
      rowptr[i] = run;
      run += row_cnt[i];
    }
    if (t == 1023) {
      rowptr[rows] = int(incl);
      if (nnz_out) *nnz_out = int(incl);
    }
    return;
  }
  const int c0 = (int(blockIdx.x) - 1) * 1024;
  // entries of all earlier columns
  int before = 0;
  for (int i = t; i < c0; i += 1024) before += col_cnt[i];
  const long long earlier = block_scan_1024(before, warp_tot);
  __shared__ long long s_base;
  if (t == 1023) s_base = earlier;
  __syncthreads();
  const int k = c0 + t;
  const int mine = k < cols ? col_cnt[k] : 0;
  const long long incl = block_scan_1024(mine, warp_tot);
  if (k < cols) colptr[k] = int(s_base + incl) - mine;
  if (k == cols - 1) colptr[cols] = int(s_base + incl);
  if (k >= cols) return;
  int run = 0;
#pragma unroll 8
  for (int s = 0; s < strips; ++s) {
    const int c = strip_cnt[(long long)s * cols + k];
    strip_off[(long long)s * cols + k] = run;
    run += c;
  }
}

__device__ __forceinline__ float residual_of(const __nv_bfloat16* x, long long idx, float lo, float hi) {
  const float v = __bfloat162float(x[idx]);
  return __fsub_rn(v, v > hi ? hi : lo);
}

// CSR: one warp per row sweeps the row's mask words; a warp scan of the words' bit counts gives
// every marked entry its place, columns ascending.
__device__ __forceinline__ void csr_fill_block(int block, const uint32_t* __restrict__ mask,
                                               const __nv_bfloat16* __restrict__ x, int rows, int cols,
                                               const float* __restrict__ thresholds, int thr_per_row,
                                               const int* __restrict__ rowptr, long long cap, int* __restrict__ csr_col,
                                               float* __restrict__ csr_val) {
  const int row = block * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  int base = rowptr[row];
  if (rowptr[row + 1] == base) return;                // nothing clamped in this row
  const int words_per_row = cols >> 5;
  const float lo = thresholds[thr_per_row ? 2 * row : 0], hi = thresholds[thr_per_row ? 2 * row + 1 : 1];
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

// CSC: one warp per (64-row strip, 32-column word of the mask).  Lane <-> row: each lane keeps the
// mask word of its row.  For every column of the word that holds a marked entry (usually one or
// two: the outlier channels), a ballot gives each marked row its rank inside the column, so all
// gathers of a column are issued at once and the order is by row by construction.
__device__ __forceinline__ void csc_fill_block(int bx, int strip, const uint32_t* __restrict__ mask,
                                               const __nv_bfloat16* __restrict__ x, int rows, int cols,
                                               const float* __restrict__ thresholds, int thr_per_row,
                                               const int* __restrict__ colptr, const int* __restrict__ strip_off,
                                               long long cap, int* __restrict__ csc_row, float* __restrict__ csc_val) {
  const int q = bx * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int words_per_row = cols >> 5;
  if (q >= words_per_row) return;
  const int r0 = strip * ENC_TM;
  const uint32_t w0 = mask[(long long)(r0 + lane) * words_per_row + q];
  const uint32_t w1 = mask[(long long)(r0 + 32 + lane) * words_per_row + q];
  const uint32_t any0 = __reduce_or_sync(0xFFFFFFFFu, w0);
  const uint32_t any1 = __reduce_or_sync(0xFFFFFFFFu, w1);
  if (!(any0 | any1)) return;
  // lane c holds the next free position of column 32 q + c
  int next = colptr[32 * q + lane] + strip_off[(long long)strip * cols + 32 * q + lane];
  const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const uint32_t w = half ? w1 : w0;
    uint32_t any = half ? any1 : any0;
    const int r = r0 + 32 * half + lane;
    const float lo = thresholds[thr_per_row ? 2 * r : 0], hi = thresholds[thr_per_row ? 2 * r + 1 : 1];
    while (any) {
      const int c = __ffs(any) - 1;
      any &= any - 1;
      const bool mine = (w >> c) & 1u;
      const uint32_t b = __ballot_sync(0xFFFFFFFFu, mine);
      const int base = __shfl_sync(0xFFFFFFFFu, next, c);
      if (mine) {
        const int pos = base + __popc(b & lt_mask);
        if (pos < cap) {
          csc_row[pos] = r;
          csc_val[pos] = residual_of(x, (long long)r * cols + 32 * q + c, lo, hi);
        }
      }
      if (lane == c) next += __popc(b);
    }
  }
}

// Launches 2 and 3 fill the CSR (8 rows per block) and the CSC (8 mask words of one strip per block).
// They share only their inputs and run on two streams where the caller offers them: the forward's
// compensation waits for the CSR alone.
__global__ void __launch_bounds__(256)
csr_fill_kernel(const uint32_t* __restrict__ mask, const __nv_bfloat16* __restrict__ x, int rows, int cols,
                const float* __restrict__ thresholds, int thr_per_row, const int* __restrict__ rowptr, long long cap,
                int* __restrict__ csr_col, float* __restrict__ csr_val) {
  csr_fill_block(blockIdx.x, mask, x, rows, cols, thresholds, thr_per_row, rowptr, cap, csr_col, csr_val);
}

__global__ void __launch_bounds__(256)
csc_fill_kernel(const uint32_t* __restrict__ mask, const __nv_bfloat16* __restrict__ x, int rows, int cols,
                const float* __restrict__ thresholds, int thr_per_row, const int* __restrict__ colptr,
                const int* __restrict__ strip_off, long long cap, int* __restrict__ csc_row,
                float* __restrict__ csc_val) {
  csc_fill_block(blockIdx.x, blockIdx.y, mask, x, rows, cols, thresholds, thr_per_row, colptr, strip_off, cap, csc_row,
                 csc_val);
}

size_t r256(size_t b) { return (b + 255) & ~size_t(255); }

struct Scratch {
  int* row_max;
  int* row_min;
  uint32_t* amax_rows;
  uint32_t* amax_cols;
  uint8_t* mask;
  int* row_cnt;
  int* col_cnt;
  uint8_t* strip_cnt;
  int* strip_off;
  float* pre_rows;
  float* pre_cols;
  bool ok;
};

Scratch carve(Arena& arena, int rows, int cols, bool occ) {
  Scratch s = {};
  s.row_max = arena.take<int>(rows);
  s.row_min = arena.take<int>(rows);
  s.amax_rows = arena.take<uint32_t>(rows);
  s.amax_cols = arena.take<uint32_t>(cols);
  s.row_cnt = arena.take<int>(rows);
  s.col_cnt = arena.take<int>(cols);
  s.pre_rows = arena.take<float>(rows);
  s.pre_cols = arena.take<float>(cols);
  if (occ) {
    s.mask = arena.take<uint8_t>(size_t(rows) * cols / 8);
    s.strip_cnt = arena.take<uint8_t>(size_t(rows / ENC_TM) * cols);
    s.strip_off = arena.take<int>(size_t(rows / ENC_TM) * cols);
  }
  s.ok = arena.ok;
  return s;
}

}  // namespace

// Counters of the quantile selection that live as long as the context: two sets, parity, ticket.
size_t quantize_persistent_bytes() { return (2 * size_t(HIST_SET_WORDS) + 64) * 4; }

size_t quantize_scratch_bytes(int64_t rows, int64_t cols) {
  size_t b = 0;
  b += 5 * r256(size_t(rows) * 4) + 4 * r256(size_t(cols) * 4);   // per-row / per-column vectors
  b += r256(size_t(rows) * size_t(cols) / 8);                    // outlier mask
  b += r256(size_t(rows / ENC_TM) * size_t(cols));               // per-strip column counts (bytes)
  b += r256(size_t(rows / ENC_TM) * size_t(cols) * 4);           // per-strip column offsets
  return b;
}

int launch_quantize(fp4_ctx* ctx, cudaStream_t stream, Arena& arena, const void* x_bf16, int64_t rows64,
                    int64_t cols64, int scale_axis, double alpha, const float* prescale, float prescale_div,
                    fp4_qtensor* out, int32_t* status, const SparseOverlap* overlap) {
  const int rows = int(rows64), cols = int(cols64);
  const long long n = (long long)rows * cols;
  const bool occ = alpha < 1.0;
  const bool e4m3 = out->format == FP4_FORMAT_E4M3 || out->format == FP4_FORMAT_E5M2;   // an FP8 format
  if (out->format != FP4_FORMAT_E2M1 && !e4m3) return FP4_ERR_ARG;
  if (e4m3 && occ) return FP4_ERR_ARG;               // outlier clamping belongs to 4-bit activations
  const uint4* x = static_cast<const uint4*>(x_bf16);
  Scratch sc = carve(arena, rows, cols, occ);
  if (!sc.ok) return FP4_ERR_WORKSPACE;

  EncodeArgs ea = {};
  ea.x = x;
  ea.rows = rows;
  ea.cols = cols;
  ea.amax_rows = sc.amax_rows;
  ea.amax_cols = sc.amax_cols;
  ea.row_max = sc.row_max;
  ea.row_min = sc.row_min;
  ea.thresholds = out->thresholds;
  ea.codes = reinterpret_cast<uint32_t*>(out->codes);
  ea.codes_t = reinterpret_cast<uint32_t*>(out->codes_t);
  ea.amax_out_rows = out->amax;
  ea.amax_out_cols = out->amax;
  ea.mask = sc.mask;
  ea.row_cnt = sc.row_cnt;
  ea.strip_cnt = sc.strip_cnt;
  ea.col_cnt = sc.col_cnt;
  ea.e5m2 = out->format == FP4_FORMAT_E5M2;
  ea.fmax = fp8_max(out->format);
  const dim3 tile_grid((cols + ENC_TK - 1) / ENC_TK, rows / ENC_TM);

  const int per_token = occ && ctx->quantile_mode == FP4_QUANTILE_TOKEN;
  if (occ) {
    const long long n_tail = llround((1.0 - alpha) * double(n));
    const long long n_vec = n / 8;
    if (per_token) {
      KernelScope scope(ctx, stream, KC_SELECT, 1);
      const int n_tail_row = int(llround((1.0 - alpha) * double(cols)));
      row_select_kernel<<<rows, 256, 0, stream>>>(x, cols / 8, n_tail_row, sc.row_max, sc.row_min, sc.row_cnt,
                                                  out->thresholds, status);
    } else {
      // The two sets of global counters, their parity and the ticket belong to the context: the
      // kernel keeps the set it is about to use zero (see there), so nothing is cleared here.
      KernelScope scope(ctx, stream, KC_SELECT, 1);
      FP4_CUDA_TRY(cudaFuncSetAttribute(hist_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        HIST_SMEM_BYTES));
      long long blocks = (n_vec + HIST_THREADS - 1) / HIST_THREADS;
      if (blocks > ctx->num_sms) blocks = ctx->num_sms;
      unsigned* parity = reinterpret_cast<unsigned*>(ctx->occ_hist + 2 * HIST_SET_WORDS);
      hist_select_kernel<<<int(blocks), HIST_THREADS, HIST_SMEM_BYTES, stream>>>(
          x, rows, cols / 8, ctx->occ_hist, parity, sc.row_max, sc.row_min, sc.row_cnt, n, n_tail, out->thresholds,
          parity + 1, status, ctx->quantile_mode == FP4_QUANTILE_ABS);
    }
    FP4_CUDA_TRY(cudaMemsetAsync(sc.col_cnt, 0, size_t(cols) * 4, stream));     // the encoder adds to it
    {
      KernelScope scope(ctx, stream, KC_ENCODE, 1);
      if (per_token)
        encode_kernel<MODE_ROWS, true, false, true><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
      else
        encode_kernel<MODE_ROWS, true, false><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
    }
    cudaStream_t sp = stream;
    if (overlap && overlap->stream) {
      sp = overlap->stream;
      FP4_CUDA_TRY(cudaEventRecord(overlap->encoded, stream));
      FP4_CUDA_TRY(cudaStreamWaitEvent(sp, overlap->encoded, 0));
    }
    const uint32_t* mask32 = reinterpret_cast<const uint32_t*>(sc.mask);
    const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x_bf16);
    const int strips = rows / ENC_TM;
    // The CSC's fill takes a stream of its own where the caller offers one.
    cudaStream_t sc2 = sp;
    {
      KernelScope scope(ctx, sp, KC_SPARSE, 2);
      sparse_prefix_kernel<<<1 + (cols + 1023) / 1024, 1024, 0, sp>>>(sc.row_cnt, rows, out->csr_rowptr, out->nnz,
                                                                    sc.col_cnt, sc.strip_cnt, cols, strips,
                                                                    out->csc_colptr, sc.strip_off);
      if (sp != stream && overlap->colptr_done) FP4_CUDA_TRY(cudaEventRecord(overlap->colptr_done, sp));
      if (sp != stream && overlap->stream_csc && overlap->colptr_done) {
        sc2 = overlap->stream_csc;
        FP4_CUDA_TRY(cudaStreamWaitEvent(sc2, overlap->colptr_done, 0));
      }
      csr_fill_kernel<<<(rows + 7) / 8, 256, 0, sp>>>(mask32, xb, rows, cols, out->thresholds, per_token, out->csr_rowptr,
                                                      out->sparse_cap, out->csr_col, out->csr_val);
    }
    if (sp != stream) FP4_CUDA_TRY(cudaEventRecord(overlap->csr_done, sp));
    {
      KernelScope scope(ctx, sc2, KC_SPARSE, 1);
      const dim3 cgrid((cols / 32 + 7) / 8, strips);
      csc_fill_kernel<<<cgrid, 256, 0, sc2>>>(mask32, xb, rows, cols, out->thresholds, per_token, out->csc_colptr, sc.strip_off,
                                              out->sparse_cap, out->csc_row, out->csc_val);
    }
    if (sp != stream && overlap->csc_done) FP4_CUDA_TRY(cudaEventRecord(overlap->csc_done, sc2));
  } else {
    if (prescale && prescale_div > 0.0f) {
      float* d = scale_axis == 0 ? sc.pre_cols : sc.pre_rows;
      const int np = scale_axis == 0 ? cols : rows;
      KernelScope scope(ctx, stream, KC_ABSMAX, 1);
      descale_kernel<<<(np + 255) / 256, 256, 0, stream>>>(prescale, np, prescale_div, d);
      prescale = d;
    }
    AbsmaxArgs aa = {};
    aa.x = x;
    aa.rows = rows;
    aa.cols = cols;
    aa.amax_rows = sc.amax_rows;
    aa.amax_cols = sc.amax_cols;
    aa.status = status;
    if (scale_axis == 0) {
      aa.pre_col = prescale;
      ea.pre_col = prescale;
      FP4_CUDA_TRY(cudaMemsetAsync(sc.amax_rows, 0, size_t(rows) * 4, stream));
      {
        KernelScope scope(ctx, stream, KC_ABSMAX, 1);
        absmax_tile_kernel<MODE_ROWS><<<tile_grid, ENC_THREADS, 0, stream>>>(aa);
      }
      KernelScope scope(ctx, stream, KC_ENCODE, 1);
      if (e4m3 && prescale)
        encode_fp8_kernel<MODE_ROWS, true><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
      else if (e4m3)
        encode_fp8_kernel<MODE_ROWS, false><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
      else if (prescale)
        encode_kernel<MODE_ROWS, false, true><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
      else
        encode_kernel<MODE_ROWS, false, false><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
    } else {
      aa.pre_row = prescale;
      ea.pre_row = prescale;
      FP4_CUDA_TRY(cudaMemsetAsync(sc.amax_cols, 0, size_t(cols) * 4, stream));
      {
        KernelScope scope(ctx, stream, KC_ABSMAX, 1);
        absmax_tile_kernel<MODE_COLS><<<tile_grid, ENC_THREADS, 0, stream>>>(aa);
      }
      KernelScope scope(ctx, stream, KC_ENCODE, 1);
      if (e4m3 && prescale)
        encode_fp8_kernel<MODE_COLS, true><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
      else if (e4m3)
        encode_fp8_kernel<MODE_COLS, false><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
      else if (prescale)
        encode_kernel<MODE_COLS, false, true><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
      else
        encode_kernel<MODE_COLS, false, false><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
    }
  }
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}

// One read of dY for both backward GEMMs: row-scaled codes of dY (.) (amax_col_pre / 6) and
// column-scaled transposed codes of dY (.) (amax_row_pre / 6).
int launch_quantize_dual(fp4_ctx* ctx, cudaStream_t stream, Arena& arena, const void* x_bf16, int64_t rows64,
                         int64_t cols64, const float* amax_col_pre, const float* amax_row_pre, uint8_t* codes_rows,
                         float* amax_rows_out, uint8_t* codes_t_cols, float* amax_cols_out, int32_t* status,
                         int format, float col_pre_div, float row_pre_div) {
  const bool e4m3 = format != FP4_FORMAT_E2M1;       // an FP8 format
  const int rows = int(rows64), cols = int(cols64);
  Scratch sc = carve(arena, rows, cols, false);
  if (!sc.ok) return FP4_ERR_WORKSPACE;
  const dim3 tile_grid((cols + ENC_TK - 1) / ENC_TK, rows / ENC_TM);
  AbsmaxArgs aa = {};
  aa.x = static_cast<const uint4*>(x_bf16);
  aa.rows = rows;
  aa.cols = cols;
  aa.pre_col = amax_col_pre;
  aa.pre_row = amax_row_pre;
  aa.pre_col_div = col_pre_div;
  aa.pre_row_div = row_pre_div;
  aa.d_col_out = sc.pre_cols;
  aa.d_row_out = sc.pre_rows;
  aa.amax_rows = sc.amax_rows;
  aa.amax_cols = sc.amax_cols;
  aa.status = status;
  // amax_rows and amax_cols are carved one behind the other: one clearing covers both
  FP4_CUDA_TRY(cudaMemsetAsync(sc.amax_rows, 0,
                               size_t(reinterpret_cast<char*>(sc.amax_cols + cols) - reinterpret_cast<char*>(sc.amax_rows)),
                               stream));
  {
    KernelScope scope(ctx, stream, KC_ABSMAX, 1);
    absmax_tile_kernel<MODE_DUAL><<<tile_grid, ENC_THREADS, 0, stream>>>(aa);
  }
  EncodeArgs ea = {};
  ea.x = aa.x;
  ea.rows = rows;
  ea.cols = cols;
  ea.pre_col = sc.pre_cols;
  ea.pre_row = sc.pre_rows;
  ea.amax_rows = sc.amax_rows;
  ea.amax_cols = sc.amax_cols;
  ea.codes = reinterpret_cast<uint32_t*>(codes_rows);
  ea.codes_t = reinterpret_cast<uint32_t*>(codes_t_cols);
  ea.amax_out_rows = amax_rows_out;
  ea.amax_out_cols = amax_cols_out;
  ea.e5m2 = format == FP4_FORMAT_E5M2;
  ea.fmax = fp8_max(format);
  KernelScope scope(ctx, stream, KC_ENCODE, 1);
  if (e4m3)
    encode_fp8_kernel<MODE_DUAL, true><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
  else
    encode_kernel<MODE_DUAL, false, true><<<tile_grid, ENC_THREADS, 0, stream>>>(ea);
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}

// ------------------------------------------------------------------------------------------
// Quantile thresholds without any allocation
// ------------------------------------------------------------------------------------------
// Scratch of fp4_quantile_thresholds_static: the 65536-bin histogram, the select kernel's segment
// sums and ticket, and the row extremes of up to FP4_STATIC_MAX_ROWS rows.  It lives in the
// library image: every GPU that loads the library holds these 769 KB until the process exits.
namespace {
constexpr size_t STATIC_HIST_BYTES = 65536 * sizeof(uint32_t);
constexpr size_t STATIC_SELECT_BYTES = 1024;      // 32 coarse counters, then (at 512) the ticket
constexpr size_t STATIC_SCRATCH_BYTES =
    STATIC_HIST_BYTES + STATIC_SELECT_BYTES + 2 * size_t(FP4_STATIC_MAX_ROWS) * sizeof(int);
constexpr int STATIC_MAX_DEVICES = 64;
}  // namespace
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

extern "C" int fp4_quantile_thresholds_static(void* stream, const void* x_bf16, int64_t rows, int64_t cols,
                                              double alpha, float* thresholds) {
  // In host code `g_static_scratch` is only a handle; the device address of this device's copy
  // is looked up once per device and cached (under a lock: host threads may race to the first call).
  static void* scratch_of_device[STATIC_MAX_DEVICES] = {};
  static int sms_of_device[STATIC_MAX_DEVICES] = {};
  static std::mutex setup_lock;
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
  std::unique_lock<std::mutex> guard(setup_lock);
  if (!scratch_of_device[device]) {
    void* ptr = nullptr;
    FP4_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
    int sms = 0;
    FP4_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    FP4_CUDA_TRY(cudaFuncSetAttribute(hist_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      HIST_SMEM_BYTES));
    sms_of_device[device] = sms;
    scratch_of_device[device] = ptr;
  }
  const int num_sms = sms_of_device[device];
  unsigned char* base = static_cast<unsigned char*>(scratch_of_device[device]);
  guard.unlock();
  uint32_t* hist = reinterpret_cast<uint32_t*>(base);
  unsigned* ticket = reinterpret_cast<unsigned*>(base + STATIC_HIST_BYTES + 512);   // behind the coarse counters
  int* row_max = reinterpret_cast<int*>(base + STATIC_HIST_BYTES + STATIC_SELECT_BYTES);
  int* row_min = row_max + FP4_STATIC_MAX_ROWS;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array keeps what the previous call left (a call that was cut short may have left counts
  // behind): the histogram and the ticket are cleared; the row extremes are written before read.
  FP4_CUDA_TRY(cudaMemsetAsync(base, 0, STATIC_HIST_BYTES + STATIC_SELECT_BYTES, st));
  const long long n_vec = n / 8;
  long long blocks = (n_vec + HIST_THREADS - 1) / HIST_THREADS;
  if (blocks > num_sms) blocks = num_sms;
  hist_select_kernel<<<int(blocks), HIST_THREADS, HIST_SMEM_BYTES, st>>>(
      static_cast<const uint4*>(x_bf16), int(rows), int(cols / 8), hist, nullptr, row_max, row_min, nullptr, n, n_tail,
      thresholds, ticket, nullptr, 0);
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}
