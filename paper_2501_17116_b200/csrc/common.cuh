// Shared declarations of the CUDA sources (internal; the public ABI is include/fp4_linear.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

#include "fp4_linear.h"

// Kernel classes reported by fp4_profile_read (values are part of the ABI, see fp4_linear.h).
enum KernelClass {
  KC_GEMM = FP4_KC_GEMM,
  KC_SELECT = FP4_KC_SELECT,
  KC_ENCODE = FP4_KC_ENCODE,
  KC_ABSMAX = FP4_KC_ABSMAX,
  KC_SPARSE = FP4_KC_SPARSE,
  KC_COMP_FWD = FP4_KC_COMP_FWD,
  KC_COMP_WGRAD = FP4_KC_COMP_WGRAD,
  KC_COUNT = FP4_KC_COUNT
};

struct ProfRecord {
  int kc;
  int launches;
  cudaEvent_t start, stop;
};

// fp4_linear_step_host keeps this many sets of device input and output buffers in flight.  Two keep
// both copy directions busy (measured: a third set changes nothing, the copies back are never short
// of finished outputs for long).
constexpr int HOST_STEP_SETS = 2;

struct fp4_ctx {
  int      device;
  int      num_sms;
  char*    workspace;
  size_t   workspace_bytes;
  void*    encode_tiled;       // cuTensorMapEncodeTiled, fetched through the runtime
  uint32_t* occ_hist;          // quantile selection: two sets of global counters, parity, ticket
  cudaStream_t side[2];        // side streams for independent kernel chains inside one call
  cudaEvent_t  ev[8];          // fork / join events of those chains
  // fp4_linear_step_host, pipelined over consecutive calls:
  cudaStream_t copy_stream;          // host-to-device copies of a call's inputs
  cudaStream_t compute_stream;       // its kernels
  cudaStream_t return_stream;        // device-to-host copies of its outputs
  cudaEvent_t  host_step_copied[HOST_STEP_SETS];  // the inputs of set i have arrived
  cudaEvent_t  host_step_computed[HOST_STEP_SETS];// the outputs of set i are complete on the device
  cudaEvent_t  host_step_done[HOST_STEP_SETS];    // the call that used set i has left the workspace
  int      host_step_parity;         // set of the next pipelined call
  int      quantile_mode;            // FP4_QUANTILE_SIGNED (the paper's clamp) or FP4_QUANTILE_ABS
  int      overlap;            // run independent kernel chains on the side streams (default on)
  uint64_t debug_wait_limit_ns;  // fp4_debug_set: limit of the GEMM's device-side waits (0: the default, 2 s)
  int      debug_skip_fill;    // fp4_debug_set: fill of shared memory that CTA 0's producer leaves out (-1: none)
  int      profile;            // record CUDA events around every kernel class
  long long launch_count;      // kernels enqueued since the last reset
  std::vector<ProfRecord>* records;
};

// Counts the kernels a launcher enqueues and, in profiling mode, brackets them with CUDA events
// on the launching stream.
struct KernelScope {
  fp4_ctx* c;
  cudaStream_t s;
  cudaEvent_t stop = nullptr;
  KernelScope(fp4_ctx* ctx, cudaStream_t stream, int kc, int launches) : c(ctx), s(stream) {
    c->launch_count += launches;
    if (c->profile && c->records) {
      ProfRecord r;
      r.kc = kc;
      r.launches = launches;
      if (cudaEventCreate(&r.start) != cudaSuccess) return;
      if (cudaEventCreate(&r.stop) != cudaSuccess) { cudaEventDestroy(r.start); return; }
      cudaEventRecord(r.start, s);
      stop = r.stop;
      c->records->push_back(r);
    }
  }
  ~KernelScope() {
    if (stop) cudaEventRecord(stop, s);
  }
};

#define FP4_CUDA_TRY(expr)                         \
  do {                                             \
    cudaError_t e__ = (expr);                      \
    if (e__ != cudaSuccess) return FP4_ERR_CUDA;   \
  } while (0)

// Bump allocator over the context's workspace; every block is 256-byte aligned.
struct Arena {
  char*  base;
  size_t size;
  size_t off = 0;
  bool   ok = true;
  Arena(char* b, size_t s) : base(b), size(s) {}
  template <typename T>
  T* take(size_t count) {
    size_t bytes = (count * sizeof(T) + 255) & ~size_t(255);
    if (off + bytes > size) { ok = false; return nullptr; }
    T* p = reinterpret_cast<T*>(base + off);
    off += bytes;
    return p;
  }
};

// DGE derivative of Eq. 8 on a scaled weight, capped at `clip`.  The E2M1 grid has steps of 0.5
// below 2, 1 on [2, 4) and 2 from 4 up, i.e. delta = 2^(max(e, 0) - 1) with e the binary exponent
// of |w| (capped at the last interval, whose formula continues past 6).  With t = |w| / delta the
// position inside the interval [g, g + delta], mapped to [-1, 1], is u = 2 (t - floor(t)) - 1.
// Branch-free: the exponent arithmetic is done on the float's bit pattern.
__device__ __forceinline__ float dge_factor(float ws, float expo, float inv_k, float clip) {
  const float a = fabsf(ws);
  int em = int(__float_as_uint(a) >> 23);
  em = min(max(em, 127), 129);                                   // exponent 0, 1 or 2
  const float inv_delta = __uint_as_float(uint32_t(255 - em) << 23);    // 2, 1 or 1/2
  const float t = a * inv_delta;                                 // exact: a power of two
  const float g = em == 129 ? 2.0f : floorf(t);                  // last interval starts at 4 = 2 delta
  const float u = fabsf(fmaf(t - g, 2.0f, -1.0f));
  // |u|^(1/k - 1) = 2^((1/k - 1) log2 |u|); u = 0 gives +inf, which the cap turns into `clip`
  // both special-function instructions as they are (2^-22 relative: far inside the tolerance of the
  // weight gradient): log2(0) = -inf, times the negative exponent +inf, 2^+inf = +inf, capped below
  float p;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p) : "f"(expo * __log2f(u)));
  const float d = inv_k * p;
  return fminf(d, clip);
}

// Work fused into the epilogue of the weight-gradient GEMM (all null / zero: plain epilogue):
//   out[k, n] = store( (acc * d_col[n] + addend[slot_of_row[k], n]) * Q'(w[k, n] * 6 / w_amax[n]) )
struct GemmEpilogue {
  const float* addend;        // compact [slots x J] fp32 rows, added before the DGE factor (or null)
  const int*   slot_of_row;   // [I]: row of `addend` that belongs to output row i, -1 for none
  const void*  w_bf16;        // [I x J] BF16 weights whose scaled values drive the DGE factor (or null)
  const float* w_amax;        // [J]
  float dge_k, dge_clip;
};

// Largest value of an operand format: what an absmax scale maps the vector's maximum to.
inline float fp8_max(int format) {
  return format == FP4_FORMAT_E5M2 ? 57344.0f : (format == FP4_FORMAT_E4M3 ? 448.0f : 6.0f);
}

// Dense tail of the forward GEMM: the residual's hot columns (outlier channels, Appendix D) as extra
// contraction columns on the tensor cores instead of per-entry gathers.  With h <= TAIL_MAX_COLS hot
// columns, `a` is [I x TAIL_WIDTH] and `b` [J x TAIL_WIDTH] FP16, row-major, made of blocks of 64
// columns: for every 64 hot columns the blocks (A_hi, A_hi, A_lo) and (B_hi, B_lo, B_hi), where
// x_hi + x_lo is the two-term FP16 split of the fp32 value x, so that the three products sum to
// A B up to 2^-21.  A = residual / (row de-scale * 4), B = 4 * weight / column de-scale: the
// epilogue's de-scales then turn the tail's sum into residual x weight.  In the two cross products
// the small factor is stored 64 times larger and the large one 64 times smaller (A_hi / 64 against
// 64 B_lo, 64 A_lo against B_hi / 64), so that x_lo, about 2^-11 x, stays a normal FP16 number for
// every |x| >= 2^-8: the smallest residual, one BF16 step beyond a threshold, is 0.0058 in these
// units, a weight of 0.1 % of its column's maximum 0.024.  *count (device) is h; 0 switches the
// tail off.
constexpr int TAIL_MAX_COLS = 128;
constexpr int TAIL_WIDTH = 3 * TAIL_MAX_COLS;
constexpr float TAIL_SCALE = 4.0f;
constexpr float TAIL_BALANCE = 64.0f;
struct GemmTail {
  const void* a;
  const void* b;
  const int* count;
};

// ---- internal launchers (each enqueues on `stream`, returns an FP4_* host code) -------------

// out[i,j] = (sum_c a[i,c] b[j,c]) * (row_amax[i]/6) * (col_amax[j]/6)
int launch_gemm_fp4(fp4_ctx* ctx, cudaStream_t stream, const uint8_t* a_codes, const uint8_t* b_codes,
                    int64_t I, int64_t J, int64_t C, const float* row_amax, const float* col_amax,
                    void* out, int out_f32, int gemm_kind, int32_t* status,
                    const GemmEpilogue* epilogue = nullptr, int a_format = FP4_FORMAT_E2M1,
                    int b_format = FP4_FORMAT_E2M1, const GemmTail* tail = nullptr);

// One GEMM, for launches that take two of them.
struct Fp4GemmDesc {
  const uint8_t* a_codes;
  const uint8_t* b_codes;
  int64_t I, J, C;
  const float* row_amax;
  const float* col_amax;
  void* out;
  int out_f32;
  const GemmEpilogue* epilogue;
  int a_format = FP4_FORMAT_E2M1;   // operand formats: E2M1 nibbles, or E4M3 / E5M2 bytes (byte-container kind only)
  int b_format = FP4_FORMAT_E2M1;
};
// Both GEMMs in one launch; the tiles of `first` are computed first.
int launch_gemm_fp4_two(fp4_ctx* ctx, cudaStream_t stream, const Fp4GemmDesc& first, const Fp4GemmDesc& second,
                        int gemm_kind, int32_t* status);

// Lets the mask -> CSR / CSC stage of a clamping quantisation run beside the caller's stream: it
// starts after `encoded` (recorded on the main stream); the pointers kernel and the CSR fill run on
// `stream`, which records `colptr_done` once row and column pointers are complete and `csr_done`
// after the CSR fill; the CSC fill runs on `stream_csc` behind `colptr_done` and records `csc_done`
// there (null: it follows the CSR fill on `stream`).  The caller joins the streams.
struct SparseOverlap {
  cudaStream_t stream;
  cudaEvent_t encoded;
  cudaEvent_t csr_done;
  cudaStream_t stream_csc;
  cudaEvent_t csc_done;
  cudaEvent_t colptr_done;    // csr_rowptr and csc_colptr are complete (or null: the CSC fill stays on `stream`)
};

// Quantiser pieces (quantize.cu)
// `prescale_div` > 0: the prescale vector holds amax values and stands for amax / prescale_div (6 for an
// E2M1 operand, 448 for an E4M3 one); 0: the vector is used as it is.  out->format selects E2M1 or E4M3.
size_t quantize_scratch_bytes(int64_t rows, int64_t cols);
size_t quantize_persistent_bytes();
int launch_quantize(fp4_ctx* ctx, cudaStream_t stream, Arena& arena, const void* x_bf16, int64_t rows,
                    int64_t cols, int scale_axis, double alpha, const float* prescale,
                    float prescale_div, fp4_qtensor* out, int32_t* status,
                    const SparseOverlap* overlap = nullptr);

// dY for both backward GEMMs in one read: row-scaled codes of x (.) (amax_col_pre / col_pre_div) with
// their row amax, and column-scaled transposed codes of x (.) (amax_row_pre / row_pre_div) with their
// column amax; E2M1 nibbles or E4M3 bytes.
int launch_quantize_dual(fp4_ctx* ctx, cudaStream_t stream, Arena& arena, const void* x_bf16, int64_t rows,
                         int64_t cols, const float* amax_col_pre, const float* amax_row_pre,
                         uint8_t* codes_rows, float* amax_rows_out, uint8_t* codes_t_cols,
                         float* amax_cols_out, int32_t* status, int format = FP4_FORMAT_E2M1, float col_pre_div = 6.0f,
                         float row_pre_div = 6.0f);

// Sparse compensation and epilogues (compensate.cu)
// y[m,:] = store( y1[m,:] + sum_{entries of row m} val * dense[col,:] )
int launch_comp_fwd(fp4_ctx* ctx, cudaStream_t stream, const float* y1, const int32_t* rowptr,
                    const int32_t* col, const float* val, const void* w_bf16, int64_t M, int64_t K,
                    int64_t N, void* y, int out_f32, const int* slot_of_col = nullptr,
                    const int* tail_count = nullptr, const void* kept = nullptr, const int* kept_end = nullptr);
// The forward GEMM's dense tail (see GemmTail): operands built from the saved activation and the weights.
size_t fwd_tail_scratch_bytes(int64_t M, int64_t K, int64_t N);
// `kept_out` / `kept_end_out`: per token, the entries the tail does not cover (null for residuals too heavy to list).
int launch_fwd_tail(fp4_ctx* ctx, cudaStream_t stream, const fp4_qtensor* a, const void* w_bf16, const float* w_amax,
                    float w_div, Arena& scratch, int64_t M, int64_t K, int64_t N, GemmTail* tail,
                    const int** slot_of_col_out, const void** kept_out, const int** kept_end_out);
// Weight-gradient compensation into a compact buffer: for every column k of the residual that
// holds entries, comp[slot_of_col[k], :] = sum_{entries of column k} val * dy[row, :].
// Lists, slots and the dense path's buffers are carved from `scratch` (comp_wgrad_scratch_bytes); the slot
// vector is handed back for the GEMM's epilogue.  `a` is the saved activation (CSC; CSR for the dense path).
int launch_comp_wgrad(fp4_ctx* ctx, cudaStream_t stream, const fp4_qtensor* a, const void* dy_bf16, Arena& scratch,
                      int** slot_of_col_out, float* comp, int64_t M, int64_t K, int64_t N, int32_t* status);
size_t comp_wgrad_scratch_bytes(int64_t M, int64_t K, int64_t N);

// Dense columns of the residual in the weight gradient, on the tensor cores (wgrad_dense_tc.cu):
// C[s, :] = sum_m V[m, s] dY[m, :] for the s < counts[0] <= DENSE_TC_MAX dense columns, as `splits`
// sets of partial sums ([splits][DENSE_TC_MAX][N], one per range of tokens) that the caller adds in
// order.  `vt` holds 3 * DENSE_TC_MAX * M BF16 values of scratch.
constexpr int DENSE_TC_MAX = 128;
int dense_tc_splits(const fp4_ctx* ctx, int64_t M, int64_t N);
size_t dense_tc_scratch_bytes(int64_t M, int64_t N);
int launch_comp_wgrad_dense_tc(fp4_ctx* ctx, cudaStream_t stream, const fp4_qtensor* a, const int* slot_of_col,
                               const int* counts, const void* dy_bf16, void* vt, float* partial, int splits,
                               int64_t M, int64_t N, int32_t* status);

