// C ABI of the library: argument validation, workspace carving and kernel sequencing.
// Every step of the path runs in the kernels of this directory; nothing here computes.
#include <cuda.h>

#include <cmath>
#include <new>

#include "common.cuh"

namespace {

bool mult128(int64_t v) { return v > 0 && (v % 128) == 0; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
bool known_format(int f) { return f == FP4_FORMAT_E2M1 || f == FP4_FORMAT_E4M3 || f == FP4_FORMAT_E5M2; }
bool is_fp8(int f) { return f == FP4_FORMAT_E4M3 || f == FP4_FORMAT_E5M2; }

size_t round256(size_t b) { return (b + 255) & ~size_t(255); }

// Bytes a call needs on top of the quantiser scratch: the fp32 GEMM result the forward compensation
// kernel consumes (the backward keeps its compact compensation rows there), both quantised copies
// of dY, and the lists of the residual's non-empty columns.
size_t linear_scratch_bytes(int64_t M, int64_t K, int64_t N) {
  size_t b = 0;
  const size_t big = size_t(M > K ? M : K) * size_t(N);
  b += round256(big * sizeof(float));                 // fwd: M x N result; bwd: up to K compensation rows of N
  b += 2 * round256(size_t(M) * size_t(N));           // dY codes, both scalings (E4M3 bytes at most)
  b += round256(size_t(M) * 4) + round256(size_t(N) * 4);   // their amax vectors
  b += 2 * round256(size_t(M > N ? M : N) * 4);       // de-scale vectors used as prescale
  b += comp_wgrad_scratch_bytes(M, K, N);             // non-empty residual columns, dense-column buffers
  b += fwd_tail_scratch_bytes(M, K, N);               // operands of the forward GEMM's dense tail
  return b;
}

int check_qtensor_dense(const fp4_qtensor* q) {
  if (!q || !q->amax) return FP4_ERR_NULL;
  if (!q->codes && !q->codes_t) return FP4_ERR_NULL;
  return FP4_OK;
}

int linear_fwd_impl(fp4_ctx* ctx, cudaStream_t st, Arena arena, const void* A_bf16, const void* W_bf16, int64_t M,
                    int64_t K, int64_t N, double alpha, int reuse, int gemm_kind, void* Y, int out_f32,
                    fp4_qtensor* savedA, fp4_qtensor* savedW, int32_t* status);
int linear_bwd_impl(fp4_ctx* ctx, cudaStream_t st, Arena arena, const void* dY_bf16, const void* W_bf16,
                    const fp4_qtensor* savedA, const fp4_qtensor* savedW, int64_t M, int64_t K, int64_t N, int dge_on,
                    float dge_k, float dge_clip, int gemm_kind, void* dA, void* dW, int out_f32, int32_t* status);

int check_qtensor_sparse(const fp4_qtensor* q, int64_t n_tail) {
  if (!q->thresholds || !q->nnz || !q->csr_rowptr || !q->csr_col || !q->csr_val || !q->csc_colptr || !q->csc_row ||
      !q->csc_val)
    return FP4_ERR_NULL;
  if (q->sparse_cap < 2 * n_tail) return FP4_ERR_CAPACITY;
  return FP4_OK;
}

}  // namespace

extern "C" {

const char* fp4_status_string(int code) {
  switch (code) {
    case FP4_OK: return "ok";
    case FP4_ERR_NULL: return "a required pointer is NULL";
    case FP4_ERR_SHAPE: return "a dimension is not a positive multiple of 128";
    case FP4_ERR_ALPHA: return "alpha outside (0.5, 1]";
    case FP4_ERR_ALIGN: return "a tensor pointer is not sufficiently aligned";
    case FP4_ERR_WORKSPACE: return "the context's workspace is too small";
    case FP4_ERR_CUDA: return "a CUDA call failed";
    case FP4_ERR_ARG: return "an argument has an unsupported value";
    case FP4_ERR_CAPACITY: return "sparse_cap is below fp4_sparse_capacity()";
    case FP4_ERR_STATIC_LIMIT: return "input exceeds the fixed scratch of the allocation-free entry point";
    default: return "unknown status";
  }
}

size_t fp4_workspace_bytes(int64_t M, int64_t K, int64_t N) {
  if (M <= 0 || K <= 0 || N <= 0) return 0;
  // forward: A and W are quantised concurrently, each in its own scratch; backward: dY alone
  size_t q = quantize_scratch_bytes(M, K) + quantize_scratch_bytes(K, N);
  const size_t qg = quantize_scratch_bytes(M, N);
  if (qg > q) q = qg;
  return q + linear_scratch_bytes(M, K, N) + 4096;
}

int fp4_create(fp4_ctx** out, int device, size_t workspace_bytes) {
  if (!out) return FP4_ERR_NULL;
  *out = nullptr;
  FP4_CUDA_TRY(cudaSetDevice(device));
  fp4_ctx* ctx = new (std::nothrow) fp4_ctx();
  if (!ctx) return FP4_ERR_CUDA;
  ctx->device = device;
  ctx->workspace = nullptr;
  ctx->workspace_bytes = 0;
  ctx->encode_tiled = nullptr;
  ctx->occ_hist = nullptr;
  ctx->profile = 0;
  ctx->debug_wait_limit_ns = 0;
  ctx->debug_skip_fill = -1;
  ctx->overlap = 1;
  ctx->launch_count = 0;
  ctx->records = new (std::nothrow) std::vector<ProfRecord>();
  for (auto& s : ctx->side) s = nullptr;
  for (auto& e : ctx->ev) e = nullptr;
  ctx->copy_stream = ctx->compute_stream = ctx->return_stream = nullptr;
  for (auto& e : ctx->host_step_done) e = nullptr;
  for (auto& e : ctx->host_step_copied) e = nullptr;
  for (auto& e : ctx->host_step_computed) e = nullptr;
  ctx->host_step_parity = 0;
  ctx->quantile_mode = FP4_QUANTILE_SIGNED;
  cudaDeviceProp prop;
  if (!ctx->records || cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
    delete ctx->records;
    delete ctx;
    return FP4_ERR_CUDA;
  }
  ctx->num_sms = prop.multiProcessorCount;
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    delete ctx->records;
    delete ctx;
    return FP4_ERR_CUDA;
  }
  ctx->encode_tiled = fn;
  if (workspace_bytes) {
    if (cudaMalloc(reinterpret_cast<void**>(&ctx->workspace), workspace_bytes) != cudaSuccess) {
      delete ctx->records;
      delete ctx;
      return FP4_ERR_CUDA;
    }
    ctx->workspace_bytes = workspace_bytes;
  }
  bool ok = true;
  // counters of the quantile selection (quantisation with clamping): cleared here, once
  ok = ok && cudaMalloc(reinterpret_cast<void**>(&ctx->occ_hist), quantize_persistent_bytes()) == cudaSuccess;
  ok = ok && cudaMemset(ctx->occ_hist, 0, quantize_persistent_bytes()) == cudaSuccess;
  for (auto& s : ctx->side) ok = ok && cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) == cudaSuccess;
  for (auto& e : ctx->ev) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&ctx->compute_stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&ctx->return_stream, cudaStreamNonBlocking) == cudaSuccess;
  for (auto& e : ctx->host_step_computed) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
  for (auto& e : ctx->host_step_done) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
  for (auto& e : ctx->host_step_copied) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    fp4_destroy(ctx);
    return FP4_ERR_CUDA;
  }
  *out = ctx;
  return FP4_OK;
}

int fp4_destroy(fp4_ctx* ctx) {
  if (!ctx) return FP4_ERR_NULL;
  cudaSetDevice(ctx->device);
  for (auto& s : ctx->side)
    if (s) cudaStreamDestroy(s);
  for (auto& e : ctx->ev)
    if (e) cudaEventDestroy(e);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  if (ctx->compute_stream) cudaStreamDestroy(ctx->compute_stream);
  if (ctx->return_stream) cudaStreamDestroy(ctx->return_stream);
  for (auto& e : ctx->host_step_computed)
    if (e) cudaEventDestroy(e);
  for (auto& e : ctx->host_step_done)
    if (e) cudaEventDestroy(e);
  for (auto& e : ctx->host_step_copied)
    if (e) cudaEventDestroy(e);
  if (ctx->workspace) cudaFree(ctx->workspace);
  if (ctx->occ_hist) cudaFree(ctx->occ_hist);
  if (ctx->records) {
    fp4_profile_reset(ctx);
    delete ctx->records;
  }
  delete ctx;
  return FP4_OK;
}

int fp4_quantize(fp4_ctx* ctx, void* stream, const void* x_bf16, int64_t rows, int64_t cols, int scale_axis,
                 double alpha, const float* prescale, fp4_qtensor* out, int32_t* status) {
  if (!ctx || !x_bf16 || !out || !status) return FP4_ERR_NULL;
  if (!mult128(rows) || !mult128(cols) || rows * cols >= (int64_t(1) << 31)) return FP4_ERR_SHAPE;
  if (scale_axis != 0 && scale_axis != 1) return FP4_ERR_ARG;
  if (!(alpha > 0.5 && alpha <= 1.0)) return FP4_ERR_ALPHA;
  int rc = check_qtensor_dense(out);
  if (rc != FP4_OK) return rc;
  if (!known_format(out->format)) return FP4_ERR_ARG;
  if (!aligned16(x_bf16) || !aligned16(out->codes) || !aligned16(out->codes_t) || !aligned16(out->amax))
    return FP4_ERR_ALIGN;
  if (alpha < 1.0) {
    if (scale_axis != 0 || prescale || out->format != FP4_FORMAT_E2M1) return FP4_ERR_ARG;
    const int64_t n = rows * cols;
    int64_t n_tail = llround((1.0 - alpha) * double(n));
    if (2 * n_tail >= n) return FP4_ERR_ALPHA;
    if (ctx->quantile_mode == FP4_QUANTILE_TOKEN) {       // per token: every row has its own two tails
      const int64_t per_row = llround((1.0 - alpha) * double(cols));
      if (2 * per_row >= cols) return FP4_ERR_ALPHA;
      n_tail = rows * per_row;
    }
    rc = check_qtensor_sparse(out, n_tail);
    if (rc != FP4_OK) return rc;
  }
  if (quantize_scratch_bytes(rows, cols) > ctx->workspace_bytes) return FP4_ERR_WORKSPACE;
  Arena arena(ctx->workspace, ctx->workspace_bytes);
  out->rows = rows;
  out->cols = cols;
  return launch_quantize(ctx, static_cast<cudaStream_t>(stream), arena, x_bf16, rows, cols, scale_axis, alpha,
                         prescale, 0.0f, out, status);
}

int fp4_gemm(fp4_ctx* ctx, void* stream, const uint8_t* a_codes, const uint8_t* b_codes, int64_t I, int64_t J,
             int64_t C, const float* row_amax, const float* col_amax, void* out, int out_f32, int gemm_kind,
             int32_t* status) {
  if (!ctx || !a_codes || !b_codes || !out || !status) return FP4_ERR_NULL;
  if (!mult128(I) || !mult128(J) || !mult128(C)) return FP4_ERR_SHAPE;
  if (!aligned16(out)) return FP4_ERR_ALIGN;
  const int e5m2_flags = gemm_kind & (FP4_GEMM_A_E5M2 | FP4_GEMM_B_E5M2);
  gemm_kind &= ~(FP4_GEMM_A_E5M2 | FP4_GEMM_B_E5M2);
  if (gemm_kind < FP4_GEMM_MXF4 || gemm_kind > FP4_GEMM_F8F6F4_A8B8) return FP4_ERR_ARG;
  const bool a8 = gemm_kind == FP4_GEMM_F8F6F4_A8 || gemm_kind == FP4_GEMM_F8F6F4_A8B8;
  const bool b8 = gemm_kind == FP4_GEMM_F8F6F4_B8 || gemm_kind == FP4_GEMM_F8F6F4_A8B8;
  // the E5M2 flags qualify an 8-bit operand
  if (((e5m2_flags & FP4_GEMM_A_E5M2) && !a8) || ((e5m2_flags & FP4_GEMM_B_E5M2) && !b8)) return FP4_ERR_ARG;
  const int a_format = a8 ? ((e5m2_flags & FP4_GEMM_A_E5M2) ? FP4_FORMAT_E5M2 : FP4_FORMAT_E4M3) : FP4_FORMAT_E2M1;
  const int b_format = b8 ? ((e5m2_flags & FP4_GEMM_B_E5M2) ? FP4_FORMAT_E5M2 : FP4_FORMAT_E4M3) : FP4_FORMAT_E2M1;
  const int kind = gemm_kind >= FP4_GEMM_F8F6F4 ? FP4_GEMM_F8F6F4 : FP4_GEMM_MXF4;
  return launch_gemm_fp4(ctx, static_cast<cudaStream_t>(stream), a_codes, b_codes, I, J, C, row_amax, col_amax, out,
                         out_f32, kind, status, nullptr, a_format, b_format);
}

int fp4_linear_fwd(fp4_ctx* ctx, void* stream, const void* A_bf16, const void* W_bf16, int64_t M, int64_t K,
                   int64_t N, double alpha, int reuse, int gemm_kind, void* Y, int out_f32, fp4_qtensor* savedA,
                   fp4_qtensor* savedW, int32_t* status) {
  if (!ctx || !A_bf16 || !W_bf16 || !Y || !savedA || !savedW || !status) return FP4_ERR_NULL;
  if (!mult128(M) || !mult128(K) || !mult128(N)) return FP4_ERR_SHAPE;
  if (M * K >= (int64_t(1) << 31) || K * N >= (int64_t(1) << 31) || M * N >= (int64_t(1) << 31)) return FP4_ERR_SHAPE;
  if (!(alpha > 0.5 && alpha <= 1.0)) return FP4_ERR_ALPHA;
  if (gemm_kind != FP4_GEMM_MXF4 && gemm_kind != FP4_GEMM_F8F6F4) return FP4_ERR_ARG;
  if (!savedA->codes || !savedA->codes_t || !savedA->amax) return FP4_ERR_NULL;
  if (!savedW->codes || !savedW->codes_t || !savedW->amax) return FP4_ERR_NULL;
  if (!aligned16(A_bf16) || !aligned16(W_bf16) || !aligned16(Y)) return FP4_ERR_ALIGN;
  const bool occ = alpha < 1.0;
  {
    const bool a8 = is_fp8(savedA->format), w8 = is_fp8(savedW->format);
    if (!known_format(savedA->format) || !known_format(savedW->format)) return FP4_ERR_ARG;
    if ((a8 || w8) && gemm_kind != FP4_GEMM_F8F6F4) return FP4_ERR_ARG;   // FP8 operands need the byte-container kind
    if (a8 && occ) return FP4_ERR_ARG;                                    // clamping belongs to 4-bit activations
  }
  if (occ) {
    int64_t n_tail = llround((1.0 - alpha) * double(M * K));
    if (2 * n_tail >= M * K) return FP4_ERR_ALPHA;
    if (ctx->quantile_mode == FP4_QUANTILE_TOKEN) {       // per token: every row has its own two tails
      const int64_t per_row = llround((1.0 - alpha) * double(K));
      if (2 * per_row >= K) return FP4_ERR_ALPHA;
      n_tail = M * per_row;
    }
    int rc = check_qtensor_sparse(savedA, n_tail);
    if (rc != FP4_OK) return rc;
  }
  if (fp4_workspace_bytes(M, K, N) > ctx->workspace_bytes) return FP4_ERR_WORKSPACE;
  return linear_fwd_impl(ctx, static_cast<cudaStream_t>(stream), Arena(ctx->workspace, ctx->workspace_bytes), A_bf16,
                         W_bf16, M, K, N, alpha, reuse, gemm_kind, Y, out_f32, savedA, savedW, status);
}

}  // extern "C"

namespace {

int linear_fwd_impl(fp4_ctx* ctx, cudaStream_t st, Arena arena, const void* A_bf16, const void* W_bf16, int64_t M,
                    int64_t K, int64_t N, double alpha, int reuse, int gemm_kind, void* Y, int out_f32,
                    fp4_qtensor* savedA, fp4_qtensor* savedW, int32_t* status) {
  const bool occ = alpha < 1.0;
  const bool reuse_w = (reuse & FP4_REUSE_W) != 0, reuse_a = (reuse & FP4_REUSE_A) != 0;
  float* y1 = occ ? arena.take<float>(size_t(M) * size_t(N)) : nullptr;
  char* scratch_a = reuse_a ? nullptr : arena.take<char>(quantize_scratch_bytes(M, K));
  char* scratch_w = reuse_w ? nullptr : arena.take<char>(quantize_scratch_bytes(K, N));
  // A heavy residual (the caller's capacity says it may hold at least 1 % of the activation, alpha <=
  // 0.995) sends its hot columns through the GEMM as a dense tail instead of per-entry gathers.
  const bool tail_on = occ && savedA->csr_rowptr && savedA->csc_colptr &&
                       savedA->sparse_cap * 100 >= M * K && M >= 512;   // a hot column holds at least 512 entries
  char* scratch_tail = tail_on ? arena.take<char>(fwd_tail_scratch_bytes(M, K, N)) : nullptr;
  if (!arena.ok) return FP4_ERR_WORKSPACE;
  int rc;

  // Independent chains: W (side stream 0), A up to its codes (caller's stream), and the
  // mask -> CSR and mask -> CSC stages of A (side streams 1 and 0), which only the compensation
  // and the backward need.
  const bool ov = ctx->overlap != 0;
  if (!reuse_w) {
    cudaStream_t s0 = ov ? ctx->side[0] : st;
    if (ov) {
      FP4_CUDA_TRY(cudaEventRecord(ctx->ev[0], st));
      FP4_CUDA_TRY(cudaStreamWaitEvent(s0, ctx->ev[0], 0));
    }
    Arena a(scratch_w, quantize_scratch_bytes(K, N));
    savedW->rows = K;
    savedW->cols = N;
    rc = launch_quantize(ctx, s0, a, W_bf16, K, N, /*scale_axis=*/1, 1.0, nullptr, 0.0f, savedW, status);
    if (rc != FP4_OK) return rc;
    if (ov) FP4_CUDA_TRY(cudaEventRecord(ctx->ev[1], s0));
  }
  if (!reuse_a) {
    Arena a(scratch_a, quantize_scratch_bytes(M, K));
    savedA->rows = M;
    savedA->cols = K;
    // CSR on side stream 1, CSC on side stream 0 (behind W's short chain, which has ended by then)
    const SparseOverlap so = {ctx->side[1], ctx->ev[2], ctx->ev[3], ctx->side[0], ctx->ev[7], ctx->ev[4]};
    rc = launch_quantize(ctx, st, a, A_bf16, M, K, /*scale_axis=*/0, alpha, nullptr, 0.0f, savedA, status,
                         occ && ov ? &so : nullptr);
    if (rc != FP4_OK) return rc;
  }
  if (!reuse_w && ov) FP4_CUDA_TRY(cudaStreamWaitEvent(st, ctx->ev[1], 0));
  // Y1 = (Q(A_c) Q(W)) * d_A[m] * d_W[n]: A codes [M x K/2], W codes transposed [N x K/2].
  const int a8 = savedA->format, w8 = savedW->format;      // operand formats (0: E2M1)
  if (!occ) {
    // Without clamping there is no residual: a saved operand that still carries the sparse
    // structure of an earlier clamped use is marked empty, so that the backward adds nothing.
    if (!reuse_a && savedA->csc_colptr && savedA->csr_rowptr && savedA->nnz) {
      FP4_CUDA_TRY(cudaMemsetAsync(savedA->csc_colptr, 0, (size_t(K) + 1) * 4, st));
      FP4_CUDA_TRY(cudaMemsetAsync(savedA->csr_rowptr, 0, (size_t(M) + 1) * 4, st));
      FP4_CUDA_TRY(cudaMemsetAsync(savedA->nnz, 0, 4, st));
    }
    return launch_gemm_fp4(ctx, st, savedA->codes, savedW->codes_t, M, N, K, savedA->amax, savedW->amax, Y, out_f32,
                           gemm_kind, status, nullptr, a8, w8);
  }
  GemmTail tail = {nullptr, nullptr, nullptr};
  const int* hot_slot_of_col = nullptr;
  const void* kept = nullptr;
  const int* kept_end = nullptr;
  if (tail_on) {
    // The tail's operands need the CSR, the CSC's column pointers and W's amax: the CSR chain and
    // the first half of the CSC chain are joined before the GEMM here; the CSC's fill runs beside it.
    if (!reuse_a && ov) {
      FP4_CUDA_TRY(cudaStreamWaitEvent(st, ctx->ev[3], 0));
      FP4_CUDA_TRY(cudaStreamWaitEvent(st, ctx->ev[4], 0));
    }
    Arena ta(scratch_tail, fwd_tail_scratch_bytes(M, K, N));
    rc = launch_fwd_tail(ctx, st, savedA, W_bf16, savedW->amax, fp8_max(w8), ta, M, K, N, &tail, &hot_slot_of_col, &kept,
                         &kept_end);
    if (rc != FP4_OK) return rc;
  }
  rc = launch_gemm_fp4(ctx, st, savedA->codes, savedW->codes_t, M, N, K, savedA->amax, savedW->amax, y1, 1, gemm_kind,
                       status, nullptr, a8, w8, tail_on ? &tail : nullptr);
  if (rc != FP4_OK) return rc;
  // Y = store(Y1 + (A - A_c) W): one rounding of the fp32 sum.  Needs the CSR.
  if (!reuse_a && ov) FP4_CUDA_TRY(cudaStreamWaitEvent(st, ctx->ev[3], 0));
  rc = launch_comp_fwd(ctx, st, y1, savedA->csr_rowptr, savedA->csr_col, savedA->csr_val, W_bf16, M, K, N, Y, out_f32,
                       hot_slot_of_col, tail.count, kept, kept_end);
  if (rc != FP4_OK) return rc;
  if (!reuse_a && ov) FP4_CUDA_TRY(cudaStreamWaitEvent(st, ctx->ev[7], 0));  // the CSC too: savedA is complete on return
  return FP4_OK;
}

}  // namespace

extern "C" {

int fp4_linear_bwd(fp4_ctx* ctx, void* stream, const void* dY_bf16, const void* W_bf16, const fp4_qtensor* savedA,
                   const fp4_qtensor* savedW, int64_t M, int64_t K, int64_t N, int dge_on, float dge_k,
                   float dge_clip, int gemm_kind, void* dA, void* dW, int out_f32, int32_t* status) {
  if (!ctx || !dY_bf16 || !W_bf16 || !savedA || !savedW || !status) return FP4_ERR_NULL;
  if (!dA && !dW) return FP4_ERR_NULL;
  if (!mult128(M) || !mult128(K) || !mult128(N)) return FP4_ERR_SHAPE;
  if (M * K >= (int64_t(1) << 31) || K * N >= (int64_t(1) << 31) || M * N >= (int64_t(1) << 31)) return FP4_ERR_SHAPE;
  {
    const int dy_flags = gemm_kind & (FP4_BWD_DY_E4M3 | FP4_BWD_DY_E5M2);
    const int kind = gemm_kind & ~(FP4_BWD_DY_E4M3 | FP4_BWD_DY_E5M2);
    if (kind != FP4_GEMM_MXF4 && kind != FP4_GEMM_F8F6F4) return FP4_ERR_ARG;
    if (dy_flags == (FP4_BWD_DY_E4M3 | FP4_BWD_DY_E5M2)) return FP4_ERR_ARG;   // one format for dY
    if (!known_format(savedA->format) || !known_format(savedW->format)) return FP4_ERR_ARG;
    const bool any8 = dy_flags || is_fp8(savedA->format) || is_fp8(savedW->format);
    if (any8 && kind != FP4_GEMM_F8F6F4) return FP4_ERR_ARG;             // FP8 operands need the byte-container kind
  }
  if (dge_on && !(dge_k > 1.0f && dge_clip > 0.0f)) return FP4_ERR_ARG;
  if (!savedA->codes_t || !savedA->amax || !savedW->codes || !savedW->amax) return FP4_ERR_NULL;
  if (!aligned16(dY_bf16) || !aligned16(W_bf16) || !aligned16(dA) || !aligned16(dW)) return FP4_ERR_ALIGN;
  if (fp4_workspace_bytes(M, K, N) > ctx->workspace_bytes) return FP4_ERR_WORKSPACE;
  return linear_bwd_impl(ctx, static_cast<cudaStream_t>(stream), Arena(ctx->workspace, ctx->workspace_bytes), dY_bf16,
                         W_bf16, savedA, savedW, M, K, N, dge_on, dge_k, dge_clip, gemm_kind, dA, dW, out_f32, status);
}

}  // extern "C"

namespace {

int linear_bwd_impl(fp4_ctx* ctx, cudaStream_t st, Arena arena, const void* dY_bf16, const void* W_bf16,
                    const fp4_qtensor* savedA, const fp4_qtensor* savedW, int64_t M, int64_t K, int64_t N, int dge_on,
                    float dge_k, float dge_clip, int gemm_kind, void* dA, void* dW, int out_f32, int32_t* status) {
  const bool has_comp = dW && savedA->csc_colptr != nullptr;
  float* comp = has_comp ? arena.take<float>(size_t(K) * size_t(N)) : nullptr;   // compact: one row per non-empty column
  // dY as FP8 bytes instead of E2M1 nibbles: its format (0: E2M1)
  const int dy8 = (gemm_kind & FP4_BWD_DY_E5M2) ? FP4_FORMAT_E5M2 : ((gemm_kind & FP4_BWD_DY_E4M3) ? FP4_FORMAT_E4M3 : 0);
  gemm_kind &= ~(FP4_BWD_DY_E4M3 | FP4_BWD_DY_E5M2);
  const int a8 = savedA->format, w8 = savedW->format;                  // operand formats (0: E2M1)
  const float a_div = fp8_max(a8), w_div = fp8_max(w8);                // de-scale = amax / MAX of the operand's format
  const size_t g_bytes = size_t(M) * size_t(N) / (dy8 ? 1 : 2);
  uint8_t* g1_codes = dA ? arena.take<uint8_t>(g_bytes) : nullptr;      // dY (.) d_W, token-wise
  uint8_t* g2_codes = dW ? arena.take<uint8_t>(g_bytes) : nullptr;      // dY (.) d_A, channel-wise
  float* g1_amax = arena.take<float>(size_t(M));
  float* g2_amax = arena.take<float>(size_t(N));
  Arena comp_arena(arena.base + arena.off, comp_wgrad_scratch_bytes(M, K, N));
  arena.take<char>(comp_wgrad_scratch_bytes(M, K, N));
  int* slot_of_col = nullptr;
  if (!arena.ok) return FP4_ERR_WORKSPACE;
  Arena q_arena(arena.base + arena.off, arena.size - arena.off);
  int rc;

  // The weight-gradient chain runs on a side stream when both gradients are wanted.  Its first
  // part, the compensation dA^T dY of the non-empty residual columns, needs neither GEMM operand.
  cudaStream_t sw = st;
  if (dA && dW && ctx->overlap) {
    sw = ctx->side[0];
    FP4_CUDA_TRY(cudaEventRecord(ctx->ev[5], st));
    FP4_CUDA_TRY(cudaStreamWaitEvent(sw, ctx->ev[5], 0));
  }
  if (has_comp) {
    rc = launch_comp_wgrad(ctx, sw, savedA, dY_bf16, comp_arena, &slot_of_col, comp, M, K, N, status);
    if (rc != FP4_OK) return rc;
  }

  // dgrad operand: G' = dY (.) d_W[n], token-wise codes [M x N/2].
  // wgrad operand: G'' = dY (.) d_A[m], channel-wise codes transposed [N x M/2].
  if (dA && dW) {
    Arena a = q_arena;
    rc = launch_quantize_dual(ctx, st, a, dY_bf16, M, N, savedW->amax, savedA->amax, g1_codes, g1_amax, g2_codes,
                              g2_amax, status, dy8, w_div, a_div);
    if (rc != FP4_OK) return rc;
    if (sw != st) {
      FP4_CUDA_TRY(cudaEventRecord(ctx->ev[6], st));
      FP4_CUDA_TRY(cudaStreamWaitEvent(sw, ctx->ev[6], 0));
    }
  } else if (dA) {
    fp4_qtensor g = {};
    g.rows = M; g.cols = N; g.codes = g1_codes; g.amax = g1_amax; g.format = dy8;
    Arena a = q_arena;
    rc = launch_quantize(ctx, st, a, dY_bf16, M, N, /*scale_axis=*/0, 1.0, savedW->amax, w_div, &g, status);
    if (rc != FP4_OK) return rc;
  } else {
    fp4_qtensor g = {};
    g.rows = M; g.cols = N; g.codes_t = g2_codes; g.amax = g2_amax; g.format = dy8;
    Arena a = q_arena;
    rc = launch_quantize(ctx, st, a, dY_bf16, M, N, /*scale_axis=*/1, 1.0, savedA->amax, a_div, &g, status);
    if (rc != FP4_OK) return rc;
  }
  // dW[k,n] = store( (d_G''[n] * sum_m Aq[m,k] G''[m,n] + comp[k,n]) * Q'(W[k,n] * 6 / amax_W[n]) ):
  // the compensation rows and the DGE factor are applied in the GEMM's epilogue.
  GemmEpilogue epi = {};
  epi.addend = comp;
  epi.slot_of_row = slot_of_col;
  epi.w_bf16 = (dge_on && !w8) ? W_bf16 : nullptr;      // the DGE factor belongs to 4-bit weights
  epi.w_amax = savedW->amax;
  epi.dge_k = dge_k;
  epi.dge_clip = dge_clip;
  // dA = d_G'[m] * sum_n G'[m,n] Wq[k,n]
  Fp4GemmDesc wgrad = {savedA->codes_t, g2_codes, K, N, M, nullptr, g2_amax, dW, out_f32, &epi};
  wgrad.a_format = a8;
  wgrad.b_format = dy8;
  Fp4GemmDesc dgrad = {g1_codes, savedW->codes, M, K, N, g1_amax, nullptr, dA, out_f32, nullptr};
  dgrad.a_format = dy8;
  dgrad.b_format = w8;
  if (dA && dW) {
    // Both GEMMs in one launch on the caller's stream, the weight gradient's tiles first (their
    // epilogue is the longer one and then runs under the other GEMM's MMAs).
    if (sw != st) {
      FP4_CUDA_TRY(cudaEventRecord(ctx->ev[7], sw));
      FP4_CUDA_TRY(cudaStreamWaitEvent(st, ctx->ev[7], 0));
    }
    return launch_gemm_fp4_two(ctx, st, wgrad, dgrad, gemm_kind, status);
  }
  if (dW) {
    rc = launch_gemm_fp4(ctx, sw, wgrad.a_codes, wgrad.b_codes, K, N, M, nullptr, g2_amax, dW, out_f32, gemm_kind,
                         status, &epi, a8, dy8);
    if (rc != FP4_OK) return rc;
  }
  if (dA) {
    rc = launch_gemm_fp4(ctx, st, g1_codes, savedW->codes, M, K, N, g1_amax, nullptr, dA, out_f32, gemm_kind, status,
                         nullptr, dy8, w8);
    if (rc != FP4_OK) return rc;
  }
  if (sw != st) {
    FP4_CUDA_TRY(cudaEventRecord(ctx->ev[7], sw));
    FP4_CUDA_TRY(cudaStreamWaitEvent(st, ctx->ev[7], 0));
  }
  return FP4_OK;
}

// Buffers of one saved operand carved from the workspace (fp4_linear_step_host).
void carve_qtensor(Arena& a, fp4_qtensor* q, int64_t rows, int64_t cols, int scale_axis, int64_t cap) {
  *q = fp4_qtensor();
  q->rows = rows;
  q->cols = cols;
  q->codes = a.take<uint8_t>(size_t(rows) * size_t(cols) / 2);
  q->codes_t = a.take<uint8_t>(size_t(rows) * size_t(cols) / 2);
  q->amax = a.take<float>(size_t(scale_axis == 0 ? rows : cols));
  q->sparse_cap = cap;
  if (cap > 0) {
    q->thresholds = a.take<float>(2 * size_t(rows));      // room for thresholds per token (fp4_set_quantile_mode)
    q->nnz = a.take<int32_t>(1);
    q->csr_rowptr = a.take<int32_t>(size_t(rows) + 1);
    q->csr_col = a.take<int32_t>(size_t(cap));
    q->csr_val = a.take<float>(size_t(cap));
    q->csc_colptr = a.take<int32_t>(size_t(cols) + 1);
    q->csc_row = a.take<int32_t>(size_t(cap));
    q->csc_val = a.take<float>(size_t(cap));
  }
}

// Residual entries a step may produce under either form of the clamp: 2 n_tail of the tensor, or
// two tails of round((1 - alpha) K) entries in every row (thresholds per token).
int64_t step_capacity(int64_t M, int64_t K, double alpha) {
  if (!(alpha < 1.0)) return 0;
  const int64_t whole = 2 * llround((1.0 - alpha) * double(M * K));
  const int64_t per_token = 2 * M * llround((1.0 - alpha) * double(K));
  return whole > per_token ? whole : per_token;
}

// fp4_linear_step_host: bytes of one set of device inputs (the outputs have the same three sizes),
// and of everything else it carves.
size_t step_host_io_bytes(int64_t M, int64_t K, int64_t N) {
  return round256(size_t(M) * K * 2) + round256(size_t(K) * N * 2) + round256(size_t(M) * N * 2);
}
size_t step_host_shared_bytes(int64_t M, int64_t K, int64_t N, double alpha) {
  const size_t cap = size_t(step_capacity(M, K, alpha));
  size_t b = 2 * round256(size_t(M) * K / 2) + 2 * round256(size_t(K) * N / 2);                          // codes
  b += round256(size_t(M) * 4) + round256(size_t(N) * 4);                                                // amax
  b += 4 * round256(cap * 4) + round256((size_t(M) + 1) * 4) + round256((size_t(K) + 1) * 4) + 3 * 256;   // sparse
  b += round256(2 * size_t(M) * 4);                                                                      // thresholds
  b += 256;                                                                                              // status
  return b + fp4_workspace_bytes(M, K, N);
}

}  // namespace

extern "C" {

size_t fp4_step_host_workspace_bytes(int64_t M, int64_t K, int64_t N, double alpha) {
  if (M <= 0 || K <= 0 || N <= 0) return 0;
  // Sized so that the pipelined layout fits: 2 HOST_STEP_SETS slots (input sets, then output sets)
  // in the first half, everything else in the second half.
  const size_t io = step_host_io_bytes(M, K, N), shared = step_host_shared_bytes(M, K, N, alpha);
  const size_t slots = 4 * HOST_STEP_SETS * io;
  return (slots > 2 * shared ? slots : 2 * shared) + 1024;
}

int fp4_linear_step_host(fp4_ctx* ctx, void* stream, const void* A_host, const void* W_host, const void* dY_host,
                         int64_t M, int64_t K, int64_t N, double alpha, int dge_on, float dge_k, float dge_clip,
                         int gemm_kind, void* Y_host, void* dA_host, void* dW_host, int32_t* status_host) {
  if (!ctx || !A_host || !W_host || !dY_host || !Y_host || !dA_host || !dW_host) return FP4_ERR_NULL;
  if (!mult128(M) || !mult128(K) || !mult128(N)) return FP4_ERR_SHAPE;
  if (M * K >= (int64_t(1) << 31) || K * N >= (int64_t(1) << 31) || M * N >= (int64_t(1) << 31)) return FP4_ERR_SHAPE;
  if (!(alpha > 0.5 && alpha <= 1.0)) return FP4_ERR_ALPHA;
  if (gemm_kind != FP4_GEMM_MXF4 && gemm_kind != FP4_GEMM_F8F6F4) return FP4_ERR_ARG;
  if (dge_on && !(dge_k > 1.0f && dge_clip > 0.0f)) return FP4_ERR_ARG;
  if (alpha < 1.0 && step_capacity(M, K, alpha) >= M * K) return FP4_ERR_ALPHA;
  const size_t io_bytes = step_host_io_bytes(M, K, N), shared_bytes = step_host_shared_bytes(M, K, N, alpha);
  if (2 * io_bytes + shared_bytes > ctx->workspace_bytes) return FP4_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  // Workspace layout.  Pipelined: 2 HOST_STEP_SETS slots in the first half of the workspace -- the
  // input sets, then the output sets -- and everything else (saved operands, scratch) in the second
  // half.  Call i uses set i % HOST_STEP_SETS: its inputs travel on the context's copy stream while call i - 1 still
  // computes, its kernels run on the context's compute stream while call i - 1 copies back on the
  // context's return stream, and `stream` waits for the copies back.  A call whose tensors do not
  // fit that layout carves the whole workspace from its start, runs on `stream` alone and is
  // ordered after everything earlier calls left in flight.
  constexpr int SETS = HOST_STEP_SETS;
  const size_t slot = (ctx->workspace_bytes / (4 * SETS)) & ~size_t(255);
  const bool pipelined = ctx->overlap && io_bytes <= slot && shared_bytes <= ctx->workspace_bytes - 2 * SETS * slot;
  const int set = ctx->host_step_parity;
  Arena in_arena = pipelined ? Arena(ctx->workspace + size_t(set) * slot, slot) : Arena(ctx->workspace, io_bytes);
  Arena out_arena = pipelined ? Arena(ctx->workspace + size_t(SETS + set) * slot, slot)
                              : Arena(ctx->workspace + io_bytes, io_bytes);
  Arena arena = pipelined ? Arena(ctx->workspace + 2 * SETS * slot, ctx->workspace_bytes - 2 * SETS * slot)
                          : Arena(ctx->workspace + 2 * io_bytes, ctx->workspace_bytes - 2 * io_bytes);
  const size_t a_bytes = size_t(M) * K * 2, w_bytes = size_t(K) * N * 2, y_bytes = size_t(M) * N * 2;
  char* dA_in = in_arena.take<char>(a_bytes);
  char* dW_in = in_arena.take<char>(w_bytes);
  char* dG_in = in_arena.take<char>(y_bytes);
  char* dY_out = out_arena.take<char>(y_bytes);
  char* dA_out = out_arena.take<char>(a_bytes);
  char* dW_out = out_arena.take<char>(w_bytes);
  int32_t* status = arena.take<int32_t>(1);
  fp4_qtensor qa, qw;
  carve_qtensor(arena, &qa, M, K, 0, step_capacity(M, K, alpha));
  carve_qtensor(arena, &qw, K, N, 1, 0);
  if (!arena.ok || !in_arena.ok || !out_arena.ok) return FP4_ERR_WORKSPACE;
  Arena rest(arena.base + arena.off, arena.size - arena.off);

  cudaStream_t s_in = st, s_cmp = st, s_out = st;      // copies in, kernels, copies back
  if (pipelined) {
    s_in = ctx->copy_stream;
    s_cmp = ctx->compute_stream;
    s_out = ctx->return_stream;
    // The copies in do not wait for `stream`: it carries the previous call's copies back, which
    // they are meant to overlap.  The host inputs must therefore be ready when the call is made.
    // Both slots of this set were last used HOST_STEP_SETS calls ago: that call's kernels have
    // to be done with the input slot before the copies in start, its copies back with the output
    // slot before this call's kernels start -- the copies in do not wait for those copies back, so
    // the two copy directions both stay busy.
    FP4_CUDA_TRY(cudaStreamWaitEvent(s_in, ctx->host_step_computed[set], 0));
    FP4_CUDA_TRY(cudaStreamWaitEvent(s_cmp, ctx->host_step_done[set], 0));
  } else {
    for (int i = 0; i < SETS; ++i) FP4_CUDA_TRY(cudaStreamWaitEvent(st, ctx->host_step_done[i], 0));
  }
  FP4_CUDA_TRY(cudaMemcpyAsync(dA_in, A_host, a_bytes, cudaMemcpyHostToDevice, s_in));
  FP4_CUDA_TRY(cudaMemcpyAsync(dW_in, W_host, w_bytes, cudaMemcpyHostToDevice, s_in));
  FP4_CUDA_TRY(cudaMemcpyAsync(dG_in, dY_host, y_bytes, cudaMemcpyHostToDevice, s_in));
  if (pipelined) {
    FP4_CUDA_TRY(cudaEventRecord(ctx->host_step_copied[set], s_in));
    FP4_CUDA_TRY(cudaStreamWaitEvent(s_cmp, ctx->host_step_copied[set], 0));
  }
  FP4_CUDA_TRY(cudaMemsetAsync(status, 0, 4, s_cmp));
  int rc = linear_fwd_impl(ctx, s_cmp, rest, dA_in, dW_in, M, K, N, alpha, 0, gemm_kind, dY_out, 0, &qa, &qw, status);
  if (rc != FP4_OK) return rc;
  rc = linear_bwd_impl(ctx, s_cmp, rest, dG_in, dW_in, &qa, &qw, M, K, N, dge_on, dge_k, dge_clip, gemm_kind, dA_out,
                       dW_out, 0, status);
  if (rc != FP4_OK) return rc;
  if (pipelined) {
    FP4_CUDA_TRY(cudaEventRecord(ctx->host_step_computed[set], s_cmp));
    FP4_CUDA_TRY(cudaStreamWaitEvent(s_out, ctx->host_step_computed[set], 0));
  }
  FP4_CUDA_TRY(cudaMemcpyAsync(Y_host, dY_out, y_bytes, cudaMemcpyDeviceToHost, s_out));
  FP4_CUDA_TRY(cudaMemcpyAsync(dA_host, dA_out, a_bytes, cudaMemcpyDeviceToHost, s_out));
  FP4_CUDA_TRY(cudaMemcpyAsync(dW_host, dW_out, w_bytes, cudaMemcpyDeviceToHost, s_out));
  if (status_host) FP4_CUDA_TRY(cudaMemcpyAsync(status_host, status, 4, cudaMemcpyDeviceToHost, s_out));
  if (pipelined) {
    FP4_CUDA_TRY(cudaEventRecord(ctx->host_step_done[set], s_out));
    FP4_CUDA_TRY(cudaStreamWaitEvent(st, ctx->host_step_done[set], 0));
    ctx->host_step_parity = (set + 1) % SETS;
  } else {
    // later pipelined calls may use either set only after this call has left the workspace
    for (int i = 0; i < SETS; ++i) {
      FP4_CUDA_TRY(cudaEventRecord(ctx->host_step_done[i], st));
      FP4_CUDA_TRY(cudaEventRecord(ctx->host_step_computed[i], st));
    }
  }
  if (status_host) FP4_CUDA_TRY(cudaStreamSynchronize(st));
  return FP4_OK;
}

int fp4_set_overlap(fp4_ctx* ctx, int on) {
  if (!ctx) return FP4_ERR_NULL;
  ctx->overlap = on ? 1 : 0;
  return FP4_OK;
}

int fp4_set_quantile_mode(fp4_ctx* ctx, int mode) {
  if (!ctx) return FP4_ERR_NULL;
  if (mode != FP4_QUANTILE_SIGNED && mode != FP4_QUANTILE_ABS && mode != FP4_QUANTILE_TOKEN) return FP4_ERR_ARG;
  ctx->quantile_mode = mode;
  return FP4_OK;
}

int fp4_debug_set(fp4_ctx* ctx, int key, int64_t value) {
  if (!ctx) return FP4_ERR_NULL;
  if (key == FP4_DEBUG_WAIT_LIMIT_US) {
    if (value < 0 || value > 10000000) return FP4_ERR_ARG;
    ctx->debug_wait_limit_ns = uint64_t(value) * 1000u;
  } else if (key == FP4_DEBUG_SKIP_FILL) {
    if (value < -1 || value > (1 << 30)) return FP4_ERR_ARG;
    ctx->debug_skip_fill = int(value);
  } else {
    return FP4_ERR_ARG;
  }
  return FP4_OK;
}

int64_t fp4_sparse_capacity(int64_t rows, int64_t cols, double alpha, int quantile_mode) {
  if (rows <= 0 || cols <= 0 || !(alpha > 0.5 && alpha <= 1.0)) return -1;
  if (quantile_mode != FP4_QUANTILE_SIGNED && quantile_mode != FP4_QUANTILE_ABS && quantile_mode != FP4_QUANTILE_TOKEN)
    return -1;
  if (!(alpha < 1.0)) return 0;
  if (quantile_mode == FP4_QUANTILE_TOKEN) return 2 * rows * llround((1.0 - alpha) * double(cols));
  return 2 * llround((1.0 - alpha) * double(rows * cols));
}

int fp4_profile_enable(fp4_ctx* ctx, int on) {
  if (!ctx) return FP4_ERR_NULL;
  ctx->profile = on ? 1 : 0;
  return FP4_OK;
}

int fp4_profile_reset(fp4_ctx* ctx) {
  if (!ctx) return FP4_ERR_NULL;
  for (ProfRecord& r : *ctx->records) {
    cudaEventDestroy(r.start);
    cudaEventDestroy(r.stop);
  }
  ctx->records->clear();
  ctx->launch_count = 0;
  return FP4_OK;
}

int fp4_profile_read(fp4_ctx* ctx, int kernel_class, double* total_ms, int64_t* launches) {
  if (!ctx || !total_ms || !launches) return FP4_ERR_NULL;
  if (kernel_class < 0 || kernel_class >= FP4_KC_COUNT) return FP4_ERR_ARG;
  double ms = 0.0;
  int64_t n = 0;
  for (ProfRecord& r : *ctx->records) {
    if (r.kc != kernel_class) continue;
    FP4_CUDA_TRY(cudaEventSynchronize(r.stop));
    float t = 0.f;
    FP4_CUDA_TRY(cudaEventElapsedTime(&t, r.start, r.stop));
    ms += t;
    n += r.launches;
  }
  *total_ms = ms;
  *launches = n;
  return FP4_OK;
}

int64_t fp4_launch_count(fp4_ctx* ctx) { return ctx ? ctx->launch_count : -1; }

}  // extern "C"
