// C ABI of the library: argument validation, workspace carving and kernel sequencing.
// Every step of the path runs in the kernels of this directory; nothing here computes.
#include <cuda.h>

#include <cmath>
#include <new>

#include "common.cuh"

namespace {

bool mult128(int64_t v) { return v > 0 && (v % 128) == 0; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

size_t round256(size_t b) { return (b + 255) & ~size_t(255); }

// Bytes the backward needs on top of the quantiser scratch: both quantised copies of dY and
// the fp32 GEMM result that the compensation / DGE epilogue kernel consumes.
size_t linear_scratch_bytes(int64_t M, int64_t K, int64_t N) {
  size_t b = 0;
  const size_t big = size_t(M > K ? M : K) * size_t(N);
  b += round256(big * sizeof(float));                 // fp32 GEMM result (fwd: M x N, wgrad: K x N)
  b += 2 * round256(size_t(M) * size_t(N) / 2);       // dY codes, both scalings
  b += round256(size_t(M) * 4) + round256(size_t(N) * 4);   // their amax vectors
  b += 2 * round256(size_t(M > N ? M : N) * 4);       // de-scale vectors used as prescale
  return b;
}

int check_qtensor_dense(const fp4_qtensor* q) {
  if (!q || !q->amax) return FP4_ERR_NULL;
  if (!q->codes && !q->codes_t) return FP4_ERR_NULL;
  return FP4_OK;
}

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
    case FP4_ERR_CAPACITY: return "sparse_cap is below 2 * n_tail";
    default: return "unknown status";
  }
}

size_t fp4_workspace_bytes(int64_t M, int64_t K, int64_t N) {
  if (M <= 0 || K <= 0 || N <= 0) return 0;
  size_t q = quantize_scratch_bytes(M, K);
  const size_t qw = quantize_scratch_bytes(K, N);
  const size_t qg = quantize_scratch_bytes(M, N);
  if (qw > q) q = qw;
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
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return FP4_ERR_CUDA; }
  ctx->num_sms = prop.multiProcessorCount;
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    delete ctx;
    return FP4_ERR_CUDA;
  }
  ctx->encode_tiled = fn;
  if (workspace_bytes) {
    if (cudaMalloc(reinterpret_cast<void**>(&ctx->workspace), workspace_bytes) != cudaSuccess) {
      delete ctx;
      return FP4_ERR_CUDA;
    }
    ctx->workspace_bytes = workspace_bytes;
  }
  *out = ctx;
  return FP4_OK;
}

int fp4_destroy(fp4_ctx* ctx) {
  if (!ctx) return FP4_ERR_NULL;
  cudaSetDevice(ctx->device);
  if (ctx->workspace) cudaFree(ctx->workspace);
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
  if (!aligned16(x_bf16) || !aligned16(out->codes) || !aligned16(out->codes_t) || !aligned16(out->amax))
    return FP4_ERR_ALIGN;
  if (alpha < 1.0) {
    if (scale_axis != 0 || prescale) return FP4_ERR_ARG;
    const int64_t n = rows * cols;
    const int64_t n_tail = llround((1.0 - alpha) * double(n));
    if (2 * n_tail >= n) return FP4_ERR_ALPHA;
    rc = check_qtensor_sparse(out, n_tail);
    if (rc != FP4_OK) return rc;
  }
  if (quantize_scratch_bytes(rows, cols) > ctx->workspace_bytes) return FP4_ERR_WORKSPACE;
  Arena arena(ctx->workspace, ctx->workspace_bytes);
  out->rows = rows;
  out->cols = cols;
  return launch_quantize(ctx, static_cast<cudaStream_t>(stream), arena, x_bf16, rows, cols, scale_axis, alpha,
                         prescale, 0, out, status);
}

int fp4_gemm(fp4_ctx* ctx, void* stream, const uint8_t* a_codes, const uint8_t* b_codes, int64_t I, int64_t J,
             int64_t C, const float* row_amax, const float* col_amax, void* out, int out_f32, int gemm_kind,
             int32_t* status) {
  if (!ctx || !a_codes || !b_codes || !out || !status) return FP4_ERR_NULL;
  if (!mult128(I) || !mult128(J) || !mult128(C)) return FP4_ERR_SHAPE;
  if (!aligned16(out)) return FP4_ERR_ALIGN;
  return launch_gemm_fp4(ctx, static_cast<cudaStream_t>(stream), a_codes, b_codes, I, J, C, row_amax, col_amax, out,
                         out_f32, gemm_kind, status);
}

int fp4_linear_fwd(fp4_ctx* ctx, void* stream, const void* A_bf16, const void* W_bf16, int64_t M, int64_t K,
                   int64_t N, double alpha, int reuse_w, int gemm_kind, void* Y, int out_f32, fp4_qtensor* savedA,
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
  if (occ) {
    const int64_t n_tail = llround((1.0 - alpha) * double(M * K));
    if (2 * n_tail >= M * K) return FP4_ERR_ALPHA;
    int rc = check_qtensor_sparse(savedA, n_tail);
    if (rc != FP4_OK) return rc;
  }
  if (fp4_workspace_bytes(M, K, N) > ctx->workspace_bytes) return FP4_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  Arena arena(ctx->workspace, ctx->workspace_bytes);
  float* y1 = occ ? arena.take<float>(size_t(M) * size_t(N)) : nullptr;
  if (!arena.ok) return FP4_ERR_WORKSPACE;
  Arena qa_arena(ctx->workspace + arena.off, ctx->workspace_bytes - arena.off);

  int rc;
  if (!reuse_w) {
    Arena a = qa_arena;
    savedW->rows = K;
    savedW->cols = N;
    rc = launch_quantize(ctx, st, a, W_bf16, K, N, /*scale_axis=*/1, 1.0, nullptr, 0, savedW, status);
    if (rc != FP4_OK) return rc;
  }
  {
    Arena a = qa_arena;
    savedA->rows = M;
    savedA->cols = K;
    rc = launch_quantize(ctx, st, a, A_bf16, M, K, /*scale_axis=*/0, alpha, nullptr, 0, savedA, status);
    if (rc != FP4_OK) return rc;
  }
  // Y1 = (Q(A_c) Q(W)) * d_A[m] * d_W[n]: A codes [M x K/2], W codes transposed [N x K/2].
  if (!occ) {
    return launch_gemm_fp4(ctx, st, savedA->codes, savedW->codes_t, M, N, K, savedA->amax, savedW->amax, Y, out_f32,
                           gemm_kind, status);
  }
  rc = launch_gemm_fp4(ctx, st, savedA->codes, savedW->codes_t, M, N, K, savedA->amax, savedW->amax, y1, 1, gemm_kind,
                       status);
  if (rc != FP4_OK) return rc;
  // Y = store(Y1 + (A - A_c) W): one rounding of the fp32 sum.
  return launch_comp_fwd(ctx, st, y1, savedA->csr_rowptr, savedA->csr_col, savedA->csr_val, W_bf16, M, K, N, Y,
                         out_f32);
}

int fp4_linear_bwd(fp4_ctx* ctx, void* stream, const void* dY_bf16, const void* W_bf16, const fp4_qtensor* savedA,
                   const fp4_qtensor* savedW, int64_t M, int64_t K, int64_t N, int dge_on, float dge_k,
                   float dge_clip, int gemm_kind, void* dA, void* dW, int out_f32, int32_t* status) {
  if (!ctx || !dY_bf16 || !W_bf16 || !savedA || !savedW || !status) return FP4_ERR_NULL;
  if (!dA && !dW) return FP4_ERR_NULL;
  if (!mult128(M) || !mult128(K) || !mult128(N)) return FP4_ERR_SHAPE;
  if (M * K >= (int64_t(1) << 31) || K * N >= (int64_t(1) << 31) || M * N >= (int64_t(1) << 31)) return FP4_ERR_SHAPE;
  if (gemm_kind != FP4_GEMM_MXF4 && gemm_kind != FP4_GEMM_F8F6F4) return FP4_ERR_ARG;
  if (dge_on && !(dge_k > 1.0f && dge_clip > 0.0f)) return FP4_ERR_ARG;
  if (!savedA->codes_t || !savedA->amax || !savedW->codes || !savedW->amax) return FP4_ERR_NULL;
  if (!aligned16(dY_bf16) || !aligned16(W_bf16) || !aligned16(dA) || !aligned16(dW)) return FP4_ERR_ALIGN;
  if (fp4_workspace_bytes(M, K, N) > ctx->workspace_bytes) return FP4_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  Arena arena(ctx->workspace, ctx->workspace_bytes);
  float* s = arena.take<float>(size_t(K) * size_t(N));
  uint8_t* g_codes = arena.take<uint8_t>(size_t(M) * size_t(N) / 2);
  float* g_amax = arena.take<float>(size_t(M > N ? M : N));
  if (!arena.ok) return FP4_ERR_WORKSPACE;
  Arena q_arena(ctx->workspace + arena.off, ctx->workspace_bytes - arena.off);
  int rc;

  if (dA) {
    // dgrad: G' = dY (.) d_W[n], token-wise codes [M x N/2]; dA = d_G'[m] * sum_n G'[m,n] Wq[k,n].
    fp4_qtensor g = {};
    g.rows = M; g.cols = N; g.codes = g_codes; g.amax = g_amax;
    Arena a = q_arena;
    rc = launch_quantize(ctx, st, a, dY_bf16, M, N, /*scale_axis=*/0, 1.0, savedW->amax, 1, &g, status);
    if (rc != FP4_OK) return rc;
    rc = launch_gemm_fp4(ctx, st, g_codes, savedW->codes, M, K, N, g_amax, nullptr, dA, out_f32, gemm_kind, status);
    if (rc != FP4_OK) return rc;
  }
  if (dW) {
    // wgrad: G'' = dY (.) d_A[m], channel-wise codes transposed [N x M/2];
    // S[k,n] = d_G''[n] * sum_m Aq[m,k] G''[m,n], then the compensation and the DGE factor.
    fp4_qtensor g = {};
    g.rows = M; g.cols = N; g.codes_t = g_codes; g.amax = g_amax;
    Arena a = q_arena;
    rc = launch_quantize(ctx, st, a, dY_bf16, M, N, /*scale_axis=*/1, 1.0, savedA->amax, 1, &g, status);
    if (rc != FP4_OK) return rc;
    rc = launch_gemm_fp4(ctx, st, savedA->codes_t, g_codes, K, N, M, nullptr, g_amax, s, 1, gemm_kind, status);
    if (rc != FP4_OK) return rc;
    rc = launch_comp_wgrad_dge(ctx, st, s, savedA->csc_colptr, savedA->csc_row, savedA->csc_val, dY_bf16, W_bf16,
                               savedW->amax, M, K, N, dge_on, dge_k, dge_clip, dW, out_f32);
    if (rc != FP4_OK) return rc;
  }
  return FP4_OK;
}

}  // extern "C"
