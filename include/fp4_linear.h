/*
 * fp4_linear.h -- C ABI of the FP4-quantized linear layer for NVIDIA B200 (sm_100a).
 *
 * The library implements the linear-layer hot path of "Optimizing Large Language Model
 * Training Using FP4 Quantization": vector-wise absmax quantisation to E2M1 (Eq. 1 with the
 * look-up quantiser of Appendix A), outlier clamping at a quantile with a sparse residual
 * (Section 3.2), the FP4 GEMM with the two de-scales applied to its result (Fig. 2,
 * Appendix C.2), the compensation product, and the backward pass with the differentiable
 * gradient estimator (Eq. 6-8).
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 *  - Every tensor pointer is a DEVICE pointer unless the parameter is documented as host.
 *    Tensors are dense, row-major and 16-byte aligned.  The caller owns every tensor; the
 *    context owns only its workspace.  Nothing is allocated after fp4_create() (outside profiling
 *    mode, fp4_profile_enable, which creates a pair of CUDA events per kernel class and call).
 *  - Notation: A[M x K] activations, W[K x N] weights (input channels x output channels),
 *    Y[M x N] = A W.  M, K and N must be multiples of 128.
 *  - E2M1 codes are sign-magnitude nibbles (bit 3 sign; 0..7 -> 0, .5, 1, 1.5, 2, 3, 4, 6),
 *    two per byte with the even element in bits 3:0.  A negative zero code is never written.
 *  - Calls are asynchronous on `stream` (a cudaStream_t passed as void*).  They return 0 or
 *    a negative FP4_ERR_* code for errors found on the host before anything is enqueued.
 *  - A context holds one workspace and a few counters that its calls share: the work of two calls
 *    on the same context must not overlap on the GPU (issue them on one stream, or order the
 *    streams); use one context per concurrent stream.
 *  - Conditions found on the device are OR-ed into the caller's device word `*status`
 *    (FP4_DEV_* bits).  When a bit is set the outputs are unspecified but every write stayed
 *    inside the caller's buffers.  Every device-side wait is bounded: a stalled pipeline
 *    sets FP4_DEV_TIMEOUT and the kernel returns.
 */
#ifndef FP4_LINEAR_H_
#define FP4_LINEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* host-side return codes */
#define FP4_OK              0
#define FP4_ERR_NULL       (-1)   /* a required pointer is NULL                              */
#define FP4_ERR_SHAPE      (-2)   /* a dimension is not a positive multiple of 128           */
#define FP4_ERR_ALPHA      (-3)   /* alpha outside (0.5, 1]                                  */
#define FP4_ERR_ALIGN      (-4)   /* a tensor pointer is not 16-byte aligned                 */
#define FP4_ERR_WORKSPACE  (-5)   /* the context's workspace is too small for this call      */
#define FP4_ERR_CUDA       (-6)   /* a CUDA runtime / driver call failed                     */
#define FP4_ERR_ARG        (-7)   /* an argument has an unsupported value                    */
#define FP4_ERR_CAPACITY   (-8)   /* sparse_cap is below fp4_sparse_capacity()               */
#define FP4_ERR_STATIC_LIMIT (-9) /* input larger than the fixed scratch of a *_static call  */

/* bits of the device status word (bit 0 is not used: the residual cannot outgrow a capacity the
 * host has accepted, see fp4_sparse_capacity) */
#define FP4_DEV_NONFINITE        2   /* an input holds an infinity or a NaN: outputs unspecified */
#define FP4_DEV_TIMEOUT          4   /* a bounded wait inside a kernel ran out               */

/* fp4_qtensor.format: how a quantised operand is stored */
#define FP4_FORMAT_E2M1  0
#define FP4_FORMAT_E4M3  1
#define FP4_FORMAT_E5M2  2

/* gemm_kind: which tcgen05.mma flavour multiplies the codes */
#define FP4_GEMM_MXF4    0   /* packed nibbles, K = 64 per instruction, unit block scales    */
#define FP4_GEMM_F8F6F4  1   /* nibbles in byte containers, K = 32 per instruction           */
/* fp4_gemm only: the byte-container kind with E4M3 bytes as one or both operands */
#define FP4_GEMM_F8F6F4_A8    2   /* a_codes are E4M3 bytes [I x C], b_codes E2M1 nibbles  */
#define FP4_GEMM_F8F6F4_B8    3   /* a_codes E2M1 nibbles, b_codes E4M3 bytes [J x C]      */
#define FP4_GEMM_F8F6F4_A8B8  4   /* both operands E4M3 bytes                              */
/* OR-ed into one of the three kinds above: that operand's bytes are E5M2 instead of E4M3 */
#define FP4_GEMM_A_E5M2       0x10
#define FP4_GEMM_B_E5M2       0x20
/* fp4_linear_bwd only, OR-ed into gemm_kind (FP4_GEMM_F8F6F4): dY is quantised to E4M3 or to
 * E5M2 bytes (one of the two) */
#define FP4_BWD_DY_E4M3       0x100
#define FP4_BWD_DY_E5M2       0x200

typedef struct fp4_ctx fp4_ctx;   /* opaque: device id, SM count, workspace */

/* One quantised operand.  Every buffer is allocated by the caller; pointers that are not
 * needed may be NULL (then that output is skipped).                                        */
typedef struct fp4_qtensor {
  int64_t  rows, cols;     /* logical shape of the source tensor                              */
  uint8_t* codes;          /* [rows x cols/2]  (r, 2j) low nibble, (r, 2j+1) high nibble      */
  uint8_t* codes_t;        /* [cols x rows/2]  (2i, c) low nibble, (2i+1, c) high nibble      */
  float*   amax;           /* [rows] if scale_axis == 0 else [cols]: exact max |x| of each
                              vector (after the clamp and the optional prescale); the scale
                              of Eq. 1 is gamma = 6 / amax and the de-scale amax / 6, each
                              rounded once to float                                           */
  float*   thresholds;     /* [2] = {lo, hi}: the (1-alpha)- and alpha-quantile (OCC only);
                              [2 * rows] under FP4_QUANTILE_TOKEN (fp4_set_quantile_mode)     */
  int32_t* csr_rowptr;     /* [rows + 1]                                                      */
  int32_t* csr_col;        /* [sparse_cap] column index, ascending within a row               */
  float*   csr_val;        /* [sparse_cap] x - clamp(x)                                       */
  int32_t* csc_colptr;     /* [cols + 1]                                                      */
  int32_t* csc_row;        /* [sparse_cap] row index, ascending within a column               */
  float*   csc_val;        /* [sparse_cap]                                                    */
  int64_t  sparse_cap;     /* capacity in entries: at least fp4_sparse_capacity(rows, cols, alpha,
                              mode), i.e. 2 * round((1-alpha) * rows * cols) for the paper's clamp */
  int32_t* nnz;            /* [1] number of residual entries                                  */
  int32_t  format;         /* set by the caller: FP4_FORMAT_E2M1 (0, as described above) or
                              FP4_FORMAT_E4M3: OCP E4M3 bytes, one per element (codes
                              [rows x cols], codes_t [cols x rows]), MAX = 448 in place of 6,
                              nearest-even rounding with saturation, no clamping: the FP8
                              operand of the W4A8 / W8A4 settings of Section 4.3; or
                              FP4_FORMAT_E5M2: OCP E5M2 bytes in the same layouts, MAX = 57344,
                              saturation to the largest finite value (never an infinity)    */
  int32_t  reserved;       /* 0                                                               */
} fp4_qtensor;

/* Create a context on `device` with a workspace of `workspace_bytes` (cudaMalloc'ed here,
 * freed by fp4_destroy).  fp4_workspace_bytes() gives a sufficient size.  `out` is host.   */
int fp4_create(fp4_ctx** out, int device, size_t workspace_bytes);
int fp4_destroy(fp4_ctx* ctx);

/* Workspace that fp4_quantize / fp4_linear_fwd / fp4_linear_bwd need for these sizes.      */
size_t fp4_workspace_bytes(int64_t M, int64_t K, int64_t N);

/* Residual entries that clamping at `alpha` can produce at most (Section 3.2: two tails of
 * n_tail = llround((1 - alpha) * rows * cols) entries; with FP4_QUANTILE_TOKEN two tails of
 * llround((1 - alpha) * cols) entries in every row): the least `sparse_cap` the calls accept.
 * 0 for alpha == 1; -1 for arguments outside their range.  `quantile_mode` is one of the
 * FP4_QUANTILE_* values below.                                                              */
int64_t fp4_sparse_capacity(int64_t rows, int64_t cols, double alpha, int quantile_mode);

/* Text of a host return code (static string).                                              */
const char* fp4_status_string(int code);

/*
 * fp4_quantize -- vector-wise absmax quantisation to E2M1 (Eq. 1; quantiser Q: Appendix A;
 * granularity: Section 4.1), optionally preceded by outlier clamping with the sparse
 * residual emitted alongside (Section 3.2).
 *
 *   x_bf16      [rows x cols] BF16
 *   scale_axis  0: one scale per row (token-wise, activations)
 *               1: one scale per column (channel-wise, weights W[c_i x c_o])
 *   alpha       1.0: no clamp.  Otherwise 0.5 < alpha < 1: with n = rows*cols and
 *               n_tail = llround((1-alpha)*n), lo and hi are the order statistics
 *               sorted[n_tail] and sorted[n-1-n_tail] of the whole tensor; x is clamped to
 *               [lo, hi] BEFORE the absmax, and every x outside [lo, hi] yields a residual
 *               entry x - clamp(x).  Requires scale_axis == 0 and prescale == NULL.
 *   prescale    optional float vector along the OTHER axis ([cols] for scale_axis 0,
 *               [rows] for scale_axis 1): x is replaced by float(x * prescale) first.
 *   out         destination buffers (host struct of device pointers); amax is required,
 *               at least one of codes / codes_t is required; with alpha < 1 thresholds,
 *               nnz, csr_* and csc_* are required.
 * Scaled value: v = float(x) * gamma with one float rounding; code = Q(v), where a value
 * equal to a threshold of the chain goes to the larger neighbour.  A zero vector gets
 * amax = 0 and all-zero codes.
 */
int fp4_quantize(fp4_ctx* ctx, void* stream, const void* x_bf16, int64_t rows, int64_t cols,
                 int scale_axis, double alpha, const float* prescale,
                 fp4_qtensor* out, int32_t* status);

/*
 * fp4_gemm -- the FP4 GEMM of Fig. 2 on E2M1 codes with the two de-scales applied to the
 * result (Appendix C.2: the GEMM consumes the scaled quantised tensors, the de-scale comes
 * afterwards):
 *     out[i, j] = (acc[i, j] * d_row[i]) * d_col[j],
 *     acc[i, j] = sum_c val(a_codes[i, c]) * val(b_codes[j, c])   (fp32 accumulation),
 *     d = amax / 6 rounded to float; a NULL amax vector means d = 1.
 *   a_codes [I x C/2], b_codes [J x C/2]: both operands have the contraction contiguous.
 *   out     [I x J], float if out_f32 != 0 else BF16.
 *   I, J, C multiples of 128.  gemm_kind: FP4_GEMM_MXF4 or FP4_GEMM_F8F6F4.
 * With FP4_GEMM_F8F6F4_A8 / _B8 / _A8B8 the named operands are OCP E4M3 bytes, one per element
 * ([rows x C]), with d = amax / 448 (the mixed-precision settings W4A8 / W8A4 of Section 4.3);
 * the accumulation is then fp32 without the exactness E2M1 products have.  FP4_GEMM_A_E5M2 /
 * FP4_GEMM_B_E5M2 OR-ed in make the named 8-bit operand OCP E5M2 (d = amax / 57344).
 */
int fp4_gemm(fp4_ctx* ctx, void* stream, const uint8_t* a_codes, const uint8_t* b_codes,
             int64_t I, int64_t J, int64_t C, const float* row_amax, const float* col_amax,
             void* out, int out_f32, int gemm_kind, int32_t* status);

/*
 * fp4_linear_fwd -- forward of the FP4 linear layer (Fig. 2, Section 3.2):
 *     Y = bf16( (Q(A_c) Q(W)) (.) d_A[m] (.) d_W[n]  +  (A - A_c) W )
 * A is clamped at the alpha-quantiles and quantised token-wise, W channel-wise; the residual
 * A - A_c multiplies the BF16 weight in fp32; both branches meet in fp32 and are rounded once.
 *   A_bf16 [M x K], W_bf16 [K x N], Y [M x N] (BF16, or float if out_f32 != 0).
 *   savedA->format / savedW->format = FP4_FORMAT_E4M3 (or FP4_FORMAT_E5M2) give the W4A8 / W8A4
 *   settings of Section 4.3 (gemm_kind must then be FP4_GEMM_F8F6F4; an 8-bit activation is not
 *   clamped: alpha must be 1).
 *   savedA, savedW: caller-allocated fp4_qtensor buffers that receive the quantised operands
 *   and are handed to fp4_linear_bwd.  savedA needs codes, codes_t, amax, thresholds, nnz,
 *   csr_*, csc_*; savedW needs codes, codes_t, amax.
 *   `reuse` is a bit mask: FP4_REUSE_W -- savedW already holds this weight's codes (weights
 *   change once per optimizer step) and is not recomputed; FP4_REUSE_A -- savedA already holds
 *   this activation quantised with the same alpha (the q/k/v projections of a layer, or its
 *   gate/up projections, read the same activation) and is not recomputed.
 *   With a heavy residual (savedA->sparse_cap at least 1 % of M * K, i.e. alpha <= 0.995) the
 *   residual's columns that at least max(M / 4, 512) tokens hit -- the outlier channels of
 *   Appendix D, up to 128 of them -- are multiplied on the tensor cores inside the GEMM (two-term
 *   FP16 splits of residual and weight); the other entries are added per entry in fp32.  The
 *   result differs from the per-entry sum by at most 4e-6 * sum_k |A - A_c|[m,k] |W|[k,n]
 *   + 2e-11 * amax_W[n] * sum_k |A - A_c|[m,k] (the second term is the resolution of W / d_W in
 *   FP16: it matters only for weights ten orders of magnitude below their column's largest).
 *   A residual value
 *   beyond 43 000 times its token's clamped absmax does not fit the FP16 operand: the call
 *   then adds every entry per entry.
 */
#define FP4_REUSE_W 1
#define FP4_REUSE_A 2
int fp4_linear_fwd(fp4_ctx* ctx, void* stream, const void* A_bf16, const void* W_bf16,
                   int64_t M, int64_t K, int64_t N, double alpha, int reuse, int gemm_kind,
                   void* Y, int out_f32, fp4_qtensor* savedA, fp4_qtensor* savedW,
                   int32_t* status);

/*
 * fp4_linear_bwd -- backward of the FP4 linear layer (Eq. 3, Eq. 6, Appendix C.2):
 *     dA = bf16( dY W_q^T )                         with the forward's W_q,
 *     dW = bf16( (Q(A_c)^T dY + (A - A_c)^T dY) (.) Q'(W (.) sf) )
 * where Q' is the DGE derivative of Eq. 8 with exponent parameter dge_k (paper: 5) capped at
 * dge_clip (paper: 3.0), evaluated on the scaled weights the forward quantised; dge_on == 0
 * selects the straight-through estimator (Q' = 1).  Both GEMMs take E2M1 operands: dY is
 * quantised token-wise after multiplication by d_W[n] (dgrad) and channel-wise after
 * multiplication by d_A[m] (wgrad), so that the forward's codes of W and A are re-used.
 *   dY_bf16 [M x N], W_bf16 [K x N], dA [M x K], dW [K x N] (BF16, or float if out_f32).
 *   dA or dW may be NULL to skip that gradient.
 *   With a heavy residual (same condition as in fp4_linear_fwd, and at least 512 tokens) the
 *   residual's dense columns -- the same outlier channels -- are multiplied with dY on the tensor
 *   cores (exact three-term BF16 split of the residual, chunks of 128 tokens added in fp32 in token
 *   order); the other entries are added per entry in fp32.  That part of dW differs from the
 *   per-entry sum by at most 4e-6 * sum_m |A - A_c|[m,k] |dY|[m,n] (times the DGE factor).
 *   gemm_kind | FP4_BWD_DY_E4M3 (or FP4_BWD_DY_E5M2) quantises both copies of dY to E4M3 (E5M2)
 *   bytes; the saved operands keep the formats the forward gave them; with an 8-bit weight Q' = 1
 *   whatever dge_on says.
 */
int fp4_linear_bwd(fp4_ctx* ctx, void* stream, const void* dY_bf16, const void* W_bf16,
                   const fp4_qtensor* savedA, const fp4_qtensor* savedW,
                   int64_t M, int64_t K, int64_t N,
                   int dge_on, float dge_k, float dge_clip, int gemm_kind,
                   void* dA, void* dW, int out_f32, int32_t* status);

/*
 * fp4_linear_step_host -- one forward + backward of the layer with HOST buffers (pinned memory
 * recommended): copies A, W, dY to the device, runs fp4_linear_fwd and fp4_linear_bwd with
 * BF16 outputs, and copies Y, dA, dW back.  It is the same path as the two calls above (Fig. 2,
 * Eq. 3, Eq. 6); only the staging is added.  Device staging and the saved quantised operands
 * live in the context's workspace: fp4_step_host_workspace_bytes() gives the size needed.
 * Ordering: the outputs are complete once the work this call enqueues on `stream` is.  The host
 * inputs must be ready when the call is made (the copies to the device need not wait for work
 * enqueued on `stream` earlier).  With a workspace of at least
 * fp4_step_host_workspace_bytes() for the call's shape the three phases run on streams of the
 * context (copies in, kernels, copies back) over two sets of device buffers, so that the inputs
 * of call i + 1 travel and its kernels run while call i copies back; the host buffers of a
 * call must stay untouched until its work on `stream` is complete, as with any asynchronous
 * copy.  A smaller workspace that still holds one set of everything is accepted and runs the
 * call on `stream` alone; fp4_set_overlap(ctx, 0) does the same.  Calls on one context must be
 * issued from one thread and on one stream (or streams ordered by the caller).
 * `status_host` (host int32, may be NULL) receives the device status word; reading it makes the
 * call wait for the stream.  All six tensor pointers are HOST pointers.
 */
size_t fp4_step_host_workspace_bytes(int64_t M, int64_t K, int64_t N, double alpha);
int fp4_linear_step_host(fp4_ctx* ctx, void* stream, const void* A_host, const void* W_host,
                         const void* dY_host, int64_t M, int64_t K, int64_t N, double alpha,
                         int dge_on, float dge_k, float dge_clip, int gemm_kind,
                         void* Y_host, void* dA_host, void* dW_host, int32_t* status_host);

/*
 * Measurement support (no counterpart in the paper).  With profiling on, every kernel class the
 * library enqueues is bracketed by CUDA events on the launching stream; fp4_profile_read waits
 * for them and returns the summed device time and the number of kernels of one class since the
 * last fp4_profile_reset.  fp4_launch_count returns the kernels enqueued since the last reset,
 * whether profiling is on or not.
 */
#define FP4_KC_GEMM        0   /* tcgen05 FP4 GEMM                                            */
#define FP4_KC_SELECT      1   /* histogram + row extremes + order statistics                 */
#define FP4_KC_ENCODE      2   /* clamp / scale / Q / pack, both layouts                      */
#define FP4_KC_ABSMAX      3   /* absmax pre-pass of tensors that are not clamped             */
#define FP4_KC_SPARSE      4   /* mask -> CSR / CSC                                           */
#define FP4_KC_COMP_FWD    5   /* residual x W + final store of Y                             */
#define FP4_KC_COMP_WGRAD  6   /* residual^T x dY + DGE factor + final store of dW            */
#define FP4_KC_COUNT       7
int fp4_profile_enable(fp4_ctx* ctx, int on);
/* Measurement support (no counterpart in the paper): a read-only kernel for measuring the bandwidth
 * of the L2 cache, the bound of the per-entry gathers of the sparse compensation (Section 3.2: one
 * row of the dense matrix per residual entry).  `blocks` blocks of 256 threads each read all of
 * `buf` (`bytes`, a multiple of 32768, at least 65536, 16-byte aligned; choose it smaller than L2)
 * `repeats` times with 16-byte loads that bypass L1, every block from its own starting offset.
 * Bytes read = blocks * repeats * bytes; the caller times the call.  `sink` is a device word the
 * kernel may write.                                                                          */
int fp4_l2_read_probe(void* stream, const void* buf, size_t bytes, int repeats, int blocks, unsigned* sink);
/* Inside one call, independent kernel chains (weight quantisation, sparse extraction, the
 * weight-gradient branch) run on side streams owned by the context and rejoin `stream` before
 * the call's work ends.  fp4_set_overlap(ctx, 0) puts every kernel on `stream` in program order
 * (used to time kernels one at a time); the results are identical either way.  Default: on.  */
int fp4_set_overlap(fp4_ctx* ctx, int on);
/* Which order statistics the clamp of an activation uses (fp4_quantize with alpha < 1 and the
 * calls built on it; not fp4_quantile_thresholds_static).  FP4_QUANTILE_SIGNED (default): the
 * paper's form (Section 3.2), lo and hi the (1-alpha)- and alpha-quantiles of the values.
 * FP4_QUANTILE_ABS, a variant outside the paper: one threshold t on the magnitudes, the order
 * statistic of |x| that at most 2 n_tail entries exceed; lo = -t, hi = t.
 * FP4_QUANTILE_TOKEN, another variant outside the paper: the signed form per token -- row m is
 * clamped between its own order statistics, round((1 - alpha) * cols) entries on either side; the
 * operand's `thresholds` then holds 2 * rows floats (lo, hi of every row) and its `sparse_cap`
 * must be at least 2 * rows * round((1 - alpha) * cols).                                       */
#define FP4_QUANTILE_SIGNED 0
#define FP4_QUANTILE_ABS    1
#define FP4_QUANTILE_TOKEN  2
int fp4_set_quantile_mode(fp4_ctx* ctx, int mode);
/* Failure-path testing (no counterpart in the paper).  FP4_DEBUG_WAIT_LIMIT_US: the limit, in
 * microseconds, of every device-side wait of the GEMM kernels this context launches from now on
 * (0 restores the default of 2 s).  FP4_DEBUG_SKIP_FILL: the producer of the GEMM's first CTA leaves
 * out its fill number `value` of the shared-memory ring (no copy, no arrival; -1: none), so that
 * the consumer's wait runs out: the kernel raises FP4_DEV_TIMEOUT, frees its tensor memory and
 * returns; the context stays usable.                                                        */
#define FP4_DEBUG_WAIT_LIMIT_US 1
#define FP4_DEBUG_SKIP_FILL     2
int fp4_debug_set(fp4_ctx* ctx, int key, int64_t value);
int fp4_profile_reset(fp4_ctx* ctx);
int fp4_profile_read(fp4_ctx* ctx, int kernel_class, double* total_ms, int64_t* launches);
int64_t fp4_launch_count(fp4_ctx* ctx);

/*
 * fp4_quantile_thresholds_static -- the two clamp thresholds of a tensor, for callers that
 * must not allocate.  (The paper has no counterpart: this is a packaging variant of the
 * threshold selection that fp4_quantize performs.)
 *
 * Who needs it: code that runs where device allocation is off limits -- inside a region that
 * forbids cudaMalloc (a memory-pool-only framework, a real-time loop, a plugin that is handed
 * tensors but no allocator) -- and that therefore cannot create an fp4_ctx, whose workspace is
 * cudaMalloc'ed.  This call takes no context.  Its scratch (the 65536-bin histogram and the
 * per-row extremes) is a fixed array inside the library image, 769 KB on every GPU that loads
 * the library, held until the process exits.  The call itself performs no cudaMalloc, no
 * cudaFree and calls no allocating library routine.
 *
 *   x_bf16      [rows x cols] BF16, device, 16-byte aligned; rows and cols multiples of 128
 *   rows        at most FP4_STATIC_MAX_ROWS, else FP4_ERR_STATIC_LIMIT is returned and nothing
 *               is enqueued
 *   alpha       0.5 < alpha < 1
 *   thresholds  device float[2]: receives {lo, hi}, bit-identical to what fp4_quantize writes
 * A NaN or an infinity in the input is not reported (the call has no status word): the thresholds
 * are then unspecified.
 * The work is enqueued on `stream` for the current device.  The first call on each device also
 * looks up the device address of the scratch array and sets a kernel attribute (once per device,
 * safe to race between host threads); make that first call before any stream capture begins.  All calls on a device share the one scratch array
 * (it is cleared at the start of each call): two calls whose work overlaps on the GPU -- issued
 * to different streams without ordering between them -- race and give wrong thresholds.
 */
#define FP4_STATIC_MAX_ROWS 65536
int fp4_quantile_thresholds_static(void* stream, const void* x_bf16, int64_t rows, int64_t cols,
                                   double alpha, float* thresholds);

#ifdef __cplusplus
}
#endif
#endif /* FP4_LINEAR_H_ */
