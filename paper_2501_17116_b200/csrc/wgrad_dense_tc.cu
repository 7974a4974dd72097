// Weight-gradient compensation of the residual's channel-dense columns on the tensor cores.
//
// Section 3.2 adds the product of the sparse residual dA = A - A_c with a dense high-precision
// matrix; in the weight gradient (Eq. 6) that product is dA^T dY.  The outlier channels of
// Appendix D make a handful of columns of dA dense (most tokens exceed the threshold there), so
// for those columns the product is a skinny dense contraction over the tokens,
//     C[s, n] = sum_m V[m, s] * dY[m, n],        s < h <= 128 dense columns,
// and it runs on tcgen05.mma instead of gathering one dY row per entry:
//   * dY is the M-side operand, read by TMA straight from the caller's BF16 tensor ([tokens x N],
//     N contiguous: an MN-major operand whose contraction runs over the box's rows);
//   * V is the N-side operand.  Its fp32 values are split exactly into three BF16 terms
//     (v = b1 + b2 + b3, each 8 significant bits), stored K-major as Vt[term][s][m]; BF16 products
//     are exact in fp32, so the tensor cores add exactly the products the fp32 kernel would form;
//   * the tensor cores accumulate one chunk of 128 tokens at a time in tensor memory (24
//     instructions, whose fp32 additions are not round-to-nearest); the epilogue warps drain each
//     chunk into registers and add the chunks in token order with ordinary fp32 additions, so the
//     number of tensor-core additions behind any output stays at 24 however many tokens there are;
//   * a CTA owns 256 output columns and a contiguous range of chunks; the ranges' partial sums go to
//     global memory and are added in range order by dense_reduce (compensate.cu): the result does
//     not depend on scheduling.
// Roles per CTA: warp 0 TMA producer, warp 1 tensor-memory allocation + MMA issue, warps 2..9
// epilogue.  Every wait is bounded (FP4_DEV_TIMEOUT).
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

constexpr int DT_TOK = 64;                       // tokens per stage
constexpr int DT_CHUNK = 2 * DT_TOK;             // tokens accumulated in tensor memory before a drain
constexpr int DT_NT = 256;                       // output columns per CTA
constexpr int DT_BOX = 64 * 64 * 2;              // one 64 x 64 BF16 box: 8 KB
constexpr int DT_DY_BYTES = (DT_NT / 64) * DT_BOX;      // 32 KB of dY per stage
constexpr int DT_THREADS = 64 + 8 * 32;
constexpr int DT_SMEM = 1024 + 3 * (DT_DY_BYTES + 3 * DT_BOX) + 256;   // fits 3 stages (one V box per term) or 2 (two)

// Shared-memory matrix descriptor of an MN-major operand tile made of 64 x 64 BF16 boxes (128-byte
// rows = 64 consecutive MN elements of one contraction index, 128-byte swizzle): groups of 8
// contraction rows are 1024 bytes apart (stride offset), blocks of 64 MN elements one box apart
// (leading offset).
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t smem_addr, uint32_t box_bytes) {
  uint64_t d = 0;
  d |= uint64_t((smem_addr & 0x3FFFFu) >> 4);
  d |= uint64_t(box_bytes >> 4) << 16;
  d |= uint64_t(1024 >> 4) << 32;
  d |= uint64_t(1) << 46;
  d |= uint64_t(2) << 61;
  return d;
}

// kind::f16, BF16 x BF16 -> fp32, A MN-major (dY), B K-major (Vt), M = 128, N = n
__device__ __forceinline__ uint32_t idesc_dense(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (uint32_t(n >> 3) << 17) | (uint32_t(128 >> 4) << 24);
}

// Vt[term][s][m]: the three BF16 terms of the dense columns' residual values, zero where a token has
// no entry.  A block owns 64 tokens: its warps walk the tokens' CSR rows into a shared tile, which
// then leaves as whole 128-byte rows.  Only rows of boxes the GEMM will load (64 per box) are written.
__global__ void __launch_bounds__(256)
dense_split_kernel(const int* __restrict__ rowptr, const int* __restrict__ col, const float* __restrict__ val,
                   const int* __restrict__ slot_of_col, const int* __restrict__ counts,
                   __nv_bfloat16* __restrict__ vt, int M) {
  extern __shared__ __align__(16) uint8_t split_smem[];
  __nv_bfloat16* tile = reinterpret_cast<__nv_bfloat16*>(split_smem);        // [3][DENSE_TC_MAX][64]
  const int n_dense = min(counts[0], DENSE_TC_MAX);
  if (n_dense == 0) return;
  const int rows = ((n_dense + 63) / 64) * 64;
  const int m0 = blockIdx.x * 64;
  uint4* t4 = reinterpret_cast<uint4*>(tile);
  for (int i = threadIdx.x; i < 3 * DENSE_TC_MAX * 64 * 2 / 16; i += blockDim.x) t4[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int tl = warp; tl < 64; tl += 8) {
    const int m = m0 + tl;
    if (m >= M) break;
    for (int e = rowptr[m] + lane; e < rowptr[m + 1]; e += 32) {
      const int slot = slot_of_col[col[e]];
      if (unsigned(slot) >= unsigned(n_dense)) continue;
      const float v = val[e];
      const __nv_bfloat16 b1 = __float2bfloat16_rn(v);
      const float r1 = v - __bfloat162float(b1);                 // exact
      const __nv_bfloat16 b2 = __float2bfloat16_rn(r1);
      const float r2 = r1 - __bfloat162float(b2);                // exact
      const __nv_bfloat16 b3 = __float2bfloat16_rn(r2);          // exact: 24 bits in three terms of 8
      tile[(0 * DENSE_TC_MAX + slot) * 64 + tl] = b1;
      tile[(1 * DENSE_TC_MAX + slot) * 64 + tl] = b2;
      tile[(2 * DENSE_TC_MAX + slot) * 64 + tl] = b3;
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 3 * rows * 8; i += blockDim.x) {
    const int t = i / (rows * 8), r = (i / 8) % rows, c = i % 8;
    const uint4 x = t4[((t * DENSE_TC_MAX + r) * 64 * 2) / 16 + c];
    *reinterpret_cast<uint4*>(vt + (size_t(t * DENSE_TC_MAX + r) * size_t(M) + size_t(m0)) + 8 * c) = x;
  }
}

struct DenseTcArgs {
  int M, N;
  int tiles;                 // blocks of DT_NT output columns
  int splits;                // ranges of chunks per tile
  const int* counts;         // counts[0] = number of dense columns (device)
  float* partial;            // [splits][DENSE_TC_MAX][N]
  int32_t* status;
};

__global__ void __launch_bounds__(DT_THREADS, 1)
comp_wgrad_dense_tc_kernel(const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_vt,
                           const __grid_constant__ DenseTcArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const int n_dense = min(__ldg(args.counts), DENSE_TC_MAX);
  if (n_dense == 0) return;                               // uniform: nothing allocated yet
  const int nb = (n_dense + 63) / 64;                     // 64-row boxes of V per term
  const int stages = nb == 1 ? 3 : 2;
  const uint32_t v_bytes = uint32_t(3 * nb * DT_BOX);
  const uint32_t stage_bytes = uint32_t(DT_DY_BYTES) + v_bytes;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_misc = smem + 3 * (DT_DY_BYTES + 3 * DT_BOX);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_misc);
  uint64_t* empty_bar = full_bar + 3;
  uint64_t* acc_full = empty_bar + 3;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* final_bar = acc_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(final_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x % args.tiles, split = blockIdx.x / args.tiles;
  const int chunks_total = (args.M + DT_CHUNK - 1) / DT_CHUNK;
  const int c_begin = int((long long)chunks_total * split / args.splits);
  const int c_end = int((long long)chunks_total * (split + 1) / args.splits);
  const int n_chunks = c_end - c_begin;
  const int n0 = tile * DT_NT;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 3; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], 8);
    }
    mbar_init(final_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_dy) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_vt) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer -------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0, fills = 0;
      bool ok = true;
      for (int c = 0; c < 2 * n_chunks && ok; ++c) {            // one stage = 64 tokens
        const int m0 = c_begin * DT_CHUNK + c * DT_TOK;
        ok = mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, args.status);
        if (!ok) break;
        uint8_t* dst = smem + stage * stage_bytes;
        mbar_arrive_expect_tx(&full_bar[stage], stage_bytes);
        for (int j = 0; j < DT_NT / 64; ++j)                    // dY: box j = columns n0 + 64 j .. + 63, 64 tokens
          tma_load_2d(dst + j * DT_BOX, &map_dy, &full_bar[stage], n0 + 64 * j, m0);
        for (int t = 0; t < 3; ++t)                             // V terms: 64 tokens x 64 rows per box
          for (int b = 0; b < nb; ++b)
            tma_load_2d(dst + DT_DY_BYTES + (t * nb + b) * DT_BOX, &map_vt, &full_bar[stage], m0,
                        t * DENSE_TC_MAX + 64 * b);
        ++fills;
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) {
        // gave up: let the copies already in flight land before shared memory is released
        const uint32_t last = fills < uint32_t(stages) ? fills : uint32_t(stages);
        for (uint32_t back = 1; back <= last; ++back) {
          const uint32_t f = fills - back;
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(&full_bar[f % stages], (f / stages) & 1u)) {
            if (global_timer_ns() - t0 > 1000000ull) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer ---------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      const uint32_t idesc = idesc_dense(64 * nb);
      for (int c = 0; c < n_chunks && ok; ++c) {
        ok = mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, args.status);
        if (!ok) break;
        tc_fence_after();
        for (int half = 0; half < 2 && ok; ++half) {            // the two stages of this chunk
          ok = mbar_wait(&full_bar[stage], phase, abort_flag, args.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t dy_addr = smem_u32(smem + stage * stage_bytes);
          const uint32_t v_addr = dy_addr + DT_DY_BYTES;
#pragma unroll
          for (int h = 0; h < 2; ++h) {                         // output columns n0 + 128 h .. + 127
            const uint32_t d_tmem = tmem_base + uint32_t(acc * 256 + h * 128);
#pragma unroll
            for (int k = 0; k < 4; ++k) {                       // 16 tokens per instruction
              const uint64_t a_desc = make_smem_desc_mn(dy_addr + uint32_t(2 * h * DT_BOX + k * 2048), DT_BOX);
#pragma unroll
              for (int t = 0; t < 3; ++t) {
                const uint64_t b_desc = make_smem_desc(v_addr + uint32_t(t * nb * DT_BOX + k * 32));
                mma_f16(d_tmem, a_desc, b_desc, idesc, (half | k | t) != 0 ? 1u : 0u);
              }
            }
          }
          tc_commit(&empty_bar[stage]);
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(&acc_full[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      tc_commit(final_bar);
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(final_bar, 0)) {
        if (global_timer_ns() - t0 > WAIT_LIMIT_NS) {
          atomicOr(args.status, FP4_DEV_TIMEOUT);
          break;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue -----------
    // Warp (h, q) owns output columns n0 + 128 h + 32 q .. + 31 (one per lane) and all dense rows.
    const int quarter = warp & 3;
    const int h = (warp - 2) >> 2;
    float run[DENSE_TC_MAX];
#pragma unroll
    for (int i = 0; i < DENSE_TC_MAX; ++i) run[i] = 0.0f;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool gave_up = false;
    for (int c = 0; c < n_chunks; ++c) {
      const bool ok = mbar_wait(&acc_full[acc], acc_phase, abort_flag, args.status);
      if (epilogue_bar_any(!ok, 8 * 32)) { gave_up = true; break; }
      tc_fence_after();
      const uint32_t t_base = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(acc * 256 + h * 128);
#pragma unroll
      for (int c0 = 0; c0 < DENSE_TC_MAX; c0 += 32) {
        if (c0 < 64 * nb) {
          uint32_t v[32];
          tmem_ld_32x32(t_base + uint32_t(c0), v);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) run[c0 + i] += __uint_as_float(v[i]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[acc]);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    const int n = n0 + 128 * h + 32 * quarter + lane;
    if (!gave_up && n < args.N) {
      float* dst = args.partial + size_t(split) * DENSE_TC_MAX * size_t(args.N) + n;
#pragma unroll
      for (int s = 0; s < DENSE_TC_MAX; ++s)
        if (s < n_dense) dst[size_t(s) * size_t(args.N)] = run[s];
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// BF16 [rows x cols] row-major, boxes of 64 columns (128 bytes) x 64 rows, 128-byte swizzle.
int make_bf16_map(fp4_ctx* ctx, CUtensorMap* map, const void* base, int64_t rows, int64_t cols) {
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
  if (!encode) return FP4_ERR_CUDA;
  if (reinterpret_cast<uintptr_t>(base) & 15) return FP4_ERR_ALIGN;
  const cuuint64_t dims[2] = {cuuint64_t(cols), cuuint64_t(rows)};
  const cuuint64_t strides[1] = {cuuint64_t(cols) * 2};
  const cuuint32_t box[2] = {64, 64};
  const cuuint32_t elem_strides[2] = {1, 1};
  const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                            elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FP4_OK : FP4_ERR_CUDA;
}

}  // namespace

// Ranges of chunks per block of output columns: the split (at most 16 ranges) whose CTAs, taken
// in rounds of one per SM, finish soonest -- rounds x chunks per CTA, plus about one chunk's time per
// round for filling the pipeline.
static int splits_for(int sms, int64_t M, int64_t N) {
  const int tiles = int((N + DT_NT - 1) / DT_NT);
  const int chunks = int((M + DT_CHUNK - 1) / DT_CHUNK);
  if (sms > 148) sms = 148;
  int best = 1;
  long long best_cost = -1;
  for (int s = 1; s <= 16 && s <= chunks; ++s) {
    const long long rounds = (tiles * s + sms - 1) / sms;
    const long long cost = rounds * ((chunks + s - 1) / s + 1);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
  }
  return best;
}

int dense_tc_splits(const fp4_ctx* ctx, int64_t M, int64_t N) { return splits_for(ctx->num_sms, M, N); }

size_t dense_tc_scratch_bytes(int64_t M, int64_t N) {
  auto r256 = [](size_t b) { return (b + 255) & ~size_t(255); };
  return r256(size_t(3) * DENSE_TC_MAX * size_t(M) * 2) + r256(size_t(splits_for(148, M, N)) * DENSE_TC_MAX * size_t(N) * 4);
}

// C[s, :] for the dense columns s < counts[0] into `partial` ([splits][DENSE_TC_MAX][N]); the caller
// adds the splits in order.  M must be a multiple of 128.
int launch_comp_wgrad_dense_tc(fp4_ctx* ctx, cudaStream_t stream, const fp4_qtensor* a, const int* slot_of_col,
                               const int* counts, const void* dy_bf16, void* vt, float* partial, int splits,
                               int64_t M, int64_t N, int32_t* status) {
  CUtensorMap map_dy, map_vt;
  int rc = make_bf16_map(ctx, &map_dy, dy_bf16, M, N);
  if (rc != FP4_OK) return rc;
  rc = make_bf16_map(ctx, &map_vt, vt, 3 * DENSE_TC_MAX, M);
  if (rc != FP4_OK) return rc;
  dense_split_kernel<<<unsigned((M + 63) / 64), 256, 3 * DENSE_TC_MAX * 64 * 2, stream>>>(
      a->csr_rowptr, a->csr_col, a->csr_val, slot_of_col, counts, static_cast<__nv_bfloat16*>(vt), int(M));
  DenseTcArgs args;
  args.M = int(M);
  args.N = int(N);
  args.tiles = int((N + DT_NT - 1) / DT_NT);
  args.splits = splits;
  args.counts = counts;
  args.partial = partial;
  args.status = status;
  FP4_CUDA_TRY(cudaFuncSetAttribute(comp_wgrad_dense_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DT_SMEM));
  comp_wgrad_dense_tc_kernel<<<unsigned(args.tiles * splits), DT_THREADS, DT_SMEM, stream>>>(map_dy, map_vt, args);
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}
