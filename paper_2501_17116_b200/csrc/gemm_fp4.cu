// FP4 GEMM on the 5th-generation tensor cores (tcgen05.mma) for sm_100a.
//
//   out[i, j] = ( sum_c val(a[i, c]) * val(b[j, c]) ) * (row_amax[i] / 6) * (col_amax[j] / 6)
//
// Both operands are E2M1 nibbles with the contraction contiguous ("K-major"), which is the
// form of all three GEMMs of the layer (Fig. 2; Eq. 3; Appendix C.2).  The two de-scales are
// applied to the accumulators in the epilogue, after the GEMM, as Appendix C.2 prescribes.
//
// Structure: persistent CTAs (one per SM), 128 x BN output tile per CTA:
//   warp 0      TMA producer: cp.async.bulk.tensor loads into 128-byte-swizzled shared memory,
//               a ring of STAGES stages guarded by full/empty mbarriers;
//   warp 1      allocates tensor memory and issues tcgen05.mma from one thread, fp32
//               accumulators in tensor memory; tcgen05.commit releases stages and publishes tiles;
//   warps 2..   epilogue (8 warps; 16 with the fused weight-gradient epilogue): tcgen05.ld the
//               accumulators (one row per thread), de-scale, write boxes into shared memory and
//               hand them to the copy engine (cp.async.bulk.tensor stores).
// Tensor memory holds two accumulator stages, so the epilogue of one tile runs under the MMAs of
// the next.  512 columns are 2 x 256; the MXF4 flavour also needs a few columns for its block
// scales, so its tile is 128 x 240 (2 x 240 accumulator columns + 16 scale columns).
// Two MMA flavours are compiled:
//   MXF4    kind::mxf4.block_scale, packed nibbles, K = 64 per instruction.  The method has no
//           block scales, so every UE8M0 scale in tensor memory is 2^0: the product is unchanged.
//   F8F6F4  kind::f8f6f4, TMA expands the packed nibbles to one per byte-container group
//           (16 nibbles + 8 bytes of padding), K = 32 per instruction.
// Every wait is bounded: on a timeout the CTA raises FP4_DEV_TIMEOUT, drains its own copies,
// frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

constexpr int BM = 128;
// Epilogue warps: two per lane quarter of tensor memory for the plain epilogue, four for the
// fused weight-gradient epilogue, whose DGE arithmetic needs the extra warps to hide its latency.
enum { EPI_PLAIN = 0, EPI_WGRAD = 1 };
__host__ __device__ constexpr int epi_warps(int epi) { return epi == EPI_WGRAD ? 16 : 8; }
__host__ __device__ constexpr int num_threads(int epi) { return 64 + 32 * epi_warps(epi); }
__host__ __device__ constexpr int stages_of(int kind) { return kind == FP4_GEMM_F8F6F4 ? 3 : 4; }
constexpr int A_STAGE_BYTES = BM * 128;
constexpr int TMEM_COLS = 512;
constexpr int ACC_STRIDE = 256;          // tensor-memory columns between the two accumulator stages
constexpr int SF_COL_B = 240;            // MXF4 only: unit block scales in the gap behind stage 0
constexpr int SF_COL_A = 248;
constexpr int STAGE_OUT_BYTES = 32768;    // epilogue staging: 4 KB per warp (plain) or 2 KB (fused)

__host__ __device__ constexpr int tile_n(int kind) { return kind == FP4_GEMM_F8F6F4 ? 256 : 240; }
__host__ __device__ constexpr int b_stage_bytes(int kind) { return tile_n(kind) * 128; }
__host__ __device__ constexpr int stage_bytes(int kind) { return A_STAGE_BYTES + b_stage_bytes(kind); }
// operand ring, epilogue staging, barriers, column de-scales [2][256], DGE column scales [2][256]
constexpr size_t smem_bytes(int kind) {
  return 1024 + size_t(stages_of(kind)) * stage_bytes(kind) + 256 + 2 * 256 * 4 + STAGE_OUT_BYTES + 2 * 256 * 4;
}

struct GemmArgs {
  int I, J;
  int num_k_blocks;
  int num_m_blocks, num_n_blocks;
  uint32_t tx_bytes;
  uint32_t idesc;              // instruction descriptor (operand formats differ per problem)
  float row_div, col_div;      // largest value of the row / column operand's format: 6 (E2M1) or 448 (E4M3)
  const float* row_amax;
  const float* col_amax;
  void* out;
  int out_f32;
  int32_t* status;
  // fused weight-gradient epilogue (EPI_WGRAD)
  const float* addend;
  const int* slot_of_row;
  const uint4* w;
  const float* w_amax;
  float inv_k, expo, clip;
  // dense tail (single-problem launches only): after the FP4 k-blocks of a tile, 3 * ceil(*tail_count / 64)
  // k-blocks of 64 FP16 columns each from the maps that otherwise describe a second problem are
  // accumulated into the same tile with kind::f16 (null: no tail)
  const int* tail_count;
  uint32_t tail_tx_bytes;
  uint32_t tail_idesc;
  // failure-path testing (fp4_debug_set): limit of every wait of this launch, and the index of one
  // fill of shared memory that the producer of CTA 0 leaves out (-1: none)
  uint64_t wait_limit_ns;
  int skip_fill;
};

// Instruction descriptors: M = 128, N = tile_n, both operands K-major, E2M1 x E2M1 -> fp32.
// kind::f8f6f4 format fields: E4M3 = 0, E2M1 = 5
// format field of the byte-container kind for an operand format of the C interface
__host__ __device__ constexpr uint32_t f8f6f4_code(int format) {
  return format == FP4_FORMAT_E4M3 ? 0u : (format == FP4_FORMAT_E5M2 ? 1u : 5u);
}
__host__ __device__ constexpr uint32_t idesc_f8f6f4(int a_format = FP4_FORMAT_E2M1, int b_format = FP4_FORMAT_E2M1) {
  return (1u << 4) | (f8f6f4_code(a_format) << 7) | (f8f6f4_code(b_format) << 10) |
         (uint32_t(tile_n(FP4_GEMM_F8F6F4) >> 3) << 17) | (uint32_t(BM >> 4) << 24);
}
// kind::f16 with FP16 operands (format 0) and fp32 accumulators, M = 128, N = the kind's tile width
__host__ __device__ constexpr uint32_t idesc_f16(int gemm_kind) {
  return (1u << 4) | (uint32_t(tile_n(gemm_kind) >> 3) << 17) | (uint32_t(BM >> 4) << 24);
}
__host__ __device__ constexpr uint32_t idesc_mxf4() {
  return (1u << 7) | (1u << 10) | (uint32_t(tile_n(FP4_GEMM_MXF4) >> 3) << 17) | (1u << 23) |
         (uint32_t(BM >> 4) << 24);
}

// Where the bulk stores of the epilogue take their boxes from and how they are described.
struct OutMaps {
  const CUtensorMap* unit;      // box of 32 rows x 64 bytes (16 floats or 32 BF16), 64-byte swizzle
  const CUtensorMap* half;      // BF16 output: box of 32 rows x 16 columns, no swizzle
};

// One 32 x W chunk of de-scaled (and, in the fused epilogue, compensated and DGE-weighted) values,
// row `lane` in y[]: write it into a staging buffer in the layout of the tensor map and let one
// lane hand the box to the copy engine.  With the 64-byte swizzle, 16-byte slot s of row r sits
// at s ^ ((r >> 1) & 3), so the row-wise writes touch every bank once.  The warp never waits for
// global memory: before a buffer is written again only the shared-memory read of the store that
// used it last must have finished.  `seq` counts the warp's stores; with NBUF = 2 they alternate
// between two 2 KB buffers.
template <int W, int NBUF>
__device__ __forceinline__ void bulk_store_chunk(const float (&y)[W], uint8_t* stage, int out_f32, const OutMaps& maps,
                                                 int row0, int col0, int lane, uint32_t& seq) {
  const int fx = (lane >> 1) & 3;
  if (out_f32) {
#pragma unroll
    for (int u = 0; u < W / 16; ++u) {              // one box per 16 columns
      uint8_t* buf = stage + (NBUF == 2 ? (seq & 1u) * 2048 : 0);
      ++seq;
      if (lane == 0) { if (NBUF == 2) tma_store_wait_read_1(); else tma_store_wait_read_0(); }
      __syncwarp();
      uint8_t* my_row = buf + lane * 64;
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<float4*>(my_row + ((j ^ fx) * 16)) =
            make_float4(y[16 * u + 4 * j], y[16 * u + 4 * j + 1], y[16 * u + 4 * j + 2], y[16 * u + 4 * j + 3]);
      fence_async_smem();
      __syncwarp();
      if (lane == 0) tma_store_2d(maps.unit, buf, col0 + 16 * u, row0);
    }
  } else {
    uint4 packed[W / 8];
#pragma unroll
    for (int j = 0; j < W / 8; ++j) {
      uint32_t w4[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        __nv_bfloat162 h = __floats2bfloat162_rn(y[8 * j + 2 * q], y[8 * j + 2 * q + 1]);
        w4[q] = *reinterpret_cast<uint32_t*>(&h);
      }
      packed[j] = make_uint4(w4[0], w4[1], w4[2], w4[3]);
    }
    // a 16-column BF16 box is 1 KB: two of them always fit the 2 KB every warp has
    constexpr bool two = NBUF == 2 || W == 16;
    uint8_t* buf = stage + (two ? (seq & 1u) * (W == 16 && NBUF == 1 ? 1024 : 2048) : 0);
    ++seq;
    if (lane == 0) { if (two) tma_store_wait_read_1(); else tma_store_wait_read_0(); }
    __syncwarp();
    if (W == 32) {
      uint8_t* my_row = buf + lane * 64;
#pragma unroll
      for (int j = 0; j < W / 8; ++j) *reinterpret_cast<uint4*>(my_row + ((j ^ fx) * 16)) = packed[j];
    } else {
      uint8_t* my_row = buf + lane * 32;
#pragma unroll
      for (int j = 0; j < W / 8; ++j) *reinterpret_cast<uint4*>(my_row + j * 16) = packed[j];
    }
    fence_async_smem();
    __syncwarp();
    if (lane == 0) tma_store_2d(W == 32 ? maps.unit : maps.half, buf, col0, row0);
  }
}

template <int W>
__device__ __forceinline__ void descale_chunk(const uint32_t (&v)[32], float d_row, const float* dcol, float (&y)[W]) {
#pragma unroll
  for (int q = 0; q < W / 4; ++q) {
    const float4 dc = *reinterpret_cast<const float4*>(dcol + 4 * q);     // same address in every lane
    y[4 * q + 0] = __fmul_rn(__fmul_rn(__uint_as_float(v[4 * q + 0]), d_row), dc.x);
    y[4 * q + 1] = __fmul_rn(__fmul_rn(__uint_as_float(v[4 * q + 1]), d_row), dc.y);
    y[4 * q + 2] = __fmul_rn(__fmul_rn(__uint_as_float(v[4 * q + 2]), d_row), dc.z);
    y[4 * q + 3] = __fmul_rn(__fmul_rn(__uint_as_float(v[4 * q + 3]), d_row), dc.w);
  }
}

// Plain epilogue of one 128 x BN block of accumulators for one warp (32 rows of it).  The warps
// that share a lane quarter take the 32-column chunks in turn (`group` g of G: chunks g, g + G,
// ...).  Chunks are read from tensor memory (the next one under the stores of the current one),
// de-scaled and stored; `row_blk` is the index of the 128-row block.
template <int BN, int G>
__device__ __forceinline__ void epilogue_tile_plain(const GemmArgs& args, int row_blk, int n_blk, uint32_t t_base,
                                                    float d_row, const float* dcol, uint8_t* stage, int quarter,
                                                    int group, int lane, const OutMaps& maps, uint32_t& seq) {
  const int n_valid = min(BN, args.J - n_blk * BN);           // ragged last tile in N (multiple of 16)
  const int row0 = row_blk * BM + quarter * 32;
  int c0 = 32 * group;
  if (c0 >= n_valid) return;
  uint32_t v[32];
  if (n_valid - c0 >= 32) tmem_ld_32x32(t_base + uint32_t(c0), v); else tmem_ld_32x16(t_base + uint32_t(c0), v);
#pragma unroll 1
  for (; c0 < n_valid; c0 += 32 * G) {
    const int width = min(32, n_valid - c0);
    const int next_width = n_valid - (c0 + 32 * G);            // <= 0: this is the warp's last chunk
    const uint32_t next_taddr = t_base + uint32_t(c0 + 32 * G);
    tmem_ld_wait();
    if (width == 32) {
      float y[32];
      descale_chunk<32>(v, d_row, dcol + c0, y);
      if (next_width >= 32) tmem_ld_32x32(next_taddr, v);      // v is dead: fetch under the stores
      else if (next_width > 0) tmem_ld_32x16(next_taddr, v);
      bulk_store_chunk<32, 2>(y, stage, args.out_f32, maps, row0, n_blk * BN + c0, lane, seq);
    } else {
      float y[16];
      descale_chunk<16>(v, d_row, dcol + c0, y);
      bulk_store_chunk<16, 2>(y, stage, args.out_f32, maps, row0, n_blk * BN + c0, lane, seq);
    }
  }
}

// Operands of the fused weight-gradient epilogue for 16 columns of this thread's row: the BF16
// weights that drive the DGE factor and the compensation row.  They are requested one chunk
// ahead, right after the previous chunk's have been consumed.
struct WgradOperands {
  uint4 w[2];            // 16 BF16 weights
  float4 add[4];         // 16 floats of the compensation row (zeros without one)
};
__device__ __forceinline__ void wgrad_fetch(WgradOperands& op, const GemmArgs& args, int row, int slot, int col) {
  if (args.w) {
    const uint4* src = args.w + ((size_t(row) * size_t(args.J) + size_t(col)) >> 3);
    op.w[0] = __ldg(src);
    op.w[1] = __ldg(src + 1);
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) op.add[j] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (slot >= 0) {
    const float4* src = reinterpret_cast<const float4*>(args.addend + size_t(slot) * size_t(args.J) + size_t(col));
#pragma unroll
    for (int j = 0; j < 4; ++j) op.add[j] = __ldg(src + j);
  }
}

// Fused weight-gradient epilogue for one warp: 16-column chunks, every thread keeps its own row
//   out[k, n] = store( (acc * d_col[n] + addend[slot[k], n]) * Q'(w[k, n] * 6 / w_amax[n]) ).
// The thread-per-row layout of tensor memory is kept throughout: the weights and the
// compensation row are read as whole 32-byte sectors per thread, the results leave through a
// bulk store.  `first` holds the operands of the warp's first chunk, requested by the caller
// before the accumulators were awaited.
template <int BN, int G>
__device__ __forceinline__ void epilogue_tile_wgrad(const GemmArgs& args, int row_blk, int n_blk, uint32_t t_base,
                                                    float d_row, const float* dcol, const float* gcol, int slot,
                                                    uint8_t* stage, int quarter, int group, int lane,
                                                    const OutMaps& maps, uint32_t& seq, WgradOperands& op) {
  const int n_valid = min(BN, args.J - n_blk * BN);
  const int row0 = row_blk * BM + quarter * 32;
  int c0 = 16 * group;
  if (c0 >= n_valid) return;
  uint32_t v[32];
  tmem_ld_32x16(t_base + uint32_t(c0), v);
#pragma unroll 1
  for (; c0 < n_valid; c0 += 16 * G) {
    const bool more = c0 + 16 * G < n_valid;
    tmem_ld_wait();
    float y[16];
    descale_chunk<16>(v, d_row, dcol + c0, y);
    if (more) tmem_ld_32x16(t_base + uint32_t(c0 + 16 * G), v);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      y[4 * j + 0] += op.add[j].x; y[4 * j + 1] += op.add[j].y; y[4 * j + 2] += op.add[j].z; y[4 * j + 3] += op.add[j].w;
    }
    if (args.w) {
      const uint32_t ww[8] = {op.w[0].x, op.w[0].y, op.w[0].z, op.w[0].w, op.w[1].x, op.w[1].y, op.w[1].z, op.w[1].w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 g4 = *reinterpret_cast<const float4*>(gcol + c0 + 4 * q);   // same address in every lane
        const float g[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = 4 * q + e;
          const float wf = __uint_as_float((c & 1) ? (ww[c >> 1] & 0xFFFF0000u) : (ww[c >> 1] << 16));
          y[c] *= dge_factor(__fmul_rn(wf, g[e]), args.expo, args.inv_k, args.clip);
        }
      }
    }
    if (more) wgrad_fetch(op, args, row0 + lane, slot, n_blk * BN + c0 + 16 * G);
    bulk_store_chunk<16, 1>(y, stage, args.out_f32, maps, row0, n_blk * BN + c0, lane, seq);
  }
}

template <int KIND, int EPI>
__global__ void __launch_bounds__(num_threads(EPI), 1)
gemm_fp4_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_out_aux,
                const __grid_constant__ GemmArgs args, const __grid_constant__ CUtensorMap map_a2,
                const __grid_constant__ CUtensorMap map_b2, const __grid_constant__ CUtensorMap map_out2,
                const __grid_constant__ CUtensorMap map_out_aux2, const __grid_constant__ GemmArgs args2) {
  constexpr int NACC = 2;
  constexpr int STAGES = stages_of(KIND);
  constexpr int BN = tile_n(KIND);
  constexpr int B_STAGE_BYTES = b_stage_bytes(KIND);
  constexpr int STAGE_BYTES = stage_bytes(KIND);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES * A_STAGE_BYTES;
  uint8_t* s_out = smem + STAGES * STAGE_BYTES;        // [8 warps][4096] staging, 1024-byte aligned
  uint8_t* smem_misc = s_out + STAGE_OUT_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_misc);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* acc_full = empty_bar + STAGES;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* final_bar = acc_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(final_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* s_dcol = reinterpret_cast<float*>(smem_misc + 256);                     // [2][256] column de-scales
  float* s_gcol = s_dcol + 2 * 256;                                              // [2][256] 6 / w_amax (DGE)

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // Two problems may share one launch (args2 with no tiles: one problem): the tiles of the first
  // come first, then those of the second, so that the epilogue of one problem's last tiles runs
  // under the MMAs of the other's first.
  const int tiles_first = args.num_m_blocks * args.num_n_blocks;
  const int num_tiles = tiles_first + args2.num_m_blocks * args2.num_n_blocks;

  int pre = 0;          // thread 0: k-blocks of its first tile already requested (see below)
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], epi_warps(EPI));
    }
    mbar_init(final_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // This thread is the producer.  The stages are empty and the barriers are its own work, so it
    // requests the first k-blocks of its first tile now: they travel while tensor memory is
    // allocated and the block synchronises.
    if (int(blockIdx.x) < num_tiles) {
      const bool second = int(blockIdx.x) >= tiles_first;
      const GemmArgs& pa = second ? args2 : args;
      const CUtensorMap* ma = second ? &map_a2 : &map_a;
      const CUtensorMap* mb = second ? &map_b2 : &map_b;
      const int tt = second ? int(blockIdx.x) - tiles_first : int(blockIdx.x);
      const int m_blk = tt % pa.num_m_blocks, n_blk = tt / pa.num_m_blocks;
      pre = pa.num_k_blocks < STAGES ? pa.num_k_blocks : STAGES;
      for (int kb = 0; kb < pre; ++kb) {
        mbar_arrive_expect_tx(&full_bar[kb], pa.tx_bytes);
        tma_load_2d(smem_a + kb * A_STAGE_BYTES, ma, &full_bar[kb], kb * 128, m_blk * BM);
        tma_load_2d(smem_b + kb * B_STAGE_BYTES, mb, &full_bar[kb], kb * 128, n_blk * BN);
      }
    }
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_out) : "memory");
    if (args.tail_count) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a2) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b2) : "memory");
    }
    if (args2.num_m_blocks) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a2) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b2) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_out2) : "memory");
    }
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (KIND == FP4_GEMM_MXF4) {
    // Unit block scales: every byte of the scale columns is 0x7F (UE8M0 2^0), so the layout the
    // instruction expects inside these columns does not matter.
    if (warp >= 2 && warp < 6) {
      const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
      for (int c = 0; c < 16; c += 8) tmem_st_32x8(tmem_base + lane_base + SF_COL_B + c, 0x7F7F7F7Fu);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
  }

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer -------
    if (lane == 0) {
      int stage = pre == STAGES ? 0 : pre;
      uint32_t phase = pre == STAGES ? 1u : 0u;
      uint32_t fills = uint32_t(pre);
      bool ok = true;
      const int tail_kb = args.tail_count ? 3 * ((min(*args.tail_count, TAIL_MAX_COLS) + 63) / 64) : 0;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        const bool second = t >= tiles_first;
        const GemmArgs& pa = second ? args2 : args;
        const CUtensorMap* ma = second ? &map_a2 : &map_a;
        const CUtensorMap* mb = second ? &map_b2 : &map_b;
        const int tt = second ? t - tiles_first : t;
        const int m_blk = tt % pa.num_m_blocks;
        const int n_blk = tt / pa.num_m_blocks;
        for (int kb = (t == int(blockIdx.x) ? pre : 0); kb < pa.num_k_blocks; ++kb) {
          ok = mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, args.status, args.wait_limit_ns);
          if (!ok) break;
          if (blockIdx.x != 0 || int(fills) != args.skip_fill) {      // a left-out fill: no copy, no arrival
            mbar_arrive_expect_tx(&full_bar[stage], pa.tx_bytes);
            tma_load_2d(smem_a + stage * A_STAGE_BYTES, ma, &full_bar[stage], kb * 128, m_blk * BM);
            tma_load_2d(smem_b + stage * B_STAGE_BYTES, mb, &full_bar[stage], kb * 128, n_blk * BN);
          }
          ++fills;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        for (int kb = 0; kb < tail_kb && ok; ++kb) {      // dense tail: FP16 columns 64 kb .. 64 kb + 63
          ok = mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, args.status, args.wait_limit_ns);
          if (!ok) break;
          mbar_arrive_expect_tx(&full_bar[stage], args.tail_tx_bytes);
          tma_load_2d(smem_a + stage * A_STAGE_BYTES, &map_a2, &full_bar[stage], kb * 64, m_blk * BM);
          tma_load_2d(smem_b + stage * B_STAGE_BYTES, &map_b2, &full_bar[stage], kb * 64, n_blk * BN);
          ++fills;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // Gave up: let the copies already in flight land before shared memory is released.
        const uint32_t last = fills < uint32_t(STAGES) ? fills : uint32_t(STAGES);
        for (uint32_t back = 1; back <= last; ++back) {
          const uint32_t f = fills - back;                 // global index of that fill
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(&full_bar[f % STAGES], (f / STAGES) & 1u)) {
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
      const int tail_kb = args.tail_count ? 3 * ((min(*args.tail_count, TAIL_MAX_COLS) + 63) / 64) : 0;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        ok = mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, args.status, args.wait_limit_ns);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + uint32_t(acc * ACC_STRIDE);
        const int num_k_blocks = t >= tiles_first ? args2.num_k_blocks : args.num_k_blocks;
        const uint32_t idesc = t >= tiles_first ? args2.idesc : args.idesc;
        for (int kb = 0; kb < num_k_blocks; ++kb) {
          ok = mbar_wait(&full_bar[stage], phase, abort_flag, args.status, args.wait_limit_ns);
          if (!ok) break;
          tc_fence_after();
          const uint64_t a_desc = make_smem_desc(smem_u32(smem_a + stage * A_STAGE_BYTES));
          const uint64_t b_desc = make_smem_desc(smem_u32(smem_b + stage * B_STAGE_BYTES));
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            // 32 bytes of the swizzled 128-byte row per instruction: +2 in the (>>4) address field
            const uint32_t accumulate = (kb | k) != 0 ? 1u : 0u;
            if (KIND == FP4_GEMM_F8F6F4) {
              mma_f8f6f4(d_tmem, a_desc + uint64_t(2 * k), b_desc + uint64_t(2 * k), idesc, accumulate);
            } else {
              mma_mxf4(d_tmem, a_desc + uint64_t(2 * k), b_desc + uint64_t(2 * k), idesc, tmem_base + SF_COL_A,
                       tmem_base + SF_COL_B, accumulate);
            }
          }
          tc_commit(&empty_bar[stage]);       // frees the stage once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        for (int kb = 0; kb < tail_kb && ok; ++kb) {
          ok = mbar_wait(&full_bar[stage], phase, abort_flag, args.status, args.wait_limit_ns);
          if (!ok) break;
          tc_fence_after();
          const uint64_t a_desc = make_smem_desc(smem_u32(smem_a + stage * A_STAGE_BYTES));
          const uint64_t b_desc = make_smem_desc(smem_u32(smem_b + stage * B_STAGE_BYTES));
#pragma unroll
          for (int k = 0; k < 4; ++k)          // 16 FP16 columns = 32 bytes of the 128-byte row per instruction
            mma_f16(d_tmem, a_desc + uint64_t(2 * k), b_desc + uint64_t(2 * k), args.tail_idesc, 1u);
          tc_commit(&empty_bar[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(&acc_full[acc]);            // accumulators of this tile are complete
        if (++acc == NACC) { acc = 0; acc_phase ^= 1u; }
      }
      // All MMAs issued by this thread must have retired before tensor memory is freed.
      tc_commit(final_bar);
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(final_bar, 0)) {
        if (global_timer_ns() - t0 > args.wait_limit_ns) {
          atomicOr(args.status, FP4_DEV_TIMEOUT);
          break;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue -----------
    constexpr int EW = epi_warps(EPI);
    constexpr int G = EW / 4;                   // warps per lane quarter
    const int quarter = warp & 3;               // the lane quarter of tensor memory this warp may read
    const int group = (warp - 2) >> 2;          // which of the G warps of this quarter
    const int et = threadIdx.x - 64;            // index among the epilogue threads
    uint8_t* stage = s_out + (warp - 2) * (STAGE_OUT_BYTES / EW);
    int acc = 0;
    uint32_t acc_phase = 0;
    uint32_t tile_parity = 0;
    uint32_t store_seq = 0;
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      const bool second = t >= tiles_first;
      const GemmArgs& pa = second ? args2 : args;
      const OutMaps out_maps = {second ? &map_out2 : &map_out, second ? &map_out_aux2 : &map_out_aux};
      const int tt = second ? t - tiles_first : t;
      const int m_blk = tt % pa.num_m_blocks;
      const int n_blk = tt / pa.num_m_blocks;
      // De-scales of this tile are fetched before the accumulators are awaited, under the MMAs.
      const int row = m_blk * BM + quarter * 32 + lane;
      const float d_row = pa.row_amax ? __fdiv_rn(__ldg(&pa.row_amax[row]), pa.row_div) : 1.0f;
      float* dcol = s_dcol + tile_parity * 256;
      float* gcol = s_gcol + tile_parity * 256;
      for (int c = et; c < BN; c += 32 * EW) {
        const int col = n_blk * BN + c;
        dcol[c] = (pa.col_amax && col < pa.J) ? __fdiv_rn(__ldg(&pa.col_amax[col]), pa.col_div) : 1.0f;
        if (EPI == EPI_WGRAD && pa.w) {
          const float am = col < pa.J ? __ldg(&pa.w_amax[col]) : 0.0f;
          gcol[c] = am > 0.0f ? __fdiv_rn(6.0f, am) : 0.0f;
        }
      }
      int slot = -1;
      WgradOperands op;
      if (EPI == EPI_WGRAD) {
        if (pa.slot_of_row) slot = __ldg(&pa.slot_of_row[row]);
        if (n_blk * BN + 16 * group < pa.J) wgrad_fetch(op, pa, row, slot, n_blk * BN + 16 * group);
      }
      const bool ok = mbar_wait(&acc_full[acc], acc_phase, abort_flag, args.status, args.wait_limit_ns);
      if (epilogue_bar_any(!ok, 32 * EW)) break;   // also publishes dcol to the other warps
      tc_fence_after();
      const uint32_t t_base = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(acc * ACC_STRIDE);
      if (EPI == EPI_WGRAD)
        epilogue_tile_wgrad<BN, G>(pa, m_blk, n_blk, t_base, d_row, dcol, gcol, slot, stage, quarter, group, lane,
                                   out_maps, store_seq, op);
      else
        epilogue_tile_plain<BN, G>(pa, m_blk, n_blk, t_base, d_row, dcol, stage, quarter, group, lane, out_maps,
                                   store_seq);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[acc]);
      if (++acc == NACC) { acc = 0; acc_phase ^= 1u; }
      tile_parity ^= 1u;
    }
    if (lane == 0) tma_store_wait_all();    // this warp's bulk stores have landed
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map over the codes of one operand with a box of 128 bytes of shared memory x box_rows:
// packed nibbles [rows x C/2 bytes] (E2M1) or bytes [rows x C] (E4M3, byte-container kind only).
int make_codes_map(fp4_ctx* ctx, CUtensorMap* map, const uint8_t* codes, int64_t rows, int64_t C, int box_rows,
                   int gemm_kind, bool e4m3 /* an FP8 format: one byte per element */) {
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
  if (!encode) return FP4_ERR_CUDA;
  const cuuint32_t elem_strides[2] = {1, 1};
  const cuuint32_t box[2] = {128, cuuint32_t(box_rows)};
  CUresult r;
  if (e4m3) {
    const cuuint64_t dims[2] = {cuuint64_t(C), cuuint64_t(rows)};
    const cuuint64_t strides[1] = {cuuint64_t(C)};
    r = encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(codes), dims, strides, box, elem_strides,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (gemm_kind == FP4_GEMM_F8F6F4) {
    // global memory packed, shared memory 16 nibbles + 8 bytes of padding per 16 bytes
    const cuuint64_t dims[2] = {cuuint64_t(C), cuuint64_t(rows)};
    const cuuint64_t strides[1] = {cuuint64_t(C / 2)};
    r = encode(map, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, 2, const_cast<uint8_t*>(codes), dims, strides, box,
               elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    const cuuint64_t dims[2] = {cuuint64_t(C / 2), cuuint64_t(rows)};
    const cuuint64_t strides[1] = {cuuint64_t(C / 2)};
    r = encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(codes), dims, strides, box, elem_strides,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  return r == CUDA_SUCCESS ? FP4_OK : FP4_ERR_CUDA;
}

// Tensor map over one operand of the dense tail: FP16 [rows x TAIL_WIDTH], a box of 64 columns (128
// bytes) x box_rows, laid out in shared memory like a stage of codes.
int make_tail_map(fp4_ctx* ctx, CUtensorMap* map, const void* base, int64_t rows, int box_rows) {
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
  if (!encode) return FP4_ERR_CUDA;
  if (reinterpret_cast<uintptr_t>(base) & 15) return FP4_ERR_ALIGN;
  const cuuint64_t dims[2] = {cuuint64_t(TAIL_WIDTH), cuuint64_t(rows)};
  const cuuint64_t strides[1] = {cuuint64_t(TAIL_WIDTH) * 2};
  const cuuint32_t box[2] = {64, cuuint32_t(box_rows)};
  const cuuint32_t elem_strides[2] = {1, 1};
  const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                            elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FP4_OK : FP4_ERR_CUDA;
}

// Tensor maps of the output [I x J] for the bulk stores of the epilogue.  `unit` is a box of 32 rows
// x 64 bytes with the 64-byte swizzle; `aux` is, for BF16 output, a box of 32 rows x 16 columns
// without swizzle (16-column chunks) and unused for fp32 output (a copy of `unit`).
int make_out_maps(fp4_ctx* ctx, CUtensorMap* unit, CUtensorMap* aux, void* out, int64_t I, int64_t J, int out_f32) {
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
  if (!encode) return FP4_ERR_CUDA;
  const size_t elt = out_f32 ? 4 : 2;
  const cuuint64_t dims[2] = {cuuint64_t(J), cuuint64_t(I)};
  const cuuint64_t strides[1] = {cuuint64_t(J) * elt};
  const cuuint32_t elem_strides[2] = {1, 1};
  const CUtensorMapDataType dt = out_f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  const cuuint32_t box_unit[2] = {cuuint32_t(64 / elt), 32};
  CUresult r = encode(unit, dt, 2, out, dims, strides, box_unit, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                      CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return FP4_ERR_CUDA;
  const cuuint32_t box_aux[2] = {16, 32};
  r = encode(aux, dt, 2, out, dims, strides, box_aux, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
             out_f32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FP4_OK : FP4_ERR_CUDA;
}

struct Problem {
  CUtensorMap map_a, map_b, map_out, map_out_aux;
  GemmArgs args;
  bool fused;
};

template <int KIND, int EPI>
int launch_kernel(int grid, cudaStream_t stream, const Problem& p, const Problem* second = nullptr) {
  constexpr size_t kSmem = smem_bytes(KIND);
  FP4_CUDA_TRY(cudaFuncSetAttribute(gemm_fp4_kernel<KIND, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    int(kSmem)));
  Problem none = p;
  none.args.num_m_blocks = none.args.num_n_blocks = 0;          // a second problem without tiles
  const Problem& q = second ? *second : none;
  gemm_fp4_kernel<KIND, EPI><<<grid, num_threads(EPI), kSmem, stream>>>(p.map_a, p.map_b, p.map_out, p.map_out_aux,
                                                                        p.args, q.map_a, q.map_b, q.map_out,
                                                                        q.map_out_aux, q.args);
  return FP4_OK;
}

// Tensor maps and arguments of one GEMM.
int make_problem(fp4_ctx* ctx, Problem* p, const Fp4GemmDesc& d, int gemm_kind, int32_t* status) {
  if (gemm_kind != FP4_GEMM_MXF4 && gemm_kind != FP4_GEMM_F8F6F4) return FP4_ERR_ARG;
  const bool a8 = d.a_format != FP4_FORMAT_E2M1, b8 = d.b_format != FP4_FORMAT_E2M1;   // FP8 bytes
  if ((a8 || b8) && gemm_kind != FP4_GEMM_F8F6F4) return FP4_ERR_ARG;   // FP8 operands need the byte-container kind
  // The byte-container form expands 32 bytes of a packed row into 64, so its rows must start on
  // 32-byte boundaries (C/2 a multiple of 32 holds for every multiple of 128).
  const uintptr_t need = gemm_kind == FP4_GEMM_F8F6F4 ? 31 : 15;
  if ((reinterpret_cast<uintptr_t>(d.a_codes) & need) || (reinterpret_cast<uintptr_t>(d.b_codes) & need))
    return FP4_ERR_ALIGN;
  int rc = make_codes_map(ctx, &p->map_a, d.a_codes, d.I, d.C, BM, gemm_kind, a8);
  if (rc != FP4_OK) return rc;
  const int BN = tile_n(gemm_kind);
  rc = make_codes_map(ctx, &p->map_b, d.b_codes, d.J, d.C, BN, gemm_kind, b8);
  if (rc != FP4_OK) return rc;
  if (reinterpret_cast<uintptr_t>(d.out) & 15) return FP4_ERR_ALIGN;
  rc = make_out_maps(ctx, &p->map_out, &p->map_out_aux, d.out, d.I, d.J, d.out_f32);
  if (rc != FP4_OK) return rc;

  GemmArgs& args = p->args;
  args.I = int(d.I);
  args.J = int(d.J);
  const int k_per_stage = gemm_kind == FP4_GEMM_F8F6F4 ? 128 : 256;   // elements per 128-byte row
  args.num_k_blocks = int((d.C + k_per_stage - 1) / k_per_stage);
  args.num_m_blocks = int(d.I / BM);
  args.num_n_blocks = int((d.J + BN - 1) / BN);
  // The transaction count of a copy is in bytes read from global memory: the byte-container form
  // fills a stage's 128-byte rows from 64 bytes of packed nibbles (E2M1) or from 128 bytes (E4M3).
  if (gemm_kind == FP4_GEMM_F8F6F4)
    args.tx_bytes = uint32_t(A_STAGE_BYTES / (a8 ? 1 : 2) + b_stage_bytes(gemm_kind) / (b8 ? 1 : 2));
  else
    args.tx_bytes = stage_bytes(gemm_kind);
  args.idesc = gemm_kind == FP4_GEMM_F8F6F4 ? idesc_f8f6f4(d.a_format, d.b_format) : idesc_mxf4();
  args.row_div = fp8_max(d.a_format);
  args.col_div = fp8_max(d.b_format);
  args.row_amax = d.row_amax;
  args.col_amax = d.col_amax;
  args.out = d.out;
  args.out_f32 = d.out_f32;
  args.status = status;
  const GemmEpilogue* epi = d.epilogue;
  const bool fused = epi && (epi->addend || epi->w_bf16);
  p->fused = fused;
  args.addend = fused ? epi->addend : nullptr;
  args.slot_of_row = fused && epi->addend ? epi->slot_of_row : nullptr;
  args.w = fused ? static_cast<const uint4*>(epi->w_bf16) : nullptr;
  args.w_amax = fused ? epi->w_amax : nullptr;
  args.inv_k = fused && epi->w_bf16 ? 1.0f / epi->dge_k : 1.0f;
  args.expo = args.inv_k - 1.0f;
  args.clip = fused ? epi->dge_clip : 0.0f;
  args.wait_limit_ns = ctx->debug_wait_limit_ns ? ctx->debug_wait_limit_ns : WAIT_LIMIT_NS;
  args.skip_fill = ctx->debug_skip_fill;
  args.tail_count = nullptr;
  args.tail_tx_bytes = uint32_t(A_STAGE_BYTES + b_stage_bytes(gemm_kind));
  args.tail_idesc = idesc_f16(gemm_kind);
  return FP4_OK;
}

}  // namespace

int launch_gemm_fp4(fp4_ctx* ctx, cudaStream_t stream, const uint8_t* a_codes, const uint8_t* b_codes, int64_t I,
                    int64_t J, int64_t C, const float* row_amax, const float* col_amax, void* out, int out_f32,
                    int gemm_kind, int32_t* status, const GemmEpilogue* epi, int a_format, int b_format,
                    const GemmTail* tail) {
  Fp4GemmDesc d = {a_codes, b_codes, I, J, C, row_amax, col_amax, out, out_f32, epi};
  d.a_format = a_format;
  d.b_format = b_format;
  Problem p;
  int rc = make_problem(ctx, &p, d, gemm_kind, status);
  if (rc != FP4_OK) return rc;
  // The dense tail's operands travel in the slots of a second problem that has no tiles.
  Problem with_tail;
  if (tail) {
    with_tail = p;
    with_tail.args.num_m_blocks = with_tail.args.num_n_blocks = 0;
    rc = make_tail_map(ctx, &with_tail.map_a, tail->a, I, BM);
    if (rc != FP4_OK) return rc;
    rc = make_tail_map(ctx, &with_tail.map_b, tail->b, J, tile_n(gemm_kind));
    if (rc != FP4_OK) return rc;
    p.args.tail_count = tail->count;
  }
  const Problem* second = tail ? &with_tail : nullptr;
  const GemmArgs& args = p.args;
  const int tiles = args.num_m_blocks * args.num_n_blocks;
  const int grid = tiles < ctx->num_sms ? tiles : ctx->num_sms;
  KernelScope scope(ctx, stream, KC_GEMM, 1);
  int rc2;
  if (gemm_kind == FP4_GEMM_F8F6F4)
    rc2 = p.fused ? launch_kernel<FP4_GEMM_F8F6F4, EPI_WGRAD>(grid, stream, p, second)
                  : launch_kernel<FP4_GEMM_F8F6F4, EPI_PLAIN>(grid, stream, p, second);
  else
    rc2 = p.fused ? launch_kernel<FP4_GEMM_MXF4, EPI_WGRAD>(grid, stream, p, second)
                  : launch_kernel<FP4_GEMM_MXF4, EPI_PLAIN>(grid, stream, p, second);
  if (rc2 != FP4_OK) return rc2;
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}

// Two GEMMs in one launch: the tiles of `first` are computed first.  Both
// run through the 16-warp epilogue; a problem without fused work simply has nothing to add.
int launch_gemm_fp4_two(fp4_ctx* ctx, cudaStream_t stream, const Fp4GemmDesc& first, const Fp4GemmDesc& second,
                        int gemm_kind, int32_t* status) {
  Problem p, q;
  int rc = make_problem(ctx, &p, first, gemm_kind, status);
  if (rc != FP4_OK) return rc;
  rc = make_problem(ctx, &q, second, gemm_kind, status);
  if (rc != FP4_OK) return rc;
  const int tiles = p.args.num_m_blocks * p.args.num_n_blocks + q.args.num_m_blocks * q.args.num_n_blocks;
  const int grid = tiles < ctx->num_sms ? tiles : ctx->num_sms;
  KernelScope scope(ctx, stream, KC_GEMM, 1);
  const int rc2 = gemm_kind == FP4_GEMM_F8F6F4 ? launch_kernel<FP4_GEMM_F8F6F4, EPI_WGRAD>(grid, stream, p, &q)
                                                : launch_kernel<FP4_GEMM_MXF4, EPI_WGRAD>(grid, stream, p, &q);
  if (rc2 != FP4_OK) return rc2;
  FP4_CUDA_TRY(cudaGetLastError());
  return FP4_OK;
}
