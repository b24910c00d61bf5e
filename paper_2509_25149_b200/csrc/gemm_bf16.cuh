// BF16 GEMM on CTA pairs (tcgen05 cta_group::2, kind::f16) for the linear layers the recipe leaves in higher
// precision (Section 4.1: the most sensitive layers stay in BF16; Appendix D: every layer late in training).
//   D[M x N] = A * B^T, FP32 accumulation in tensor memory, bf16 or fp32 output, optional accumulation into D.
// Same persistent structure as the block-scaled pair kernel (256 x 256 tiles, each CTA holding its 128 rows of A
// and half of the B tile) minus the scale path; the tensor-memory columns the scales would take hold a second
// accumulator, so a tile's epilogue runs entirely under the next tile's main loop.
//
// Operand layouts.  An operand is "K-major" when the contraction index is contiguous in memory (A stored [M][K],
// B stored [N][K]) and "MN-major" when the output index is (A stored [K][M], B stored [K][N]).  The three GEMMs of a
// layer with row-major X [M x K], W [N x K], dY [M x N] need no transposed copies:
//   Fprop  Y  = X  W^T : A = X  K-major,  B = W  K-major
//   Dgrad  dX = dY W   : A = dY K-major,  B = W  MN-major (contraction over N, W's rows)
//   Wgrad  dW = dY^T X : A = dY MN-major, B = X  MN-major (contraction over the tokens, the rows of both)
// Shared-memory tiles per stage (K = 64 elements): K-major  128 rows x 128 bytes, 128-byte swizzle, 8-row groups
// 1024 bytes apart; MN-major two boxes of 64 k-rows x 128 bytes (64 contiguous output indices each), 8 KB apart.
// One instruction covers K = 16: 32 bytes further along a K-major row, two 8-row groups further in an MN-major box.
// Included by gemm.cu only.
#pragma once

#include "gemm_2cta.cuh"

namespace nvfp4 {
namespace dense {

constexpr int kThreads = 320;       // producer, MMA issuer, 2 x 4 epilogue warps
constexpr int kStages = 6;
constexpr int kOperandBytes = 128 * 128;           // 128 rows (or output indices) x 64 bf16
constexpr int kStageBytes = 2 * kOperandBytes;     // A, this CTA's half of B
constexpr int kStagingBytes = 2 * 16384;
constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024 /*alignment*/ + 256 /*barriers*/;
constexpr uint32_t kTmemCols = 512;                // two 256-column accumulators

struct Args {
  int M, N, K;
  int a_mn, b_mn;  // 1 = the operand is stored with the output index contiguous
  int d_is_fp32, accumulate;
};

// kind::f16 instruction descriptor: FP32 accumulator (bit 4), BF16 x BF16 (format 1 at bits 7 and 10), operand
// major-ness at bits 15 / 16 (0 = K-major), N >> 3 at bit 17, M >> 4 at bit 24
__host__ __device__ constexpr uint32_t instr_desc_bf16(int m, int n, int a_mn, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ void tc2_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
    gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                          const __grid_constant__ CUtensorMap map_d, const __grid_constant__ Args g) {
  using namespace pair;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t staging = base + dense::kStages * dense::kStageBytes;
  const uint32_t bar_base = staging + dense::kStagingBytes;
  constexpr int S = dense::kStages;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };              // leader only: both CTAs' operands landed
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };       // one per CTA
  auto accf_bar = [&](int b) { return bar_base + 8u * (2 * S + b); };    // one per CTA and accumulator
  auto acce_bar = [&](int b) { return bar_base + 8u * (2 * S + 2 + b); };  // leader only, 16 arrivals
  const uint32_t done_bar = bar_base + 8u * (2 * S + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(
      base_ptr + S * dense::kStageBytes + dense::kStagingBytes + 8 * (2 * S + 5));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader
  const bool leader = rank == 0;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  // ragged edges: loads beyond the operands read zeros, stores beyond D are clipped (both by the tensor maps)
  const int tiles_m = (g.M + 255) / 256, tiles_n = (g.N + 255) / 256, n_tiles = tiles_m * tiles_n;
  const int k_blocks = (g.K + 63) / 64;
  // groups of eight row-blocks sweep all column-blocks before the next group starts (L2 reuse of A and B)
  constexpr int kGroupM = 8;
  auto tile_coords = [&](int tile, int& m_blk, int& n_blk) {
    const int per_group = kGroupM * tiles_n;
    const int grp = tile / per_group, in_grp = tile - grp * per_group;
    const int m0 = grp * kGroupM;
    const int gm = (tiles_m - m0 < kGroupM) ? (tiles_m - m0) : kGroupM;
    m_blk = m0 + in_grp % gm;
    n_blk = in_grp / gm;
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 2);  // one arrive.expect_tx from each CTA's producer
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), 1);
      mbar_init(acce_bar(b), 16);  // eight epilogue warps in each CTA
    }
    mbar_init(done_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(dense::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers are initialised before any remote signal
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer ----
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair_id; tile < n_tiles && ok; tile += n_pairs) {
        int m_blk, n_blk;
        tile_coords(tile, m_blk, n_blk);
        const int row_a = m_blk * 256 + (int)rank * 128;  // this CTA's rows of A
        const int row_b = n_blk * 256 + (int)rank * 128;  // this CTA's half of the B tile
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 0x900u + stage))) break;
          const uint32_t st = base + stage * dense::kStageBytes;
          const uint32_t bar = map_to_cta(full_bar(stage), 0);  // the leader's barrier counts both CTAs' operands
          mbar_expect_tx_cluster(bar, dense::kStageBytes);
          if (g.a_mn) {
            tma_load_2d_pair(st, &map_a, row_a, kb * 64, bar);
            tma_load_2d_pair(st + 8192, &map_a, row_a + 64, kb * 64, bar);
          } else {
            tma_load_2d_pair(st, &map_a, kb * 64, row_a, bar);
          }
          if (g.b_mn) {
            tma_load_2d_pair(st + dense::kOperandBytes, &map_b, row_b, kb * 64, bar);
            tma_load_2d_pair(st + dense::kOperandBytes + 8192, &map_b, row_b + 64, kb * 64, bar);
          } else {
            tma_load_2d_pair(st + dense::kOperandBytes, &map_b, kb * 64, row_b, bar);
          }
          if (++stage == S) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (leader) ----
    if (leader && lane == 0) {
      int stage = 0;
      uint32_t phase = 0, acc_phase = 0;  // bit b: phase of accumulator b's barrier
      bool ok = true;
      const uint32_t idesc = instr_desc_bf16(256, 256, g.a_mn, g.b_mn);
      // descriptor halves: start address and leading byte offset (low word), stride byte offset / version /
      // 128-byte swizzle (high word).  K-major: 8-row groups 1024 bytes apart, leading offset unused.  MN-major:
      // 64-index boxes 8192 bytes apart (leading), 8-row k groups 1024 bytes apart (stride).
      const uint32_t a_lo0 = ((base >> 4) & 0x3fffu) | ((g.a_mn ? (8192u >> 4) : 1u) << 16);
      const uint32_t b_lo0 = (((base + dense::kOperandBytes) >> 4) & 0x3fffu) | ((g.b_mn ? (8192u >> 4) : 1u) << 16);
      const uint32_t a_step = g.a_mn ? (2048u >> 4) : (32u >> 4);  // one K = 16 instruction further
      const uint32_t b_step = g.b_mn ? (2048u >> 4) : (32u >> 4);
      int it = 0;
      for (int tile = pair_id; tile < n_tiles && ok; tile += n_pairs, ++it) {
        const int buf = it & 1;
        if (!(ok = mbar_wait_cluster(acce_bar(buf), ((acc_phase >> buf) & 1u) ^ 1u, abort_flag, 0xB00u + buf))) break;
        tc_fence_after();
        const uint32_t d_t = tmem + buf * 256;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait_cluster(full_bar(stage), phase, abort_flag, 0xA00u + stage))) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + stage * (dense::kStageBytes >> 4);
          const uint32_t b_lo = b_lo0 + stage * (dense::kStageBytes >> 4);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            tc2_mma_bf16(d_t, make_desc(a_lo + j * a_step, kDescHiOperand), make_desc(b_lo + j * b_step, kDescHiOperand),
                         idesc, (kb > 0 || j > 0) ? 1u : 0u);
          tc2_commit_both(empty_bar(stage), 3);  // both CTAs' stages are free once these MMAs have read them
          if (++stage == S) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        tc2_commit_both(accf_bar(buf), 3);  // this accumulator is complete in both CTAs
        acc_phase ^= 1u << buf;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2-9) ----
    const int quad = warp & 3;              // tensor-memory lanes this warp may read
    const int half = (warp - 2) >> 2;       // column half / epilogue group
    const int et = (threadIdx.x - 64) & 127;  // 0..127 inside the group
    const int bar_id = 1 + half;
    uint32_t acc_phase = 0;
    const int row_in_tile = quad * 32 + lane;
    const uint32_t stage_buf = staging + half * 16384;
    int it = 0;
    for (int tile = pair_id; tile < n_tiles; tile += n_pairs, ++it) {
      const int buf = it & 1;
      int m_blk, n_blk;
      tile_coords(tile, m_blk, n_blk);
      mbar_wait_cluster(accf_bar(buf), (acc_phase >> buf) & 1u, abort_flag, 0xC00u + buf);
      // agree on giving up: a warp that timed out still joins this barrier, and all 128 threads take ONE decision
      if (group_gave_up(abort_flag, bar_id, 128)) break;
      tc_fence_after();
      const int row0 = m_blk * 256 + (int)rank * 128;
      const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16) + buf * 256 + half * 128;
      uint32_t r[128];
#pragma unroll
      for (int q = 0; q < 8; ++q) tc_ld16(t_row + q * 16, *reinterpret_cast<uint32_t(*)[16]>(&r[q * 16]));
      tc_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(acce_bar(buf), 0));
      if (g.d_is_fp32)
        store_half<true>(r, 1.0f, et, bar_id, row_in_tile, stage_buf, &map_d, n_blk * 256 + half * 128, row0,
                         g.accumulate);
      else
        store_half<false>(r, 1.0f, et, bar_id, row_in_tile, stage_buf, &map_d, n_blk * 256 + half * 128, row0,
                          g.accumulate);
      acc_phase ^= 1u << buf;
    }
    if (et == 0) bulk_wait_all<0>();  // all stores have left shared memory and are visible
  }

  // ------------------------------------------------------------------ teardown ----
  // Neither CTA may leave while the other can still signal its barriers or read its shared memory.
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    mbar_arrive_cluster(map_to_cta(done_bar, rank ^ 1u));
    mbar_wait_cluster(done_bar, 0, abort_flag, 0xD00u);
  }
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 100; ++i) __nanosleep(1000);
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(dense::kTmemCols) : "memory");
  }
}

}  // namespace dense
}  // namespace nvfp4
