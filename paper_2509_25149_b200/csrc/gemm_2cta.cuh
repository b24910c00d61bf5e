// Block-scaled NVFP4 GEMM on CTA pairs (tcgen05 cta_group::2): a cluster of two CTAs on one TPC computes a
// 256 x 256 output tile.  Each CTA keeps its own 128 rows of A, HALF of the B tile (128 of its 256 rows) and the
// accumulator of its 128 output rows in its own tensor memory; the pair's tensor cores exchange the B halves, so
// every byte of B is fetched from L2 and read from shared memory once per pair.  That halving of the operand
// traffic per flop is the point: the one-CTA kernel is bound by shared-memory bandwidth, not by the tensor pipe.
//
// Roles per CTA (14 warps): 0 TMA producer (both CTAs; every load signals the LEADER's "full" barrier),
// 1 MMA issuer (leader only; allocates tensor memory in both), 2 and 11-13 scale warps (both CTAs; shared memory ->
// registers -> tensor memory, one warp per 32-lane quadrant), 3-10 epilogue (both; two groups of four warps, one per
// 128-column half: tensor memory -> registers -> swizzled staging -> TMA store; the accumulator is released as
// soon as it has been read).
// Included by gemm.cu only.
#pragma once

#include <cuda_bf16.h>

#include "gemm.h"
#include "tc_ptx.cuh"

namespace nvfp4 {
namespace pair {

constexpr int kThreads = 448;      // producer, MMA, 2 x 4 epilogue warps, 4 scale warps (2, 11, 12, 13)
constexpr int kStages = 5;
constexpr int kABytes = 128 * 128;   // 128 rows x 256 K elements
constexpr int kBBytes = 128 * 128;   // this CTA's half of the 256-row B tile
constexpr int kSfaBytes = 4 * 512;   // own 128 rows, four K64 steps
constexpr int kSfbBytes = 8 * 512;   // all 256 rows of B (both CTAs need them), four K64 steps
constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;  // 38 KB
constexpr int kStagingBytes = 2 * 16384;  // one 128 x 128-byte store buffer per epilogue group
constexpr int kBetaBytes = 2 * 128 * 4;   // column scales of the tile, one half per epilogue group (row-scaled B)
constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024 /*alignment*/ + 256 /*barriers*/ + kBetaBytes;
constexpr uint32_t kTmemCols = 512;
constexpr int kSfCol = 256;          // after the 256 accumulator columns: one 48-column slot per stage
constexpr int kSfSlotCols = 48;      // SFA 4 x 4, SFB 4 x 8
static_assert(kSfCol + kStages * kSfSlotCols <= 512, "tensor memory budget");
static_assert(kStageBytes % 1024 == 0, "stages must keep the 1024-byte swizzle alignment");

struct Problem {
  int M, N, K;
  const uint8_t* sfa;  // swizzled scale atoms of A and B (global memory)
  const uint8_t* sfb;
  const float* a_global;
  const float* b_global;
  int d_is_fp32, accumulate;
  // Global scale per row instead of per tensor (Appendix B.1, closing remark): {amax, s_dec} pairs, one per row of
  // the operand; NULL = the operand carries the usual per-tensor words in a_global / b_global
  const float* a_rows;
  const float* b_rows;
};
// One launch works through the tiles of up to two independent GEMMs (problem 0 first): Dgrad and Wgrad of a
// linear layer share no output, so their tiles can fill the same persistent grid and the partial last round of
// the first problem is not paid twice.
struct Args {
  Problem p[2];
  int n_tiles0;  // tiles of problem 0
  int n_tiles;   // tiles of both problems
  // Measurement aids (0 / NULL in normal operation).  exp: bit 0 = the issuer skips the MMAs, bit 1 = the producer
  // skips the operand loads, bit 2 = scale atoms are neither loaded nor copied to tensor memory, bit 3 = the epilogue hands the
  // accumulator back unread and stores nothing, bit 4 = the issuer does not wait for the accumulator (results are
  // meaningless with any bit set; the barriers are signalled as usual).  probe: per pair eight 64-bit words, five
  // written by the issuer: SM cycles and nanoseconds of its main loop, k-blocks and tiles it went through, and the
  // cycles it spent, after issuing a tile's last MMA, waiting for the accumulator to be handed back.
  int exp;
  unsigned long long* probe;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  // default semantics: the explicitly cluster-scoped release form costs ~0.5 us per call on this part, and the
  // tensor-memory accesses this arrival orders are already fenced with tcgen05.fence::before_thread_sync
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded wait with cluster-scope acquire (the barrier receives arrivals from the peer CTA)
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                  uint32_t code) {
  if (mbar_try_cluster(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_cluster(bar, parity)) return true;
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = code;
        atomicCAS(&g_device_status, 0u, code);
        return false;
      }
    }
  }
}

// pair-aware TMA load: the data lands in this CTA's shared memory, the bytes are counted on `bar`, which may be
// the peer's barrier (cluster address)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x), "r"(y),
               "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map),
               "r"(x), "r"(y), "r"(src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_all() {
  asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void tc2_commit_local(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// arrives on the barrier at the same offset in every CTA of `mask` once all earlier tcgen05 operations of the
// issuing thread have completed
__device__ __forceinline__ void tc2_commit_both(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask)
               : "memory");
}
// registers -> tensor memory: this warp's 32 lanes x 16 consecutive columns
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
// one 512-byte scale atom (32 rows x 16 bytes) shared memory -> four columns of tensor memory, replicated to the four
// lane quadrants, in both CTAs of the pair (each from its own shared memory at the same offset)
__device__ __forceinline__ void tc2_cp_sf(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tc2_mma_nvf4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                             uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tc2_mma_mxf4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                             uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate)
      : "memory");
}

// Epilogue helper: 128 accumulator columns of one row per thread (registers) -> alpha, conversion -> 128-byte
// swizzled rows of the group's staging buffer -> TMA store (or reduce-add) of 128 x 128-byte boxes.  A group has
// ONE 16 KB buffer: a chunk is converted only after the store of the previous chunk has finished reading it.
// BETA: the 128 columns additionally carry their own factors (float[128] in shared memory at `beta`).
template <bool FP32, bool BETA = false>
__device__ __forceinline__ void store_half(const uint32_t (&r)[128], float alpha, int et, int bar_id, int row_in_tile,
                                           uint32_t stage_buf, const CUtensorMap* map_d, int x0, int row0,
                                           int accumulate, const float* beta = nullptr, int skip = 0) {
  // skip (measurement aid): bit 0 = the converted values are not written to the staging buffer, bit 1 = no TMA store
  constexpr int kChunks = FP32 ? 4 : 2;
  constexpr int kChunkCols = FP32 ? 32 : 64;
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    if (et == 0) bulk_wait_read<0>();
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    const uint32_t srow = stage_buf + row_in_tile * 128;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      uint32_t p[4];
      if (FP32) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = __uint_as_float(r[c * 32 + 4 * j + e]) * alpha;
          if (BETA) v *= beta[c * 32 + 4 * j + e];
          p[e] = __float_as_uint(v);
        }
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v0 = __uint_as_float(r[c * 64 + 8 * j + 2 * e]) * alpha;
          float v1 = __uint_as_float(r[c * 64 + 8 * j + 2 * e + 1]) * alpha;
          if (BETA) {
            v0 *= beta[c * 64 + 8 * j + 2 * e];
            v1 *= beta[c * 64 + 8 * j + 2 * e + 1];
          }
          __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
          p[e] = *reinterpret_cast<uint32_t*>(&h);
        }
      }
      if (!(skip & 1) || (p[0] ^ p[1] ^ p[2] ^ p[3]) == 0x9E3779B9u)  // (the aid keeps the conversion alive)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(srow + ((j ^ (row_in_tile & 7)) << 4)), "r"(p[0]),
                     "r"(p[1]), "r"(p[2]), "r"(p[3])
                     : "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    if (et == 0 && !(skip & 2)) {
      if (accumulate)
        tma_reduce_add_2d(map_d, x0 + c * kChunkCols, row0, stage_buf);
      else
        tma_store_2d(map_d, x0 + c * kChunkCols, row0, stage_buf);
      bulk_commit();
    }
  }
}

// MX = false: NVFP4 (E4M3 scale per 16 elements: one 512-byte atom per 128 rows and K = 64).
// MX = true : MXFP4 (UE8M0 scale per 32 elements: one atom per 128 rows and K = 128, so half the atoms, the same
//             slots in shared and tensor memory half used, and the byte pair picked by the instruction descriptor).
// ROWS = true: at least one operand carries its global scale per row (a_rows / b_rows); the epilogue then applies a
// factor per output row and / or per output column.  A separate instantiation so that the common kernel keeps its
// register budget.
template <bool MX, bool ROWS = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
    gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_b0,
                     const __grid_constant__ CUtensorMap map_d0, const __grid_constant__ CUtensorMap map_a1,
                     const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_d1,
                     const __grid_constant__ Args g) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t staging = base + kStages * kStageBytes;
  const uint32_t bar_base = staging + kStagingBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };                  // leader only: both CTAs' operands landed
  auto sff_bar = [&](int s) { return bar_base + 8u * (kStages + s); };       // leader only: scales of both CTAs in TMEM
  auto empty_bar = [&](int s) { return bar_base + 8u * (2 * kStages + s); }; // one per CTA
  auto sfl_bar = [&](int s) { return bar_base + 8u * (3 * kStages + s); };   // one per CTA: own scale atoms landed
  const uint32_t accf_bar = bar_base + 8u * (4 * kStages);                   // one per CTA
  const uint32_t acce_bar = bar_base + 8u * (4 * kStages + 1);               // leader only, 16 arrivals
  const uint32_t done_bar = bar_base + 8u * (4 * kStages + 2);               // one per CTA, peer arrives
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(base_ptr + kStages * kStageBytes + kStagingBytes + 8 * (4 * kStages + 3));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader
  const bool leader = rank == 0;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_tiles = g.n_tiles;
  // Tile order inside a problem: groups of kGroupM row-blocks sweep all column-blocks before the next group
  // starts, so the group's rows of A and all of B stay in L2 while they are reused.
  constexpr int kGroupM = 8;
  auto tile_coords = [&](int tile, int& prob, int& m_blk, int& n_blk) {
    prob = tile >= g.n_tiles0 ? 1 : 0;
    if (prob) tile -= g.n_tiles0;
    const int tiles_m = g.p[prob].M / 256, tiles_n = g.p[prob].N / 256;
    const int per_group = kGroupM * tiles_n;
    const int grp = tile / per_group, in_grp = tile - grp * per_group;
    const int m0 = grp * kGroupM;
    const int gm = (tiles_m - m0 < kGroupM) ? (tiles_m - m0) : kGroupM;
    m_blk = m0 + in_grp % gm;
    n_blk = in_grp / gm;
  };
  auto k_blocks_of = [&](int tile) { return g.p[tile >= g.n_tiles0 ? 1 : 0].K / 256; };
  // Tiles go to the pairs in rounds, odd rounds in reverse pair order (a snake): with two problems of different
  // depth in one launch, the pairs that drew the deeper or the extra tiles of one round draw the shallower ones, or
  // none, in the next.  A balance measure only: on one problem it times the same as the plain round-robin.
  auto next_tile = [&](int rnd) { return rnd * n_pairs + ((rnd & 1) ? n_pairs - 1 - pair_id : pair_id); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 2);   // one arrive.expect_tx from each CTA's producer
      mbar_init(sff_bar(s), 8);    // four scale warps in each CTA
      mbar_init(empty_bar(s), 1);
      mbar_init(sfl_bar(s), 1);
    }
    mbar_init(accf_bar, 1);
    mbar_init(acce_bar, 16);       // eight epilogue warps in each CTA
    mbar_init(done_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers are initialised before any remote signal
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // Launched behind the quantizer of the same call, the CTA reaches this point while that kernel still runs: from
  // here on every role touches what it wrote (operands, scales, global scales), so all of them wait for it to end.
  griddep_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer ----
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int rnd = 0, tile = pair_id; tile < n_tiles && ok; tile = next_tile(++rnd)) {
        int prob, m_blk, n_blk;
        tile_coords(tile, prob, m_blk, n_blk);
        const Problem& pr = g.p[prob];
        const CUtensorMap* map_a = prob ? &map_a1 : &map_a0;
        const CUtensorMap* map_b = prob ? &map_b1 : &map_b0;
        const int k_blocks = pr.K / 256;
        const int sf_atoms_k = pr.K / (MX ? 128 : 64);  // atoms along K per 128-row group
        constexpr int kAtomsKb = MX ? 2 : 4;              // atoms per 256-deep k-block and 128-row group
        const int row_a = m_blk * 256 + (int)rank * 128;       // this CTA's A rows
        const int row_b = n_blk * 256 + (int)rank * 128;       // this CTA's half of the B tile
        const uint8_t* sfa = pr.sfa + (int64_t)(m_blk * 2 + (int)rank) * sf_atoms_k * 512;  // own 128 rows
        const uint8_t* sfb = pr.sfb + (int64_t)(n_blk * 2) * sf_atoms_k * 512;               // all 256 rows of B
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 0x100u + stage))) break;
          const uint32_t st = base + stage * kStageBytes;
          const uint32_t bar = map_to_cta(full_bar(stage), 0);  // the leader's barrier counts both CTAs' operands
          if (g.exp & 2) {
            mbar_expect_tx_cluster(bar, 0);  // measurement aid: no operand loads
          } else {
            mbar_expect_tx_cluster(bar, kABytes + kBBytes);
            tma_load_2d_pair(st, map_a, kb * 128, row_a, bar);
            tma_load_2d_pair(st + kABytes, map_b, kb * 128, row_b, bar);
          }
          // scale atoms: plain bulk copies counted on this CTA's own barrier (its scale warps wait on it)
          if (g.exp & 4) {
            mbar_expect_tx(sfl_bar(stage), 0);  // measurement aid: no scale loads
          } else {
            mbar_expect_tx(sfl_bar(stage), 3 * kAtomsKb * 512);
            bulk_load(st + kABytes + kBBytes, sfa + (int64_t)kb * kAtomsKb * 512, kAtomsKb * 512, sfl_bar(stage));
            bulk_load(st + kABytes + kBBytes + kSfaBytes, sfb + (int64_t)kb * kAtomsKb * 512, kAtomsKb * 512,
                      sfl_bar(stage));
            bulk_load(st + kABytes + kBBytes + kSfaBytes + 2048, sfb + ((int64_t)sf_atoms_k + kb * kAtomsKb) * 512,
                      kAtomsKb * 512, sfl_bar(stage));
          }
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 2 || warp >= 11) {
    // ------------------------------- scale atoms: shared memory -> registers -> tensor memory (both CTAs) ----
    // One warp per 32-lane quadrant of tensor memory (warps 2, 11, 12, 13 -> quadrants 2, 3, 0, 1).  Lane l of
    // every quadrant holds row l of each 512-byte atom: columns [4j, 4j+4) of the stage's slot for SFA of K64-step
    // j, columns [16 + 8j + 4g, ..) for SFB of step j and 128-row group g.  The tensor-memory copy engine
    // (tcgen05.cp) moves one atom per instruction and was the bottleneck of the main loop; twelve 16-byte loads
    // and three tcgen05.st per warp do the same work off the critical path.
    const int quad = warp & 3;
    int stage = 0;
    uint32_t phase = 0;
    const uint32_t sff_leader = map_to_cta(sff_bar(0), 0);
    for (int rnd = 0, tile = pair_id; tile < n_tiles; tile = next_tile(++rnd)) {
      bool ok = true;
      const int k_blocks = k_blocks_of(tile);
      for (int kb = 0; kb < k_blocks; ++kb) {
        ok = mbar_wait(sfl_bar(stage), phase, abort_flag, 0x500u + stage);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        if (g.exp & (4 | 32)) {  // measurement aids: no scale copies / the issuer copies, this warp only relays
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(sff_leader + 8u * stage);
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
          continue;
        }
        const uint32_t sf_s = base + stage * kStageBytes + kABytes + kBBytes + lane * 16;
        uint32_t r[48];
        constexpr int kAtomsKb = MX ? 2 : 4;  // atoms per k-block and 128-row group
#pragma unroll
        for (int j = 0; j < kAtomsKb; ++j) {
          const uint4 a = lds128(sf_s + j * 512);
          r[4 * j] = a.x; r[4 * j + 1] = a.y; r[4 * j + 2] = a.z; r[4 * j + 3] = a.w;
        }
        const uint32_t sf_t = tmem + ((uint32_t)(quad * 32) << 16) + kSfCol + stage * kSfSlotCols;
#pragma unroll
        for (int j = 0; j < kAtomsKb; ++j)
#pragma unroll
          for (int grp = 0; grp < 2; ++grp) {
            const uint4 b = lds128(sf_s + kSfaBytes + grp * 2048 + j * 512);
            r[16 + 8 * j + 4 * grp] = b.x; r[16 + 8 * j + 4 * grp + 1] = b.y;
            r[16 + 8 * j + 4 * grp + 2] = b.z; r[16 + 8 * j + 4 * grp + 3] = b.w;
          }
        if (MX) {
          asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(sf_t), "r"(r[0]),
                       "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                       : "memory");
          tc_st16(sf_t + 16, &r[16]);
        } else {
          tc_st16(sf_t, &r[0]);
          tc_st16(sf_t + 16, &r[16]);
          tc_st16(sf_t + 32, &r[32]);
        }
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(sff_leader + 8u * stage);
        if (++stage == kStages) {
          stage = 0;
          phase ^= 1u;
        }
      }
      if (!ok) break;
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (leader) ----
    if (leader && lane == 0) {
      int stage = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      constexpr uint32_t idesc = instr_desc_nvf4(256, 256);
      constexpr uint32_t idesc_mx[2] = {instr_desc_mxf4(256, 256, 0), instr_desc_mxf4(256, 256, 2)};
      const uint32_t a_lo0 = ((base >> 4) & 0x3fffu) | (1u << 16);
      const uint32_t b_lo0 = (((base + kABytes) >> 4) & 0x3fffu) | (1u << 16);
      const long long probe_c0 = g.probe ? clock64() : 0;
      const unsigned long long probe_t0 = g.probe ? globaltimer_ns() : 0;
      unsigned long long probe_kb = 0, probe_tiles = 0;
      long long probe_wait = 0, probe_mark = probe_c0;  // cycles spent waiting for the accumulator to be handed back
      for (int rnd = 0, tile = pair_id; tile < n_tiles && ok; tile = next_tile(++rnd)) {
        if (!(g.exp & 16) && !(ok = mbar_wait_cluster(acce_bar, acc_phase ^ 1u, abort_flag, 0x300u))) break;
        if (g.probe) probe_wait += clock64() - probe_mark;
        tc_fence_after();
        const int k_blocks = k_blocks_of(tile);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait_cluster(full_bar(stage), phase, abort_flag, 0x200u + stage))) break;
          if (!(ok = mbar_wait_cluster(sff_bar(stage), phase, abort_flag, 0x280u + stage))) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + stage * (kStageBytes >> 4);
          const uint32_t b_lo = b_lo0 + stage * (kStageBytes >> 4);
          const uint32_t sf_t = tmem + kSfCol + stage * kSfSlotCols;
          if (g.exp & 32) {  // measurement aid: the scale atoms go through the copy engine, issued here
            const uint32_t sf_lo = (((base + kABytes + kBBytes) >> 4) & 0x3fffu) + stage * (kStageBytes >> 4);
            constexpr int kAtomsKb = MX ? 2 : 4;
#pragma unroll
            for (int j = 0; j < kAtomsKb; ++j) {
              tc2_cp_sf(sf_t + j * 4, make_desc(sf_lo + j * 32, kDescHiSf));
#pragma unroll
              for (int grp = 0; grp < 2; ++grp)
                tc2_cp_sf(sf_t + 16 + 8 * j + 4 * grp, make_desc(sf_lo + (kSfaBytes >> 4) + grp * 128 + j * 32, kDescHiSf));
            }
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (g.exp & 1) break;  // measurement aid: no MMAs
            if (MX)  // one atom (4 columns) serves two K = 64 steps: bytes 0-1, then bytes 2-3
              tc2_mma_mxf4(tmem, make_desc(a_lo + 2 * j, kDescHiOperand), make_desc(b_lo + 2 * j, kDescHiOperand),
                           idesc_mx[j & 1], sf_t + (j >> 1) * 4, sf_t + 16 + (j >> 1) * 8, (kb > 0 || j > 0) ? 1u : 0u);
            else
              tc2_mma_nvf4(tmem, make_desc(a_lo + 2 * j, kDescHiOperand), make_desc(b_lo + 2 * j, kDescHiOperand), idesc,
                           sf_t + j * 4, sf_t + 16 + j * 8, (kb > 0 || j > 0) ? 1u : 0u);
          }
          tc2_commit_both(empty_bar(stage), 3);  // both CTAs' stages are free once these MMAs have read them
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        tc2_commit_both(accf_bar, 3);  // accumulators of both CTAs complete
        acc_phase ^= 1u;
        probe_kb += (unsigned long long)k_blocks;
        ++probe_tiles;
        if (g.probe) probe_mark = clock64();
      }
      if (g.probe) {
        // the last commit has been issued, not completed: wait for the accumulator hand-over of the last tile so that
        // the interval covers the work (bounded like every other wait)
        mbar_wait_cluster(acce_bar, acc_phase ^ 1u, abort_flag, 0x380u);
        probe_wait += clock64() - probe_mark;
        g.probe[8 * pair_id] = (unsigned long long)(clock64() - probe_c0);
        g.probe[8 * pair_id + 1] = globaltimer_ns() - probe_t0;
        g.probe[8 * pair_id + 2] = probe_kb;
        g.probe[8 * pair_id + 3] = probe_tiles;
        g.probe[8 * pair_id + 4] = (unsigned long long)probe_wait;
      }
    }
  } else if (warp >= 3 && warp <= 10) {
    // ------------------------------------------------------------------ epilogue ----
    // Two groups of four warps; group h drains columns [128h, 128h + 128) of the accumulator through its own
    // pair of staging buffers, so the two halves leave tensor memory concurrently.
    const int quad = warp & 3;              // tensor-memory lanes this warp may read
    const int half = (warp - 3) >> 2;       // column half / epilogue group
    const int et = (threadIdx.x - 96) & 127;  // 0..127 inside the group
    const int bar_id = 1 + half;
    uint32_t acc_phase = 0;
    // per-tensor decode scales; an operand with per-row scales contributes 1 here and its vector below
    const float alpha0 = __fmul_rn((ROWS && g.p[0].a_rows) ? 1.f : g.p[0].a_global[1], (ROWS && g.p[0].b_rows) ? 1.f : g.p[0].b_global[1]);
    const float alpha1 = __fmul_rn((ROWS && g.p[1].a_rows) ? 1.f : g.p[1].a_global[1], (ROWS && g.p[1].b_rows) ? 1.f : g.p[1].b_global[1]);
    float* beta = reinterpret_cast<float*>(base_ptr + kStages * kStageBytes + kStagingBytes + 256) + half * 128;
    const uint32_t acce_leader = map_to_cta(acce_bar, 0);
    const int row_in_tile = quad * 32 + lane;
    const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16) + half * 128;
    const uint32_t stage_buf = staging + half * 16384;
    for (int rnd = 0, tile = pair_id; tile < n_tiles; tile = next_tile(++rnd)) {
      int prob, m_blk, n_blk;
      tile_coords(tile, prob, m_blk, n_blk);
      const CUtensorMap* map_d = prob ? &map_d1 : &map_d0;
      float alpha = prob ? alpha1 : alpha0;
      const int d_is_fp32 = g.p[prob].d_is_fp32, accumulate = g.p[prob].accumulate;
      const float* a_rows = ROWS ? g.p[prob].a_rows : nullptr;
      const float* b_rows = ROWS ? g.p[prob].b_rows : nullptr;
      if (a_rows) alpha *= a_rows[2 * (int64_t)(m_blk * 256 + (int)rank * 128 + quad * 32 + lane) + 1];
      // the group's 128 column factors; the first barrier inside store_half orders this write before their use, its
      // last one orders their use before the next tile's write
      if (b_rows) beta[et] = b_rows[2 * (int64_t)(n_blk * 256 + half * 128 + et) + 1];
      mbar_wait_cluster(accf_bar, acc_phase, abort_flag, 0x400u);
      // agree on giving up: a warp that timed out still joins this barrier, and all 128 threads take ONE decision
      if (group_gave_up(abort_flag, bar_id, 128)) break;
      tc_fence_after();
      if (g.exp & 8) {  // measurement aid: the accumulator is handed back unread, nothing is stored
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acce_leader);
        acc_phase ^= 1u;
        continue;
      }
      const int row0 = m_blk * 256 + (int)rank * 128;
      // read this warp's 32 lanes x 128 columns in one go and hand the accumulator back at once: the MMA issuer
      // can start the next tile while the values are converted and stored from registers
      uint32_t r[128];
      // sixteen columns per load: measured per tile 1830 cycles of hand-over with x16 loads against 2400 with x32
      // and 3500 with x64 (wider loads want longer runs of consecutive registers)
#pragma unroll
      for (int q = 0; q < 8; ++q) tc_ld16(t_row + q * 16, *reinterpret_cast<uint32_t(*)[16]>(&r[q * 16]));
      tc_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acce_leader);
      if (ROWS && b_rows) {
        if (d_is_fp32)
          store_half<true, true>(r, alpha, et, bar_id, row_in_tile, stage_buf, map_d, n_blk * 256 + half * 128,
                                 row0, accumulate, beta);
        else
          store_half<false, true>(r, alpha, et, bar_id, row_in_tile, stage_buf, map_d, n_blk * 256 + half * 128,
                                  row0, accumulate, beta);
      } else if (d_is_fp32) {
        store_half<true>(r, alpha, et, bar_id, row_in_tile, stage_buf, map_d, n_blk * 256 + half * 128, row0,
                         accumulate, nullptr, (g.exp >> 6) & 3);
      } else {
        store_half<false>(r, alpha, et, bar_id, row_in_tile, stage_buf, map_d, n_blk * 256 + half * 128, row0,
                          accumulate, nullptr, (g.exp >> 6) & 3);
      }
      acc_phase ^= 1u;
    }
    if (et == 0) bulk_wait_all<0>();  // all stores have left shared memory and are visible
  }

  // ------------------------------------------------------------------ teardown ----
  // Neither CTA may leave while the other can still signal its barriers or read its shared memory: each tells
  // the peer it is done and waits (bounded) for the peer's word.
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    mbar_arrive_cluster(map_to_cta(done_bar, rank ^ 1u));
    mbar_wait_cluster(done_bar, 0, abort_flag, 0x600u);
  }
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 100; ++i) __nanosleep(1000);
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

}  // namespace pair
}  // namespace nvfp4
