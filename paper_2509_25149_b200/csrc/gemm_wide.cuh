// Block-scaled FP4 GEMM on CTA pairs with 256 x 384 output tiles.
//
// The largest tile a CTA pair can hold: tensor memory has 512 columns, enough for a 384-column FP32 accumulator plus
// two 64-column slots for the scale factors.  A 256 x 384 tile moves (256 + 384) / (256 * 384) operand rows per
// output, 17 % less than the 256 x 256 tile of gemm_2cta.cuh, and has a third fewer accumulator hand-overs per
// output.  With all 148 SMs on the tensor pipe the part is power-capped, so less data movement per flop shows up as
// a little more clock rather than as a shorter k-block; the price is a coarser schedule, which is why the host
// picks the tile width per problem from an estimate of the schedule.  N is cut into 384-wide tiles plus zero, one
// or two 256-wide ones (N = 128 q = 384 a + 256 b); both widths run through the same code.
//
// Per K = 64 step the 384 columns take two instructions (N = 256 and N = 128; the B tile of a CTA is its 128 rows
// of the first 256 and its 64 rows of the last 128).  Roles as in the pair kernel; differences:
//   - four stages of 48 KB (A 16, B 24, scale atoms 8);
//   - the scale slots in tensor memory are a ring of two, freed by the same event that frees the shared-memory
//     stage of two k-blocks earlier (the scale warps wait on that stage's "empty" barrier);
//   - the epilogue drains its half of the tile in passes of 64 columns (3 or 2), releasing the accumulator after
//     the last read, and stores each pass through its staging buffer with TMA (fp32 outputs: in 64-byte-wide chunks
//     through the two halves of the buffer in turn, so that no chunk waits for the store of the chunk before it).
// Included by gemm.cu only.
#pragma once

#include "gemm_2cta.cuh"

namespace nvfp4 {
namespace wide {

using namespace pair;  // PTX wrappers and cluster helpers

constexpr int kWThreads = 448;  // producer, MMA, 2 x 4 epilogue warps, 4 scale warps (2, 11, 12, 13)
constexpr int kWStages = 4;
constexpr int kWABytes = 128 * 128;   // 128 rows x 256 K elements
constexpr int kWBBytes = 192 * 128;   // this CTA's rows of the B tile: 128 of the first 256 + 64 of the last 128
constexpr int kWSfaBytes = 4 * 512;
constexpr int kWSfbBytes = 12 * 512;  // three 128-row groups x four K64 steps
constexpr int kWStageBytes = kWABytes + kWBBytes + kWSfaBytes + kWSfbBytes;  // 48 KB
constexpr int kWStagingBytes = 2 * 16384;
constexpr int kWSmemBytes = kWStages * kWStageBytes + kWStagingBytes + 1024 /*alignment*/ + 256 /*barriers*/;
constexpr uint32_t kWTmemCols = 512;
constexpr int kWSfCol = 384;      // after the accumulator columns
constexpr int kWSfSlotCols = 64;  // SFA 4 x 4, SFB 4 x 12
static_assert(kWSfCol + 2 * kWSfSlotCols <= 512, "tensor memory budget");
static_assert(kWStageBytes % 1024 == 0, "stages must keep the 1024-byte swizzle alignment");
static_assert(kWSmemBytes <= 232448, "shared memory budget");

struct WProblem {
  int M, N, K;
  const uint8_t* sfa;
  const uint8_t* sfb;
  const float* a_global;
  const float* b_global;
  int d_is_fp32, accumulate;
  int n_wide;   // 384-wide column tiles (they come first)
  int tiles_n;  // all column tiles
};
struct WArgs {
  WProblem p[2];
  int n_tiles0;  // tiles of problem 0
  int n_tiles;   // tiles of both problems
};

// 64 accumulator columns of one row per thread -> alpha, conversion -> swizzled staging -> TMA store / reduce-add.
// bf16: one chunk of 128-byte rows through the group's 16 KB buffer, converted once the store issued before it has
// finished reading the buffer.
// fp32: four chunks of 64-byte rows (16 columns) through the two 8 KB halves of the same buffer in turn: before a chunk
// is written, the store issued from its half two chunks ago has finished reading it, while the latest store (from the
// other half) may still be in flight, so the tensor-memory reads between the chunks do not wait for a store.  (The same
// scheme for bf16 outputs, with 32-column chunks, was measured slower than the single buffer: twice the barriers and
// stores of half the width.)  n_chunks counts the group's fp32 chunks; the caller drains all stores before a tile.
template <bool FP32>
__device__ __forceinline__ void store_cols64(const uint32_t (&r)[64], float alpha, int et, int bar_id, int row_in_tile,
                                             uint32_t stage_buf16k, uint32_t& n_chunks, const CUtensorMap* map_d, int x0,
                                             int row0, int accumulate) {
  if (FP32) {
#pragma unroll
    for (int c = 0; c < 4; ++c, ++n_chunks) {
      const uint32_t stage_buf = stage_buf16k + (n_chunks & 1u) * 8192u;
      if (et == 0) bulk_wait_read<1>();
      asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
      const uint32_t srow = stage_buf + row_in_tile * 64;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t p[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) p[e] = __float_as_uint(__uint_as_float(r[c * 16 + 4 * j + e]) * alpha);
        // 64-byte swizzle: the 16-byte unit index is XORed with bits 7-8 of the address, i.e. with (row >> 1) & 3
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(srow + ((j ^ ((row_in_tile >> 1) & 3)) << 4)),
                     "r"(p[0]), "r"(p[1]), "r"(p[2]), "r"(p[3])
                     : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
      if (et == 0) {
        if (accumulate)
          tma_reduce_add_2d(map_d, x0 + c * 16, row0, stage_buf);
        else
          tma_store_2d(map_d, x0 + c * 16, row0, stage_buf);
        bulk_commit();
      }
    }
  } else {
    if (et == 0) bulk_wait_read<0>();  // the store issued from this buffer before has finished reading it
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    const uint32_t srow = stage_buf16k + row_in_tile * 128;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      uint32_t p[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * j + 2 * e]) * alpha,
                                                 __uint_as_float(r[8 * j + 2 * e + 1]) * alpha);
        p[e] = *reinterpret_cast<uint32_t*>(&h);
      }
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(srow + ((j ^ (row_in_tile & 7)) << 4)), "r"(p[0]),
                   "r"(p[1]), "r"(p[2]), "r"(p[3])
                   : "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    if (et == 0) {
      tma_store_2d(map_d, x0, row0, stage_buf16k);
      bulk_commit();
    }
  }
}

template <bool MX>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kWThreads, 1)
    gemm_wide_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_b0,
                     const __grid_constant__ CUtensorMap map_c0, const __grid_constant__ CUtensorMap map_d0,
                     const __grid_constant__ CUtensorMap map_a1, const __grid_constant__ CUtensorMap map_b1,
                     const __grid_constant__ CUtensorMap map_c1, const __grid_constant__ CUtensorMap map_d1,
                     const __grid_constant__ WArgs g) {
  // map_b: B codes with 128-row boxes, map_c: the same array with 64-row boxes
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t staging = base + kWStages * kWStageBytes;
  const uint32_t bar_base = staging + kWStagingBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };                   // leader only: both CTAs' operands landed
  auto sff_bar = [&](int s) { return bar_base + 8u * (kWStages + s); };       // leader only: scales of both CTAs in TMEM
  auto empty_bar = [&](int s) { return bar_base + 8u * (2 * kWStages + s); }; // one per CTA
  auto sfl_bar = [&](int s) { return bar_base + 8u * (3 * kWStages + s); };   // one per CTA: own scale atoms landed
  const uint32_t accf_bar = bar_base + 8u * (4 * kWStages);                   // one per CTA
  const uint32_t acce_bar = bar_base + 8u * (4 * kWStages + 1);               // leader only, 16 arrivals
  const uint32_t done_bar = bar_base + 8u * (4 * kWStages + 2);               // one per CTA, peer arrives
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(
      base_ptr + kWStages * kWStageBytes + kWStagingBytes + 8 * (4 * kWStages + 3));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader
  const bool leader = rank == 0;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_tiles = g.n_tiles;
  // Tile order inside a problem: groups of kGroupM row-blocks sweep all column tiles before the next group starts.
  constexpr int kGroupM = 8;
  // -> problem, row block, first column and width (384 or 256) of a tile
  auto tile_coords = [&](int tile, int& prob, int& m_blk, int& n0, int& width) {
    prob = tile >= g.n_tiles0 ? 1 : 0;
    if (prob) tile -= g.n_tiles0;
    const int tiles_m = g.p[prob].M / 256, tiles_n = g.p[prob].tiles_n, n_wide = g.p[prob].n_wide;
    const int per_group = kGroupM * tiles_n;
    const int grp = tile / per_group, in_grp = tile - grp * per_group;
    const int m0 = grp * kGroupM;
    const int gm = (tiles_m - m0 < kGroupM) ? (tiles_m - m0) : kGroupM;
    m_blk = m0 + in_grp % gm;
    const int n_idx = in_grp / gm;
    width = n_idx < n_wide ? 384 : 256;
    n0 = n_idx < n_wide ? n_idx * 384 : n_wide * 384 + (n_idx - n_wide) * 256;
  };
  auto k_blocks_of = [&](int tile) { return g.p[tile >= g.n_tiles0 ? 1 : 0].K / 256; };
  // Tiles go to the pairs in rounds, odd rounds in reverse pair order (a snake): the pairs that got the larger or
  // the extra tiles of one round get the smaller ones, or none, in the next.  A balance measure only: with equal
  // tiles it times the same as the plain round-robin.
  auto next_tile = [&](int rnd) { return rnd * n_pairs + ((rnd & 1) ? n_pairs - 1 - pair_id : pair_id); };
  constexpr int kAtomsKb = MX ? 2 : 4;  // scale atoms per 256-deep k-block and 128-row group

  if (threadIdx.x == 0) {
    for (int s = 0; s < kWStages; ++s) {
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
                 "r"(kWTmemCols)
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
        int prob, m_blk, n0, width;
        tile_coords(tile, prob, m_blk, n0, width);
        const WProblem& pr = g.p[prob];
        const CUtensorMap* map_a = prob ? &map_a1 : &map_a0;
        const CUtensorMap* map_b = prob ? &map_b1 : &map_b0;
        const CUtensorMap* map_c = prob ? &map_c1 : &map_c0;
        const bool is_wide = width == 384;
        const int k_blocks = pr.K / 256;
        const int sf_atoms_k = pr.K / (MX ? 128 : 64);  // atoms along K per 128-row group
        const int row_a = m_blk * 256 + (int)rank * 128;  // this CTA's A rows
        const int row_b = n0 + (int)rank * 128;            // its 128 rows of the tile's first 256 columns
        const int row_c = n0 + 256 + (int)rank * 64;       // its 64 rows of the last 128 columns (wide tiles)
        const int groups = width / 128;
        const uint8_t* sfa = pr.sfa + (int64_t)(m_blk * 2 + (int)rank) * sf_atoms_k * 512;  // own 128 rows
        const uint8_t* sfb = pr.sfb + (int64_t)(n0 / 128) * sf_atoms_k * 512;               // all rows of the B tile
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 0x100u + stage))) break;
          const uint32_t st = base + stage * kWStageBytes;
          const uint32_t bar = map_to_cta(full_bar(stage), 0);  // the leader's barrier counts both CTAs' operands
          mbar_expect_tx_cluster(bar, kWABytes + 128 * 128 + (is_wide ? 64 * 128 : 0));
          tma_load_2d_pair(st, map_a, kb * 128, row_a, bar);
          tma_load_2d_pair(st + kWABytes, map_b, kb * 128, row_b, bar);
          if (is_wide) tma_load_2d_pair(st + kWABytes + 128 * 128, map_c, kb * 128, row_c, bar);
          // scale atoms: plain bulk copies counted on this CTA's own barrier (its scale warps wait on it)
          mbar_expect_tx(sfl_bar(stage), (1 + groups) * kAtomsKb * 512);
          const uint32_t sf_s = st + kWABytes + kWBBytes;
          bulk_load(sf_s, sfa + (int64_t)kb * kAtomsKb * 512, kAtomsKb * 512, sfl_bar(stage));
          for (int grp = 0; grp < groups; ++grp)
            bulk_load(sf_s + kWSfaBytes + grp * 2048, sfb + ((int64_t)grp * sf_atoms_k + kb * kAtomsKb) * 512,
                      kAtomsKb * 512, sfl_bar(stage));
          if (++stage == kWStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 2 || warp >= 11) {
    // ------------------------------- scale atoms: shared memory -> registers -> tensor memory (both CTAs) ----
    // One warp per 32-lane quadrant (warps 2, 11, 12, 13 -> quadrants 2, 3, 0, 1).  Slot layout: columns [4j, 4j+4)
    // SFA of atom j, columns [16 + 12j + 4g, ..) SFB of atom j and 128-row group g.  The two slots alternate per
    // k-block; slot reuse waits for the MMAs of two k-blocks earlier (that stage's "empty" barrier).
    const int quad = warp & 3;
    int stage = 0;
    uint32_t phase = 0, it = 0;  // it: k-blocks processed so far (selects the slot)
    const uint32_t sff_leader = map_to_cta(sff_bar(0), 0);
    uint32_t r[64];  // the slot's 64 columns; entries of a narrow tile's third group keep stale (unused) values
#pragma unroll
    for (int i = 0; i < 64; ++i) r[i] = 0u;
    for (int rnd = 0, tile = pair_id; tile < n_tiles; tile = next_tile(++rnd)) {
      bool ok = true;
      int prob, m_blk, n0, width;
      tile_coords(tile, prob, m_blk, n0, width);
      const bool is_wide = width == 384;
      const int k_blocks = g.p[prob].K / 256;
      for (int kb = 0; kb < k_blocks; ++kb, ++it) {
        ok = mbar_wait(sfl_bar(stage), phase, abort_flag, 0x500u + stage);
        if (ok && it >= 2) {
          const uint32_t prev = it - 2;  // the k-block that used this slot before
          ok = mbar_wait_cluster(empty_bar(prev & 3u), (prev >> 2) & 1u, abort_flag, 0x540u + (prev & 3u));
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        tc_fence_after();
        const uint32_t sf_s = base + stage * kWStageBytes + kWABytes + kWBBytes + lane * 16;
#pragma unroll
        for (int j = 0; j < kAtomsKb; ++j) {
          const uint4 a = lds128(sf_s + j * 512);
          r[4 * j] = a.x; r[4 * j + 1] = a.y; r[4 * j + 2] = a.z; r[4 * j + 3] = a.w;
#pragma unroll
          for (int grp = 0; grp < 3; ++grp) {
            if (grp < 2 || is_wide) {
              const uint4 b = lds128(sf_s + kWSfaBytes + grp * 2048 + j * 512);
              r[16 + 12 * j + 4 * grp] = b.x; r[16 + 12 * j + 4 * grp + 1] = b.y;
              r[16 + 12 * j + 4 * grp + 2] = b.z; r[16 + 12 * j + 4 * grp + 3] = b.w;
            }
          }
        }
        const uint32_t sf_t = tmem + ((uint32_t)(quad * 32) << 16) + kWSfCol + (it & 1u) * kWSfSlotCols;
        tc_st16(sf_t, &r[0]);
        tc_st16(sf_t + 16, &r[16]);
        tc_st16(sf_t + 32, &r[32]);
        if (!MX) tc_st16(sf_t + 48, &r[48]);  // MXFP4 has two atoms per k-block: columns up to 16 + 12 + 12
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(sff_leader + 8u * stage);
        if (++stage == kWStages) {
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
      uint32_t phase = 0, acc_phase = 0, it = 0;
      bool ok = true;
      constexpr uint32_t id256 = instr_desc_nvf4(256, 256), id128 = instr_desc_nvf4(256, 128);
      constexpr uint32_t id256_mx[2] = {instr_desc_mxf4(256, 256, 0), instr_desc_mxf4(256, 256, 2)};
      constexpr uint32_t id128_mx[2] = {instr_desc_mxf4(256, 128, 0), instr_desc_mxf4(256, 128, 2)};
      const uint32_t a_lo0 = ((base >> 4) & 0x3fffu) | (1u << 16);
      const uint32_t b_lo0 = (((base + kWABytes) >> 4) & 0x3fffu) | (1u << 16);
      for (int rnd = 0, tile = pair_id; tile < n_tiles && ok; tile = next_tile(++rnd)) {
        int prob, m_blk, n0, width;
        tile_coords(tile, prob, m_blk, n0, width);
        const bool is_wide = width == 384;
        if (!(ok = mbar_wait_cluster(acce_bar, acc_phase ^ 1u, abort_flag, 0x300u))) break;
        tc_fence_after();
        const int k_blocks = k_blocks_of(tile);
        for (int kb = 0; kb < k_blocks; ++kb, ++it) {
          if (!(ok = mbar_wait_cluster(full_bar(stage), phase, abort_flag, 0x200u + stage))) break;
          if (!(ok = mbar_wait_cluster(sff_bar(stage), phase, abort_flag, 0x280u + stage))) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + stage * (kWStageBytes >> 4);
          const uint32_t b_lo = b_lo0 + stage * (kWStageBytes >> 4);
          const uint32_t c_lo = b_lo + ((128 * 128) >> 4);  // the 64 rows of the last 128 columns
          const uint32_t sf_t = tmem + kWSfCol + (it & 1u) * kWSfSlotCols;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t acc = (kb > 0 || j > 0) ? 1u : 0u;
            const uint64_t ad = make_desc(a_lo + 2 * j, kDescHiOperand);
            if (MX) {  // one atom (4 columns per group) serves two K = 64 steps: bytes 0-1, then bytes 2-3
              const uint32_t sfa_t = sf_t + (j >> 1) * 4, sfb_t = sf_t + 16 + (j >> 1) * 12;
              tc2_mma_mxf4(tmem, ad, make_desc(b_lo + 2 * j, kDescHiOperand), id256_mx[j & 1], sfa_t, sfb_t, acc);
              if (is_wide)
                tc2_mma_mxf4(tmem + 256, ad, make_desc(c_lo + 2 * j, kDescHiOperand), id128_mx[j & 1], sfa_t, sfb_t + 8,
                             acc);
            } else {
              const uint32_t sfa_t = sf_t + j * 4, sfb_t = sf_t + 16 + j * 12;
              tc2_mma_nvf4(tmem, ad, make_desc(b_lo + 2 * j, kDescHiOperand), id256, sfa_t, sfb_t, acc);
              if (is_wide)
                tc2_mma_nvf4(tmem + 256, ad, make_desc(c_lo + 2 * j, kDescHiOperand), id128, sfa_t, sfb_t + 8, acc);
            }
          }
          tc2_commit_both(empty_bar(stage), 3);  // both CTAs' stages (and the scale slot) are free after these MMAs
          if (++stage == kWStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        tc2_commit_both(accf_bar, 3);  // accumulators of both CTAs complete
        acc_phase ^= 1u;
      }
    }
  } else if (warp >= 3 && warp <= 10) {
    // ------------------------------------------------------------------ epilogue ----
    // Two groups of four warps; group h drains columns [h * W / 2, (h + 1) * W / 2) of the accumulator in passes
    // of 64 columns through its own staging buffer.
    const int quad = warp & 3;                // tensor-memory lanes this warp may read
    const int half = (warp - 3) >> 2;         // column half / epilogue group
    const int et = (threadIdx.x - 96) & 127;  // 0..127 inside the group
    const int bar_id = 1 + half;
    uint32_t acc_phase = 0;
    const float alpha0 = __fmul_rn(g.p[0].a_global[1], g.p[0].b_global[1]);
    const float alpha1 = __fmul_rn(g.p[1].a_global[1], g.p[1].b_global[1]);
    const uint32_t acce_leader = map_to_cta(acce_bar, 0);
    const int row_in_tile = quad * 32 + lane;
    const uint32_t stage_bufs = staging + half * 16384;
    uint32_t n_chunks = 0;  // chunks this group has stored so far (selects the buffer)
    for (int rnd = 0, tile = pair_id; tile < n_tiles; tile = next_tile(++rnd)) {
      int prob, m_blk, n0, width;
      tile_coords(tile, prob, m_blk, n0, width);
      const CUtensorMap* map_d = prob ? &map_d1 : &map_d0;
      const float alpha = prob ? alpha1 : alpha0;
      const int d_is_fp32 = g.p[prob].d_is_fp32, accumulate = g.p[prob].accumulate;
      const int cols_half = width >> 1, passes = cols_half >> 6;  // 192 / 3 or 128 / 2
      mbar_wait_cluster(accf_bar, acc_phase, abort_flag, 0x400u);
      // agree on giving up: a warp that timed out still joins this barrier, and all 128 threads take ONE decision
      if (group_gave_up(abort_flag, bar_id, 128)) break;
      tc_fence_after();
      const int row0 = m_blk * 256 + (int)rank * 128;
      const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16) + half * cols_half;
      // the previous tile's stores have long left the staging buffer; waiting for all of them here lets a tile with
      // another output type (two problems in one launch) use the buffer its own way
      if (et == 0) bulk_wait_read<0>();
      for (int p = 0; p < passes; ++p) {
        uint32_t r[64];
#pragma unroll
        for (int q = 0; q < 4; ++q) tc_ld16(t_row + p * 64 + q * 16, *reinterpret_cast<uint32_t(*)[16]>(&r[q * 16]));
        tc_wait_ld();
        if (p == passes - 1) {  // the accumulator has been read: the MMA issuer may start the next tile
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acce_leader);
        }
        const int x0 = n0 + half * cols_half + p * 64;
        if (d_is_fp32)
          store_cols64<true>(r, alpha, et, bar_id, row_in_tile, stage_bufs, n_chunks, map_d, x0, row0, accumulate);
        else
          store_cols64<false>(r, alpha, et, bar_id, row_in_tile, stage_bufs, n_chunks, map_d, x0, row0, accumulate);
      }
      acc_phase ^= 1u;
    }
    if (et == 0) bulk_wait_all<0>();  // all stores have left shared memory and are visible
  }

  // ------------------------------------------------------------------ teardown ----
  // Neither CTA may leave while the other can still signal its barriers or read its shared memory.
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
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kWTmemCols) : "memory");
  }
}

}  // namespace wide
}  // namespace nvfp4
