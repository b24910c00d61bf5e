// Block-scaled NVFP4 GEMM for sm_100a: D[M x N] = alpha * A[M x K] * B[N x K]^T  (Eq. 5 of the paper:
// per 16-element block partial dot products times the two E4M3 block scales, accumulated in FP32;
// alpha = s_dec^A * s_dec^B applied once on the result).
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0   producer: TMA loads of the code tiles (128-byte swizzle) and bulk copies of the scale atoms
//   warp 1   MMA issuer: tcgen05.mma kind::mxf4nvf4.block_scale.scale_vec::4X (M 128, N = BN, K 64 per
//            instruction), accumulator in tensor memory
//   warp 2   scale-atom copier: tcgen05.cp of the E4M3 atoms shared -> tensor memory (its own warp because
//            instruction issue by a single thread, not the tensor pipe, was the bottleneck with both in one)
//   warps 3-6 epilogue: tcgen05.ld of the FP32 accumulator, alpha, conversion, global stores
// Every wait is bounded: when one expires the kernel records a code in a device status word, every role
// leaves its loop, tensor memory is released and the kernel returns.
//
// This file holds the one-CTA kernel (shapes with M or N not a multiple of 256), the tensor-map helpers and the
// launchers of both kernels; the CTA-pair kernel that carries the large shapes is in gemm_2cta.cuh.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include <algorithm>
#include <mutex>
#include <vector>

#include "gemm.h"
#include "tc_ptx.cuh"
#include "gemm_2cta.cuh"
#include "gemm_wide.cuh"
#include "gemm_bf16.cuh"

namespace nvfp4 {

EncodeTiledFn tensor_map_encoder() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Encoding a tensor map is pure host arithmetic in the driver (about a microsecond each, three to eight per GEMM
// launch): the result depends only on the arguments, so a small per-thread cache keyed by them returns repeats (the
// same buffers launch after launch, as in a training loop) without the call.
bool make_map_2d(CUtensorMap* map, CUtensorMapDataType dtype, int elem_bytes, const void* base, uint64_t inner_elems,
                 uint64_t rows, uint64_t row_pitch_bytes, uint32_t box_inner, uint32_t box_rows, int swizzle) {
  (void)elem_bytes;
  struct Entry {
    uint64_t key[6];
    bool valid;
    CUtensorMap map;
  };
  constexpr int kEntries = 64;
  static thread_local Entry cache[kEntries] = {};
  const uint64_t key[6] = {reinterpret_cast<uint64_t>(base), inner_elems, rows, row_pitch_bytes,
                           ((uint64_t)box_inner << 32) | box_rows, ((uint64_t)dtype << 2) | (uint64_t)(swizzle & 3)};
  uint64_t h = 0x9E3779B97F4A7C15ull;
  for (uint64_t k : key) h = (h ^ k) * 0xFF51AFD7ED558CCDull + (h >> 29);
  Entry& e = cache[(h >> 20) % kEntries];
  if (e.valid && std::equal(key, key + 6, e.key)) {
    *map = e.map;
    return true;
  }
  EncodeTiledFn fn = tensor_map_encoder();
  if (!fn) return false;
  cuuint64_t dims[2] = {inner_elems, rows};
  cuuint64_t strides[1] = {row_pitch_bytes};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  if (fn(map, dtype, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
         swizzle == 1 ? CU_TENSOR_MAP_SWIZZLE_128B : swizzle == 2 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE,
         CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  std::copy(key, key + 6, e.key);
  e.map = *map;
  e.valid = true;
  return true;
}

namespace {

constexpr int BM = 128;
constexpr int BK_BYTES = 128;           // bytes of codes per row per stage = 256 elements of K
constexpr int BK = 256;
constexpr int kThreads = 224;
constexpr uint32_t kTmemCols = 512;

template <int BN>
struct Cfg {
  static constexpr int kStages = (BN == 256) ? 4 : 6;
  static constexpr int kAccStages = (BN == 256) ? 1 : 2;
  static constexpr int kABytes = BM * BK_BYTES;             // 16 KB
  static constexpr int kBBytes = BN * BK_BYTES;             // 16 / 32 KB
  static constexpr int kSfaBytes = 4 * 512;                 // 4 K64-steps x one 128-row atom
  static constexpr int kSfbBytes = (BN / 128) * 4 * 512;
  static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
  // tensor memory columns
  static constexpr int kAccCol = 0;
  static constexpr int kSfCol = kAccStages * BN;            // one slot of (SFA 16 + SFB 4*BN/32) columns per stage
  static constexpr int kSfaCols = 16;
  static constexpr int kSfbCols = 4 * (BN / 32);
  static constexpr int kSfBufCols = kSfaCols + kSfbCols;
  static_assert(kSfCol + kStages * kSfBufCols <= 512, "tensor memory budget");
};

// ------------------------------------------------------------------------------------ kernel ----
// MX = true: MXFP4 operands (UE8M0 scale per 32 elements): half the scale atoms per k-block, one atom serving two
// K = 64 steps through the scale-id field of the instruction descriptor (see gemm_2cta.cuh).
template <int BN, bool MX>
__global__ void __launch_bounds__(kThreads, 1)
    gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const GemmArgs g) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  // barriers live after the stages
  const uint32_t bar_base = base + C::kStages * C::kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };                      // operands + scale atoms landed
  auto sff_bar = [&](int s) { return bar_base + 8u * (C::kStages + s); };        // scale atoms are in tensor memory
  auto empty_bar = [&](int s) { return bar_base + 8u * (2 * C::kStages + s); };  // MMAs have consumed the stage
  auto accf_bar = [&](int s) { return bar_base + 8u * (3 * C::kStages + s); };
  auto acce_bar = [&](int s) { return bar_base + 8u * (3 * C::kStages + C::kAccStages + s); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(
      base_ptr + C::kStages * C::kStageBytes + 8 * (3 * C::kStages + 2 * C::kAccStages));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = g.M / BM, tiles_n = g.N / BN;
  const int n_tiles = tiles_m * tiles_n;
  const int k_blocks = g.K / BK;
  const int64_t sf_atoms_per_row_group = g.K / (MX ? 128 : 64);
  constexpr int kAtomsKb = MX ? 2 : 4;  // scale atoms per 256-deep k-block and 128-row group

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(sff_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int s = 0; s < C::kAccStages; ++s) {
      mbar_init(accf_bar(s), 1);
      mbar_init(acce_bar(s), 4);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer ----
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int m_blk = tile % tiles_m, n_blk = tile / tiles_m;
        const uint8_t* sfa = g.sfa + (int64_t)m_blk * sf_atoms_per_row_group * 512;
        const uint8_t* sfb = g.sfb + (int64_t)n_blk * (BN / 128) * sf_atoms_per_row_group * 512;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 0x100u + stage))) break;
          const uint32_t st = base + stage * C::kStageBytes;
          mbar_expect_tx(full_bar(stage), C::kABytes + C::kBBytes + (1 + BN / 128) * kAtomsKb * 512);
          tma_load_2d(st, &map_a, kb * BK_BYTES, m_blk * BM, full_bar(stage));
          tma_load_2d(st + C::kABytes, &map_b, kb * BK_BYTES, n_blk * BN, full_bar(stage));
          bulk_load(st + C::kABytes + C::kBBytes, sfa + (int64_t)kb * kAtomsKb * 512, kAtomsKb * 512, full_bar(stage));
#pragma unroll
          for (int grp = 0; grp < BN / 128; ++grp)
            bulk_load(st + C::kABytes + C::kBBytes + C::kSfaBytes + grp * 2048,
                      sfb + ((int64_t)grp * sf_atoms_per_row_group + (int64_t)kb * kAtomsKb) * 512, kAtomsKb * 512,
                      full_bar(stage));
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------- scale atoms: shared -> tensor memory ----
    // SFA of K64-step j goes to columns [4j, 4j+4) of the stage's slot; SFB of step j to
    // [16 + j*BN/32, ...), 4 columns per 128 rows of B.  The slot of a stage is free again when the
    // stage's operands are (empty -> producer -> full), so no extra barrier guards it.
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint32_t sf_lo0 = (base + C::kABytes + C::kBBytes) >> 4;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag, 0x500u + stage))) break;
          tc_fence_after();
          const uint32_t lo = sf_lo0 + stage * (C::kStageBytes >> 4);
          const uint32_t sf_t = tmem + C::kSfCol + stage * C::kSfBufCols;
#pragma unroll
          for (int j = 0; j < kAtomsKb; ++j) {
            tc_cp_sf(sf_t + j * 4, make_desc(lo + j * 32, kDescHiSf));
#pragma unroll
            for (int grp = 0; grp < BN / 128; ++grp)
              tc_cp_sf(sf_t + C::kSfaCols + j * (BN / 32) + grp * 4,
                       make_desc(lo + (C::kSfaBytes >> 4) + grp * 128 + j * 32, kDescHiSf));
          }
          tc_commit(sff_bar(stage));
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer ----
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      constexpr uint32_t idesc = instr_desc_nvf4(BM, BN);
      constexpr uint32_t idesc_mx[2] = {instr_desc_mxf4(BM, BN, 0), instr_desc_mxf4(BM, BN, 2)};
      const uint32_t a_lo0 = ((base >> 4) & 0x3fffu) | (1u << 16);
      const uint32_t b_lo0 = (((base + C::kABytes) >> 4) & 0x3fffu) | (1u << 16);
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        if (!(ok = mbar_wait(acce_bar(acc), acc_phase ^ 1u, abort_flag, 0x300u + acc))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem + C::kAccCol + acc * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait(sff_bar(stage), phase, abort_flag, 0x200u + stage))) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + stage * (C::kStageBytes >> 4);
          const uint32_t b_lo = b_lo0 + stage * (C::kStageBytes >> 4);
          const uint32_t sf_t = tmem + C::kSfCol + stage * C::kSfBufCols;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            // advancing 64 elements of K = 32 bytes inside the 128-byte swizzle span: +2 in the address field
            if (MX)
              tc_mma_mxf4(d_tmem, make_desc(a_lo + 2 * j, kDescHiOperand), make_desc(b_lo + 2 * j, kDescHiOperand),
                          idesc_mx[j & 1], sf_t + (j >> 1) * 4, sf_t + C::kSfaCols + (j >> 1) * (BN / 32),
                          (kb > 0 || j > 0) ? 1u : 0u);
            else
              tc_mma_nvf4(d_tmem, make_desc(a_lo + 2 * j, kDescHiOperand), make_desc(b_lo + 2 * j, kDescHiOperand), idesc,
                          sf_t + j * 4, sf_t + C::kSfaCols + j * (BN / 32), (kb > 0 || j > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));  // frees the stage once the MMAs above have read it
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        tc_commit(accf_bar(acc));  // accumulator complete
        if (++acc == C::kAccStages) {
          acc = 0;
          acc_phase ^= 1u;
        }
      }
    }
  } else if (warp >= 3) {
    // ------------------------------------------------------------------ epilogue ----
    const int quad = warp & 3;  // the 32 tensor-memory lanes this warp may read
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    const float alpha = __fmul_rn(g.a_global[1], g.b_global[1]);
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      const int m_blk = tile % tiles_m, n_blk = tile / tiles_m;
      ok = mbar_wait(accf_bar(acc), acc_phase, abort_flag, 0x400u + acc);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      tc_fence_after();
      const int64_t row = (int64_t)m_blk * BM + quad * 32 + lane;
      const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16) + C::kAccCol + acc * BN;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tc_ld32(t_row + c * 32, r);
        tc_wait_ld();
        const int64_t col = (int64_t)n_blk * BN + c * 32;
        if (g.d_is_fp32) {
          float* dst = reinterpret_cast<float*>(g.d) + row * g.ldd + col;
#pragma unroll
          for (int v = 0; v < 8; ++v) {
            float4 o = make_float4(__uint_as_float(r[4 * v]) * alpha, __uint_as_float(r[4 * v + 1]) * alpha,
                                   __uint_as_float(r[4 * v + 2]) * alpha, __uint_as_float(r[4 * v + 3]) * alpha);
            if (g.accumulate) {
              float4 old = *reinterpret_cast<const float4*>(dst + 4 * v);
              o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
            }
            *reinterpret_cast<float4*>(dst + 4 * v) = o;
          }
        } else {
          __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(g.d) + row * g.ldd + col;
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint32_t p[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * v + 2 * e]) * alpha,
                                                       __uint_as_float(r[8 * v + 2 * e + 1]) * alpha);
              p[e] = *reinterpret_cast<uint32_t*>(&h);
            }
            *reinterpret_cast<uint4*>(dst + 8 * v) = make_uint4(p[0], p[1], p[2], p[3]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acce_bar(acc));
      if (++acc == C::kAccStages) {
        acc = 0;
        acc_phase ^= 1u;
      }
    }
  }

  // ------------------------------------------------------------------ teardown ----
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is handed back
    for (int i = 0; i < 100; ++i) __nanosleep(1000);
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ------------------------------------------------------------------------------- host side ----
// codes [rows][k_bytes] uint8, box = 128 bytes x box_rows, 128-byte swizzle
bool make_code_map(CUtensorMap* map, const void* codes, int64_t rows, int64_t k_bytes, int box_rows) {
  return make_map_2d(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes, (uint64_t)k_bytes, (uint64_t)rows, (uint64_t)k_bytes,
                     BK_BYTES, (uint32_t)box_rows, true);
}

template <int BN, bool MX>
cudaError_t launch_t(const GemmArgs& g, const void* a_codes, const void* b_codes, int num_sms, cudaStream_t s) {
  using C = Cfg<BN>;
  CUtensorMap map_a, map_b;
  if (!make_code_map(&map_a, a_codes, g.M, g.K / 2, BM) || !make_code_map(&map_b, b_codes, g.N, g.K / 2, BN))
    return cudaErrorInvalidValue;
  auto kern = gemm_kernel<BN, MX>;
  static std::atomic<uint64_t> configured{0};  // per call site (template instantiation) and device
  int dev;
  if (device_needs_config(configured, &dev)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    device_configured(configured, dev);
  }
  const int n_tiles = (g.M / BM) * (g.N / BN);
  const int grid = n_tiles < num_sms ? n_tiles : num_sms;
  kern<<<grid, kThreads, C::kSmemBytes, s>>>(map_a, map_b, g);
  count_launch();
  return cudaGetLastError();
}

bool make_pair_maps(const GemmArgs& g, const void* a_codes, const void* b_codes, CUtensorMap* map_a, CUtensorMap* map_b,
                    CUtensorMap* map_d) {
  bool ok = make_code_map(map_a, a_codes, g.M, g.K / 2, 128) && make_code_map(map_b, b_codes, g.N, g.K / 2, 128);
  if (g.d_is_fp32)
    ok = ok && make_map_2d(map_d, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, g.d, (uint64_t)g.N, (uint64_t)g.M,
                           (uint64_t)g.ldd * 4, 32, 128, true);
  else
    ok = ok && make_map_2d(map_d, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, g.d, (uint64_t)g.N, (uint64_t)g.M,
                           (uint64_t)g.ldd * 2, 64, 128, true);
  return ok;
}

// measurement aids of the CTA-pair kernel (set_gemm_experiment)
std::atomic<int> g_exp_mode{0}, g_exp_max_pairs{0};
std::atomic<unsigned long long*> g_exp_probe{nullptr};

pair::Problem pair_problem(const GemmArgs& g) {
  return pair::Problem{g.M, g.N, g.K, g.sfa, g.sfb, g.a_global, g.b_global, g.d_is_fp32, g.accumulate, g.a_rows, g.b_rows};
}

// g1 == nullptr: one problem
cudaError_t launch_pair(const GemmArgs& g0, const void* a0, const void* b0, const GemmArgs* g1, const void* a1,
                        const void* b1, int num_sms, cudaStream_t s) {
  CUtensorMap m[6];
  if (!make_pair_maps(g0, a0, b0, &m[0], &m[1], &m[2])) return cudaErrorInvalidValue;
  if (g1) {
    if (!make_pair_maps(*g1, a1, b1, &m[3], &m[4], &m[5])) return cudaErrorInvalidValue;
  } else {
    m[3] = m[0]; m[4] = m[1]; m[5] = m[2];
  }
  if (g1 && g1->mx != g0.mx) return cudaErrorInvalidValue;
  static std::atomic<uint64_t> configured{0};  // per call site (template instantiation) and device
  int dev;
  if (device_needs_config(configured, &dev)) {
    cudaError_t e = cudaFuncSetAttribute(pair::gemm_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         pair::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(pair::gemm_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             pair::kSmemBytes);
    if (e != cudaSuccess) return e;
    device_configured(configured, dev);
  }
  pair::Args a{};
  a.p[0] = pair_problem(g0);
  a.p[1] = pair_problem(g1 ? *g1 : g0);
  a.n_tiles0 = (g0.M / 256) * (g0.N / 256);
  a.n_tiles = a.n_tiles0 + (g1 ? (g1->M / 256) * (g1->N / 256) : 0);
  int max_pairs = num_sms / 2;
  const int cap = g_exp_max_pairs.load(std::memory_order_relaxed);  // measurement aids, 0 / NULL normally
  if (cap > 0 && cap < max_pairs) max_pairs = cap;
  a.exp = g_exp_mode.load(std::memory_order_relaxed);
  a.probe = g_exp_probe.load(std::memory_order_relaxed);
  const int pairs = a.n_tiles < max_pairs ? a.n_tiles : max_pairs;
  const bool rows = a.p[0].a_rows || a.p[0].b_rows || a.p[1].a_rows || a.p[1].b_rows;
  if (rows) {
    if (g0.mx) return cudaErrorInvalidValue;
    static std::atomic<uint64_t> configured_rows{0};
    if (device_needs_config(configured_rows, &dev)) {
      cudaError_t e = cudaFuncSetAttribute(pair::gemm_pair_kernel<false, true>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, pair::kSmemBytes);
      if (e != cudaSuccess) return e;
      device_configured(configured_rows, dev);
    }
  }
  const bool chained = g0.chained != 0;
  const dim3 grid(2 * pairs), block(pair::kThreads);
  cudaError_t le;
  if (rows)
    le = launch_kernel(pair::gemm_pair_kernel<false, true>, grid, block, pair::kSmemBytes, s, chained, m[0], m[1], m[2],
                       m[3], m[4], m[5], a);
  else if (g0.mx)
    le = launch_kernel(pair::gemm_pair_kernel<true>, grid, block, pair::kSmemBytes, s, chained, m[0], m[1], m[2], m[3],
                       m[4], m[5], a);
  else
    le = launch_kernel(pair::gemm_pair_kernel<false>, grid, block, pair::kSmemBytes, s, chained, m[0], m[1], m[2], m[3],
                       m[4], m[5], a);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

// N = 128 q = 384 a + 256 b with b in {0, 1, 2}: a wide column tiles, b narrow ones (q >= 2)
bool wide_split(int N, int* n_wide, int* n_narrow) {
  if (N % 128 != 0 || N < 256) return false;
  const int q = N / 128;
  const int b = (q % 3 == 0) ? 0 : (q % 3 == 1) ? 2 : 1;
  if (q - 2 * b < 0) return false;
  *n_wide = (q - 2 * b) / 3;
  *n_narrow = b;
  return true;
}

bool wide_eligible(const GemmArgs& g) {
  int a, b;
  return g.M % 256 == 0 && g.K % 256 == 0 && wide_split(g.N, &a, &b);
}

wide::WProblem wide_problem(const GemmArgs& g) {
  int a = 0, b = 0;
  wide_split(g.N, &a, &b);
  return wide::WProblem{g.M, g.N, g.K, g.sfa, g.sfb, g.a_global, g.b_global, g.d_is_fp32, g.accumulate, a, a + b};
}

bool make_wide_maps(const GemmArgs& g, const void* a_codes, const void* b_codes, CUtensorMap* m) {
  // m[0] A (128-row boxes), m[1] B (128-row boxes), m[2] B (64-row boxes), m[3] D
  bool ok = make_code_map(&m[0], a_codes, g.M, g.K / 2, 128) && make_code_map(&m[1], b_codes, g.N, g.K / 2, 128) &&
            make_code_map(&m[2], b_codes, g.N, g.K / 2, 64);
  // D: the epilogue's store chunks, 128 rows x 64 bytes with the 64-byte swizzle (fp32) or x 128 bytes (bf16)
  if (g.d_is_fp32)
    ok = ok && make_map_2d(&m[3], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, g.d, (uint64_t)g.N, (uint64_t)g.M,
                           (uint64_t)g.ldd * 4, 16, 128, 2);
  else
    ok = ok && make_map_2d(&m[3], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, g.d, (uint64_t)g.N, (uint64_t)g.M,
                           (uint64_t)g.ldd * 2, 64, 128, 1);
  return ok;
}

// Estimated makespan (in units of one 256-deep k-block of a 256 x 256 tile) of the static round-robin schedule
// the pair kernels use, for one or two problems: round r hands tiles r * pairs .. to the pairs in order, odd rounds
// in reverse order.  A tile
// costs its k-blocks times its width factor plus the accumulator hand-over.
double pair_makespan(const GemmArgs* const* gs, int n_problems, bool wide_tiles, int pairs) {
  std::vector<double> load((size_t)pairs, 0.0);
  constexpr int kGroupM = 8;
  int64_t t = 0;
  for (int pi = 0; pi < n_problems; ++pi) {
    const GemmArgs& g = *gs[pi];
    int n_wide = 0, n_narrow = g.N / 256;
    if (wide_tiles) wide_split(g.N, &n_wide, &n_narrow);
    const int tiles_m = g.M / 256, tiles_n = n_wide + n_narrow;
    const double kb = g.K / 256.0;
    for (int m0 = 0; m0 < tiles_m; m0 += kGroupM) {
      const int gm = tiles_m - m0 < kGroupM ? tiles_m - m0 : kGroupM;
      for (int n_idx = 0; n_idx < tiles_n; ++n_idx) {
        const bool w = n_idx < n_wide;
        // hand-over per tile in k-block units, fitted to 24 layer shapes timed with both tile widths (the fp32 figure
        // of the wide tile refitted after its store chunks stopped waiting for each other)
        const double cost = w ? 1.5 * kb + (g.d_is_fp32 ? 3.8 : 3.3) : kb + (wide_tiles ? 2.9 : 2.5);
        for (int i = 0; i < gm; ++i, ++t) {
          const int64_t rnd = t / pairs, p = t % pairs;
          load[(size_t)((rnd & 1) ? pairs - 1 - p : p)] += cost;  // odd rounds run through the pairs in reverse
        }
      }
    }
  }
  double worst = 0.0;
  for (double v : load) worst = v > worst ? v : worst;
  // the wide tiles move 17 % fewer operand bytes per flop; under the power cap that showed as ~3 % more clock
  return wide_tiles ? worst * 0.97 : worst;
}

// g1 == nullptr: one problem
cudaError_t launch_wide(const GemmArgs& g0, const void* a0, const void* b0, const GemmArgs* g1, const void* a1,
                        const void* b1, int num_sms, cudaStream_t s) {
  CUtensorMap m[8];
  if (!make_wide_maps(g0, a0, b0, &m[0])) return cudaErrorInvalidValue;
  if (g1) {
    if (!make_wide_maps(*g1, a1, b1, &m[4])) return cudaErrorInvalidValue;
  } else {
    for (int i = 0; i < 4; ++i) m[4 + i] = m[i];
  }
  if (g1 && g1->mx != g0.mx) return cudaErrorInvalidValue;
  static std::atomic<uint64_t> configured{0};  // per device
  int dev;
  if (device_needs_config(configured, &dev)) {
    cudaError_t e = cudaFuncSetAttribute(wide::gemm_wide_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         wide::kWSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(wide::gemm_wide_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             wide::kWSmemBytes);
    if (e != cudaSuccess) return e;
    device_configured(configured, dev);
  }
  wide::WArgs a{};
  a.p[0] = wide_problem(g0);
  a.p[1] = wide_problem(g1 ? *g1 : g0);
  a.n_tiles0 = (g0.M / 256) * a.p[0].tiles_n;
  a.n_tiles = a.n_tiles0 + (g1 ? (g1->M / 256) * a.p[1].tiles_n : 0);
  const int max_pairs = num_sms / 2;
  const int pairs = a.n_tiles < max_pairs ? a.n_tiles : max_pairs;
  const dim3 grid(2 * pairs), block(wide::kWThreads);
  const cudaError_t le =
      g0.mx ? launch_kernel(wide::gemm_wide_kernel<true>, grid, block, wide::kWSmemBytes, s, g0.chained != 0, m[0], m[1],
                            m[2], m[3], m[4], m[5], m[6], m[7], a)
            : launch_kernel(wide::gemm_wide_kernel<false>, grid, block, wide::kWSmemBytes, s, g0.chained != 0, m[0], m[1],
                            m[2], m[3], m[4], m[5], m[6], m[7], a);
  count_launch();
  return le != cudaSuccess ? le : cudaGetLastError();
}

cudaError_t sm_count(int* n) {
  static std::atomic<int> cache[64] = {};  // per device ordinal
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  int v = (dev >= 0 && dev < 64) ? cache[dev].load(std::memory_order_relaxed) : 0;
  if (!v) {
    e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) cache[dev].store(v, std::memory_order_relaxed);
  }
  *n = v;
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_gemm(const GemmArgs& g, const void* a_codes, const void* b_codes, int tile_n, cudaStream_t s) {
  int num_sms = 0;
  cudaError_t e = sm_count(&num_sms);
  if (e != cudaSuccess) return e;
  if (g.a_rows || g.b_rows) {  // scale vectors are applied by the 256 x 256 pair kernel's epilogue only
    if (g.M % 256 != 0 || g.N % 256 != 0) return cudaErrorInvalidValue;
    return launch_pair(g, a_codes, b_codes, nullptr, nullptr, nullptr, num_sms, s);
  }
  if (tile_n == 768 && wide_eligible(g)) return launch_wide(g, a_codes, b_codes, nullptr, nullptr, nullptr, num_sms, s);
  if ((tile_n == 512 || tile_n == 768) && g.M % 256 == 0 && g.N % 256 == 0)
    return launch_pair(g, a_codes, b_codes, nullptr, nullptr, nullptr, num_sms, s);
  if (tile_n == 256 && g.N % 256 == 0)
    return g.mx ? launch_t<256, true>(g, a_codes, b_codes, num_sms, s) : launch_t<256, false>(g, a_codes, b_codes, num_sms, s);
  return g.mx ? launch_t<128, true>(g, a_codes, b_codes, num_sms, s) : launch_t<128, false>(g, a_codes, b_codes, num_sms, s);
}

cudaError_t launch_gemm_two(const GemmArgs& g0, const void* a0, const void* b0, const GemmArgs& g1, const void* a1,
                            const void* b1, bool wide_tiles, cudaStream_t s) {
  int num_sms = 0;
  cudaError_t e = sm_count(&num_sms);
  if (e != cudaSuccess) return e;
  if (wide_tiles && wide_eligible(g0) && wide_eligible(g1)) return launch_wide(g0, a0, b0, &g1, a1, b1, num_sms, s);
  return launch_pair(g0, a0, b0, &g1, a1, b1, num_sms, s);
}

bool prefer_wide_tiles(const GemmArgs& g0, const GemmArgs* g1) {
  if (!wide_eligible(g0) || (g1 && !wide_eligible(*g1))) return false;
  if (g0.N % 256 != 0 || (g1 && g1->N % 256 != 0)) return true;  // only the wide kernel takes N = 128 (2k + 1)
  int num_sms = 0;
  if (sm_count(&num_sms) != cudaSuccess) return false;
  // the estimate walks every tile of both schedules: remember the answers for the shapes seen (a training loop
  // repeats a handful of them)
  struct Entry { int key[8]; bool wide; };
  static std::mutex mu;
  static std::vector<Entry> seen;
  // (the output type is part of the key: an fp32 output changes the hand-over cost and with it the choice)
  const int key[8] = {g0.M, g0.N, g0.K, g1 ? g1->M : 0, g1 ? g1->N : 0, g1 ? g1->K : 0, num_sms,
                      (g0.d_is_fp32 ? 1 : 0) | (g1 && g1->d_is_fp32 ? 2 : 0)};
  {
    std::lock_guard<std::mutex> lock(mu);
    for (const Entry& e : seen)
      if (std::equal(key, key + 8, e.key)) return e.wide;
  }
  const GemmArgs* gs[2] = {&g0, g1};
  const int n = g1 ? 2 : 1, pairs = num_sms / 2;
  const bool wide = pair_makespan(gs, n, true, pairs) < pair_makespan(gs, n, false, pairs);
  std::lock_guard<std::mutex> lock(mu);
  if (seen.size() < 256) {
    Entry e{};
    std::copy(key, key + 8, e.key);
    e.wide = wide;
    seen.push_back(e);
  }
  return wide;
}

cudaError_t launch_gemm_bf16(const DenseGemmArgs& g, cudaStream_t s) {
  int num_sms = 0;
  cudaError_t e = sm_count(&num_sms);
  if (e != cudaSuccess) return e;
  CUtensorMap map_a, map_b, map_d;
  const CUtensorMapDataType bf = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  bool ok = g.a_mn ? make_map_2d(&map_a, bf, 2, g.a, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.lda * 2, 64, 64, true)
                   : make_map_2d(&map_a, bf, 2, g.a, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda * 2, 64, 128, true);
  ok = ok && (g.b_mn ? make_map_2d(&map_b, bf, 2, g.b, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.ldb * 2, 64, 64, true)
                     : make_map_2d(&map_b, bf, 2, g.b, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.ldb * 2, 64, 128, true));
  if (g.d_is_fp32)
    ok = ok && make_map_2d(&map_d, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, g.d, (uint64_t)g.N, (uint64_t)g.M,
                           (uint64_t)g.ldd * 4, 32, 128, true);
  else
    ok = ok && make_map_2d(&map_d, bf, 2, g.d, (uint64_t)g.N, (uint64_t)g.M, (uint64_t)g.ldd * 2, 64, 128, true);
  if (!ok) return cudaErrorInvalidValue;
  static std::atomic<uint64_t> configured{0};  // per device
  int dev;
  if (device_needs_config(configured, &dev)) {
    e = cudaFuncSetAttribute(dense::gemm_bf16_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             dense::kSmemBytes);
    if (e != cudaSuccess) return e;
    device_configured(configured, dev);
  }
  dense::Args a{g.M, g.N, g.K, g.a_mn, g.b_mn, g.d_is_fp32, g.accumulate};
  const int n_tiles = ((g.M + 255) / 256) * ((g.N + 255) / 256), max_pairs = num_sms / 2;
  const int pairs = n_tiles < max_pairs ? n_tiles : max_pairs;
  dense::gemm_bf16_pair_kernel<<<2 * pairs, dense::kThreads, dense::kSmemBytes, s>>>(map_a, map_b, map_d, a);
  count_launch();
  return cudaGetLastError();
}

// Test aid: one warp waits, with the given limit, on a barrier nobody arrives at.  The wait runs out, the code lands
// in the status word, the abort word stops the other lanes, and the kernel returns by itself.
__global__ void wait_probe_kernel(unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0u;
  }
  __syncthreads();
  mbar_wait_limit(smem_u32(&bar), 0u, &abort_flag, kWaitProbeCode, limit_ns);
}

cudaError_t launch_wait_probe(unsigned long long limit_ns, cudaStream_t s) {
  wait_probe_kernel<<<1, 32, 0, s>>>(limit_ns);
  count_launch();
  return cudaGetLastError();
}

void set_gemm_experiment(int mode, int max_pairs, unsigned long long* probe) {
  g_exp_mode.store(mode, std::memory_order_relaxed);
  g_exp_max_pairs.store(max_pairs, std::memory_order_relaxed);
  g_exp_probe.store(probe, std::memory_order_relaxed);
}

cudaError_t device_status_word(unsigned int** word) {
  static std::atomic<unsigned int*> cache[64] = {};  // per device ordinal
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  unsigned int* p = (dev >= 0 && dev < 64) ? cache[dev].load(std::memory_order_acquire) : nullptr;
  if (!p) {
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_device_status);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) cache[dev].store(p, std::memory_order_release);
  }
  *word = p;
  return cudaSuccess;
}

cudaError_t read_device_status(cudaStream_t s, uint32_t* code) {
  cudaError_t e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return e;
  unsigned int v = 0;
  e = cudaMemcpyFromSymbol(&v, g_device_status, sizeof(v));
  if (e != cudaSuccess) return e;
  if (v) {
    unsigned int zero = 0;
    e = cudaMemcpyToSymbol(g_device_status, &zero, sizeof(zero));
  }
  *code = v;
  return e;
}

}  // namespace nvfp4
