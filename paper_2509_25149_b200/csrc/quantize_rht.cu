// NVFP4 quantizer with a random Hadamard transform of another size (Appendix E.4.2 of the paper compares 2 x 2,
// 4 x 4, 16 x 16 and 128 x 128 matrices on the Wgrad inputs): d = 2, 4, 8 or 128 instead of the recipe's 16.
// Blocks, scales and rounding are those of the main quantizer (Appendix B, Section 4.4); only the rotation differs:
// every aligned chunk of d elements along a copy's contraction dimension is multiplied by S * H_d / sqrt(d).
//
// One kernel serves both passes over a 128 x 128 source tile (MODE 0: tensor amax in the rotated space, MODE 1:
// scale + round + pack), so the values whose maximum was taken are bit for bit the values that get encoded.
//   d <= 16 : the first log2(d) stages of the 16-point register butterfly, per 1 x 16 chunk.
//   d = 128 : H_128 = H_8 (x) H_16.  Row-wise copy: the eight chunks of a 128-chunk sit in eight lanes of a warp, so
//             three shuffle stages follow the register butterfly.  Transposed copy: the eight 16-row groups of a
//             column belong to the eight warps, so a first pass does the three cross-group stages through an FP32
//             tile in shared memory and the usual 16-row pass finishes the transform.
// The normalisation 1/sqrt(d) is one FP32 multiply per element (exact for d = 4).  These are ablation variants: the
// structure follows the main kernel (phases 1-3, same staging layouts) without its instruction-level tuning.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "async_ptx.cuh"
#include "common.cuh"
#include "quantize.h"
#include "quantize_common.cuh"

namespace nvfp4 {

namespace {

struct RhtSmem {
  static constexpr int kColCodes = 0;                 // 128 columns x 64 B
  static constexpr int kSfRow = kColCodes + 8192;     // 1 KB
  static constexpr int kSfCol = kSfRow + 1024;        // 1 KB
  static constexpr int kGlobalScales = kSfCol + 1024; // 4 floats
  static constexpr int kRed = kGlobalScales + 64;     // 2 x 8 floats (amax pass)
  static constexpr int kRand = kRed + 64;             // 128 rows x 128 B
  static constexpr int kTile = kRand + 16384;         // d <= 16: 128 rows x 256 B of bf16
  static constexpr int kU = kTile;                    // d = 128 (transposed copy): 128 x 128 floats instead
  static constexpr int kBytesSmall = kTile + 32768;
  static constexpr int kBytesBig = kU + 65536;
};

// stages h < limit of the 16-point butterfly (limit = min(d, 16); 1 = no transform)
__device__ __forceinline__ void fwht16_partial(float (&v)[16], int limit) {
#pragma unroll
  for (int h = 1; h < 16; h <<= 1) {
    if (h < limit) {
#pragma unroll
      for (int i = 0; i < 16; ++i)
        if ((i & h) == 0) {
          const float a = v[i], b = v[i | h];
          v[i] = a + b;
          v[i | h] = a - b;
        }
    }
  }
}

// sign bits of the sixteen elements at positions [16 * c16, 16 * c16 + 16) of a chunk
__device__ __forceinline__ uint32_t chunk_signs(const RhtArgs& ra, int c16) {
  return ra.d == 128 ? ((ra.sign_words[c16 >> 1] >> ((c16 & 1) * 16)) & 0xffffu) : ra.mask16;
}

template <int MODE, bool SR>
__global__ void __launch_bounds__(256, 3) quantize_rht_kernel(const RhtArgs ra) {
  const QuantArgs& a = ra.q;
  extern __shared__ __align__(128) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = MODE == 0 ? (int)blockIdx.x : (int)(gridDim.x - 1 - blockIdx.x);  // pass 2 walks backwards (L2)
  griddep_launch_dependents();  // the GEMM of a composed call may set itself up while the last CTAs run
  const int64_t row0 = (int64_t)(tile / a.tiles_c) * 128;
  const int64_t col0 = (int64_t)(tile % a.tiles_c) * 128;
  const int64_t n_cb = a.cols >> 4, n_rb = a.rows >> 4;
  const bool has_row = ra.has_row, has_col = ra.has_col;
  const int d_row = ra.rht_row ? ra.d : 1, d_col = ra.rht_col ? ra.d : 1;
  const float norm_row = ra.rht_row ? ra.norm : 1.f, norm_col = ra.rht_col ? ra.norm : 1.f;

  float* g_sc = reinterpret_cast<float*>(smem + RhtSmem::kGlobalScales);
  if (MODE == 1 && threadIdx.x == 0) {
    float re = 1.f, rd = 1.f, ce = 1.f, cd = 1.f;
    if (has_row) global_scales(a.r_global[0], re, rd);
    if (has_col) global_scales(a.c_global[0], ce, cd);
    g_sc[0] = re; g_sc[1] = rd; g_sc[2] = ce; g_sc[3] = cd;
    if (blockIdx.x == 0) {
      if (has_row) a.r_global[1] = rd;
      if (has_col) a.c_global[1] = cd;
    }
  }

  // ------------------------------------------------------------------ phase 1: load, row-wise copy ----
  const int cb = lane & 7;
  uint32_t raw[4][8];
  bool ok[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = warp * 16 + i * 4 + (lane >> 3);
    ok[i] = (row0 + r < a.rows) && (col0 + cb * 16 < a.cols);
    if (ok[i]) {
      ldg256_stream(a.x + (row0 + r) * a.ld + col0 + cb * 16, raw[i]);
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) raw[i][k] = 0u;
    }
    if (has_col && d_col == 128) {  // FP32 tile: the cross-group stages run in place on it
      float* dst = reinterpret_cast<float*>(smem + RhtSmem::kU) + r * 128 + cb * 16;
#pragma unroll
      for (int k = 0; k < 4; ++k)
        *reinterpret_cast<float4*>(dst + 4 * k) = make_float4(bf16_lo(raw[i][2 * k]), bf16_hi(raw[i][2 * k]),
                                                              bf16_lo(raw[i][2 * k + 1]), bf16_hi(raw[i][2 * k + 1]));
    } else if (has_col) {  // halves written in lane-dependent order so that a quarter warp covers all 32 banks
      uint8_t* dst = smem + RhtSmem::kTile + r * 256 + cb * 32;
      const int first = ((lane >> 2) & 1) * 16;
      *reinterpret_cast<uint4*>(dst + first) =
          first ? make_uint4(raw[i][4], raw[i][5], raw[i][6], raw[i][7]) : make_uint4(raw[i][0], raw[i][1], raw[i][2], raw[i][3]);
      *reinterpret_cast<uint4*>(dst + (16 - first)) =
          first ? make_uint4(raw[i][0], raw[i][1], raw[i][2], raw[i][3]) : make_uint4(raw[i][4], raw[i][5], raw[i][6], raw[i][7]);
    }
  }
  __syncthreads();
  const float r_senc = g_sc[0], r_sdec = g_sc[1], c_senc = g_sc[2], c_sdec = g_sc[3];
  float m_row = 0.f, m_col = 0.f;

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = warp * 16 + i * 4 + (lane >> 3);
    uint32_t rnd[4] = {0u, 0u, 0u, 0u};
    if (MODE == 1 && SR) {
      const uint64_t g = (uint64_t)(row0 + r) * (uint64_t)n_cb + (uint64_t)((col0 >> 4) + cb);
      const uint4 q = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), a.off_lo, a.off_hi, a.rk);
      rnd[0] = q.x; rnd[1] = q.y; rnd[2] = q.z; rnd[3] = q.w;
      if (has_col) {
        uint4 qc = q;
        if (a.off_hi_col != a.off_hi) qc = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), a.off_lo, a.off_hi_col, a.rk);
        *reinterpret_cast<uint4*>(smem + RhtSmem::kRand + r * 128 + cb * 16) = qc;
      }
    }
    if (has_row) {
      const uint32_t sg = ra.rht_row ? chunk_signs(ra, cb) : 0u;
      float f[16];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint32_t word = raw[i][k] ^ sign_pair(sg, 2 * k, 2 * k + 1);
        f[2 * k] = bf16_lo(word);
        f[2 * k + 1] = bf16_hi(word);
      }
      fwht16_partial(f, d_row < 16 ? d_row : 16);
      if (d_row == 128) {  // the other seven chunks of this 128-chunk are in the lanes that differ in bits 0-2
#pragma unroll
        for (int m = 1; m < 8; m <<= 1) {
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            const float other = __shfl_xor_sync(0xffffffffu, f[k], m);
            f[k] = (lane & m) ? (other - f[k]) : (f[k] + other);
          }
        }
      }
#pragma unroll
      for (int k = 0; k < 16; ++k) f[k] = __fmul_rn(f[k], norm_row);
      if (MODE == 0) {
        m_row = fmaxf(m_row, amax16(f));
      } else {
        uint32_t byte;
        float enc;
        block_scales(amax16(f), r_senc, r_sdec, byte, enc);
        const uint2 codes = convert16<SR>(f, enc, Nu14FromWords{rnd});
        if (ok[i])
          *reinterpret_cast<uint2*>(a.r_codes + (row0 + r) * (a.cols >> 1) + ((col0 + cb * 16) >> 1)) = codes;
        const int pos = a.r_swz ? ((cb >> 2) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (cb & 3)) : (r * 8 + cb);
        smem[RhtSmem::kSfRow + pos] = (uint8_t)byte;
      }
    }
  }

  // ------------------------------------------------------------------ phase 2: transposed copy ----
  // A warp reads back only what the same warp stored above (the random bytes of its own 16 rows; the tile was
  // staged before the barrier), so a warp-level barrier orders it; d = 128 adds a CTA barrier after its first pass.
  __syncwarp();
  if (has_col) {
    float* U = reinterpret_cast<float*>(smem + RhtSmem::kU);
    if (d_col == 128) {
      // cross-group stages: for row offset j and column pair cp, the eight rows j + 16 g (g = 0..7)
#pragma unroll 1
      for (int k = 0; k < 4; ++k) {
        const int id = threadIdx.x + 256 * k;
        const int j = id >> 6, cp = id & 63;
        float2 v[8];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const int p = 16 * g + j;  // position in the 128-chunk = row inside the tile
          const float2 x = *reinterpret_cast<const float2*>(U + p * 128 + 2 * cp);
          const bool neg = (ra.sign_words[p >> 5] >> (p & 31)) & 1u;
          v[g] = neg ? make_float2(-x.x, -x.y) : x;
        }
#pragma unroll
        for (int h = 1; h < 8; h <<= 1)
#pragma unroll
          for (int g = 0; g < 8; ++g)
            if ((g & h) == 0) {
              const float2 x = v[g], y = v[g | h];
              v[g] = make_float2(x.x + y.x, x.y + y.y);
              v[g | h] = make_float2(x.x - y.x, x.y - y.y);
            }
#pragma unroll
        for (int g = 0; g < 8; ++g) *reinterpret_cast<float2*>(U + (16 * g + j) * 128 + 2 * cp) = v[g];
      }
      __syncthreads();
    }
    const int q = warp;  // 16-row group
#pragma unroll 1
    for (int it = 0; it < 2; ++it) {
      const int cp = lane + 32 * it;
      float f0[16], f1[16];
      if (d_col == 128) {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float2 v = *reinterpret_cast<const float2*>(U + (q * 16 + j) * 128 + 2 * cp);
          f0[j] = v.x;
          f1[j] = v.y;
        }
      } else {
        const uint32_t sg = ra.rht_col ? ra.mask16 : 0u;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          uint32_t word = *reinterpret_cast<const uint32_t*>(smem + RhtSmem::kTile + (q * 16 + j) * 256 + cp * 4);
          word ^= sign_pair(sg, j, j);
          f0[j] = bf16_lo(word);
          f1[j] = bf16_hi(word);
        }
      }
      fwht16_partial(f0, d_col < 16 ? d_col : 16);
      fwht16_partial(f1, d_col < 16 ? d_col : 16);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        f0[j] = __fmul_rn(f0[j], norm_col);
        f1[j] = __fmul_rn(f1[j], norm_col);
      }
      if (MODE == 0) {
        m_col = fmaxf(m_col, fmaxf(amax16(f0), amax16(f1)));
      } else {
        uint32_t byte0, byte1;
        float enc0, enc1;
        block_scales(amax16(f0), c_senc, c_sdec, byte0, enc0);
        block_scales(amax16(f1), c_senc, c_sdec, byte1, enc1);
        uint32_t two[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) two[j] = 0u;
        if (SR) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            two[j] = *reinterpret_cast<const uint16_t*>(smem + RhtSmem::kRand + (q * 16 + j) * 128 + cp * 2);
        }
        const uint2 codes0 = convert16<SR>(f0, enc0, Nu14FromPairs<0>{two});
        const uint2 codes1 = convert16<SR>(f1, enc1, Nu14FromPairs<1>{two});
#pragma unroll
        for (int odd = 0; odd < 2; ++odd) {
          const int c = 2 * cp + odd;
          // unit q of column c sits at slot (q ^ (c >> 1)) & 7: neighbouring lanes hit different banks
          *reinterpret_cast<uint2*>(smem + RhtSmem::kColCodes + c * 64 + (((q ^ (c >> 1)) & 7) << 3)) = odd ? codes1 : codes0;
          const uint32_t byte = odd ? byte1 : byte0;
          const int pos = a.c_swz ? ((q >> 2) * 512 + (c & 31) * 16 + (c >> 5) * 4 + (q & 3)) : (c * 8 + q);
          smem[RhtSmem::kSfCol + pos] = (uint8_t)byte;
        }
      }
    }
  }

  if (MODE == 0) {
    float* red = reinterpret_cast<float*>(smem + RhtSmem::kRed);
    m_row = warp_max(m_row);
    m_col = warp_max(m_col);
    if (lane == 0) {
      red[warp] = m_row;
      red[8 + warp] = m_col;
    }
    __syncthreads();
    if (threadIdx.x < 2) {
      float m = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) m = fmaxf(m, red[threadIdx.x * 8 + w]);
      const uint32_t bits = __float_as_uint(m);  // non-negative floats order like their bit patterns
      if (threadIdx.x == 0 && has_row) atomicMax(reinterpret_cast<unsigned int*>(a.r_global), bits);
      if (threadIdx.x == 1 && has_col) atomicMax(reinterpret_cast<unsigned int*>(a.c_global), bits);
    }
    return;
  }
  __syncthreads();

  // ------------------------------------------------------------------ phase 3: staged outputs ----
  if (has_col) {
    const int64_t pitch = a.rows >> 1;  // bytes per row of the transposed copy
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int unit = threadIdx.x + 256 * k;
      const int c = unit >> 3, qq = unit & 7;  // column, 16-row group
      if (col0 + c >= a.cols || row0 + 16 * qq >= a.rows) continue;
      *reinterpret_cast<uint2*>(a.c_codes + (col0 + c) * pitch + (row0 >> 1) + qq * 8) =
          *reinterpret_cast<const uint2*>(smem + RhtSmem::kColCodes + c * 64 + (((qq ^ (c >> 1)) & 7) << 3));
    }
  }
#pragma unroll
  for (int which = 0; which < 2; ++which) {
    if (which == 0 ? !has_row : !has_col) continue;
    const uint8_t* src = smem + (which == 0 ? RhtSmem::kSfRow : RhtSmem::kSfCol);
    uint8_t* dst = which == 0 ? a.r_scales : a.c_scales;
    const int swz = which == 0 ? a.r_swz : a.c_swz;
    const int64_t R0 = which == 0 ? row0 : col0, K0 = which == 0 ? (col0 >> 4) : (row0 >> 4);
    const int64_t Rn = which == 0 ? a.rows : a.cols, n_kb = which == 0 ? n_cb : n_rb;
    if (swz) {
      if (threadIdx.x < 64) {
        const int atom = threadIdx.x >> 5;
        if (K0 + atom * 4 < n_kb) {
          const int64_t off = ((R0 >> 7) * (n_kb >> 2) + (K0 >> 2) + atom) * 512 + (threadIdx.x & 31) * 16;
          *reinterpret_cast<uint4*>(dst + off) = *reinterpret_cast<const uint4*>(src + threadIdx.x * 16);
        }
      }
    } else {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int idx = threadIdx.x * 4 + k;
        const int r = idx >> 3, kb = idx & 7;
        if (R0 + r < Rn && K0 + kb < n_kb) dst[(R0 + r) * n_kb + K0 + kb] = src[idx];
      }
    }
  }
}

template <int MODE, bool SR>
cudaError_t launch_mode(const RhtArgs& ra, cudaStream_t s) {
  auto kern = quantize_rht_kernel<MODE, SR>;
  static std::atomic<uint64_t> configured{0};  // per call site (template instantiation) and device
  int dev;
  if (device_needs_config(configured, &dev)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, RhtSmem::kBytesBig);
    if (e != cudaSuccess) return e;
    device_configured(configured, dev);
  }
  const int smem = (ra.d == 128 && ra.has_col && ra.rht_col) ? RhtSmem::kBytesBig : RhtSmem::kBytesSmall;
  kern<<<(unsigned)((int64_t)ra.q.tiles_r * ra.q.tiles_c), 256, smem, s>>>(ra);
  count_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_quantize_rht(const RhtArgs& ra, bool amax_provided, bool sr, cudaStream_t s) {
  cudaError_t e;
  if (!amax_provided && ra.d <= 16 && ra.has_col && ra.rht_col && !ra.rht_row) {
    // the recipe's case (plain row-wise copy, transformed transposed copy): pass 1 on the tensor cores, HBM-bound
    if ((e = launch_amax_rot_col_small(ra.q, ra.has_row != 0, ra.mask16, ra.d, ra.norm, s)) != cudaSuccess) return e;
  } else if (!amax_provided) {
    if (ra.has_row && (e = cudaMemsetAsync(ra.q.r_global, 0, sizeof(float), s)) != cudaSuccess) return e;
    if (ra.has_col && (e = cudaMemsetAsync(ra.q.c_global, 0, sizeof(float), s)) != cudaSuccess) return e;
    if ((e = launch_mode<0, false>(ra, s)) != cudaSuccess) return e;
  }
  return sr ? launch_mode<1, true>(ra, s) : launch_mode<1, false>(ra, s);
}

}  // namespace nvfp4
