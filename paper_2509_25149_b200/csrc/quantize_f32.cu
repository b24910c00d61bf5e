// NVFP4 quantizer for a binary32 source (Appendix B names FP32 as well as BF16 as the precision converted from),
// e.g. weights quantized straight from their FP32 master copy.  Same two passes and the same arithmetic as the bf16
// kernels of quantize.cu, only the element read differs: the tile is staged as FP32 (64 KB), a chunk is two 32-byte
// loads.  No Hadamard transform (the recipe transforms activations and gradients, which are bf16).
#include "quantize.h"
#include "quantize_common.cuh"

namespace nvfp4 {

__device__ __forceinline__ void ldg256_stream_f(const float* p, float (&r)[8]) {
  asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
               : "l"(p));
}

// Pass 1: plain tensor amax.  CTA tile 128 rows x 128 columns; a warp owns 16 rows, a lane 4 columns of each.
__global__ void __launch_bounds__(256) amax_f32_kernel(const float* __restrict__ x, int64_t rows, int64_t cols,
                                                       int64_t ld, int tiles_c, float* __restrict__ out0,
                                                       float* __restrict__ out1) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t tr = blockIdx.x / tiles_c, tc = blockIdx.x % tiles_c;
  const int64_t r0 = tr * 128 + warp * 16, c0 = tc * 128 + lane * 4;
  float m = 0.f;
  if (r0 < rows && c0 < cols) {  // rows % 16 == 0, cols % 16 == 0
    uint4 v[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = ldg128_stream(x + (r0 + j) * ld + c0);
#pragma unroll
    for (int j = 0; j < 16; ++j)
      m = fmaxf(fmaxf(m, fmaxf(fabsf(__uint_as_float(v[j].x)), fabsf(__uint_as_float(v[j].y)))),
                fmaxf(fabsf(__uint_as_float(v[j].z)), fabsf(__uint_as_float(v[j].w))));
  }
  __shared__ float red[8];
  m = warp_max(m);
  if (lane == 0) red[warp] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) t = fmaxf(t, red[w]);
    const uint32_t bits = __float_as_uint(t);  // non-negative floats order like their bit patterns
    if (out0) atomicMax(reinterpret_cast<unsigned int*>(out0), bits);
    if (out1) atomicMax(reinterpret_cast<unsigned int*>(out1), bits);
  }
}

struct F32Smem {
  static constexpr int kTile = 0;                    // 128 rows x 512 B of FP32
  static constexpr int kColCodes = 65536;            // 128 columns x 64 B
  static constexpr int kSfRow = kColCodes + 8192;    // 1 KB
  static constexpr int kSfCol = kSfRow + 1024;       // 1 KB
  static constexpr int kBlkEnc = kSfCol + 1024;      // 64 floats (16x16 mode)
  static constexpr int kBlkByte = kBlkEnc + 256;     // 64 bytes
  static constexpr int kGlobalScales = kBlkByte + 64;
  static constexpr int kRand = kGlobalScales + 64;   // 128 rows x 128 B, chunk cb of row r at slot cb ^ ((r >> 2) & 7)
  static constexpr int kBytesNoRand = kRand;
  static constexpr int kBytesRand = kRand + 16384;
};

// Pass 2: one CTA per 128 x 128 tile, phases as in quantize_kernel (row-wise copy from registers + staging,
// transposed copy from the staged tile, 16-byte stores of codes and scale atoms).
template <bool HAS_ROW, bool HAS_COL, bool BLOCK2D, bool SR>
__global__ void __launch_bounds__(256, 2) quantize_f32_kernel(const QuantArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  const float* __restrict__ src = reinterpret_cast<const float*>(a.x);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = (int)(gridDim.x - 1 - blockIdx.x);  // reverse order: the tail of pass 1 is still in L2
  const int64_t row0 = (int64_t)(tile / a.tiles_c) * 128;
  const int64_t col0 = (int64_t)(tile % a.tiles_c) * 128;
  const int64_t n_cb = a.cols >> 4, n_rb = a.rows >> 4;

  float* g_sc = reinterpret_cast<float*>(smem + F32Smem::kGlobalScales);
  if (threadIdx.x == 0) {  // Eq. 1 once per CTA
    float re = 1.f, rd = 1.f, ce = 1.f, cd = 1.f;
    if (HAS_ROW || BLOCK2D) global_scales(HAS_ROW ? a.r_global[0] : a.c_global[0], re, rd);
    if (HAS_COL) {
      if (BLOCK2D && HAS_ROW) {
        ce = re;
        cd = rd;
      } else {
        global_scales(a.c_global[0], ce, cd);
      }
    }
    g_sc[0] = re; g_sc[1] = rd; g_sc[2] = ce; g_sc[3] = cd;
    if (blockIdx.x == 0) {
      if (HAS_ROW) a.r_global[1] = rd;
      if (HAS_COL) a.c_global[1] = cd;
    }
  }

  // ------------------------------------------------------------------ phase 1 ----
  const int cb = lane & 7;
  float f[4][16];
  bool ok[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = warp * 16 + i * 4 + (lane >> 3);
    ok[i] = (row0 + r < a.rows) && (col0 + cb * 16 < a.cols);
    if (ok[i]) {
      const float* p = src + (row0 + r) * a.ld + col0 + cb * 16;
      ldg256_stream_f(p, *reinterpret_cast<float(*)[8]>(&f[i][0]));
      ldg256_stream_f(p + 8, *reinterpret_cast<float(*)[8]>(&f[i][8]));
    } else {
#pragma unroll
      for (int k = 0; k < 16; ++k) f[i][k] = 0.f;
    }
  }
  if (HAS_COL) {
    // stage the tile; quarter s (16 bytes) of a 64-byte chunk sits at slot s ^ ((cb >> 1) & 3), so that the eight
    // lanes of a quarter warp (chunks 64 bytes apart) cover all banks with every store
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = warp * 16 + i * 4 + (lane >> 3);
      uint8_t* dst = smem + F32Smem::kTile + r * 512 + cb * 64;
#pragma unroll
      for (int s = 0; s < 4; ++s)
        *reinterpret_cast<float4*>(dst + ((s ^ ((cb >> 1) & 3)) << 4)) =
            make_float4(f[i][4 * s], f[i][4 * s + 1], f[i][4 * s + 2], f[i][4 * s + 3]);
    }
  }
  __syncthreads();
  const float r_senc = g_sc[0], r_sdec = g_sc[1], c_senc = g_sc[2], c_sdec = g_sc[3];

  uint32_t blk_byte = 0;
  float blk_enc = 0.f;
  if (BLOCK2D) {
    float m = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) m = fmaxf(m, amax16(f[i]));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 8));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 16));
    block_scales(m, r_senc, r_sdec, blk_byte, blk_enc);
    if (lane < 8) {
      reinterpret_cast<float*>(smem + F32Smem::kBlkEnc)[warp * 8 + cb] = blk_enc;
      smem[F32Smem::kBlkByte + warp * 8 + cb] = (uint8_t)blk_byte;
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = warp * 16 + i * 4 + (lane >> 3);
    uint32_t rnd[4] = {0u, 0u, 0u, 0u};
    if (SR) {
      const uint64_t g = (uint64_t)(row0 + r) * (uint64_t)n_cb + (uint64_t)((col0 >> 4) + cb);
      uint4 q = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), a.off_lo, a.off_hi, a.rk);
      rnd[0] = q.x; rnd[1] = q.y; rnd[2] = q.z; rnd[3] = q.w;
      if (HAS_COL) {
        uint4 qc = q;
        if (a.off_hi_col != a.off_hi)
          qc = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), a.off_lo, a.off_hi_col, a.rk);
        *reinterpret_cast<uint4*>(smem + F32Smem::kRand + r * 128 + ((cb ^ ((r >> 2) & 7)) << 4)) = qc;
      }
    }
    if (HAS_ROW) {
      uint32_t byte;
      float enc;
      if (BLOCK2D) {
        byte = blk_byte;
        enc = blk_enc;
      } else {
        block_scales(amax16(f[i]), r_senc, r_sdec, byte, enc);
      }
      const uint2 codes = convert16<SR>(f[i], enc, Nu14FromWords{rnd});
      if (ok[i])
        *reinterpret_cast<uint2*>(a.r_codes + (row0 + r) * (a.cols >> 1) + ((col0 + cb * 16) >> 1)) = codes;
      const int pos = a.r_swz ? ((cb >> 2) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (cb & 3)) : (r * 8 + cb);
      smem[F32Smem::kSfRow + pos] = (uint8_t)byte;
    }
  }
  __syncthreads();

  // ------------------------------------------------------------------ phase 2 ----
  if (HAS_COL) {
    const int q = warp;  // 16-row group inside the tile
#pragma unroll 1
    for (int it = 0; it < 2; ++it) {
      const int cp = lane + 32 * it;  // column pair: tile columns 2cp, 2cp+1
      float f0[16], f1[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        // columns 2cp, 2cp+1: chunk cp >> 3, quarter (cp >> 1) & 3 at its swizzled slot
        const float2 w = *reinterpret_cast<const float2*>(
            smem + F32Smem::kTile + (q * 16 + j) * 512 + (cp >> 3) * 64 +
            (((((cp >> 1) & 3) ^ ((cp >> 4) & 3))) << 4) + (cp & 1) * 8);
        f0[j] = w.x;
        f1[j] = w.y;
      }
      uint32_t byte0, byte1;
      float enc0, enc1;
      if (BLOCK2D) {
        enc0 = enc1 = reinterpret_cast<const float*>(smem + F32Smem::kBlkEnc)[q * 8 + (cp >> 3)];
        byte0 = byte1 = smem[F32Smem::kBlkByte + q * 8 + (cp >> 3)];
      } else {
        block_scales(amax16(f0), c_senc, c_sdec, byte0, enc0);
        block_scales(amax16(f1), c_senc, c_sdec, byte1, enc1);
      }
      uint32_t two[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        two[j] = 0u;
        if (SR)
          two[j] = *reinterpret_cast<const uint16_t*>(smem + F32Smem::kRand + (q * 16 + j) * 128 +
                                                      (((cp >> 3) ^ ((4 * q + (j >> 2)) & 7)) << 4) + (cp & 7) * 2);
      }
      const uint2 codes0 = convert16<SR>(f0, enc0, Nu14FromPairs<0>{two});
      const uint2 codes1 = convert16<SR>(f1, enc1, Nu14FromPairs<1>{two});
      const int sel = (lane >> 3) & 1;
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        const int odd = s ^ sel;
        const int c = 2 * cp + odd;
        const uint2 val = odd ? codes1 : codes0;
        *reinterpret_cast<uint2*>(smem + F32Smem::kColCodes + c * 64 + (((q ^ (c >> 1)) & 7) << 3)) = val;
        const uint32_t byte = odd ? byte1 : byte0;
        const int pos = a.c_swz ? ((q >> 2) * 512 + (c & 31) * 16 + (c >> 5) * 4 + (q & 3)) : (c * 8 + q);
        smem[F32Smem::kSfCol + pos] = (uint8_t)byte;
      }
    }
  }
  __syncthreads();

  // ------------------------------------------------------------------ phase 3 ----
  if (HAS_COL) {
    const int64_t pitch = a.rows >> 1;
    const bool vec16 = (a.rows & 31) == 0;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int unit = threadIdx.x + 256 * k;
      const int c = unit >> 2, m = unit & 3;
      if (col0 + c >= a.cols) continue;
      const int x = (c >> 1) & 7;
      uint4 v = *reinterpret_cast<const uint4*>(smem + F32Smem::kColCodes + c * 64 + ((((2 * m) ^ x) & 6) << 3));
      if (x & 1) v = make_uint4(v.z, v.w, v.x, v.y);
      uint8_t* dst = a.c_codes + (col0 + c) * pitch + (row0 >> 1) + m * 16;
      const int64_t rr = row0 + 32 * m;
      if (rr + 16 < a.rows && vec16) {
        *reinterpret_cast<uint4*>(dst) = v;
      } else {
        if (rr < a.rows) *reinterpret_cast<uint2*>(dst) = make_uint2(v.x, v.y);
        if (rr + 16 < a.rows) *reinterpret_cast<uint2*>(dst + 8) = make_uint2(v.z, v.w);
      }
    }
  }
#pragma unroll
  for (int which = 0; which < 2; ++which) {
    if (which == 0 && !HAS_ROW) continue;
    if (which == 1 && !HAS_COL) continue;
    const uint8_t* sp = smem + (which == 0 ? F32Smem::kSfRow : F32Smem::kSfCol);
    uint8_t* dst = which == 0 ? a.r_scales : a.c_scales;
    const int swz = which == 0 ? a.r_swz : a.c_swz;
    const int64_t R0 = which == 0 ? row0 : col0, K0 = which == 0 ? (col0 >> 4) : (row0 >> 4);
    const int64_t Rn = which == 0 ? a.rows : a.cols, n_kb = which == 0 ? n_cb : n_rb;
    if (swz) {
      if (threadIdx.x < 64) {
        const int atom = threadIdx.x >> 5;
        if (K0 + atom * 4 < n_kb) {
          const int64_t off = ((R0 >> 7) * (n_kb >> 2) + (K0 >> 2) + atom) * 512 + (threadIdx.x & 31) * 16;
          *reinterpret_cast<uint4*>(dst + off) = *reinterpret_cast<const uint4*>(sp + threadIdx.x * 16);
        }
      }
    } else {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int idx = threadIdx.x * 4 + k;
        const int r = idx >> 3, kb = idx & 7;
        if (R0 + r < Rn && K0 + kb < n_kb) dst[(R0 + r) * n_kb + K0 + kb] = sp[idx];
      }
    }
  }
}

cudaError_t launch_amax_f32(const QuantArgs& a, bool has_row, bool has_col, cudaStream_t s) {
  cudaError_t e;
  if (has_row && (e = cudaMemsetAsync(a.r_global, 0, sizeof(float), s)) != cudaSuccess) return e;
  if (has_col && (e = cudaMemsetAsync(a.c_global, 0, sizeof(float), s)) != cudaSuccess) return e;
  const int tiles_c = (int)((a.cols + 127) / 128);
  const unsigned tiles = (unsigned)(((a.rows + 127) / 128) * tiles_c);
  amax_f32_kernel<<<tiles, 256, 0, s>>>(reinterpret_cast<const float*>(a.x), a.rows, a.cols, a.ld, tiles_c,
                                        has_row ? a.r_global : nullptr, has_col ? a.c_global : nullptr);
  count_launch();
  return cudaGetLastError();
}

template <bool HR, bool HC, bool B2, bool SR>
static cudaError_t launch_f32_t(const QuantArgs& a, cudaStream_t s) {
  auto kern = quantize_f32_kernel<HR, HC, B2, SR>;
  const int smem = (SR && HC) ? F32Smem::kBytesRand : F32Smem::kBytesNoRand;
  static std::atomic<uint64_t> configured{0};  // per call site (template instantiation) and device
  int dev;
  if (device_needs_config(configured, &dev)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, F32Smem::kBytesRand);
    if (e != cudaSuccess) return e;
    device_configured(configured, dev);
  }
  kern<<<(unsigned)((int64_t)a.tiles_r * a.tiles_c), 256, smem, s>>>(a);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_quantize_f32(const QuantArgs& a, bool has_row, bool has_col, bool block2d, bool sr, cudaStream_t s) {
#define NVFP4_F32Q(HR, HC, B2, SRV) \
  if (has_row == HR && has_col == HC && block2d == B2 && sr == SRV) return launch_f32_t<HR, HC, B2, SRV>(a, s);
#define NVFP4_F32Q_COPIES(B2, SRV) \
  NVFP4_F32Q(true, false, B2, SRV)  \
  NVFP4_F32Q(false, true, B2, SRV)  \
  NVFP4_F32Q(true, true, B2, SRV)
  NVFP4_F32Q_COPIES(true, false)
  NVFP4_F32Q_COPIES(true, true)
  NVFP4_F32Q_COPIES(false, false)
  NVFP4_F32Q_COPIES(false, true)
#undef NVFP4_F32Q_COPIES
#undef NVFP4_F32Q
  return cudaErrorInvalidValue;
}

}  // namespace nvfp4
