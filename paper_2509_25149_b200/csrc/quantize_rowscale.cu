// Single-pass NVFP4 quantizer with the FP32 "global" scale taken per ROW instead of per tensor (the closing remark of
// Appendix B.1: a global scale spanning a row or a block of elements avoids the extra trip through device memory
// that the tensor amax costs).  Row-wise copy only: a scale per row of the copy is constant along the contraction
// dimension, so the GEMM can apply it in its epilogue as a vector; the transposed copy of the same tensor would need
// a statistic over all source rows, i.e. the pass this variant exists to remove.
//
// CTAs of four warps.  A row of up to 5120 elements is held in the registers of ONE warp between the amax step and the
// encoding (ten 16-element chunks per lane), a row of up to 10240 / 20480 elements in those of two / four warps, which
// exchange their partial maxima through shared memory: one read from HBM in every case.  Longer rows are read a second
// time (from L1 / L2).  Eq. 1 per row, Eq. 2-4 as in the main quantizer; stochastic-rounding draws are keyed by the
// element's position in the source, as everywhere.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "quantize.h"
#include "quantize_common.cuh"

namespace nvfp4 {

namespace {

constexpr int kKeep = 10;  // chunks of 16 elements a lane holds: 10 * 32 * 16 = 5120 elements per warp

__device__ __forceinline__ void ldg256_cached(const void* p, uint32_t (&r)[8]) {
  const uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
  const uint4 b = __ldg(reinterpret_cast<const uint4*>(p) + 1);
  r[0] = a.x; r[1] = a.y; r[2] = a.z; r[3] = a.w; r[4] = b.x; r[5] = b.y; r[6] = b.z; r[7] = b.w;
}

template <bool SR>
__device__ __forceinline__ void encode_chunk(const QuantArgs& a, const uint32_t (&raw)[8], int64_t row, int64_t cb,
                                             int64_t n_cb, float s_enc, float s_dec) {
  uint32_t acc = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) acc = absmax_bf16x2(acc, raw[k]);
  uint32_t byte;
  float enc;
  block_scales(fmaxf(bf16_lo(acc), bf16_hi(acc)), s_enc, s_dec, byte, enc);
  float f[16];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    f[2 * k] = bf16_lo(raw[k]);
    f[2 * k + 1] = bf16_hi(raw[k]);
  }
  uint32_t rnd[4] = {0u, 0u, 0u, 0u};
  if (SR) {
    const uint64_t g = (uint64_t)row * (uint64_t)n_cb + (uint64_t)cb;
    const uint4 q = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), a.off_lo, a.off_hi, a.rk);
    rnd[0] = q.x; rnd[1] = q.y; rnd[2] = q.z; rnd[3] = q.w;
  }
  const uint2 codes = convert16<SR>(f, enc, Nu14FromWords{rnd});
  *reinterpret_cast<uint2*>(a.r_codes + row * (a.cols >> 1) + cb * 8) = codes;
  a.r_scales[a.r_swz ? sf_swizzled_offset(row, cb, n_cb) : (row * n_cb + cb)] = (uint8_t)byte;
}

// WPR warps per row (1, 2 or 4): warp w of the CTA holds chunks [(w % WPR) * 320, ...) of row (4 / WPR) * i + w / WPR.
template <bool SR, int WPR>
__global__ void __launch_bounds__(128, 4) quantize_rowscale_kernel(const QuantArgs a) {
  __shared__ float part[2][4];  // partial maxima, double-buffered across iterations
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kRowsPerCta = 4 / WPR;
  const int seg = warp % WPR, sub = warp / WPR;
  const int64_t n_cb = a.cols >> 4;
  int it = 0;
  // every warp of a CTA runs the same number of iterations (rows are padded), so the barriers below are uniform
  for (int64_t base = (int64_t)blockIdx.x * kRowsPerCta; base < a.rows; base += (int64_t)gridDim.x * kRowsPerCta, ++it) {
    const int64_t row = base + sub;
    const bool live = row < a.rows;
    const uint16_t* src = a.x + (live ? row : 0) * a.ld;
    uint32_t keep[kKeep][8];
    uint32_t acc = 0;
#pragma unroll
    for (int i = 0; i < kKeep; ++i) {
      const int64_t cb = (int64_t)seg * (kKeep * 32) + lane + 32 * i;
      if (live && cb < n_cb) {
        ldg256_stream(src + cb * 16, keep[i]);
      } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) keep[i][k] = 0u;
      }
    }
#pragma unroll
    for (int i = 0; i < kKeep; ++i)
#pragma unroll
      for (int k = 0; k < 8; ++k) acc = absmax_bf16x2(acc, keep[i][k]);
    float amax = warp_max(fmaxf(bf16_lo(acc), bf16_hi(acc)));
    if (WPR > 1) {
      if (lane == 0) part[it & 1][warp] = amax;
      __syncthreads();
#pragma unroll
      for (int w = 0; w < WPR; ++w) amax = fmaxf(amax, part[it & 1][sub * WPR + w]);
    }
    float s_enc, s_dec;
    global_scales(amax, s_enc, s_dec);  // Eq. 1 with the row's amax
    if (live && seg == 0 && lane == 0) {
      a.r_global[2 * row] = amax;
      a.r_global[2 * row + 1] = s_dec;
    }
    if (live) {
#pragma unroll
      for (int i = 0; i < kKeep; ++i) {
        const int64_t cb = (int64_t)seg * (kKeep * 32) + lane + 32 * i;
        if (cb < n_cb) encode_chunk<SR>(a, keep[i], row, cb, n_cb, s_enc, s_dec);
      }
    }
  }
}

// rows longer than 4 * 5120 elements: one warp per row, two sweeps (the second one from L1 / L2)
template <bool SR>
__global__ void __launch_bounds__(256) quantize_rowscale_long_kernel(const QuantArgs a) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t n_cb = a.cols >> 4;
  for (int64_t row = (int64_t)blockIdx.x * 8 + warp; row < a.rows; row += (int64_t)gridDim.x * 8) {
    const uint16_t* src = a.x + row * a.ld;
    uint32_t acc = 0;
    for (int64_t cb0 = 0; cb0 < n_cb; cb0 += 128) {  // four independent loads per lane in flight
      uint32_t raw[4][8];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int64_t cb = cb0 + lane + 32 * u;
        if (cb < n_cb) {
          ldg256_cached(src + cb * 16, raw[u]);  // allocate in L1: the second sweep comes back for it
        } else {
#pragma unroll
          for (int k = 0; k < 8; ++k) raw[u][k] = 0u;
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int k = 0; k < 8; ++k) acc = absmax_bf16x2(acc, raw[u][k]);
    }
    const float amax = warp_max(fmaxf(bf16_lo(acc), bf16_hi(acc)));
    float s_enc, s_dec;
    global_scales(amax, s_enc, s_dec);
    if (lane == 0) {
      a.r_global[2 * row] = amax;
      a.r_global[2 * row + 1] = s_dec;
    }
    for (int64_t cb0 = 0; cb0 < n_cb; cb0 += 64) {
      uint32_t raw[2][8];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int64_t cb = cb0 + lane + 32 * u;
        if (cb < n_cb) ldg256_cached(src + cb * 16, raw[u]);
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int64_t cb = cb0 + lane + 32 * u;
        if (cb < n_cb) encode_chunk<SR>(a, raw[u], row, cb, n_cb, s_enc, s_dec);
      }
    }
  }
}

template <bool SR>
cudaError_t launch_t(const QuantArgs& a, int sms, cudaStream_t s) {
  const int64_t per_warp = (int64_t)kKeep * 32 * 16;
  if (a.cols > 4 * per_warp) {
    const int64_t want = (a.rows + 7) / 8, cap = (int64_t)sms * 6;
    quantize_rowscale_long_kernel<SR><<<(unsigned)(want < cap ? want : cap), 256, 0, s>>>(a);
    return cudaGetLastError();
  }
  const int wpr = a.cols <= per_warp ? 1 : (a.cols <= 2 * per_warp ? 2 : 4);
  const int64_t want = (a.rows * wpr + 3) / 4, cap = (int64_t)sms * 4 * 4;  // four CTAs per SM, four rounds
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  if (wpr == 1) quantize_rowscale_kernel<SR, 1><<<grid, 128, 0, s>>>(a);
  else if (wpr == 2) quantize_rowscale_kernel<SR, 2><<<grid, 128, 0, s>>>(a);
  else quantize_rowscale_kernel<SR, 4><<<grid, 128, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_quantize_rowscale(const QuantArgs& a, bool sr, cudaStream_t s) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  e = sr ? launch_t<true>(a, sms, s) : launch_t<false>(a, sms, s);
  count_launch();
  return e;
}

}  // namespace nvfp4
