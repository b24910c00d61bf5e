// Quantization-error reductions (Appendix E.2 of the paper: error metrics as a way to decide which linear layers
// stay in higher precision).  Two HBM-bound kernels:
//   quant_error_kernel : sum (x - decode(q))^2 and sum x^2 of a row-wise quantized copy against its bf16 source,
//                        decoding on the fly (2 + 0.5 + 1/16 bytes per element);
//   sq_error_kernel    : the same two sums between two dense tensors (bf16 or fp32 each), e.g. a weight gradient
//                        from the FP4 GEMM against the one from the BF16 GEMM.
// A thread sums 16 elements in FP32 and adds that into an FP64 partial; warps and CTAs are combined in FP64 and
// leave through one atomicAdd pair per CTA.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "quantize.h"
#include "quantize_common.cuh"

namespace nvfp4 {

namespace {

__device__ __forceinline__ void block_reduce_add(double err, double ref, double* out) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    err += __shfl_xor_sync(0xffffffffu, err, o);
    ref += __shfl_xor_sync(0xffffffffu, ref, o);
  }
  __shared__ double red[2][8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    red[0][warp] = err;
    red[1][warp] = ref;
  }
  __syncthreads();
  if (threadIdx.x < 2) {
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += red[threadIdx.x][w];
    atomicAdd(out + threadIdx.x, s);
  }
}

// i = r * n + c with c < n: 32-bit division whenever the index allows (the 64-bit one costs as much as the rest of a
// 16-element chunk)
__device__ __forceinline__ void split_index(int64_t i, int64_t n, int64_t& r, int64_t& c) {
  if (i <= 0xffffffffll && n <= 0xffffffffll) {
    const uint32_t q = (uint32_t)i / (uint32_t)n;
    r = q;
    c = (uint32_t)i - q * (uint32_t)n;
  } else {
    r = i / n;
    c = i - r * n;
  }
}

// one byte of codes -> its two E2M1 values (low nibble first)
__device__ __forceinline__ float2 e2m1x2_values(uint32_t byte) {
  uint32_t h2;
  asm("{\n\t.reg .b8 lo, hi;\n\t"
      "mov.b16 {lo, hi}, %1;\n\t"
      "cvt.rn.f16x2.e2m1x2 %0, lo;\n\t}"
      : "=r"(h2)
      : "h"((uint16_t)byte));
  return __half22float2(*reinterpret_cast<__half2*>(&h2));
}

template <bool MX>
__global__ void __launch_bounds__(256) quant_error_kernel(const uint16_t* __restrict__ x, int64_t rows, int64_t cols,
                                                          int64_t ld, const uint8_t* __restrict__ codes,
                                                          const uint8_t* __restrict__ scales,
                                                          const float* __restrict__ global, int swz,
                                                          int per_row, double* __restrict__ out) {
  const int64_t n_cb = cols >> 4;                 // 16-element chunks per row
  const int64_t n_sb = MX ? (cols >> 5) : n_cb;   // scale blocks per row
  const int64_t n_chunks = rows * n_cb;
  const float s_dec_t = MX ? 1.f : global[1];
  double err = 0.0, ref = 0.0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n_chunks; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t r, cb;
    split_index(i, n_cb, r, cb);
    uint32_t raw[8];
    ldg256_stream(x + r * ld + cb * 16, raw);
    const uint2 c = *reinterpret_cast<const uint2*>(codes + r * (cols >> 1) + cb * 8);
    const int64_t sb = MX ? (cb >> 1) : cb;
    const uint32_t byte = scales[swz ? sf_swizzled_offset(r, sb, n_sb) : (r * n_sb + sb)];
    float sf;
    if (MX) {
      sf = byte == 0 ? __uint_as_float(0x00400000u) : __uint_as_float(byte << 23);  // 2^(byte - 127)
    } else {
      uint32_t h2;
      asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)byte));
      sf = __half2float(__ushort_as_half((unsigned short)(h2 & 0xffffu)));
    }
    const float scale = __fmul_rn(sf, per_row ? global[2 * r + 1] : s_dec_t);  // per_row: {amax, s_dec} per row
    float e = 0.f, n = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float2 q = e2m1x2_values(((k < 4 ? c.x : c.y) >> (8 * (k & 3))) & 0xffu);
      const float x0 = bf16_lo(raw[k]), x1 = bf16_hi(raw[k]);
      const float d0 = x0 - q.x * scale, d1 = x1 - q.y * scale;
      e = fmaf(d0, d0, e);
      e = fmaf(d1, d1, e);
      n = fmaf(x0, x0, n);
      n = fmaf(x1, x1, n);
    }
    err += (double)e;
    ref += (double)n;
  }
  block_reduce_add(err, ref, out);
}

template <bool FP32>
__device__ __forceinline__ void load8(const void* base, int64_t elem, float (&v)[8]) {
  if (FP32) {
    const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(base) + elem);
    const float4 a = __ldg(p), b = __ldg(p + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  } else {
    const uint4 a = ldg128_stream(static_cast<const uint16_t*>(base) + elem);
    v[0] = bf16_lo(a.x); v[1] = bf16_hi(a.x); v[2] = bf16_lo(a.y); v[3] = bf16_hi(a.y);
    v[4] = bf16_lo(a.z); v[5] = bf16_hi(a.z); v[6] = bf16_lo(a.w); v[7] = bf16_hi(a.w);
  }
}

template <bool REF32, bool TEST32>
__global__ void __launch_bounds__(256) sq_error_kernel(const void* __restrict__ refp, int64_t ld_ref,
                                                       const void* __restrict__ testp, int64_t ld_test, int64_t rows,
                                                       int64_t cols, double* __restrict__ out) {
  const int64_t n_c8 = cols >> 3, n_units = rows * n_c8;  // units of 8 elements
  double err = 0.0, ref = 0.0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n_units; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t r, c8;
    split_index(i, n_c8, r, c8);
    float a[8], b[8];
    load8<REF32>(refp, r * ld_ref + c8 * 8, a);
    load8<TEST32>(testp, r * ld_test + c8 * 8, b);
    float e = 0.f, n = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float d = a[k] - b[k];
      e = fmaf(d, d, e);
      n = fmaf(a[k], a[k], n);
    }
    err += (double)e;
    ref += (double)n;
  }
  block_reduce_add(err, ref, out);
}

cudaError_t grid_for(int64_t units, unsigned* grid) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const int64_t want = (units + 255) / 256, cap = (int64_t)sms * 8;  // eight resident CTAs per SM
  *grid = (unsigned)(want < cap ? (want > 0 ? want : 1) : cap);
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_quant_error(const void* x, int64_t rows, int64_t cols, int64_t ld, const nvfp4_tensor& q,
                               double* out, cudaStream_t s) {
  cudaError_t e = cudaMemsetAsync(out, 0, 2 * sizeof(double), s);
  if (e != cudaSuccess) return e;
  unsigned grid;
  if ((e = grid_for(rows * (cols >> 4), &grid)) != cudaSuccess) return e;
  const int swz = q.sf_layout == NVFP4_SF_SWIZZLED;
  if (q.format == NVFP4_FORMAT_MXFP4)
    quant_error_kernel<true><<<grid, 256, 0, s>>>(static_cast<const uint16_t*>(x), rows, cols, ld, q.codes, q.scales,
                                                  q.global, swz, 0, out);
  else
    quant_error_kernel<false><<<grid, 256, 0, s>>>(static_cast<const uint16_t*>(x), rows, cols, ld, q.codes, q.scales,
                                                   q.global, swz, q.format == NVFP4_FORMAT_NVFP4_ROWSCALE, out);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_sq_error(const void* ref, bool ref_fp32, int64_t ld_ref, const void* test, bool test_fp32,
                            int64_t ld_test, int64_t rows, int64_t cols, double* out, cudaStream_t s) {
  cudaError_t e = cudaMemsetAsync(out, 0, 2 * sizeof(double), s);
  if (e != cudaSuccess) return e;
  unsigned grid;
  if ((e = grid_for(rows * (cols >> 3), &grid)) != cudaSuccess) return e;
#define NVFP4_SQ(R, T)                                                                                        \
  if (ref_fp32 == R && test_fp32 == T)                                                                        \
    sq_error_kernel<R, T><<<grid, 256, 0, s>>>(ref, ld_ref, test, ld_test, rows, cols, out);
  NVFP4_SQ(false, false)
  NVFP4_SQ(false, true)
  NVFP4_SQ(true, false)
  NVFP4_SQ(true, true)
#undef NVFP4_SQ
  count_launch();
  return cudaGetLastError();
}

}  // namespace nvfp4
