// Device helpers shared by the NVFP4 and the MXFP4 quantizer kernels (included by quantize.cu and quantize_mx.cu).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace nvfp4 {

// ---------------------------------------------------------------------------------------------
// small PTX helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void ldg256_stream(const void* p, uint32_t (&r)[8]) {
  asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
                 "=r"(r[7])
               : "l"(p));
}
__device__ __forceinline__ uint4 ldg128_stream(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

__device__ __forceinline__ uint32_t absmax_bf16x2(uint32_t acc, uint32_t v) {
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&acc);
  uint32_t m = v & 0x7fff7fffu;
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&m);
  __nv_bfloat162 r = __hmax2(a, b);
  return *reinterpret_cast<uint32_t*>(&r);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// sign word for a bf16 pair whose two elements are inputs j0 and j1 of a Hadamard chunk
__device__ __forceinline__ uint32_t sign_pair(uint32_t mask, int j0, int j1) {
  return (((mask >> j0) & 1u) << 15) | (((mask >> j1) & 1u) << 31);
}

// 16 scaled values -> 16 E2M1 nibbles (element 0 in the lowest nibble of .x).  For stochastic rounding `nu14(i)`
// returns the complemented 8-bit draw of element i placed in bits [21, 29).
template <bool SR, class Nu14>
__device__ __forceinline__ uint2 convert16(const float (&f)[16], float s_enc_b, Nu14 nu14) {
  uint2 out;
  float v[16];
#pragma unroll
  for (int i = 0; i < 16; i += 2) {  // Eq. 4: v = fl(y * s_enc,b), two lanes per instruction
    const float2 p = mul2(make_float2(f[i], f[i + 1]), make_float2(s_enc_b, s_enc_b));
    v[i] = p.x;
    v[i + 1] = p.y;
  }
  if (!SR) {
    const float(&lo)[8] = *reinterpret_cast<const float(*)[8]>(&v[0]);
    const float(&hi)[8] = *reinterpret_cast<const float(*)[8]>(&v[8]);
    out.x = e2m1x8_rne(lo);
    out.y = e2m1x8_rne(hi);
  } else {
    out.x = e2m1x8_sr(&v[0], nu14, 0);
    out.y = e2m1x8_sr(&v[8], nu14, 8);
  }
  return out;
}

// draws packed four to a word, byte i = element i (the row-wise copy: straight from the Philox output)
struct Nu14FromWords {
  const uint32_t (&rnd)[4];
  __device__ __forceinline__ uint32_t operator()(int i) const {
    const uint32_t nr = ~rnd[i >> 2];
    const int b = i & 3;
    return (b == 0 ? (nr << 21) : b == 1 ? (nr << 13) : b == 2 ? (nr << 5) : (nr >> 3)) & 0x1FE00000u;
  }
};
// draws of two adjacent columns, 16 bits per row (the transposed copy: read back from shared memory)
template <int COL>
struct Nu14FromPairs {
  const uint32_t (&two)[16];
  __device__ __forceinline__ uint32_t operator()(int i) const {
    return (COL == 0 ? (~two[i] << 21) : (~two[i] << 13)) & 0x1FE00000u;
  }
};

__device__ __forceinline__ float amax16(const float (&f)[16]) {
  float m = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(f[i]));
  return m;
}

}  // namespace nvfp4
