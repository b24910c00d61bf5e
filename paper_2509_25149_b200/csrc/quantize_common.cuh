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

// Eq. 4 for sixteen values: v = fl(y * s_enc,b), two lanes per instruction; for stochastic rounding the result is
// then moved one binary32 towards zero, which is what e2m1x2_sr() expects.
template <bool SR>
__device__ __forceinline__ void scale16(const float (&f)[16], float s_enc_b, float (&v)[16]) {
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    float2 p = mul2(make_float2(f[i], f[i + 1]), make_float2(s_enc_b, s_enc_b));
    if (SR) p = mul2_rz(p, make_float2(kSrTowardsZero, kSrTowardsZero));
    v[i] = p.x;
    v[i + 1] = p.y;
  }
}

// 16 scaled values -> 16 E2M1 nibbles (element 0 in the lowest nibble of .x).  For stochastic rounding
// `draws.rbits(i, j)` returns the random word of e2m1x2_sr() for elements i (low) and j (high).
template <bool SR, class Draws>
__device__ __forceinline__ uint2 convert16(const float (&f)[16], float s_enc_b, Draws draws) {
  uint2 out;
  float v[16];
  scale16<SR>(f, s_enc_b, v);
  if (!SR) {
    const float(&lo)[8] = *reinterpret_cast<const float(*)[8]>(&v[0]);
    const float(&hi)[8] = *reinterpret_cast<const float(*)[8]>(&v[8]);
    out.x = e2m1x8_rne(lo);
    out.y = e2m1x8_rne(hi);
  } else {
    // nibbles 0 and 2 of each 16-bit half: elements (4k, 4k + 2) in `even`, (4k + 1, 4k + 3) in `odd`, k = 0, 1 | 2, 3
    const uint32_t even01 = e2m1x2_sr_pair(v[0], v[2], draws.rbits(0, 2), v[4], v[6], draws.rbits(4, 6));
    const uint32_t odd01 = e2m1x2_sr_pair(v[1], v[3], draws.rbits(1, 3), v[5], v[7], draws.rbits(5, 7));
    const uint32_t even23 = e2m1x2_sr_pair(v[8], v[10], draws.rbits(8, 10), v[12], v[14], draws.rbits(12, 14));
    const uint32_t odd23 = e2m1x2_sr_pair(v[9], v[11], draws.rbits(9, 11), v[13], v[15], draws.rbits(13, 15));
    out.x = even01 + odd01 * 16u;  // disjoint nibbles: the sum is the union
    out.y = even23 + odd23 * 16u;
  }
  return out;
}

// draws packed four to a word, byte i = element i (the row-wise copy: straight from the Philox output)
struct Nu14FromWords {
  const uint32_t (&rnd)[4];
  __device__ __forceinline__ uint32_t rbits(int i, int j) const {  // i, j in the same word, i even <=> j even
    return __byte_perm(~rnd[i >> 2], 0x80808080u, (i & 1) ? 0x3144u : 0x2044u);
  }
};
// draws of two adjacent columns, 16 bits per row (the transposed copy: read back from shared memory)
template <int COL>
struct Nu14FromPairs {
  const uint32_t (&two)[16];
  __device__ __forceinline__ uint32_t rbits(int i, int j) const {
    const uint32_t picked = __byte_perm(two[i], two[j], COL == 0 ? 0x4000u : 0x5100u);  // bytes 2, 3 = draws of i, j
    return (~picked & 0xFFFF0000u) | 0x8080u;
  }
};

// Two columns of sixteen rows at once (the transposed copy of the main kernel): element j of both columns goes into
// one conversion.  ntwo[j]: low byte = 255 - draw of (row j, first column), next byte = the same for the second one.
__device__ __forceinline__ void convert16x2_sr(const float (&f0)[16], const float (&f1)[16], float enc0, float enc1,
                                               const uint32_t (&ntwo)[16], uint2& out0, uint2& out1) {
  float v0[16], v1[16];
  scale16<true>(f0, enc0, v0);
  scale16<true>(f1, enc1, v1);
  // rows (r, r + 1) of both columns: byte 0 = first column, byte 1 = second column; rows (r + 2, r + 3) in bytes 2, 3
  uint32_t e[4];
#pragma unroll
  for (int m = 0; m < 4; ++m) {
    const int r = 4 * m;
    const uint32_t a = e2m1x2_sr_pair(v0[r], v1[r], __byte_perm(ntwo[r], 0x80808080u, 0x1044u), v0[r + 2], v1[r + 2],
                                      __byte_perm(ntwo[r + 2], 0x80808080u, 0x1044u));
    const uint32_t b = e2m1x2_sr_pair(v0[r + 1], v1[r + 1], __byte_perm(ntwo[r + 1], 0x80808080u, 0x1044u), v0[r + 3],
                                      v1[r + 3], __byte_perm(ntwo[r + 3], 0x80808080u, 0x1044u));
    e[m] = a + b * 16u;  // disjoint nibbles
  }
  out0 = make_uint2(__byte_perm(e[0], e[1], 0x6420u), __byte_perm(e[2], e[3], 0x6420u));
  out1 = make_uint2(__byte_perm(e[0], e[1], 0x7531u), __byte_perm(e[2], e[3], 0x7531u));
}

__device__ __forceinline__ float amax16(const float (&f)[16]) {
  float m = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(f[i]));
  return m;
}

}  // namespace nvfp4
