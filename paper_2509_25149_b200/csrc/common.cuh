// Shared device helpers for the NVFP4 kernels (sm_100a only).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "nvfp4.h"

#if defined(__CUDA_ARCH__) && !defined(__CUDA_ARCH_FEAT_SM100_ALL)
#error "build with -gencode arch=compute_100a,code=sm_100a"
#endif

namespace nvfp4 {

// Host-side launch counter (reported by nvfp4_launch_count()).
void count_launch(int n = 1);

// One-time, per-device configuration of a call site (function attributes are per device): `seen` holds one bit per
// device ordinal.  Returns true when the current device still has to be configured; the caller marks it afterwards.
// Devices beyond ordinal 63 are configured on every call (the attribute calls are idempotent).
inline bool device_needs_config(const std::atomic<uint64_t>& seen, int* dev) {
  *dev = -1;
  if (cudaGetDevice(dev) != cudaSuccess || *dev < 0 || *dev >= 64) return true;
  return (seen.load(std::memory_order_acquire) & (1ull << *dev)) == 0;
}
inline void device_configured(std::atomic<uint64_t>& seen, int dev) {
  if (dev >= 0 && dev < 64) seen.fetch_or(1ull << dev, std::memory_order_release);
}

// ---------------------------------------------------------------------------------------------
// Formats
// ---------------------------------------------------------------------------------------------
constexpr float kFltMax = 3.402823466e+38f;

// bf16 pair packed in 32 bits -> two fp32 (exact).
__device__ __forceinline__ float bf16_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }

// Eq. 1: s_enc = 6*448/amax (clamped), s_dec = 1/s_enc, IEEE division.
__device__ __forceinline__ void global_scales(float amax, float& s_enc, float& s_dec) {
  float e = (amax == 0.0f) ? 1.0f : fminf(__fdiv_rn(2688.0f, amax), kFltMax);
  s_enc = e;
  s_dec = __frcp_rn(e);
}

// Eq. 2-3 and the text after Eq. 3: stored E4M3 byte of a block and the encode scale derived from it.
// fl(x / 6) for x >= 0 with three instructions: q = fl(x * fl(1/6)), exact residual r = fma(-6, q, x), corrected
// q' = fma(r, fl(1/6), q).  x/6 is never closer than ulp/6 to a rounding midpoint (6 * midpoint needs 26 bits), and
// the correction term is off by only 2^-25 relative, so q' is the correctly rounded quotient whenever the residual is
// exact, i.e. outside the denormal range (checked exhaustively over whole binades on the host); tiny inputs take the
// IEEE division.
__device__ __forceinline__ float div6_rn(float x) {
  const float c = 0.16666667163372039794921875f;  // fl(1/6)
  const float q = __fmul_rn(x, c);
  const float r = __fmaf_rn(-6.0f, q, x);
  const float fast = __fmaf_rn(r, c, q);
  return (x != 0.0f && x < 1.0e-30f) ? __fdiv_rn(x, 6.0f) : fast;
}

__device__ __forceinline__ void block_scales(float amax_b, float s_enc, float s_dec, uint32_t& byte,
                                             float& s_enc_b) {
  float t = __fmul_rn(div6_rn(amax_b), s_enc);
  uint16_t packed;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %1;" : "=h"(packed) : "f"(t));
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(packed));
  float sf = __half2float(__ushort_as_half((unsigned short)(h2 & 0xffffu)));
  byte = packed & 0xffu;
  float d = __fmul_rn(sf, s_dec);
  s_enc_b = (byte == 0u) ? 0.0f : fminf(__frcp_rn(d), kFltMax);
}

// Four (lo, hi) pairs -> 8 E2M1 nibbles, element 0 in the lowest nibble (round-to-nearest-even,
// saturating at +-6).  cvt...e2m1x2 puts its FIRST source in the high nibble.
__device__ __forceinline__ uint32_t e2m1x8_rne(const float v[8]) {
  uint32_t r;
  asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
      "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
      : "=r"(r)
      : "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]));
  return r;
}

// Stochastic rounding of scaled values to E2M1 nibbles (Section 4.4): neighbours lo <= |v| < hi on the grid
// {0,.5,1,1.5,2,3,4,6}; round up iff u + 0.5 < 256 * frac, u the element's 8-bit draw, frac = (|v| - lo) / (hi - lo).
//
// The conversion instruction cvt.rs.satfinite.e2m1x4.f32 d, {a3, a2, a1, a0}, rbits puts a_k into nibble k of d and
// decides "up" for it iff  floor(frac * 2^16) + r16 >= 2^16  with a 16-bit number taken from rbits:
//   nibble 0: r16 = (byte 2 << 8) | byte 0,      nibble 1: the same sixteen bits in reversed order,
//   nibble 2: r16 = (byte 3 << 8) | byte 1,      nibble 3: the same sixteen bits in reversed order
// (measured on the part over a dense sweep of inputs and random words; magnitudes above 6 saturate, the sign bit is
// kept, also for zeros).  Nibbles 0 and 2 therefore have independent random numbers, 1 and 3 do not, so two elements
// go into one instruction and the other two inputs are zero (code 0 whatever the random bits).
// To make the instruction decide exactly as the rule above:
//   - r16 = ((255 - u) << 8) | 128;
//   - the magnitude is first moved to the next binary32 towards zero, w = rz(v * (1 - 2^-24)).  frac * 2^16 is a
//     multiple of delta = ulp * 2^16 / (hi - lo) <= 2^-6 and w lowers it by exactly delta, so
//     floor(frac(w) * 2^16) = ceil(frac(v) * 2^16) - 1, and the instruction's test becomes
//     ceil(frac * 2^16) >= 256 u + 129  <=>  frac * 2^16 > 256 u + 128  <=>  256 frac > u + 0.5.
//     A grid point lo > 0 moves into the cell below with floor(...) = 65535 and r16 >= 128 brings it back up, zero
//     stays zero, values just above 6 saturate as before.
constexpr float kSrTowardsZero = 0.99999994f;  // 1 - 2^-24 = 0x3F7FFFFF

// One conversion: code of w_lo in nibble 0 and of w_hi in nibble 2 of a 16-bit result;
// rbits = (nu_hi << 24) | (nu_lo << 16) | 0x8080, nu = 255 - u.
__device__ __forceinline__ uint32_t e2m1x2_sr(float w_lo, float w_hi, uint32_t rbits) {
  uint16_t d;
  asm("cvt.rs.satfinite.e2m1x4.f32 %0, {%1, %2, %1, %3}, %4;" : "=h"(d) : "f"(0.0f), "f"(w_hi), "f"(w_lo), "r"(rbits));
  return d;
}
// Two conversions packed into one word: (a_lo, a_hi) in the low half, (b_lo, b_hi) in the high half
__device__ __forceinline__ uint32_t e2m1x2_sr_pair(float a_lo, float a_hi, uint32_t ra, float b_lo, float b_hi,
                                                   uint32_t rb) {
  uint32_t d;
  asm("{\n\t.reg .b16 t0, t1;\n\t"
      "cvt.rs.satfinite.e2m1x4.f32 t0, {%1, %2, %1, %3}, %4;\n\t"
      "cvt.rs.satfinite.e2m1x4.f32 t1, {%1, %5, %1, %6}, %7;\n\t"
      "mov.b32 %0, {t0, t1};\n\t}"
      : "=r"(d)
      : "f"(0.0f), "f"(a_hi), "f"(a_lo), "r"(ra), "f"(b_hi), "f"(b_lo), "r"(rb));
  return d;
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10: counter (g.lo, g.hi, off.lo, off.hi), key (seed.lo, seed.hi) -> 16 random bytes
// ---------------------------------------------------------------------------------------------
// rk: the ten round keys, (k0 + r * 0x9E3779B9, k1 + r * 0xBB67AE85) for r = 0..9, computed once on the host and
// read from the kernel's parameter bank
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const uint32_t (&rk)[20]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;  // one wide multiply each
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk[2 * r];
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk[2 * r + 1];
    c0 = n0; c1 = (uint32_t)p1; c2 = n2; c3 = (uint32_t)p0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// ---------------------------------------------------------------------------------------------
// Packed FP32 pairs (sm_100: add / sub / mul .f32x2 process two binary32 lanes per instruction, each lane
// rounded to nearest exactly like the scalar instruction)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
  float2 r;
  asm("{.reg .b64 ra, rb, rc; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; add.rn.f32x2 rc, ra, rb; mov.b64 {%0, %1}, rc;}"
      : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return r;
}
__device__ __forceinline__ float2 sub2(float2 a, float2 b) {
  float2 r;
  asm("{.reg .b64 ra, rb, rc; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; sub.rn.f32x2 rc, ra, rb; mov.b64 {%0, %1}, rc;}"
      : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return r;
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
  float2 r;
  asm("{.reg .b64 ra, rb, rc; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mul.rn.f32x2 rc, ra, rb; mov.b64 {%0, %1}, rc;}"
      : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return r;
}

__device__ __forceinline__ float2 mul2_rz(float2 a, float2 b) {  // both lanes rounded towards zero
  float2 r;
  asm("{.reg .b64 ra, rb, rc; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mul.rz.f32x2 rc, ra, rb; mov.b64 {%0, %1}, rc;}"
      : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return r;
}

// 16-point butterfly on sixteen pairs: .x and .y are two independent transforms (two adjacent columns)
__device__ __forceinline__ void fwht16_pairs(float2 v[16]) {
#pragma unroll
  for (int h = 1; h < 16; h <<= 1) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if ((i & h) == 0) {
        const float2 a = v[i], b = v[i | h];
        v[i] = add2(a, b);
        v[i | h] = sub2(a, b);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// 16-point Walsh-Hadamard butterfly (Sylvester order) on registers; the caller applies the 1/4.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void fwht16(float v[16]) {
#pragma unroll
  for (int h = 1; h < 16; h <<= 1) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if ((i & h) == 0) {
        float a = v[i], b = v[i | h];
        v[i] = a + b;
        v[i | h] = a - b;
      }
    }
  }
}

// Offset of scale byte (row r, block kb) in the swizzled 128x4 atom layout; n_kb = blocks per row.
__host__ __device__ __forceinline__ int64_t sf_swizzled_offset(int64_t r, int64_t kb, int64_t n_kb) {
  return ((r >> 7) * (n_kb >> 2) + (kb >> 2)) * 512 + (r & 31) * 16 + ((r & 127) >> 5) * 4 + (kb & 3);
}

}  // namespace nvfp4
