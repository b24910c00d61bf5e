// Test-only helper: exposes the CUDA toolkit's HOST conversion routines so the oracle's
// E2M1 / E4M3 rounding can be cross-checked against a library implementation.
#include <cuda_fp4.h>
#include <cuda_fp8.h>
extern "C" unsigned char nv_host_e2m1_rne(float x) {
  return (unsigned char)__nv_cvt_float_to_fp4(x, __NV_E2M1, cudaRoundNearest);
}
extern "C" unsigned char nv_host_e4m3_satfinite(float x) {
  return (unsigned char)__nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3);
}
