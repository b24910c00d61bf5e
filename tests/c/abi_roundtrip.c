/* Plain-C client of the library: no Python, no torch.  Quantizes two small bf16 matrices whose values lie on the
 * E2M1 grid (so quantization is exact, Appendix B), multiplies them with the block-scaled GEMM (Eq. 5) and with the
 * BF16 GEMM, and compares both results with the integer product computed here on the host.
 * Build: gcc abi_roundtrip.c -I<repo>/include -I<cuda>/include -L<libdir> -lnvfp4_b200 -L<cuda>/lib64 -lcudart
 * Exit code 0 = all checks passed. */
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "nvfp4.h"

#define M 256
#define N 256
#define K 512

static uint16_t bf16_of(float f) { /* exact for the small values used here */
  uint32_t u;
  memcpy(&u, &f, 4);
  return (uint16_t)(u >> 16);
}
static float f32_of_bf16(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}
#define CK(call)                                                          \
  do {                                                                    \
    cudaError_t e_ = (call);                                              \
    if (e_ != cudaSuccess) {                                              \
      fprintf(stderr, "%s: %s\n", #call, cudaGetErrorString(e_));         \
      return 2;                                                           \
    }                                                                     \
  } while (0)
#define NV(call)                                                          \
  do {                                                                    \
    nvfp4_status s_ = (call);                                             \
    if (s_ != NVFP4_OK) {                                                 \
      fprintf(stderr, "%s: %s\n", #call, nvfp4_status_string(s_));        \
      return 3;                                                           \
    }                                                                     \
  } while (0)

static int alloc_copy(nvfp4_tensor* t, int64_t rows, int64_t cols) {
  memset(t, 0, sizeof *t);
  t->rows = rows;
  t->cols = cols;
  t->sf_layout = NVFP4_SF_SWIZZLED;
  t->format = NVFP4_FORMAT_NVFP4;
  if (cudaMalloc((void**)&t->codes, (size_t)(rows * cols / 2)) != cudaSuccess) return 1;
  if (cudaMalloc((void**)&t->scales, (size_t)(rows * cols / 16)) != cudaSuccess) return 1;
  if (cudaMalloc((void**)&t->global, 2 * sizeof(float)) != cudaSuccess) return 1;
  return 0;
}

int main(void) {
  static const float grid[8] = {0.f, 0.5f, 1.f, 1.5f, 2.f, 3.f, 4.f, 6.f};
  static uint16_t ha[M * K], hb[N * K], hd[M * N];
  static float fa[M * K], fb[N * K], ref[M * N];
  uint32_t lcg = 12345u;
  for (int i = 0; i < M * K; ++i) {
    lcg = lcg * 1664525u + 1013904223u;
    float v = grid[(lcg >> 24) & 7] * (((lcg >> 20) & 1) ? -1.f : 1.f);
    if (i % 16 == 0) v = 6.f; /* every block holds the maximum: all block scales equal, decode is exact */
    fa[i] = v;
    ha[i] = bf16_of(v);
  }
  for (int i = 0; i < N * K; ++i) {
    lcg = lcg * 1664525u + 1013904223u;
    float v = grid[(lcg >> 24) & 7] * (((lcg >> 20) & 1) ? -1.f : 1.f);
    if (i % 16 == 0) v = 6.f;
    fb[i] = v;
    hb[i] = bf16_of(v);
  }
  for (int i = 0; i < M; ++i)
    for (int j = 0; j < N; ++j) {
      double acc = 0.0;
      for (int k = 0; k < K; ++k) acc += (double)fa[i * K + k] * (double)fb[j * K + k];
      ref[i * N + j] = (float)acc; /* multiples of 1/4 below 2^15: exact */
    }

  void *da, *db, *dd, *dd32;
  CK(cudaMalloc(&da, sizeof ha));
  CK(cudaMalloc(&db, sizeof hb));
  CK(cudaMalloc(&dd, sizeof hd));
  CK(cudaMalloc(&dd32, sizeof ref));
  CK(cudaMemcpy(da, ha, sizeof ha, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(db, hb, sizeof hb, cudaMemcpyHostToDevice));
  nvfp4_tensor qa, qb;
  if (alloc_copy(&qa, M, K) || alloc_copy(&qb, N, K)) return 2;

  nvfp4_quant_opts o;
  memset(&o, 0, sizeof o);
  o.block_rows = 1;
  o.rounding = NVFP4_ROUND_NEAREST_EVEN;
  NV(nvfp4_quantize(da, M, K, K, &o, &qa, NULL, NULL));
  NV(nvfp4_quantize(db, N, K, K, &o, &qb, NULL, NULL));

  /* block-scaled FP4 product, fp32 output: the quantized operands decode to a tiny multiple of the originals
   * (the tensor decode scale 1/448 is not a binary32 number), so compare to 1e-6 relative */
  static float out32[M * N];
  NV(nvfp4_gemm(&qa, &qb, dd32, 1, N, 0, NULL));
  NV(nvfp4_device_status(NULL, NULL));
  CK(cudaMemcpy(out32, dd32, sizeof out32, cudaMemcpyDeviceToHost));
  int bad = 0;
  for (int i = 0; i < M * N; ++i) {
    float tol = 1e-5f * (float)K * 36.f;
    float d = out32[i] - ref[i];
    if (d < -tol || d > tol) ++bad;
  }
  if (bad) {
    fprintf(stderr, "FP4 GEMM: %d of %d outputs off\n", bad, M * N);
    return 4;
  }

  /* BF16 product of the same operands, bf16 output: integers and quarters below 256 are exact, larger values round */
  NV(nvfp4_gemm_bf16(da, NVFP4_K_MAJOR, K, db, NVFP4_K_MAJOR, K, M, N, K, dd, 0, N, 0, NULL));
  NV(nvfp4_device_status(NULL, NULL));
  CK(cudaMemcpy(hd, dd, sizeof hd, cudaMemcpyDeviceToHost));
  for (int i = 0; i < M * N; ++i) {
    float got = f32_of_bf16(hd[i]), want = ref[i];
    float tol = (want < 0 ? -want : want) / 256.f + 1e-6f;
    float d = got - want;
    if (d < -tol || d > tol) ++bad;
  }
  if (bad) {
    fprintf(stderr, "BF16 GEMM: %d of %d outputs off\n", bad, M * N);
    return 5;
  }

  /* error metric: the grid values quantize without error */
  double* dm;
  double hm[2];
  CK(cudaMalloc((void**)&dm, sizeof hm));
  NV(nvfp4_quant_error(da, M, K, K, &qa, dm, NULL));
  CK(cudaMemcpy(hm, dm, sizeof hm, cudaMemcpyDeviceToHost));
  if (!(hm[0] <= 1e-12 * hm[1]) || !(hm[1] > 0.0)) {
    fprintf(stderr, "quant_error: %g / %g\n", hm[0], hm[1]);
    return 6;
  }
  printf("ok launches=%llu\n", (unsigned long long)nvfp4_launch_count());
  return 0;
}
