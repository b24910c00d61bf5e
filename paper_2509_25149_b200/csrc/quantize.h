// Internal launch interface of the quantizer kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "nvfp4.h"

namespace nvfp4 {

struct QuantArgs {
  const uint16_t* x;  // bf16 source [rows x cols], leading dimension ld (binary32 when the f32 launchers are used)
  int64_t rows, cols, ld;
  uint8_t* r_codes;   // row-wise copy
  uint8_t* r_scales;
  float* r_global;
  uint8_t* c_codes;   // column-wise (transposed) copy
  uint8_t* c_scales;
  float* c_global;
  int r_swz, c_swz;   // 1 = swizzled scale layout
  uint32_t sign_mask;
  uint32_t seed_lo, seed_hi, off_lo, off_hi, off_hi_col;
  uint32_t rk[20];       // Philox round keys (seed_lo + r * W0, seed_hi + r * W1), r = 0..9, filled by the host
  int tiles_r, tiles_c;  // 128 x 128 tiles of the source
  unsigned int* status;  // device status word: a bounded wait that expired leaves its code here (may be NULL)
  int chained;  // host side: the previous launch on the stream is a kernel of the same call (see launch_kernel)
  // side job of launch_quantize_with_amax_of: 128 x 128 tiles of the second tensor and where its amax goes
  int side_tiles_r, side_tiles_c;
  float* side_out0;
  float* side_out1;
};

// A second bf16 tensor whose plain amax (pass 1 of its own quantization) a quantize launch takes on the side
struct SideAmax {
  const void* x;
  int64_t rows, cols, ld;
  float* out0;  // both receive the amax (the row-wise and the transposed copy's global[0]); either may be NULL
  float* out1;
};

// Another transform size (quantize_rht.cu): d = 2, 4, 8 or 128 on the copies flagged rht_row / rht_col
struct RhtArgs {
  QuantArgs q;
  int d;
  int has_row, has_col, rht_row, rht_col;
  uint32_t mask16;         // d <= 16: the d sign bits repeated over sixteen positions
  uint32_t sign_words[4];  // d = 128: sign bit of position p is bit (p & 31) of word p >> 5
  float norm;              // fl(1 / sqrt(d))
};
cudaError_t launch_quantize_rht(const RhtArgs& ra, bool amax_provided, bool sr, cudaStream_t s);
cudaError_t launch_amax_rot_col_small(const QuantArgs& a, bool has_row, uint32_t mask16, int d, float norm,
                                      cudaStream_t s);

cudaError_t launch_amax(const QuantArgs& a, bool has_row, bool has_col, bool rht_row, bool rht_col,
                        cudaStream_t s);
cudaError_t launch_quantize(const QuantArgs& a, bool has_row, bool has_col, bool block2d, bool rht_row,
                            bool rht_col, bool sr, cudaStream_t s);
// The row-wise copy (and, with has_col, the transformed transposed copy) of a, round-to-nearest, 1 x 16 blocks, and
// on the side the plain amax of `side`: the memory-bound pass 1 of the next tensor rides on this issue-bound kernel.
cudaError_t launch_quantize_with_amax_of(const QuantArgs& a, bool has_col, const SideAmax& side, cudaStream_t s);
cudaError_t zero_side_amax(const SideAmax& side, cudaStream_t s);  // before the launches that lead up to it
// MXFP4 outputs (quantize_mx.cu): one pass, no tensor-level scale
cudaError_t launch_quantize_mx(const QuantArgs& a, bool has_row, bool has_col, bool block2d, bool rht_col, bool sr,
                               cudaStream_t s);
// binary32 source (quantize_f32.cu): plain amax pass and the quantize pass, no transform
cudaError_t launch_amax_f32(const QuantArgs& a, bool has_row, bool has_col, cudaStream_t s);
cudaError_t launch_quantize_f32(const QuantArgs& a, bool has_row, bool has_col, bool block2d, bool sr, cudaStream_t s);
cudaError_t launch_dequantize(const nvfp4_tensor& t, float* out, cudaStream_t s);
cudaError_t launch_e2m1_sr(const float* v, const uint8_t* u, int64_t n, uint8_t* codes, cudaStream_t s);
cudaError_t launch_rht16(const void* x, int64_t rows, int64_t cols, int64_t ld, int colwise, uint32_t mask,
                         float* out, cudaStream_t s);

// quantize_rowscale.cu: row-wise copy with {amax, s_dec} per row in a.r_global[2 * rows], one pass
cudaError_t launch_quantize_rowscale(const QuantArgs& a, bool sr, cudaStream_t s);
// metrics.cu: out = {sum (x - decode(q))^2, sum x^2} of a row-wise copy; {sum (ref - test)^2, sum ref^2} of two tensors
cudaError_t launch_quant_error(const void* x, int64_t rows, int64_t cols, int64_t ld, const nvfp4_tensor& q,
                               double* out, cudaStream_t s);
cudaError_t launch_sq_error(const void* ref, bool ref_fp32, int64_t ld_ref, const void* test, bool test_fp32,
                            int64_t ld_test, int64_t rows, int64_t cols, double* out, cudaStream_t s);

}  // namespace nvfp4
