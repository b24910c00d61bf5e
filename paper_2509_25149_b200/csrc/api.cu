// C-ABI entry points: argument validation and the stream-ordered composition of the kernels.
#include <atomic>
#include <cmath>

#include "common.cuh"
#include "gemm.h"
#include "quantize.h"

namespace nvfp4 {
static std::atomic<uint64_t> g_launches{0};
static std::atomic<int> g_tile_n{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
}  // namespace nvfp4

using namespace nvfp4;

// Scratch of nvfp4_linear_fwd_noalloc: the row-wise NVFP4 copy of X lives here instead of in caller memory.
// Every GPU that loads the library holds this array until the process exits.
#define NVFP4_NOALLOC_SCRATCH_BYTES (16u << 20)
static __device__ __align__(256) unsigned char g_noalloc_scratch[NVFP4_NOALLOC_SCRATCH_BYTES];

namespace {

inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

nvfp4_status check_copy(const nvfp4_tensor* t, int64_t rows, int64_t cols) {
  if (!t->codes || !t->scales || !t->global) return NVFP4_ERR_NULL;
  if (t->rows != rows || t->cols != cols) return NVFP4_ERR_SHAPE;
  if (t->sf_layout != NVFP4_SF_LINEAR && t->sf_layout != NVFP4_SF_SWIZZLED) return NVFP4_ERR_ARG;
  if (t->format != NVFP4_FORMAT_NVFP4 && t->format != NVFP4_FORMAT_MXFP4 && t->format != NVFP4_FORMAT_NVFP4_ROWSCALE)
    return NVFP4_ERR_ARG;
  const int64_t atom_cols = t->format == NVFP4_FORMAT_MXFP4 ? 128 : 64;  // four blocks of 32 / 16 elements
  if (t->sf_layout == NVFP4_SF_SWIZZLED && (rows % 128 != 0 || cols % atom_cols != 0)) return NVFP4_ERR_SHAPE;
  if (!aligned(t->codes, 16) || !aligned(t->scales, 16) || !aligned(t->global, 8)) return NVFP4_ERR_ALIGN;
  return NVFP4_OK;
}

// check_only: every argument check of the call, no launch (the composed calls validate all their steps first, so
// that a rejected call has enqueued nothing)
nvfp4_status quantize_impl(const void* x, int64_t rows, int64_t cols, int64_t ld, const nvfp4_quant_opts* o,
                           const nvfp4_tensor* rowwise, const nvfp4_tensor* colwise, cudaStream_t s,
                           bool check_only = false, const SideAmax* side = nullptr, bool chained = false) {
  if (!x || !o) return NVFP4_ERR_NULL;
  if (!rowwise && !colwise) return NVFP4_ERR_NULL;
  if (rows <= 0 || cols <= 0 || rows % 16 != 0 || cols % 16 != 0) return NVFP4_ERR_SHAPE;
  if (ld < cols) return NVFP4_ERR_SHAPE;
  if (ld % 16 != 0 || !aligned(x, 32)) return NVFP4_ERR_ALIGN;
  const int32_t fmt = rowwise ? rowwise->format : colwise->format;
  if (fmt == NVFP4_FORMAT_NVFP4_ROWSCALE) {
    // one pass, row-wise copy only (a scale per row of the transposed copy would be a statistic over all source rows)
    if (colwise) return NVFP4_ERR_ARG;
    if (o->block_rows != 1 || o->rht_rowwise || o->rht_colwise) return NVFP4_ERR_ARG;
    if (o->rounding != NVFP4_ROUND_NEAREST_EVEN && o->rounding != NVFP4_ROUND_STOCHASTIC) return NVFP4_ERR_ARG;
    if (o->flags & ~NVFP4_SR_INDEPENDENT_COPIES) return NVFP4_ERR_ARG;
    if (rows > (int64_t)1 << 30 || cols > (int64_t)1 << 30) return NVFP4_ERR_SHAPE;
    nvfp4_status st0 = check_copy(rowwise, rows, cols);
    if (st0 != NVFP4_OK) return st0;
    if (check_only) return NVFP4_OK;
    QuantArgs a{};
    a.x = static_cast<const uint16_t*>(x);
    a.rows = rows; a.cols = cols; a.ld = ld;
    a.r_codes = rowwise->codes; a.r_scales = rowwise->scales; a.r_global = rowwise->global;
    a.r_swz = rowwise->sf_layout == NVFP4_SF_SWIZZLED;
    a.seed_lo = (uint32_t)o->seed; a.seed_hi = (uint32_t)(o->seed >> 32);
    for (uint32_t r = 0; r < 10; ++r) {  // Philox key schedule
      a.rk[2 * r] = a.seed_lo + r * 0x9E3779B9u;
      a.rk[2 * r + 1] = a.seed_hi + r * 0xBB67AE85u;
    }
    a.off_lo = (uint32_t)o->sr_offset; a.off_hi = (uint32_t)(o->sr_offset >> 32);
    return launch_quantize_rowscale(a, o->rounding == NVFP4_ROUND_STOCHASTIC, s) == cudaSuccess ? NVFP4_OK
                                                                                                  : NVFP4_ERR_CUDA;
  }
  if (fmt != NVFP4_FORMAT_NVFP4 && fmt != NVFP4_FORMAT_MXFP4) return NVFP4_ERR_ARG;
  if (rowwise && colwise && rowwise->format != colwise->format) return NVFP4_ERR_ARG;
  const bool mx = fmt == NVFP4_FORMAT_MXFP4;
  const int32_t blk = mx ? 32 : 16;  // block length along the contraction dimension, and the 2D block size
  if (mx && (rows % 32 != 0 || cols % 32 != 0)) return NVFP4_ERR_SHAPE;
  if (o->block_rows != 1 && o->block_rows != blk) return NVFP4_ERR_ARG;
  if (o->rounding != NVFP4_ROUND_NEAREST_EVEN && o->rounding != NVFP4_ROUND_STOCHASTIC) return NVFP4_ERR_ARG;
  if ((o->rht_rowwise | o->rht_colwise) & ~1) return NVFP4_ERR_ARG;
  if (o->block_rows == blk && (o->rht_rowwise || o->rht_colwise)) return NVFP4_ERR_ARG;
  if (mx && o->rht_rowwise) return NVFP4_ERR_UNIMPLEMENTED;  // the recipe transforms the transposed copies only
  if (o->flags & ~(NVFP4_SR_INDEPENDENT_COPIES | NVFP4_AMAX_PROVIDED | NVFP4_INPUT_FP32)) return NVFP4_ERR_ARG;
  const bool f32 = (o->flags & NVFP4_INPUT_FP32) != 0;
  if (f32 && (mx || o->rht_rowwise || o->rht_colwise)) return NVFP4_ERR_UNIMPLEMENTED;
  // transform size: 0 = the format's own (16, or 32 for MXFP4); 2, 4, 8, 128 are the sizes of Appendix E.4.2
  const int32_t rd = o->rht_dim;
  const bool any_rht = o->rht_rowwise || o->rht_colwise;
  const bool other_dim = any_rht && rd != 0 && rd != (mx ? 32 : 16);
  if (rd != 0 && rd != 2 && rd != 4 && rd != 8 && rd != 16 && rd != 32 && rd != 128) return NVFP4_ERR_ARG;
  if (other_dim && (mx || rd == 32 || rd == 16)) return NVFP4_ERR_UNIMPLEMENTED;
  if (other_dim && rd == 128 && ((o->rht_rowwise && rowwise && cols % 128 != 0) || (o->rht_colwise && colwise && rows % 128 != 0)))
    return NVFP4_ERR_SHAPE;
  if (rows > (int64_t)1 << 30 || cols > (int64_t)1 << 30 || ((rows + 127) / 128) * ((cols + 127) / 128) > 0x7fffffff)
    return NVFP4_ERR_SHAPE;
  nvfp4_status st;
  if (rowwise && (st = check_copy(rowwise, rows, cols)) != NVFP4_OK) return st;
  if (colwise && (st = check_copy(colwise, cols, rows)) != NVFP4_OK) return st;
  if (check_only) return NVFP4_OK;

  QuantArgs a{};
  a.x = static_cast<const uint16_t*>(x);
  a.rows = rows; a.cols = cols; a.ld = ld;
  if (rowwise) {
    a.r_codes = rowwise->codes; a.r_scales = rowwise->scales; a.r_global = rowwise->global;
    a.r_swz = rowwise->sf_layout == NVFP4_SF_SWIZZLED;
  }
  if (colwise) {
    a.c_codes = colwise->codes; a.c_scales = colwise->scales; a.c_global = colwise->global;
    a.c_swz = colwise->sf_layout == NVFP4_SF_SWIZZLED;
  }
  a.sign_mask = mx ? o->rht_sign_mask : (o->rht_sign_mask & 0xffffu);
  a.seed_lo = (uint32_t)o->seed; a.seed_hi = (uint32_t)(o->seed >> 32);
  for (uint32_t r = 0; r < 10; ++r) {  // Philox key schedule
    a.rk[2 * r] = a.seed_lo + r * 0x9E3779B9u;
    a.rk[2 * r + 1] = a.seed_hi + r * 0xBB67AE85u;
  }
  a.off_lo = (uint32_t)o->sr_offset; a.off_hi = (uint32_t)(o->sr_offset >> 32);
  a.off_hi_col = (o->flags & NVFP4_SR_INDEPENDENT_COPIES) ? (a.off_hi | 0x80000000u) : a.off_hi;
  a.tiles_r = (int)((rows + 127) / 128);
  a.tiles_c = (int)((cols + 127) / 128);
  if (device_status_word(&a.status) != cudaSuccess) return NVFP4_ERR_CUDA;

  const bool hr = rowwise != nullptr, hc = colwise != nullptr;
  const bool b2 = o->block_rows == blk, sr = o->rounding == NVFP4_ROUND_STOCHASTIC;
  if (mx)  // no tensor-level scale, hence no amax pass
    return launch_quantize_mx(a, hr, hc, b2, o->rht_colwise != 0, sr, s) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
  if (f32) {
    if (!(o->flags & NVFP4_AMAX_PROVIDED) && launch_amax_f32(a, hr, hc, s) != cudaSuccess) return NVFP4_ERR_CUDA;
    return launch_quantize_f32(a, hr, hc, b2, sr, s) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
  }
  if (other_dim) {
    RhtArgs ra{};
    ra.q = a;
    ra.d = rd;
    ra.has_row = hr; ra.has_col = hc;
    ra.rht_row = hr && o->rht_rowwise; ra.rht_col = hc && o->rht_colwise;
    ra.sign_words[0] = o->rht_sign_mask;
    for (int i = 0; i < 3; ++i) ra.sign_words[1 + i] = o->rht_sign_mask_ext[i];
    if (rd < 16) {
      const uint32_t low = o->rht_sign_mask & ((1u << rd) - 1u);
      for (int p = 0; p < 16; p += rd) ra.mask16 |= low << p;
    }
    ra.norm = (float)(1.0 / sqrt((double)rd));
    return launch_quantize_rht(ra, (o->flags & NVFP4_AMAX_PROVIDED) != 0, sr, s) == cudaSuccess ? NVFP4_OK
                                                                                                  : NVFP4_ERR_CUDA;
  }
  // pass 2 may become resident while the previous kernel of this call drains (its own pass 1, or the caller's launch)
  a.chained = chained;
  // only the forward pass's activation quantize carries a side job (see side_amax_fits); checked before any launch
  if (side && (!hr || b2 || sr || o->rht_rowwise || (hc && !o->rht_colwise))) return NVFP4_ERR_ARG;
  if (side && zero_side_amax(*side, s) != cudaSuccess) return NVFP4_ERR_CUDA;  // not between pass 1 and pass 2
  if (!(o->flags & NVFP4_AMAX_PROVIDED)) {
    if (launch_amax(a, hr, hc, o->rht_rowwise != 0, o->rht_colwise != 0, s) != cudaSuccess) return NVFP4_ERR_CUDA;
    a.chained = 1;
  }
  if (side) {
    return launch_quantize_with_amax_of(a, hc, *side, s) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
  }
  if (launch_quantize(a, hr, hc, b2, o->rht_rowwise != 0, o->rht_colwise != 0, sr, s) != cudaSuccess)
    return NVFP4_ERR_CUDA;
  return NVFP4_OK;
}

// Whether a quantize of the composed calls (options xo) runs `quantize_kernel`, the kernel that can take a second
// tensor's plain amax on the side and lets the next kernel of the call set itself up early: bf16 source, NVFP4, the
// 16-point transform or none.
bool side_amax_fits(int32_t fmt, const nvfp4_quant_opts& xo) {
  return fmt == NVFP4_FORMAT_NVFP4 && (xo.rht_dim == 0 || xo.rht_dim == 16) && !(xo.flags & NVFP4_INPUT_FP32);
}

// argument checks of one GEMM and its launch description
nvfp4_status gemm_prepare(const nvfp4_tensor* A, const nvfp4_tensor* B, void* D, int32_t d_is_fp32, int64_t ldd,
                          int32_t accumulate, GemmArgs& g) {
  if (!A || !B || !D) return NVFP4_ERR_NULL;
  if (!A->codes || !A->scales || !A->global || !B->codes || !B->scales || !B->global) return NVFP4_ERR_NULL;
  if (A->cols != B->cols) return NVFP4_ERR_SHAPE;
  const int64_t M = A->rows, N = B->rows, K = A->cols;
  if (M <= 0 || N <= 0 || K <= 0 || M % 128 != 0 || N % 128 != 0 || K % 256 != 0) return NVFP4_ERR_SHAPE;
  if (M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff || (M / 128) * (N / 128) > 0x7fffffff) return NVFP4_ERR_SHAPE;
  if (A->sf_layout != NVFP4_SF_SWIZZLED || B->sf_layout != NVFP4_SF_SWIZZLED) return NVFP4_ERR_ARG;
  const bool a_rs = A->format == NVFP4_FORMAT_NVFP4_ROWSCALE, b_rs = B->format == NVFP4_FORMAT_NVFP4_ROWSCALE;
  // a row-scaled NVFP4 operand mixes with a tensor-scaled one; MXFP4 only with MXFP4
  if ((a_rs ? NVFP4_FORMAT_NVFP4 : A->format) != (b_rs ? NVFP4_FORMAT_NVFP4 : B->format)) return NVFP4_ERR_ARG;
  if (!a_rs && A->format != NVFP4_FORMAT_NVFP4 && A->format != NVFP4_FORMAT_MXFP4) return NVFP4_ERR_ARG;
  if ((a_rs || b_rs) && (M % 256 != 0 || N % 256 != 0)) return NVFP4_ERR_SHAPE;
  if (accumulate && !d_is_fp32) return NVFP4_ERR_ARG;
  if (ldd < N) return NVFP4_ERR_SHAPE;
  const int64_t esz = d_is_fp32 ? 4 : 2;
  if ((ldd * esz) % 16 != 0 || !aligned(D, 16)) return NVFP4_ERR_ALIGN;
  if (!aligned(A->codes, 16) || !aligned(B->codes, 16) || !aligned(A->scales, 16) || !aligned(B->scales, 16))
    return NVFP4_ERR_ALIGN;
  g = GemmArgs{};
  g.sfa = A->scales; g.sfb = B->scales;
  g.a_global = A->global; g.b_global = B->global;
  g.d = D; g.ldd = ldd;
  g.M = (int)M; g.N = (int)N; g.K = (int)K;
  g.d_is_fp32 = d_is_fp32 != 0; g.accumulate = accumulate != 0;
  g.mx = A->format == NVFP4_FORMAT_MXFP4;
  g.a_rows = a_rs ? A->global : nullptr;
  g.b_rows = b_rs ? B->global : nullptr;
  return NVFP4_OK;
}

int gemm_tile(const GemmArgs& g) {
  const int M = g.M, N = g.N, K = g.K;
  const int d_is_fp32 = g.d_is_fp32;
  // CTA pairs on 256 x 256 tiles whenever the shape allows (half the operand traffic per flop, half the
  // scale-copy and MMA issue work per SM).  Otherwise one CTA per tile: 128 x 256 tiles hold one accumulator
  // (exposed epilogue), 128 x 128 tiles two (the epilogue overlaps the next tile), so the wide tile pays off
  // once the main loop is long enough to amortise the epilogue.
  int tile_n = g_tile_n.load(std::memory_order_relaxed);
  if (tile_n != 128 && tile_n != 256 && tile_n != 512 && tile_n != 768) {
    if (M % 256 == 0 && N % 256 == 0)
      tile_n = prefer_wide_tiles(g, nullptr) ? 768 : 512;  // CTA pairs: the tile width with the shorter schedule
    else if (M % 256 == 0 && N % 128 == 0 && N >= 256)
      tile_n = 768;
    else
      tile_n = (K >= (d_is_fp32 ? 16384 : 8192)) ? 256 : 128;
  }
  return tile_n;
}

nvfp4_status gemm_impl(const nvfp4_tensor* A, const nvfp4_tensor* B, void* D, int32_t d_is_fp32, int64_t ldd,
                       int32_t accumulate, cudaStream_t s, bool chained = false) {
  GemmArgs g;
  nvfp4_status st = gemm_prepare(A, B, D, d_is_fp32, ldd, accumulate, g);
  if (st != NVFP4_OK) return st;
  g.chained = chained;
  if (launch_gemm(g, A->codes, B->codes, gemm_tile(g), s) != cudaSuccess) return NVFP4_ERR_CUDA;
  return NVFP4_OK;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline size_t copy_bytes(int64_t rows, int64_t cols) {
  return align_up((size_t)(rows * cols / 2), 256) + align_up((size_t)(rows * cols / 16), 256) + 256;
}
// the same with room for {amax, s_dec} per row (forward-only calls with row scales)
inline size_t copy_bytes_rows(int64_t rows, int64_t cols) {
  return align_up((size_t)(rows * cols / 2), 256) + align_up((size_t)(rows * cols / 16), 256) +
         align_up((size_t)rows * 8, 256);
}
// carve one swizzled-scale copy [rows x cols] out of a workspace
nvfp4_tensor carve(uint8_t*& p, int64_t rows, int64_t cols, int32_t format = NVFP4_FORMAT_NVFP4) {
  nvfp4_tensor t{};
  t.codes = p;
  p += align_up((size_t)(rows * cols / 2), 256);
  t.scales = p;
  p += align_up((size_t)(rows * cols / 16), 256);
  t.global = reinterpret_cast<float*>(p);
  p += 256;
  t.rows = rows; t.cols = cols; t.sf_layout = NVFP4_SF_SWIZZLED;
  t.format = format;
  return t;
}

}  // namespace

extern "C" {

nvfp4_status nvfp4_quantize(const void* x_bf16, int64_t rows, int64_t cols, int64_t ld, const nvfp4_quant_opts* opts,
                            const nvfp4_tensor* rowwise, const nvfp4_tensor* colwise, void* cuda_stream) {
  return quantize_impl(x_bf16, rows, cols, ld, opts, rowwise, colwise, static_cast<cudaStream_t>(cuda_stream));
}

nvfp4_status nvfp4_gemm(const nvfp4_tensor* A, const nvfp4_tensor* B, void* D, int32_t d_is_fp32, int64_t ldd,
                        int32_t accumulate, void* cuda_stream) {
  return gemm_impl(A, B, D, d_is_fp32, ldd, accumulate, static_cast<cudaStream_t>(cuda_stream));
}

size_t nvfp4_linear_fwd_workspace_bytes(int64_t M, int64_t K) { return copy_bytes_rows(M, K); }
size_t nvfp4_linear_bwd_workspace_bytes(int64_t M, int64_t N) { return 2 * copy_bytes(M, N); }

nvfp4_status nvfp4_linear_fwd(const void* X, const void* W, int64_t M, int64_t N, int64_t K,
                              const nvfp4_quant_opts* opts, void* Y_bf16, const nvfp4_tensor* X_col_saved,
                              const nvfp4_tensor* W_row, const nvfp4_tensor* W_col_saved, int32_t w_is_cached,
                              void* workspace, size_t workspace_bytes, void* cuda_stream) {
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (!X || !opts || !Y_bf16 || !W_row) return NVFP4_ERR_NULL;
  if (!w_is_cached && !W) return NVFP4_ERR_NULL;
  if (M <= 0 || N <= 0 || K <= 0 || M % 256 || N % 256 || K % 256) return NVFP4_ERR_SHAPE;
  if (!workspace || workspace_bytes < nvfp4_linear_fwd_workspace_bytes(M, K)) return NVFP4_ERR_WORKSPACE;
  if (!aligned(workspace, 256)) return NVFP4_ERR_ALIGN;
  nvfp4_status st;
  if ((st = check_copy(W_row, N, K)) != NVFP4_OK) return st;
  if (W_col_saved && (st = check_copy(W_col_saved, K, N)) != NVFP4_OK) return st;
  if (X_col_saved && (st = check_copy(X_col_saved, K, M)) != NVFP4_OK) return st;
  if (W_row->sf_layout != NVFP4_SF_SWIZZLED) return NVFP4_ERR_ARG;
  // the format of the layer is the format of its weight copy (MXFP4: 32-element blocks, transform size 32)
  const int32_t fmt = W_row->format;
  if (fmt != NVFP4_FORMAT_NVFP4 && fmt != NVFP4_FORMAT_MXFP4) return NVFP4_ERR_ARG;  // per-tensor scales only
  if ((W_col_saved && W_col_saved->format != fmt) || (X_col_saved && X_col_saved->format != fmt)) return NVFP4_ERR_ARG;

  nvfp4_quant_opts wo{};
  wo.block_rows = fmt == NVFP4_FORMAT_MXFP4 ? 32 : 16;
  wo.rounding = NVFP4_ROUND_NEAREST_EVEN;
  uint8_t* p = static_cast<uint8_t*>(workspace);
  if (opts->flags & NVFP4_LINEAR_ROW_SCALES) {
    // forward-only call: X gets a global scale per row in one pass (Appendix B.1, closing remark) and Fprop applies
    // the vector in its epilogue.  No transposed copy can be made this way, so none may be requested.
    if (X_col_saved || fmt != NVFP4_FORMAT_NVFP4) return NVFP4_ERR_ARG;
    nvfp4_tensor x_rows{};
    x_rows.codes = p;
    p += align_up((size_t)(M * K / 2), 256);
    x_rows.scales = p;
    p += align_up((size_t)(M * K / 16), 256);
    x_rows.global = reinterpret_cast<float*>(p);
    x_rows.rows = M; x_rows.cols = K; x_rows.sf_layout = NVFP4_SF_SWIZZLED;
    x_rows.format = NVFP4_FORMAT_NVFP4_ROWSCALE;
    nvfp4_quant_opts ro{};
    ro.block_rows = 1;
    ro.rounding = NVFP4_ROUND_NEAREST_EVEN;
    GemmArgs gy;  // every step is validated before the first launch
    if (!w_is_cached && (st = quantize_impl(W, N, K, K, &wo, W_row, W_col_saved, s, true)) != NVFP4_OK) return st;
    if ((st = quantize_impl(X, M, K, K, &ro, &x_rows, nullptr, s, true)) != NVFP4_OK) return st;
    if ((st = gemm_prepare(&x_rows, W_row, Y_bf16, 0, N, 0, gy)) != NVFP4_OK) return st;
    if (!w_is_cached && (st = quantize_impl(W, N, K, K, &wo, W_row, W_col_saved, s)) != NVFP4_OK) return st;
    if ((st = quantize_impl(X, M, K, K, &ro, &x_rows, nullptr, s)) != NVFP4_OK) return st;
    return gemm_impl(&x_rows, W_row, Y_bf16, 0, N, 0, s);
  }
  nvfp4_tensor x_row = carve(p, M, K, fmt);
  nvfp4_quant_opts xo{};
  xo.block_rows = 1;
  xo.rounding = NVFP4_ROUND_NEAREST_EVEN;
  xo.rht_colwise = 1;
  xo.rht_sign_mask = opts->rht_sign_mask;
  xo.rht_dim = opts->rht_dim;  // 0 = the format's own size; Appendix E.4.2's other sizes pass through
  for (int i = 0; i < 3; ++i) xo.rht_sign_mask_ext[i] = opts->rht_sign_mask_ext[i];
  GemmArgs gy;  // every step is validated before the first launch
  if (!w_is_cached && (st = quantize_impl(W, N, K, K, &wo, W_row, W_col_saved, s, true)) != NVFP4_OK) return st;
  if ((st = quantize_impl(X, M, K, K, &xo, &x_row, X_col_saved, s, true)) != NVFP4_OK) return st;
  if ((st = gemm_prepare(&x_row, W_row, Y_bf16, 0, N, 0, gy)) != NVFP4_OK) return st;
  if (!w_is_cached && side_amax_fits(fmt, xo)) {
    // pass 1 of W (memory-bound) rides on pass 2 of X (issue-bound); W's pass 2 then finds its amax in place
    const SideAmax w_amax{W, N, K, K, W_row->global, W_col_saved ? W_col_saved->global : nullptr};
    if ((st = quantize_impl(X, M, K, K, &xo, &x_row, X_col_saved, s, false, &w_amax)) != NVFP4_OK) return st;
    wo.flags |= NVFP4_AMAX_PROVIDED;
    if ((st = quantize_impl(W, N, K, K, &wo, W_row, W_col_saved, s, false, nullptr, true)) != NVFP4_OK) return st;
    return gemm_impl(&x_row, W_row, Y_bf16, 0, N, 0, s, true);
  }
  if (!w_is_cached && (st = quantize_impl(W, N, K, K, &wo, W_row, W_col_saved, s)) != NVFP4_OK) return st;
  if ((st = quantize_impl(X, M, K, K, &xo, &x_row, X_col_saved, s)) != NVFP4_OK) return st;
  // behind a quantizer of this call the GEMM may set itself up while that kernel drains
  return gemm_impl(&x_row, W_row, Y_bf16, 0, N, 0, s, true);
}

nvfp4_status nvfp4_linear_bwd(const void* dY, const nvfp4_tensor* X_col_saved, const nvfp4_tensor* W_col_saved,
                              int64_t M, int64_t N, int64_t K, const nvfp4_quant_opts* opts, void* dX_bf16,
                              float* dW_fp32, int32_t accumulate_dw, void* workspace, size_t workspace_bytes,
                              void* cuda_stream) {
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (!dY || !opts) return NVFP4_ERR_NULL;
  if (!dX_bf16 && !dW_fp32) return NVFP4_ERR_NULL;
  if (dX_bf16 && !W_col_saved) return NVFP4_ERR_NULL;
  if (dW_fp32 && !X_col_saved) return NVFP4_ERR_NULL;
  if (M <= 0 || N <= 0 || K <= 0 || M % 256 || N % 256 || K % 256) return NVFP4_ERR_SHAPE;
  if (!workspace || workspace_bytes < nvfp4_linear_bwd_workspace_bytes(M, N)) return NVFP4_ERR_WORKSPACE;
  if (!aligned(workspace, 256)) return NVFP4_ERR_ALIGN;
  nvfp4_status st;
  if (W_col_saved && (st = check_copy(W_col_saved, K, N)) != NVFP4_OK) return st;
  if (X_col_saved && (st = check_copy(X_col_saved, K, M)) != NVFP4_OK) return st;

  const int32_t fmt = W_col_saved ? W_col_saved->format : X_col_saved->format;
  if (fmt != NVFP4_FORMAT_NVFP4 && fmt != NVFP4_FORMAT_MXFP4) return NVFP4_ERR_ARG;  // per-tensor scales only
  if (W_col_saved && X_col_saved && W_col_saved->format != X_col_saved->format) return NVFP4_ERR_ARG;
  uint8_t* p = static_cast<uint8_t*>(workspace);
  nvfp4_tensor g_row = carve(p, M, N, fmt);
  nvfp4_tensor g_col = carve(p, N, M, fmt);
  nvfp4_quant_opts go{};
  go.block_rows = 1;
  go.rounding = NVFP4_ROUND_STOCHASTIC;
  go.rht_colwise = 1;
  go.rht_sign_mask = opts->rht_sign_mask;
  go.rht_dim = opts->rht_dim;
  for (int i = 0; i < 3; ++i) go.rht_sign_mask_ext[i] = opts->rht_sign_mask_ext[i];
  go.seed = opts->seed;
  go.sr_offset = opts->sr_offset;
  go.flags = opts->flags & NVFP4_SR_INDEPENDENT_COPIES;
  {  // every step is validated before the first launch
    GemmArgs gchk;
    if ((st = quantize_impl(dY, M, N, N, &go, dX_bf16 ? &g_row : nullptr, dW_fp32 ? &g_col : nullptr, s, true)) != NVFP4_OK)
      return st;
    if (dX_bf16 && (st = gemm_prepare(&g_row, W_col_saved, dX_bf16, 0, K, 0, gchk)) != NVFP4_OK) return st;
    if (dW_fp32 && (st = gemm_prepare(&g_col, X_col_saved, dW_fp32, 1, K, accumulate_dw, gchk)) != NVFP4_OK) return st;
  }
  if ((st = quantize_impl(dY, M, N, N, &go, dX_bf16 ? &g_row : nullptr, dW_fp32 ? &g_col : nullptr, s)) != NVFP4_OK)
    return st;
  if (dX_bf16 && dW_fp32) {
    // Dgrad and Wgrad are independent: when both run on CTA pairs they share one launch, the longer contraction
    // first, so the partial last round of one is filled with tiles of the other
    GemmArgs gd, gw;
    if ((st = gemm_prepare(&g_row, W_col_saved, dX_bf16, 0, K, 0, gd)) != NVFP4_OK) return st;
    if ((st = gemm_prepare(&g_col, X_col_saved, dW_fp32, 1, K, accumulate_dw, gw)) != NVFP4_OK) return st;
    gd.chained = gw.chained = 1;  // behind the quantizer of dY
    const int td = gemm_tile(gd), tw = gemm_tile(gw);
    if ((td == 512 || td == 768) && (tw == 512 || tw == 768)) {
      const bool forced = g_tile_n.load(std::memory_order_relaxed) != 0;
      const bool dgrad_first = gd.K >= gw.K;
      const bool wide = forced ? td == 768 : prefer_wide_tiles(dgrad_first ? gd : gw, dgrad_first ? &gw : &gd);
      const cudaError_t e =
          dgrad_first ? launch_gemm_two(gd, g_row.codes, W_col_saved->codes, gw, g_col.codes, X_col_saved->codes, wide, s)
                      : launch_gemm_two(gw, g_col.codes, X_col_saved->codes, gd, g_row.codes, W_col_saved->codes, wide, s);
      return e == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
    }
  }
  if (dX_bf16 && (st = gemm_impl(&g_row, W_col_saved, dX_bf16, 0, K, 0, s, true)) != NVFP4_OK) return st;
  if (dW_fp32 && (st = gemm_impl(&g_col, X_col_saved, dW_fp32, 1, K, accumulate_dw, s)) != NVFP4_OK) return st;
  return NVFP4_OK;
}

size_t nvfp4_linear_fwd_noalloc_max_bytes(void) { return NVFP4_NOALLOC_SCRATCH_BYTES; }

nvfp4_status nvfp4_linear_fwd_noalloc(const void* X, const void* W, int64_t M, int64_t N, int64_t K,
                                      const nvfp4_quant_opts* opts, void* Y_bf16, const nvfp4_tensor* X_col_saved,
                                      const nvfp4_tensor* W_row, const nvfp4_tensor* W_col_saved, int32_t w_is_cached,
                                      void* cuda_stream) {
  if (M <= 0 || K <= 0 || M % 256 || K % 256) return NVFP4_ERR_SHAPE;
  // the request must fit the built-in array: refuse larger problems instead of touching memory we do not own
  if (nvfp4_linear_fwd_workspace_bytes(M, K) > (size_t)NVFP4_NOALLOC_SCRATCH_BYTES) return NVFP4_ERR_WORKSPACE;
  // `g_noalloc_scratch` names a host-side handle in host code, not a device address: ask the runtime for the
  // address once per device (with that device current) and hand that pointer to the kernels.
  constexpr int kMaxDevices = 64;
  static std::atomic<void*> scratch_of_device[kMaxDevices] = {};  // two host threads may make the first call at once
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NVFP4_ERR_CUDA;
  void* scratch = scratch_of_device[dev].load(std::memory_order_acquire);
  if (!scratch) {
    if (cudaGetSymbolAddress(&scratch, g_noalloc_scratch) != cudaSuccess || !scratch) return NVFP4_ERR_CUDA;
    scratch_of_device[dev].store(scratch, std::memory_order_release);  // every thread computes the same address
  }
  return nvfp4_linear_fwd(X, W, M, N, K, opts, Y_bf16, X_col_saved, W_row, W_col_saved, w_is_cached, scratch,
                          NVFP4_NOALLOC_SCRATCH_BYTES, cuda_stream);
}

nvfp4_status nvfp4_gemm_bf16(const void* A, int32_t a_layout, int64_t lda, const void* B, int32_t b_layout, int64_t ldb,
                             int64_t M, int64_t N, int64_t K, void* D, int32_t d_is_fp32, int64_t ldd,
                             int32_t accumulate, void* cuda_stream) {
  if (!A || !B || !D) return NVFP4_ERR_NULL;
  if ((a_layout != NVFP4_K_MAJOR && a_layout != NVFP4_MN_MAJOR) || (b_layout != NVFP4_K_MAJOR && b_layout != NVFP4_MN_MAJOR))
    return NVFP4_ERR_ARG;
  if (M <= 0 || N <= 0 || K <= 0 || M % 8 != 0 || N % 8 != 0 || K % 8 != 0) return NVFP4_ERR_SHAPE;
  if (M > 0x7fffff00 || N > 0x7fffff00 || K > 0x7fffff00 || ((M + 255) / 256) * ((N + 255) / 256) > 0x7fffffff)
    return NVFP4_ERR_SHAPE;
  if (lda < (a_layout == NVFP4_MN_MAJOR ? M : K) || ldb < (b_layout == NVFP4_MN_MAJOR ? N : K) || ldd < N)
    return NVFP4_ERR_SHAPE;
  if (accumulate && !d_is_fp32) return NVFP4_ERR_ARG;
  const int64_t esz = d_is_fp32 ? 4 : 2;
  if (lda % 8 != 0 || ldb % 8 != 0 || (ldd * esz) % 16 != 0 || !aligned(A, 16) || !aligned(B, 16) || !aligned(D, 16))
    return NVFP4_ERR_ALIGN;
  DenseGemmArgs g{};
  g.a = A; g.b = B; g.d = D;
  g.lda = lda; g.ldb = ldb; g.ldd = ldd;
  g.M = (int)M; g.N = (int)N; g.K = (int)K;
  g.a_mn = a_layout == NVFP4_MN_MAJOR; g.b_mn = b_layout == NVFP4_MN_MAJOR;
  g.d_is_fp32 = d_is_fp32 != 0; g.accumulate = accumulate != 0;
  return launch_gemm_bf16(g, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_linear_bf16_fwd(const void* X, const void* W, int64_t M, int64_t N, int64_t K, void* Y_bf16,
                                   void* cuda_stream) {
  return nvfp4_gemm_bf16(X, NVFP4_K_MAJOR, K, W, NVFP4_K_MAJOR, K, M, N, K, Y_bf16, 0, N, 0, cuda_stream);
}

nvfp4_status nvfp4_linear_bf16_bwd(const void* dY, const void* X, const void* W, int64_t M, int64_t N, int64_t K,
                                   void* dX_bf16, float* dW_fp32, int32_t accumulate_dw, void* cuda_stream) {
  if (!dY) return NVFP4_ERR_NULL;
  if (!dX_bf16 && !dW_fp32) return NVFP4_ERR_NULL;
  nvfp4_status st;
  // Dgrad: dX[M x K] = dY[M x N] W[N x K]; the contraction runs over W's rows
  if (dX_bf16 && (st = nvfp4_gemm_bf16(dY, NVFP4_K_MAJOR, N, W, NVFP4_MN_MAJOR, K, M, K, N, dX_bf16, 0, K, 0,
                                       cuda_stream)) != NVFP4_OK)
    return st;
  // Wgrad: dW[N x K] = dY^T X; the contraction runs over the tokens, the rows of both operands
  if (dW_fp32 && (st = nvfp4_gemm_bf16(dY, NVFP4_MN_MAJOR, N, X, NVFP4_MN_MAJOR, K, N, K, M, dW_fp32, 1, K,
                                       accumulate_dw, cuda_stream)) != NVFP4_OK)
    return st;
  return NVFP4_OK;
}

nvfp4_status nvfp4_quant_error(const void* x_bf16, int64_t rows, int64_t cols, int64_t ld, const nvfp4_tensor* q,
                               double* out2, void* cuda_stream) {
  if (!x_bf16 || !q || !out2) return NVFP4_ERR_NULL;
  if (rows <= 0 || cols <= 0 || ld < cols) return NVFP4_ERR_SHAPE;
  nvfp4_status st = check_copy(q, rows, cols);
  if (st != NVFP4_OK) return st;
  if (cols % (q->format == NVFP4_FORMAT_MXFP4 ? 32 : 16) != 0) return NVFP4_ERR_SHAPE;
  if (!aligned(x_bf16, 32) || ld % 16 != 0 || !aligned(out2, 8)) return NVFP4_ERR_ALIGN;
  return launch_quant_error(x_bf16, rows, cols, ld, *q, out2, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? NVFP4_OK
             : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_sq_error(const void* ref, int32_t ref_is_fp32, int64_t ld_ref, const void* test,
                            int32_t test_is_fp32, int64_t ld_test, int64_t rows, int64_t cols, double* out2,
                            void* cuda_stream) {
  if (!ref || !test || !out2) return NVFP4_ERR_NULL;
  if (rows <= 0 || cols <= 0 || cols % 8 != 0 || ld_ref < cols || ld_test < cols) return NVFP4_ERR_SHAPE;
  if (!aligned(ref, ref_is_fp32 ? 32 : 16) || !aligned(test, test_is_fp32 ? 32 : 16) || ld_ref % 8 != 0 ||
      ld_test % 8 != 0 || !aligned(out2, 8))
    return NVFP4_ERR_ALIGN;
  return launch_sq_error(ref, ref_is_fp32 != 0, ld_ref, test, test_is_fp32 != 0, ld_test, rows, cols, out2,
                         static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? NVFP4_OK
             : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_dequantize(const nvfp4_tensor* t, float* out, void* cuda_stream) {
  if (!t || !out || !t->codes || !t->scales || !t->global) return NVFP4_ERR_NULL;
  nvfp4_status st = check_copy(t, t->rows, t->cols);
  if (st != NVFP4_OK) return st;
  if (t->rows <= 0 || t->cols <= 0 || t->cols % (t->format == NVFP4_FORMAT_MXFP4 ? 32 : 16)) return NVFP4_ERR_SHAPE;
  return launch_dequantize(*t, out, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_rht16(const void* x_bf16, int64_t rows, int64_t cols, int64_t ld, int32_t colwise,
                         uint32_t sign_mask, float* out, void* cuda_stream) {
  if (!x_bf16 || !out) return NVFP4_ERR_NULL;
  if (rows <= 0 || cols <= 0 || ld < cols) return NVFP4_ERR_SHAPE;
  if ((colwise ? rows : cols) % 16 != 0) return NVFP4_ERR_SHAPE;
  return launch_rht16(x_bf16, rows, cols, ld, colwise != 0, sign_mask & 0xffffu, out,
                      static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? NVFP4_OK
             : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_e2m1_sr(const float* v, const uint8_t* u, int64_t n, uint8_t* codes, void* cuda_stream) {
  if (!v || !u || !codes) return NVFP4_ERR_NULL;
  if (n <= 0) return NVFP4_ERR_SHAPE;
  return launch_e2m1_sr(v, u, n, codes, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? NVFP4_OK
                                                                                                 : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_device_status(void* cuda_stream, uint32_t* detail) {
  uint32_t code = 0;
  if (read_device_status(static_cast<cudaStream_t>(cuda_stream), &code) != cudaSuccess) return NVFP4_ERR_CUDA;
  if (detail) *detail = code;
  return code ? NVFP4_ERR_TIMEOUT : NVFP4_OK;
}

nvfp4_status nvfp4_test_wait_timeout(uint64_t limit_ns, void* cuda_stream) {
  if (limit_ns == 0 || limit_ns > 100000000ull) return NVFP4_ERR_ARG;  // at most 0.1 s
  return launch_wait_probe(limit_ns, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

int32_t nvfp4_set_gemm_experiment(int32_t mode, int32_t max_pairs, void* probe) {
  if (mode < 0 || mode > 255 || max_pairs < 0) return -1;
  set_gemm_experiment(mode, max_pairs, static_cast<unsigned long long*>(probe));
  return 0;
}

int32_t nvfp4_set_gemm_tile_n(int32_t tile_n) {
  if (tile_n != 0 && tile_n != 128 && tile_n != 256 && tile_n != 512 && tile_n != 768) return -1;
  g_tile_n.store(tile_n, std::memory_order_relaxed);
  return 0;
}

const char* nvfp4_status_string(nvfp4_status s) {
  switch (s) {
    case NVFP4_OK: return "ok";
    case NVFP4_ERR_NULL: return "a required pointer is NULL";
    case NVFP4_ERR_SHAPE: return "unsupported shape";
    case NVFP4_ERR_ALIGN: return "insufficient alignment";
    case NVFP4_ERR_ARG: return "unsupported option";
    case NVFP4_ERR_WORKSPACE: return "workspace missing or too small (or the problem exceeds the built-in scratch)";
    case NVFP4_ERR_CUDA: return "CUDA call failed";
    case NVFP4_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case NVFP4_ERR_UNIMPLEMENTED: return "not implemented";
  }
  return "unknown status";
}

uint64_t nvfp4_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
