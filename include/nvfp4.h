/*
 * nvfp4.h -- C ABI of the B200 (sm_100a) NVFP4 quantize + block-scaled FP4 GEMM library.
 *
 * The calls follow the paper's statement of the problem ("Pretraining Large Language
 * Models with NVFP4"): a high-precision tensor is converted to E2M1 codes, one E4M3
 * decode scale per block and one FP32 per-tensor decode scale (Appendix B, Eq. 1-4);
 * two such tensors are multiplied with block and tensor scales into BF16/FP32
 * (Eq. 5 and the sentence after it); a linear layer does this three times (Section 4.1,
 * the compute-flow figure).
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers on the current CUDA device and are owned by the
 *     caller; the library allocates no device memory and keeps no per-call state.  The
 *     nvfp4_tensor / nvfp4_quant_opts structs themselves live in HOST memory.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = the legacy
 *     default stream).  No call synchronises with the host or copies device data back.
 *   - Arguments are validated before anything is launched; a non-zero nvfp4_status means
 *     nothing was enqueued (except NVFP4_ERR_CUDA, which reports a failed launch).
 *   - Inputs must be finite; the result for NaN/Inf inputs is unspecified.
 */
#ifndef NVFP4_H_
#define NVFP4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define NVFP4_API __attribute__((visibility("default")))
#else
#define NVFP4_API
#endif

typedef enum nvfp4_status {
  NVFP4_OK = 0,
  NVFP4_ERR_NULL = 1,          /* a required pointer is NULL                                  */
  NVFP4_ERR_SHAPE = 2,         /* a dimension is not a multiple of what the layout needs      */
  NVFP4_ERR_ALIGN = 3,         /* a pointer or leading dimension is not sufficiently aligned  */
  NVFP4_ERR_ARG = 4,           /* an option has an unsupported value or combination           */
  NVFP4_ERR_WORKSPACE = 5,     /* workspace missing or smaller than the *_workspace_bytes()   */
  NVFP4_ERR_CUDA = 6,          /* a CUDA runtime / driver call failed                         */
  NVFP4_ERR_TIMEOUT = 7,       /* a bounded device-side wait expired (see device_status)      */
  NVFP4_ERR_UNIMPLEMENTED = 8
} nvfp4_status;

enum { NVFP4_ROUND_NEAREST_EVEN = 0, NVFP4_ROUND_STOCHASTIC = 1 };
enum { NVFP4_SF_LINEAR = 0, NVFP4_SF_SWIZZLED = 1 };
/* Element / scale format of a copy.  NVFP4 is the paper's format (Section 2, Appendix B).  MXFP4 is the
   format the paper compares against (Section 2, Section 5, Appendix B.4): E2M1 elements with one UE8M0
   power-of-two scale per 32 elements, the decode scale amax_b / 6 rounded UP to a power of two, no
   tensor-level scale (global = {0, 1}), transform size 32 on the weight-gradient operands, 32x32 blocks
   for weights.
   NVFP4_ROWSCALE is NVFP4 with the FP32 "global" scale taken per ROW of the copy instead of per tensor (the
   closing remark of Appendix B.1: with one global scale per row no separate amax sweep over the whole tensor is needed): global holds rows pairs {amax of the row, s_dec of the row}, Eq. 1 per row,
   Eq. 2-4 unchanged.  Row-wise copies only; nvfp4_quantize makes them in ONE pass and nvfp4_gemm applies the
   vectors in its epilogue (D[i][j] = s_dec^A[i] * s_dec^B[j] * sum ...). */
enum { NVFP4_FORMAT_NVFP4 = 0, NVFP4_FORMAT_MXFP4 = 1, NVFP4_FORMAT_NVFP4_ROWSCALE = 2 };
enum {
  /* the column-wise copy draws its stochastic-rounding bits from a second stream (bit 63 of
     sr_offset set) instead of sharing the draw of the same source element with the row-wise copy */
  NVFP4_SR_INDEPENDENT_COPIES = 1,
  /* global[0] of each requested copy already holds the tensor amax: skip the reduction pass */
  NVFP4_AMAX_PROVIDED = 2,
  /* the source is binary32 instead of bf16 (Appendix B names FP32 as well as BF16 as the precision converted from), e.g. weights
     quantized from their FP32 master copy.  NVFP4 outputs without the Hadamard transform only; ld counts floats */
  NVFP4_INPUT_FP32 = 4,
  /* nvfp4_linear_fwd only, forward-only calls (X_col_saved == NULL): quantize X with a global scale per row in
     one pass (NVFP4_FORMAT_NVFP4_ROWSCALE) and apply the scale vector in the Fprop epilogue */
  NVFP4_LINEAR_ROW_SCALES = 8
};

/*
 * One quantized copy of a tensor (Appendix B.3: what is kept in memory is the codes, the block decode scales and
 * the tensor decode scale).  The copy is a row-major [rows x cols] matrix whose
 * columns are the dot-product (contraction) dimension of the GEMM that will read it.
 *   codes : rows * cols/2 bytes; element (r, c) is the E2M1 nibble of byte [r][c/2], even c in
 *           the low nibble.  E2M1 = sign, 2 exponent bits, 1 mantissa bit (Section 2).
 *   scales: rows * cols/16 bytes of E4M3 (bias 7, max 448) block decode scales, Eq. 3.
 *           NVFP4_SF_LINEAR  : byte of (r, kb) at r * cols/16 + kb.
 *           NVFP4_SF_SWIZZLED: the layout the block-scaled tensor-core instruction reads: 512-byte
 *             atoms of 128 rows x 4 blocks, atoms ordered along the row's blocks first:
 *             ((r/128) * (cols/64) + kb/4) * 512 + (r%32) * 16 + ((r%128)/32) * 4 + kb%4.
 *             Needs rows % 128 == 0 and cols % 64 == 0.
 *   global: float[2] = { amax of the (transformed) tensor, s_dec = 1 / (6*448/amax) }, Eq. 1.
 */
typedef struct nvfp4_tensor {
  uint8_t* codes;
  uint8_t* scales;
  float* global;
  int64_t rows, cols;
  int32_t sf_layout;
  int32_t format;   /* NVFP4_FORMAT_NVFP4 (0) or NVFP4_FORMAT_MXFP4; MXFP4: scales hold rows * cols/32 UE8M0
                       bytes (byte b = 2^(b-127)), same two layouts with 32-element blocks (swizzled needs
                       cols % 128 == 0), global is written as {0, 1} and not used;
                       NVFP4_FORMAT_NVFP4_ROWSCALE: global is float[2 * rows] */
} nvfp4_tensor;

/*
 * Quantization recipe (Section 4: 1x16 blocks for activations and gradients, 16x16 blocks for
 * weights; 16x16 random Hadamard transform on weight-gradient GEMM inputs; stochastic rounding
 * for gradients, round-to-nearest-even otherwise).
 */
typedef struct nvfp4_quant_opts {
  int32_t block_rows;     /* 1: one scale per 1x16 block; 16: one scale per 16x16 block (Sec. 4.3),  */
                          /*    replicated to the 16 1x16 blocks it covers in either copy            */
                          /*    (MXFP4 outputs: 1 or 32, blocks of 1x32 / 32x32)                      */
  int32_t rounding;       /* NVFP4_ROUND_NEAREST_EVEN or NVFP4_ROUND_STOCHASTIC (Sec. 4.4)            */
  int32_t rht_rowwise;    /* 1: rotate every aligned 16-chunk of each row of the row-wise copy by     */
  int32_t rht_colwise;    /*    S*H_16 before scaling (Appendix C); same for the column-wise copy     */
  uint32_t rht_sign_mask; /* low 16 bits: bit j set => the j-th input of a chunk is negated (S_d);    */
                          /* MXFP4 outputs use all 32 bits (transform size 32, Section 5)             */
  int32_t flags;          /* NVFP4_SR_INDEPENDENT_COPIES | NVFP4_AMAX_PROVIDED | NVFP4_INPUT_FP32     */
  uint64_t seed;          /* Philox4x32-10 key                                                        */
  uint64_t sr_offset;     /* Philox counter words 2..3; words 0..1 = (row-major source index) >> 4,   */
                          /* and the element uses byte (index & 15) of the 16 output bytes            */
  int32_t rht_dim;        /* size d of the transform: 0 = the format's own (16; 32 for MXFP4); 2, 4,  */
                          /* 8 or 128 = the other sizes of Appendix E.4.2 (NVFP4 outputs, bf16 source,*/
                          /* 1x16 blocks): every aligned d-chunk along the copy's contraction         */
                          /* dimension is multiplied by S * H_d / sqrt(d); d = 128 needs that         */
                          /* dimension to be a multiple of 128.  Sign bit of chunk position j is bit  */
                          /* j of rht_sign_mask (j < 32), else bit (j & 31) of                        */
  uint32_t rht_sign_mask_ext[3]; /* rht_sign_mask_ext[(j >> 5) - 1]                                   */
} nvfp4_quant_opts;

/*
 * nvfp4_quantize -- Appendix B (Eq. 1-4) with the recipe options of Section 4.
 *   x_bf16  : device, bf16 [rows x cols] row-major with leading dimension ld (elements);
 *             32-byte aligned, ld % 16 == 0, rows % 16 == 0, cols % 16 == 0.
 *             With NVFP4_INPUT_FP32 in opts->flags the same for a binary32 array.
 *   rowwise : (nullable) receives the copy whose blocks run along the source columns:
 *             rowwise->rows == rows, rowwise->cols == cols.
 *   colwise : (nullable) receives the quantized TRANSPOSE (blocks along the source rows,
 *             Section 4.3: the backward pass contracts over the other dimension):
 *             colwise->rows == cols, colwise->cols == rows.
 *   At least one copy must be requested.  With block_rows == 16 both copies hold the same
 *   quantized values (transposed) and no Hadamard transform is allowed.
 *   rowwise->format == NVFP4_FORMAT_NVFP4_ROWSCALE: one pass, colwise must be NULL, block_rows 1, no transform,
 *   bf16 source; rowwise->global receives 2 * rows floats.
 * Two passes over x: a tensor-amax reduction (in the rotated space for a transformed copy),
 * then transform + scale + round + pack.  Stochastic rounding rounds up iff
 * u + 0.5 < 256 * frac, u = the 8-bit Philox draw of the source position, frac = the position of
 * the scaled value between its two E2M1 neighbours.
 * Errors: NULL / SHAPE / ALIGN / ARG as described at nvfp4_status; nothing is enqueued on error.
 */
NVFP4_API nvfp4_status nvfp4_quantize(const void* x_bf16, int64_t rows, int64_t cols, int64_t ld,
                                      const nvfp4_quant_opts* opts, const nvfp4_tensor* rowwise,
                                      const nvfp4_tensor* colwise, void* cuda_stream);

/*
 * nvfp4_gemm -- Eq. 5: D[i][j] = s_dec^A * s_dec^B * sum_blocks S^A[i,b] S^B[j,b] sum_{k in b} a[i,k] b[j,k]
 *   A [M x K], B [N x K]: quantized copies whose columns are the contraction dimension, scales in
 *   the NVFP4_SF_SWIZZLED layout, M % 128 == 0, N % 128 == 0, K % 256 == 0 (K = A->cols = B->cols).
 *   Shapes with M % 256 == 0 run on CTA pairs (256 x 256 or 256 x 384 tiles), others on one CTA per tile.
 *   D: device, row-major [M x N] with leading dimension ldd (elements, >= N, ldd*elemsize % 16 == 0),
 *   bf16 (round-to-nearest-even) when d_is_fp32 == 0, else fp32.  Partial sums are accumulated in
 *   FP32 by the tensor cores; the product of the two tensor decode scales is applied once at the end.
 *   accumulate != 0 adds the product to the existing contents of an fp32 D (gradient accumulation,
 *   Section 4.1); it is rejected for bf16 outputs.
 *   Both operands must have the same format (MXFP4 operands carry no tensor-level scale and power-of-two
 *   block scales per 32 elements); an NVFP4_ROWSCALE operand combines with an NVFP4 or another NVFP4_ROWSCALE
 *   operand and needs M % 256 == 0 and N % 256 == 0 (the scale vectors are applied by the CTA-pair kernel).
 */
NVFP4_API nvfp4_status nvfp4_gemm(const nvfp4_tensor* A, const nvfp4_tensor* B, void* D,
                                  int32_t d_is_fp32, int64_t ldd, int32_t accumulate,
                                  void* cuda_stream);

/*
 * nvfp4_gemm_bf16 -- the GEMM of a linear layer that is kept in BF16 (Section 4.1: a small share of the layers,
 * the last ones above all, stay in higher precision; Appendix D: all of them late in training).
 *   D[M x N] = op(A) op(B)^T, products of bf16 values accumulated in FP32 by the tensor cores.
 *   A: device bf16.  a_layout NVFP4_K_MAJOR : stored [M][K], leading dimension lda >= K (contraction contiguous);
 *                    a_layout NVFP4_MN_MAJOR: stored [K][M], lda >= M (the operand is read transposed).
 *   B: device bf16.  b_layout NVFP4_K_MAJOR : stored [N][K], ldb >= K;  NVFP4_MN_MAJOR: stored [K][N], ldb >= N.
 *   D: device, row-major [M x N], ldd >= N, bf16 (round-to-nearest-even) or fp32 (d_is_fp32 != 0);
 *      accumulate != 0 adds into an fp32 D.
 *   M, N, K multiples of 8 (the kernel works on 256 x 256 x 64 tiles; ragged edges are zero-filled on load and
 *   clipped on store by the tensor maps); pointers 16-byte aligned, lda, ldb multiples of 8, ldd * elemsize of 16.
 *   Nothing is enqueued on error.
 */
enum { NVFP4_K_MAJOR = 0, NVFP4_MN_MAJOR = 1 };
NVFP4_API nvfp4_status nvfp4_gemm_bf16(const void* A, int32_t a_layout, int64_t lda, const void* B, int32_t b_layout,
                                       int64_t ldb, int64_t M, int64_t N, int64_t K, void* D, int32_t d_is_fp32,
                                       int64_t ldd, int32_t accumulate, void* cuda_stream);

/*
 * The same layer as nvfp4_linear_fwd / _bwd without quantization (Section 4.1, Appendix D), on the same row-major
 * operands X [M x K], W [N x K], dY [M x N], all contiguous bf16; no transposed copies are made:
 *   fwd: Y  = X W^T (bf16);   bwd: dX = dY W (bf16), dW = dY^T X (fp32, accumulate_dw != 0 adds into it);
 *   dX or dW may be NULL to skip that GEMM.  M, N, K multiples of 8.
 */
NVFP4_API nvfp4_status nvfp4_linear_bf16_fwd(const void* X, const void* W, int64_t M, int64_t N, int64_t K,
                                             void* Y_bf16, void* cuda_stream);
NVFP4_API nvfp4_status nvfp4_linear_bf16_bwd(const void* dY, const void* X, const void* W, int64_t M, int64_t N,
                                             int64_t K, void* dX_bf16, float* dW_fp32, int32_t accumulate_dw,
                                             void* cuda_stream);

/*
 * Quantization-error metrics (Appendix E.2: the layers whose FP4 weight gradients carry the largest quantization
 * error are the ones worth keeping in higher precision; such a metric can drive that choice).
 *
 * nvfp4_quant_error: out2 = { sum (x - x^)^2, sum x^2 } over the tensor, x^ the decoded row-wise copy q of the bf16
 *   source x [rows x cols] (leading dimension ld; same alignment rules as nvfp4_quantize).  q is NVFP4 or MXFP4,
 *   scales linear or swizzled, and must be a copy WITHOUT the Hadamard transform (a transformed copy lives in the
 *   rotated space).  The ratio of the two sums is the relative squared quantization error.
 * nvfp4_sq_error: out2 = { sum (ref - test)^2, sum ref^2 } of two dense row-major [rows x cols] tensors, each bf16 or
 *   fp32 (e.g. dW from nvfp4_linear_bwd against dW from nvfp4_linear_bf16_bwd).  cols % 8 == 0, leading dimensions
 *   multiples of 8, pointers 16-byte (bf16) / 32-byte (fp32) aligned.
 * out2: DEVICE double[2], written in stream order (zeroed, then accumulated in FP64; the order of the additions, and
 *   with it the last bits, vary from run to run).
 */
NVFP4_API nvfp4_status nvfp4_quant_error(const void* x_bf16, int64_t rows, int64_t cols, int64_t ld,
                                         const nvfp4_tensor* q, double* out2, void* cuda_stream);
NVFP4_API nvfp4_status nvfp4_sq_error(const void* ref, int32_t ref_is_fp32, int64_t ld_ref, const void* test,
                                      int32_t test_is_fp32, int64_t ld_test, int64_t rows, int64_t cols,
                                      double* out2, void* cuda_stream);

/*
 * Linear layer, Section 4.1 (three GEMMs, each quantizing its inputs):
 *   X [M x K] bf16 (tokens x in-features), W [N x K] bf16, dY [M x N] bf16, all contiguous.
 *   M, N, K multiples of 256.
 *
 * nvfp4_linear_fwd: Y = X W^T (bf16).  Quantizes X row-wise (1x16, RNE) for Fprop and, when
 *   X_col_saved is given, column-wise with the Hadamard transform for the later Wgrad; quantizes W
 *   with 16x16 blocks into W_row (Fprop) and W_col_saved (Dgrad) unless w_is_cached != 0, in which
 *   case W_row must already hold the quantized weight.  opts supplies rht_sign_mask (and rht_dim, when another
 *   transform size than the format's own is wanted: the same value must then be given to nvfp4_linear_bwd), and the flag
 *   NVFP4_LINEAR_ROW_SCALES for forward-only calls (then X_col_saved must be NULL).
 *   workspace: device scratch of nvfp4_linear_fwd_workspace_bytes(M, K) for the row-wise copy of X.
 * nvfp4_linear_bwd: dX = dY W (bf16), dW = dY^T X (fp32).  Quantizes dY with stochastic rounding
 *   (opts->seed, opts->sr_offset) row-wise for Dgrad and column-wise with the Hadamard transform
 *   for Wgrad.  dX or dW may be NULL to skip that GEMM.  accumulate_dw != 0 adds into dW.
 *   workspace: device scratch of nvfp4_linear_bwd_workspace_bytes(M, N) for the two copies of dY.
 *   When both GEMMs are requested they run in one launch of the CTA-pair kernel.
 * Ordering: both calls are stream-ordered as a whole (everything enqueued before them on the stream has
 *   finished before their first kernel starts, and their results are complete for whatever is enqueued after
 *   them).  Inside a call the kernels overlap only their set-up with the tail of the kernel before them
 *   (programmatic dependent launch) and never read each other's output early; in the NVFP4 bf16 path the tensor
 *   amax of W (Appendix B.1) is taken inside the kernel that quantizes X.  Results are bit-identical to the
 *   same steps issued one by one through nvfp4_quantize and nvfp4_gemm.
 * Format: the layer runs in the format of the copies it is given (W_row / W_col_saved / X_col_saved must
 *   agree).  With MXFP4 copies the same sequence uses 1x32 and 32x32 blocks and the 32-point transform
 *   (Section 5); opts->rht_sign_mask then supplies 32 sign bits.
 */
NVFP4_API size_t nvfp4_linear_fwd_workspace_bytes(int64_t M, int64_t K);
NVFP4_API size_t nvfp4_linear_bwd_workspace_bytes(int64_t M, int64_t N);
NVFP4_API nvfp4_status nvfp4_linear_fwd(const void* X, const void* W, int64_t M, int64_t N,
                                        int64_t K, const nvfp4_quant_opts* opts, void* Y_bf16,
                                        const nvfp4_tensor* X_col_saved, const nvfp4_tensor* W_row,
                                        const nvfp4_tensor* W_col_saved, int32_t w_is_cached,
                                        void* workspace, size_t workspace_bytes, void* cuda_stream);
NVFP4_API nvfp4_status nvfp4_linear_bwd(const void* dY, const nvfp4_tensor* X_col_saved,
                                        const nvfp4_tensor* W_col_saved, int64_t M, int64_t N,
                                        int64_t K, const nvfp4_quant_opts* opts, void* dX_bf16,
                                        float* dW_fp32, int32_t accumulate_dw, void* workspace,
                                        size_t workspace_bytes, void* cuda_stream);

/*
 * nvfp4_linear_fwd_noalloc -- the forward pass for callers that cannot hand over scratch memory.
 * (The paper has no counterpart: this is a packaging variant of nvfp4_linear_fwd, same arithmetic.)
 *
 * Some callers have no way to allocate device memory at the point where they run a layer: code inside a
 * real-time or inference-server callback that must not call cudaMalloc (it synchronises the device and may
 * fail under memory pressure), plug-ins that are handed only their input and output buffers, or hosts whose
 * allocator is owned by another component.  For them the row-wise NVFP4 copy of X, which nvfp4_linear_fwd
 * keeps in caller-provided workspace, is placed in an array built into the library's device image.
 *
 *   - Arguments are those of nvfp4_linear_fwd without `workspace` / `workspace_bytes`; inputs and outputs
 *     (X, W, Y, the saved copies) are still the caller's.
 *   - Limit: nvfp4_linear_fwd_workspace_bytes(M, K) must not exceed nvfp4_linear_fwd_noalloc_max_bytes()
 *     (16 MiB: M * K up to about 29.8 million elements, e.g. 4096 x 5120); larger problems return
 *     NVFP4_ERR_WORKSPACE and nothing is enqueued.  Every GPU that loads the library carries these 16 MiB
 *     until the process exits.
 *   - The call allocates nothing: no cudaMalloc / cudaFree and no allocating library routine.  Its first call
 *     on a device looks up the array's device address (a host-side query, no allocation) with that device
 *     current; make that first call before any stream capture begins.
 *   - All calls share the one array and find the previous call's contents in it; what must start from zero
 *     (the amax word of the reduction) is cleared by the call itself.  Two calls whose work overlaps on the
 *     GPU (different streams, or different threads on the same device) race on the array: serialise them.
 */
NVFP4_API size_t nvfp4_linear_fwd_noalloc_max_bytes(void);
NVFP4_API nvfp4_status nvfp4_linear_fwd_noalloc(const void* X, const void* W, int64_t M, int64_t N,
                                                int64_t K, const nvfp4_quant_opts* opts, void* Y_bf16,
                                                const nvfp4_tensor* X_col_saved, const nvfp4_tensor* W_row,
                                                const nvfp4_tensor* W_col_saved, int32_t w_is_cached,
                                                void* cuda_stream);

/*
 * Test aids (not on the hot path).
 * nvfp4_dequantize: out[r][c] = code * fp32(block scale) * s_dec as fp32 (the decode of Section 2).
 * nvfp4_rht16: the transformed values y = x*(S*H_16) of the row-wise (colwise == 0, out [rows x cols])
 *   or column-wise (colwise != 0, out [cols x rows]) copy, fp32, as the quantizer sees them.
 * nvfp4_e2m1_sr: codes[i] = the E2M1 code (4 bits in a byte) of the already scaled value v[i] under the
 *   stochastic-rounding rule of Section 4.4 with the 8-bit draw u[i], computed by the device routine the
 *   quantizer kernels use; v, u, codes are device arrays of n elements.
 */
NVFP4_API nvfp4_status nvfp4_dequantize(const nvfp4_tensor* t, float* out, void* cuda_stream);
NVFP4_API nvfp4_status nvfp4_e2m1_sr(const float* v, const uint8_t* u, int64_t n, uint8_t* codes,
                                     void* cuda_stream);
NVFP4_API nvfp4_status nvfp4_rht16(const void* x_bf16, int64_t rows, int64_t cols, int64_t ld,
                                   int32_t colwise, uint32_t sign_mask, float* out,
                                   void* cuda_stream);

/*
 * Every device-side wait in the GEMM is bounded; when one expires the kernel records a code in a
 * device status word and returns.  This call synchronises `cuda_stream`, reads and clears that word
 * and returns NVFP4_ERR_TIMEOUT (with *detail = the recorded code, if detail != NULL) or NVFP4_OK.
 */
NVFP4_API nvfp4_status nvfp4_device_status(void* cuda_stream, uint32_t* detail);

/*
 * Test aid for that path: enqueues a one-warp kernel that waits, for at most `limit_ns` nanoseconds
 * (1 .. 100 000 000), on a barrier nobody arrives at.  The wait runs out, the kernel records the code
 * 0x7E570001 in the status word and returns by itself; the next nvfp4_device_status() reports
 * NVFP4_ERR_TIMEOUT with that code, and the device stays usable.  NVFP4_ERR_ARG for a limit out of range.
 */
NVFP4_API nvfp4_status nvfp4_test_wait_timeout(uint64_t limit_ns, void* cuda_stream);

/* Tuning knob: which GEMM tiling to use.  128 / 256 = one CTA per 128 x 128 / 128 x 256 output tile;
 * 512 = a CTA pair per 256 x 256 tile (needs M % 256 == 0 and N % 256 == 0, otherwise 128 is used);
 * 768 = a CTA pair per 256 x 384 tile, plus up to two 256-wide tiles per row of tiles (needs M % 256 == 0,
 * N % 128 == 0 and N >= 256, otherwise as 512);
 * 0 = choose by shape (for the pair kernels: the tile width whose static schedule is estimated shorter).
 * Returns 0, or -1 for any other value.  Process-wide; results do not depend on it
 * beyond FP32 summation order. */
NVFP4_API int32_t nvfp4_set_gemm_tile_n(int32_t tile_n);

/*
 * Measurement aid for the main loop of the CTA-pair GEMM with 256 x 256 tiles (what bounds a 256-deep k-block):
 * affects that kernel's later launches in this process; (0, 0, NULL) restores normal operation.
 *   mode      bit 0: the issuer skips the MMAs; bit 1: the producer skips the operand loads; bit 2: the scale atoms
 *             are neither loaded nor copied to tensor memory; bit 3: the epilogue hands the accumulator back
 *             unread and stores nothing; bit 4: the issuer does not wait for the accumulator to be handed back.
 *             bit 5: the scale atoms reach tensor memory through the copy engine (twelve tcgen05.cp per k-block,
 *             issued by the MMA issuer in front of the k-block's MMAs) instead of through the scale warps'
 *             registers; alone, this bit leaves the output CORRECT.
 *             bit 6: the epilogue converts but does not write its staging buffer; bit 7: it issues no TMA store.
 *             With any of bits 0-4, 6, 7 set the OUTPUT IS MEANINGLESS (timing
 *             only); every barrier is still signalled, so the kernel runs to its end.
 *   max_pairs > 0: at most that many CTA pairs (SM pairs) take part.
 *   probe     device array of 8 x uint64 per pair; each pair's issuer writes five: SM cycles and nanoseconds of its
 *             main loop, the k-blocks and the tiles it went through, and the cycles it spent between issuing a
 *             tile's last MMA and getting the accumulator back from the epilogue.
 * Returns 0, or -1 for a value out of range.
 */
NVFP4_API int32_t nvfp4_set_gemm_experiment(int32_t mode, int32_t max_pairs, void* probe);

NVFP4_API const char* nvfp4_status_string(nvfp4_status s);
/* Number of kernel launches this process has enqueued through the library so far. */
NVFP4_API uint64_t nvfp4_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* NVFP4_H_ */
