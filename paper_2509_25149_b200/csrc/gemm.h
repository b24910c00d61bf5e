// Internal launch interface of the block-scaled GEMM kernel.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace nvfp4 {

struct GemmArgs {
  const uint8_t* sfa;     // swizzled scale atoms of A [M x K/16]
  const uint8_t* sfb;     // swizzled scale atoms of B [N x K/16]
  const float* a_global;  // {amax, s_dec}
  const float* b_global;
  void* d;                // [M x N], bf16 or fp32
  int64_t ldd;
  int M, N, K;
  int d_is_fp32, accumulate;
  int mx;                 // operands are MXFP4 (UE8M0 scale per 32 elements) instead of NVFP4
  const float* a_rows;    // per-row {amax, s_dec} pairs of A / B when their global scale is taken per row, else NULL
  const float* b_rows;    // (CTA-pair kernel with 256 x 256 tiles only)
  int chained;            // the previous launch on the stream is a kernel of the same call (see launch_kernel)
};

// tile_n: 128 or 256 (one CTA per tile; 256 needs N % 256 == 0, otherwise 128 is used), 512 (CTA pairs, 256 x 256
// tiles; M, N % 256 == 0) or 768 (CTA pairs, 256 x 384 tiles; M % 256 == 0, N % 128 == 0, N >= 256)
cudaError_t launch_gemm(const GemmArgs& g, const void* a_codes, const void* b_codes, int tile_n, cudaStream_t s);
// Two independent GEMMs in one launch of the CTA-pair kernel (all of M, N multiples of 256, K of 256): the tiles of
// g0 are worked through first, then those of g1, on one persistent grid.
// wide_tiles: 256 x 384 tiles (gemm_wide.cuh) when both shapes allow, else 256 x 256.
cudaError_t launch_gemm_two(const GemmArgs& g0, const void* a0, const void* b0, const GemmArgs& g1, const void* a1,
                            const void* b1, bool wide_tiles, cudaStream_t s);
// Scheduling estimate: do 256 x 384 tiles beat 256 x 256 tiles for this problem (or pair of problems in one launch)?
bool prefer_wide_tiles(const GemmArgs& g0, const GemmArgs* g1);
// Measurement aids of the CTA-pair kernel with 256 x 256 tiles (0, 0, NULL = normal operation): mode bit 0 = no MMAs,
// bit 1 = no operand loads, bit 2 = no scale loads / copies, bit 3 = accumulator handed back unread and nothing
// stored, bit 4 = the issuer does not wait for the accumulator (results meaningless with any bit set); max_pairs caps the
// persistent grid; probe = device array of eight 64-bit words per pair (SM cycles and nanoseconds of the issuer's main
// loop, k-blocks, tiles, cycles waiting for the accumulator hand-over; three unused).
void set_gemm_experiment(int mode, int max_pairs, unsigned long long* probe);
cudaError_t read_device_status(cudaStream_t s, uint32_t* code);
// test aid: a bounded wait that is made to run out (a barrier nobody arrives at); leaves kWaitProbeCode in the
// status word and returns by itself
constexpr uint32_t kWaitProbeCode = 0x7E570001u;
cudaError_t launch_wait_probe(unsigned long long limit_ns, cudaStream_t s);
// device address of the status word on the current device (for kernels of other translation units)
cudaError_t device_status_word(unsigned int** word);

// BF16 GEMM D[M x N] = A B^T on CTA pairs (gemm_bf16.cuh) for layers kept in higher precision.
// a_mn / b_mn = 0: the operand is stored [M or N][K] (contraction contiguous); 1: stored [K][M or N].
// M, N, K multiples of 8 (tiles of 256 x 256 x 64 with zero-filled / clipped edges); leading dimensions in elements.
struct DenseGemmArgs {
  const void* a;
  const void* b;
  void* d;
  int64_t lda, ldb, ldd;
  int M, N, K;
  int a_mn, b_mn;
  int d_is_fp32, accumulate;
};
cudaError_t launch_gemm_bf16(const DenseGemmArgs& g, cudaStream_t s);

}  // namespace nvfp4
