// NVFP4 quantizer for sm_100a: tensor-amax reduction (pass 1) and the fused
// transform + scale + round + pack kernel producing the row-wise and/or the transposed copy (pass 2).
//
// Paper: Appendix B (Eq. 1-4), Appendix C (16x16 random Hadamard transform), Section 4.3 (16x16
// weight blocks, two copies for the two passes), Section 4.4 (stochastic rounding).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "async_ptx.cuh"
#include "common.cuh"
#include "quantize.h"
#include "quantize_common.cuh"

namespace nvfp4 {

// ---------------------------------------------------------------------------------------------
// Pass 1: tensor amax (Appendix B.1), plain and / or in the rotated space of a transformed copy.
// CTA tile 128 rows x 256 columns; a warp owns 16 rows, a lane 8 columns of each of them.
// ---------------------------------------------------------------------------------------------
template <bool PLAIN, bool ROT_ROW, bool ROT_COL>
__global__ void __launch_bounds__(256) amax_kernel(const uint16_t* __restrict__ x, int64_t rows,
                                                   int64_t cols, int64_t ld, uint32_t sign_mask,
                                                   int tiles_c, float* __restrict__ out_plain0,
                                                   float* __restrict__ out_plain1,
                                                   float* __restrict__ out_rot_row,
                                                   float* __restrict__ out_rot_col) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t tr = blockIdx.x / tiles_c, tc = blockIdx.x % tiles_c;
  const int64_t r0 = tr * 128 + warp * 16;
  const int64_t c0 = tc * 256 + lane * 8;
  const bool in_range = (r0 < rows) && (c0 < cols);  // rows % 16 == 0, cols % 8 == 0
  griddep_launch_dependents();  // pass 2 may set itself up while the last CTAs of this pass run

  uint4 raw[16];
  if (in_range) {
    const uint16_t* p = x + r0 * ld + c0;
#pragma unroll
    for (int j = 0; j < 16; ++j) raw[j] = ldg128_stream(p + j * ld);
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j) raw[j] = make_uint4(0, 0, 0, 0);
  }

  float m_plain = 0.f, m_row = 0.f, m_col = 0.f;
  if (PLAIN) {
    uint32_t acc = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      acc = absmax_bf16x2(acc, raw[j].x);
      acc = absmax_bf16x2(acc, raw[j].y);
      acc = absmax_bf16x2(acc, raw[j].z);
      acc = absmax_bf16x2(acc, raw[j].w);
    }
    m_plain = fmaxf(bf16_lo(acc), bf16_hi(acc));
  }
  if (ROT_COL) {
    // chunks run down the 16 rows of the warp's slab: one transform per column
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      float a[16], b[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        uint32_t word = (w == 0) ? raw[j].x : (w == 1) ? raw[j].y : (w == 2) ? raw[j].z : raw[j].w;
        word ^= sign_pair(sign_mask, j, j);
        a[j] = bf16_lo(word);
        b[j] = bf16_hi(word);
      }
      fwht16(a);
      fwht16(b);
#pragma unroll
      for (int j = 0; j < 16; ++j) m_col = fmaxf(m_col, fmaxf(fabsf(a[j]), fabsf(b[j])));
    }
    m_col *= 0.25f;
  }
  if (ROT_ROW) {
    // a chunk is 16 consecutive columns = the 8 columns of an even lane and of the next odd lane
    const int half = lane & 1;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      float v[8];
      const uint32_t w4[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        uint32_t word = w4[k] ^ sign_pair(sign_mask, half * 8 + 2 * k, half * 8 + 2 * k + 1);
        v[2 * k] = bf16_lo(word);
        v[2 * k + 1] = bf16_hi(word);
      }
#pragma unroll
      for (int h = 1; h < 8; h <<= 1)
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if ((i & h) == 0) {
            float a = v[i], b = v[i | h];
            v[i] = a + b;
            v[i | h] = a - b;
          }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float other = __shfl_xor_sync(0xffffffffu, v[i], 1);
        float y = half ? (other - v[i]) : (v[i] + other);
        m_row = fmaxf(m_row, fabsf(y));
      }
    }
    m_row *= 0.25f;
  }

  __shared__ float red[3][8];
  m_plain = warp_max(m_plain);
  m_row = warp_max(m_row);
  m_col = warp_max(m_col);
  if (lane == 0) {
    red[0][warp] = m_plain;
    red[1][warp] = m_row;
    red[2][warp] = m_col;
  }
  __syncthreads();
  if (threadIdx.x < 3) {
    float m = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) m = fmaxf(m, red[threadIdx.x][w]);
    // non-negative floats order like their bit patterns
    uint32_t bits = __float_as_uint(m);
    if (threadIdx.x == 0 && PLAIN) {
      if (out_plain0) atomicMax(reinterpret_cast<unsigned int*>(out_plain0), bits);
      if (out_plain1) atomicMax(reinterpret_cast<unsigned int*>(out_plain1), bits);
    }
    if (threadIdx.x == 1 && ROT_ROW) atomicMax(reinterpret_cast<unsigned int*>(out_rot_row), bits);
    if (threadIdx.x == 2 && ROT_COL) atomicMax(reinterpret_cast<unsigned int*>(out_rot_col), bits);
  }
}

// ---------------------------------------------------------------------------------------------
// Pass 1 for a copy transformed down the rows (the transposed copy of a Wgrad operand, Appendix C): the
// 16-point transform of 8 columns at a time is one bf16 tensor-core product  Y(16x8) = A(16x16) * X(16x8)  with
// A[k][j] = s_j * h(k, j) (entries +-1, exact in bf16; FP32 accumulation) and the 1/4 applied to the maximum.
// A lane loads 16 columns of one row; its eight words are fragments of eight 8x8 matrices whose "columns" are an
// interleaved subset of the 64 columns a quad covers - columns are independent under this transform, so any
// assignment works - and movmatrix turns each into the k-pair layout the product wants.
// CTA tile 128 rows x 256 columns; a warp owns 16 rows.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t v) {
  uint32_t r;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(v));
  return r;
}

// d, norm: size of the transform (2, 4, 8 or 16: H_16 is replaced by the block-diagonal matrix of 16 / d copies of
// H_d) and its normalisation 1 / sqrt(d), applied to the maximum.
template <bool PLAIN>
__global__ void __launch_bounds__(256) amax_rot_col_kernel(const uint16_t* __restrict__ x, int64_t rows,
                                                           int64_t cols, int64_t ld, uint32_t sign_mask,
                                                           int tiles_c, float* __restrict__ out_plain0,
                                                           float* __restrict__ out_plain1,
                                                           float* __restrict__ out_rot_col, int d, float norm) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t tr = blockIdx.x / tiles_c, tc = blockIdx.x % tiles_c;
  const int64_t r0 = tr * 128 + warp * 16;
  griddep_launch_dependents();  // pass 2 may set itself up while the last CTAs of this pass run

  uint32_t lo[4][8], hi[4][8];  // rows g and g + 8 of the slab, 16 columns each, four 64-column steps
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int64_t c = tc * 256 + q * 64 + t * 16;
    if (r0 < rows && c < cols) {  // rows % 16 == 0, cols % 16 == 0
      ldg256_stream(x + (r0 + g) * ld + c, lo[q]);
      ldg256_stream(x + (r0 + 8 + g) * ld + c, hi[q]);
    } else {
#pragma unroll
      for (int w = 0; w < 8; ++w) lo[q][w] = hi[q][w] = 0u;
    }
  }

  // A fragments: entry (k, j) = +-1 as bf16 inside the d x d diagonal blocks (0 outside), negative iff
  // popc(k & j) is odd XOR sign bit j
  auto entry = [&](int k, int j) -> uint32_t {
    if ((k ^ j) >= d) return 0u;
    return ((__popc(k & j & (d - 1)) ^ (sign_mask >> j)) & 1u) ? 0xBF80u : 0x3F80u;
  };
  const uint32_t a0 = entry(g, 2 * t) | (entry(g, 2 * t + 1) << 16);
  const uint32_t a1 = entry(g + 8, 2 * t) | (entry(g + 8, 2 * t + 1) << 16);
  const uint32_t a2 = entry(g, 2 * t + 8) | (entry(g, 2 * t + 9) << 16);
  const uint32_t a3 = entry(g + 8, 2 * t + 8) | (entry(g + 8, 2 * t + 9) << 16);

  float m_col = 0.f;
  uint32_t acc = 0u;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      if (PLAIN) {
        acc = absmax_bf16x2(acc, lo[q][w]);
        acc = absmax_bf16x2(acc, hi[q][w]);
      }
      const uint32_t b0 = movmatrix_trans(lo[q][w]);
      const uint32_t b1 = movmatrix_trans(hi[q][w]);
      float d0, d1, d2, d3;
      asm volatile(
          "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
          "{%10,%10,%10,%10};"
          : "=f"(d0), "=f"(d1), "=f"(d2), "=f"(d3)
          : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
      m_col = fmaxf(fmaxf(m_col, fmaxf(fabsf(d0), fabsf(d1))), fmaxf(fabsf(d2), fabsf(d3)));
    }
  }
  m_col *= norm;
  float m_plain = PLAIN ? fmaxf(bf16_lo(acc), bf16_hi(acc)) : 0.f;

  __shared__ float red[2][8];
  m_plain = warp_max(m_plain);
  m_col = warp_max(m_col);
  if (lane == 0) {
    red[0][warp] = m_plain;
    red[1][warp] = m_col;
  }
  __syncthreads();
  if (threadIdx.x < 2) {
    float m = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) m = fmaxf(m, red[threadIdx.x][w]);
    const uint32_t bits = __float_as_uint(m);  // non-negative floats order like their bit patterns
    if (threadIdx.x == 0 && PLAIN) {
      if (out_plain0) atomicMax(reinterpret_cast<unsigned int*>(out_plain0), bits);
      if (out_plain1) atomicMax(reinterpret_cast<unsigned int*>(out_plain1), bits);
    }
    if (threadIdx.x == 1) atomicMax(reinterpret_cast<unsigned int*>(out_rot_col), bits);
  }
}

// ---------------------------------------------------------------------------------------------
// Pass 2: persistent CTAs (two per SM), each working through 128 x 128 tiles of the source.  The tiles arrive by
// TMA (cp.async.bulk.tensor, this GPU's memory, no multicast) in a ring of two 32 KB buffers: the load of tile
// k + 2 is issued as soon as tile k has been consumed, so a tile is in flight during the whole of the previous one;
// out-of-range parts of a ragged tile are zero-filled by the copy.
//   set-up   once per CTA: Eq. 1, and the table  E4M3 byte -> encode scale  of each copy (the text after Eq. 3:
//            s_enc,b = 1 / (fp32(S_b) * s_dec) has only 127 possible values per tensor), so a block costs one
//            conversion and one shared-memory read instead of an IEEE reciprocal;
//   phase 1  each thread owns four 1x16 chunks of the tile and produces the row-wise copy (and, for stochastic
//            rounding, stages the random bytes of its chunks in shared memory);
//   phase 2  each thread owns 16 rows x 2 columns of the tile and produces the transposed copy into a swizzled
//            staging buffer;
//   phase 3  staged codes and scale bytes leave with 16-byte stores.
// A warp's phase 2 reads only what the same warp staged in phase 1, and the buffers phase 3 reads are double
// buffered, so a tile needs one CTA barrier.  Tiles are visited in reverse order so that the end of the tensor,
// which pass 1 touched last, is read first while it may still sit in L2.
// ---------------------------------------------------------------------------------------------
struct QuantSmem {
  static constexpr int kTile = 0;                     // 2 x (128 rows x 256 B of bf16), filled by TMA
  static constexpr int kColCodes = 65536;             // 2 x (128 columns x 64 B)
  static constexpr int kSfRow = kColCodes + 2 * 8192; // 2 x 1 KB
  static constexpr int kSfCol = kSfRow + 2 * 1024;    // 2 x 1 KB
  static constexpr int kBlkEnc = kSfCol + 2 * 1024;   // 64 floats (16x16 mode)
  static constexpr int kBlkByte = kBlkEnc + 256;      // 64 bytes
  static constexpr int kGlobalScales = kBlkByte + 64; // s_enc, s_dec of the row-wise and the column-wise copy
  static constexpr int kEncRow = kGlobalScales + 64;  // 128 floats: encode scale by E4M3 byte, row-wise copy
  static constexpr int kEncCol = kEncRow + 512;       // the same for the transposed copy
  static constexpr int kBars = kEncCol + 512;         // two "tile landed" barriers, then the abort word
  static constexpr int kRand = kBars + 32;            // 128 rows x 128 B of complemented draws (stochastic rounding),
                                                      // or 128 rows x 64 B of row-wise codes (16x16 blocks, both copies)
  static constexpr int kTileBytes = 32768;
  static constexpr int bytes(bool rand, bool row_codes) { return kRand + (rand ? 16384 : row_codes ? 8192 : 0); }
};

// Bounded wait for a tile (2 s): on expiry the abort word of the CTA and the device status word are set.
constexpr uint32_t kQuantWaitCode = 0x51000001u;
__device__ __forceinline__ bool quant_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                           unsigned int* status) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = kQuantWaitCode;
        if (status) atomicCAS(status, 0u, kQuantWaitCode);
        return false;
      }
    }
  }
}

// max(m, |a|, |b|)
__device__ __forceinline__ float amax3(float m, float a, float b) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(m), "f"(fabsf(a)), "f"(fabsf(b)));
  return r;
}
__device__ __forceinline__ float amax16_3(const float (&f)[16]) {
  float m = 0.f;
#pragma unroll
  for (int i = 0; i < 16; i += 2) m = amax3(m, f[i], f[i + 1]);
  return m;
}

// Eq. 2-3: the stored E4M3 byte of a block, S_b = e4m3(fl(fl(amax_b / 6) * s_enc))
__device__ __forceinline__ uint32_t block_scale_byte(float amax_b, float s_enc) {
  const float t = __fmul_rn(div6_rn(amax_b), s_enc);
  uint16_t packed;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %1;" : "=h"(packed) : "f"(t));
  return packed & 0xffu;
}
// the text after Eq. 3: encode scale of a block from its stored byte, fl(1 / fl(fp32(S_b) * s_dec)), 0 for S_b = 0
__device__ __forceinline__ float encode_scale_of_byte(uint32_t byte, float s_dec) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)byte));
  const float sf = __half2float(__ushort_as_half((unsigned short)(h2 & 0xffffu)));
  const float d = __fmul_rn(sf, s_dec);
  return (byte == 0u) ? 0.0f : fminf(__frcp_rn(d), kFltMax);
}

template <bool HAS_ROW, bool HAS_COL, bool BLOCK2D, bool RHT_ROW, bool RHT_COL, bool SR, bool SIDE = false>
__global__ void __launch_bounds__(256, 2) quantize_kernel(const __grid_constant__ CUtensorMap src_map,
                                                          const __grid_constant__ CUtensorMap side_map,
                                                          const QuantArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_cb = (int)(a.cols >> 4);  // 16-blocks per source row
  const int n_rb = (int)(a.rows >> 4);  // 16-blocks per source column
  // 16x16 blocks with both copies requested: the transposed copy holds the very codes of the row-wise one
  // (Section 4.3), so it is made by transposing nibbles; the raw tile is not needed a second time
  constexpr bool kNibbleTranspose = BLOCK2D && HAS_ROW && HAS_COL;
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + QuantSmem::kBars + 16);
  const uint32_t bar0 = smem_u32(smem + QuantSmem::kBars), tile0 = smem_u32(smem + QuantSmem::kTile);

  const int total = a.tiles_r * a.tiles_c, stride = (int)gridDim.x;
  const int first = total - 1 - (int)blockIdx.x;         // this CTA's tiles: first, first - stride, ...
  const int n_mine = first >= 0 ? first / stride + 1 : 0;
  // SIDE: the CTA also streams its share of a second tensor's tiles through the same ring and takes their plain
  // amax (pass 1 of that tensor, Appendix B.1): memory-bound work riding on an issue-bound kernel.  Side tiles go
  // front to back (the tensor's own pass 2 starts from its end), interleaved in proportion with the CTA's own tiles.
  const int side_total = SIDE ? a.side_tiles_r * a.side_tiles_c : 0;
  const int m_mine = (int)blockIdx.x < side_total ? (side_total - 1 - (int)blockIdx.x) / stride + 1 : 0;
  const int n_jobs = n_mine + m_mine;
  // with k own tiles and sk side tiles behind it, the CTA's next job is a side tile iff ...
  auto side_next = [&](int k, int sk) {
    return SIDE && sk < m_mine && (k >= n_mine || (long long)sk * n_mine < (long long)k * m_mine);
  };
  auto issue_load = [&](int j, int k, int sk) {  // job j (own tile k or side tile sk) into buffer j & 1 (one thread)
    const uint32_t bar = bar0 + 8 * (j & 1), dst = tile0 + (j & 1) * QuantSmem::kTileBytes;
    mbar_expect_tx(bar, QuantSmem::kTileBytes);
    if (side_next(k, sk)) {
      const int t = (int)blockIdx.x + sk * stride, tr = t / a.side_tiles_c, tc = t - tr * a.side_tiles_c;
      tma_load_2d(dst, &side_map, tc * 128, tr * 128, bar);
    } else {
      const int t = first - k * stride, tr = t / a.tiles_c, tc = t - tr * a.tiles_c;
      tma_load_2d(dst, &src_map, tc * 128, tr * 128, bar);
    }
  };
  int ahead_k = 0, ahead_sk = 0;  // thread 0: own / side tiles among the jobs already issued
  auto issue_next = [&](int j) {
    issue_load(j, ahead_k, ahead_sk);
    if (side_next(ahead_k, ahead_sk)) ++ahead_sk; else ++ahead_k;
  };

  // ------------------------------------------------------------------ set-up ----
  float* g_sc = reinterpret_cast<float*>(smem + QuantSmem::kGlobalScales);
  if (threadIdx.x == 0) {
    mbar_init(bar0, 1);
    mbar_init(bar0 + 8, 1);
    *abort_flag = 0u;
    fence_mbarrier_init();
    fence_proxy_async_smem();
    if (n_jobs > 0) issue_next(0);
    if (n_jobs > 1) issue_next(1);
    // the source tiles above are nobody's output in this call; the tensor amax below is the previous kernel's.
    // Every other thread passes the barrier below only after this wait, so no output is written before it either.
    griddep_wait();
    // Eq. 1 (two IEEE divisions per copy)
    float re = 1.f, rd = 1.f, ce = 1.f, cd = 1.f;
    if (HAS_ROW || BLOCK2D) global_scales(HAS_ROW ? a.r_global[0] : a.c_global[0], re, rd);
    if (HAS_COL) {
      if (BLOCK2D && HAS_ROW) {
        ce = re;
        cd = rd;
      } else {
        global_scales(a.c_global[0], ce, cd);
      }
    }
    g_sc[0] = re; g_sc[1] = rd; g_sc[2] = ce; g_sc[3] = cd;
    if (blockIdx.x == 0) {
      if (HAS_ROW) a.r_global[1] = rd;
      if (HAS_COL) a.c_global[1] = cd;
    }
  }
  __syncthreads();
  griddep_launch_dependents();
  const float r_senc = g_sc[0], r_sdec = g_sc[1], c_senc = g_sc[2], c_sdec = g_sc[3];
  const float* enc_row = reinterpret_cast<const float*>(smem + QuantSmem::kEncRow);
  const float* enc_col = reinterpret_cast<const float*>(smem + QuantSmem::kEncCol);
  if (!BLOCK2D) {
    // with the transform the kernel works on 4 * y: the 1/4 is folded into the block amax and the encode scale (exact)
    if (threadIdx.x < 128) {
      if (HAS_ROW)
        reinterpret_cast<float*>(smem + QuantSmem::kEncRow)[threadIdx.x] =
            encode_scale_of_byte(threadIdx.x, r_sdec) * (RHT_ROW ? 0.25f : 1.0f);
    } else {
      if (HAS_COL)
        reinterpret_cast<float*>(smem + QuantSmem::kEncCol)[threadIdx.x - 128] =
            encode_scale_of_byte(threadIdx.x - 128, c_sdec) * (RHT_COL ? 0.25f : 1.0f);
    }
    __syncthreads();
  }

  // per-thread constants of phase 1: chunk column cb, row rl + 4 i for chunk i
  const int cb = lane & 7, rl = warp * 16 + (lane >> 3);
  const uint32_t tile_ld = rl * 256 + cb * 32;     // chunk i of the thread inside a tile buffer: + 1024 i
  const uint32_t rand_st = QuantSmem::kRand + rl * 128 + cb * 16;  // + 512 i
  // sign of source row j of a 16-row group (the transform of the transposed copy negates whole source rows: input j
  // of a chunk = row j of the group) for both halves of a bf16 pair: bits 15 and 31 of sign2 << (15 - j)
  const uint32_t sign2 = (a.sign_mask & 0xffffu) * 0x10001u;
  const int sf_row_pos = a.r_swz ? ((cb >> 2) * 512 + (rl & 31) * 16 + (rl >> 5) * 4 + (cb & 3)) : (rl * 8 + cb);
  const int sf_row_step = a.r_swz ? 64 : 32;
  const int64_t r_pitch = a.cols >> 1;  // bytes per row of the row-wise codes

  // hoisted constants of phase 2: where a thread stages its two columns' codes and scale bytes (iteration it, column
  // parity odd); the 16-byte unit of column pair cp and 16-row group q sits at cp * 128 + ((q ^ cp) & 7) * 16
  const int col_codes_st = lane * 128 + (((warp ^ lane) & 7) << 4);  // + 4096 it
  const int sf_col_pos = a.c_swz ? ((warp >> 2) * 512 + (lane & 15) * 32 + (lane >> 4) * 4 + (warp & 3)) : (lane * 16 + warp);
  const int sf_col_odd = a.c_swz ? 16 : 8, sf_col_it = a.c_swz ? 8 : 512;

  const int step_r = stride / a.tiles_c, step_c = stride - step_r * a.tiles_c;  // tile coordinates move by these
  int tr = first >= 0 ? first / a.tiles_c : 0, tc = first >= 0 ? first - tr * a.tiles_c : 0;
  int k = 0, sk = 0, j = 0;  // own tiles done, side tiles done, jobs done (the ring position)
  uint32_t side_acc = 0;     // |.| maximum of the side tiles, two bf16 lanes
  for (; j < n_jobs; ++j) {
    const uint8_t* const tile_buf = smem + QuantSmem::kTile + (j & 1) * QuantSmem::kTileBytes;
    quant_wait(bar0 + 8 * (j & 1), (uint32_t)(j >> 1) & 1u, abort_flag, a.status);  // the tile has landed
    if (SIDE && side_next(k, sk)) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {  // zero fill outside the tensor leaves the maximum alone
        const uint4 v = *reinterpret_cast<const uint4*>(tile_buf + i * 4096 + threadIdx.x * 16);
        side_acc = absmax_bf16x2(absmax_bf16x2(side_acc, v.x), v.y);
        side_acc = absmax_bf16x2(absmax_bf16x2(side_acc, v.z), v.w);
      }
      __syncthreads();
      if (*abort_flag) break;
      if (threadIdx.x == 0 && j + 2 < n_jobs) issue_next(j + 2);
      ++sk;
      continue;
    }
    const int buf = k & 1;  // staging buffers alternate with the CTA's own tiles
    const int64_t row0 = (int64_t)tr * 128, col0 = (int64_t)tc * 128;
    const bool full_tile = (row0 + 128 <= a.rows) && (col0 + 128 <= a.cols);
    uint8_t* const col_codes = smem + QuantSmem::kColCodes + buf * 8192;
    uint8_t* const sf_row = smem + QuantSmem::kSfRow + buf * 1024;
    uint8_t* const sf_col = smem + QuantSmem::kSfCol + buf * 1024;

    auto phases_1_2 = [&](auto full_c) {
      constexpr bool FULL = decltype(full_c)::value;
      // ---------------------------------------------------------------- phase 1 ----
      const int rows_left = FULL ? 128 : (int)(a.rows - row0) - rl;         // chunk i exists iff 4 i < rows_left
      const bool col_ok = FULL || (col0 + cb * 16 < a.cols);
      uint32_t raw[4][8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 h0 = *reinterpret_cast<const uint4*>(tile_buf + tile_ld + i * 1024);
        const uint4 h1 = *reinterpret_cast<const uint4*>(tile_buf + tile_ld + i * 1024 + 16);
        raw[i][0] = h0.x; raw[i][1] = h0.y; raw[i][2] = h0.z; raw[i][3] = h0.w;
        raw[i][4] = h1.x; raw[i][5] = h1.y; raw[i][6] = h1.z; raw[i][7] = h1.w;
      }

      uint32_t blk_byte = 0;
      float blk_enc = 0.f;
      if (BLOCK2D) {  // amax of the lane's chunk column over the warp's 16 rows: one scale per 16 x 16 block
        float blk_amax = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t acc = 0;
#pragma unroll
          for (int k = 0; k < 8; ++k) acc = absmax_bf16x2(acc, raw[i][k]);
          blk_amax = fmaxf(blk_amax, fmaxf(bf16_lo(acc), bf16_hi(acc)));
        }
        blk_amax = fmaxf(blk_amax, __shfl_xor_sync(0xffffffffu, blk_amax, 8));
        blk_amax = fmaxf(blk_amax, __shfl_xor_sync(0xffffffffu, blk_amax, 16));
        block_scales(blk_amax, r_senc, r_sdec, blk_byte, blk_enc);
        if (lane < 8) {
          reinterpret_cast<float*>(smem + QuantSmem::kBlkEnc)[warp * 8 + cb] = blk_enc;
          smem[QuantSmem::kBlkByte + warp * 8 + cb] = (uint8_t)blk_byte;
        }
      }

      uint64_t g = 0;  // Philox counter of chunk 0: the chunk's index in the source, 16-blocks numbered row by row
      if (SR) g = (uint64_t)(row0 + rl) * (uint64_t)n_cb + (uint64_t)((col0 >> 4) + cb);
      uint8_t* r_out = HAS_ROW ? a.r_codes + (row0 + rl) * r_pitch + ((col0 + cb * 16) >> 1) : nullptr;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t rnd[4] = {0u, 0u, 0u, 0u};
        if (SR) {
          const uint64_t gi = g + (uint64_t)(4 * i) * (uint64_t)n_cb;
          uint4 q = philox4x32_10((uint32_t)gi, (uint32_t)(gi >> 32), a.off_lo, a.off_hi, a.rk);
          rnd[0] = q.x; rnd[1] = q.y; rnd[2] = q.z; rnd[3] = q.w;
          if (HAS_COL && !kNibbleTranspose) {
            uint4 qc = q;
            if (a.off_hi_col != a.off_hi)
              qc = philox4x32_10((uint32_t)gi, (uint32_t)(gi >> 32), a.off_lo, a.off_hi_col, a.rk);
            // staged complemented: the conversion wants 255 - draw
            *reinterpret_cast<uint4*>(smem + rand_st + i * 512) = make_uint4(~qc.x, ~qc.y, ~qc.z, ~qc.w);
          }
        }
        if (HAS_ROW) {
          float f[16];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            uint32_t word = raw[i][k];
            if (RHT_ROW) word ^= sign_pair(a.sign_mask, 2 * k, 2 * k + 1);
            f[2 * k] = bf16_lo(word);
            f[2 * k + 1] = bf16_hi(word);
          }
          if (RHT_ROW) fwht16(f);  // values are 4 * y from here on
          uint32_t byte;
          float enc;
          if (BLOCK2D) {
            byte = blk_byte;
            enc = blk_enc;
          } else {
            const float m = amax16_3(f);
            byte = block_scale_byte(RHT_ROW ? 0.25f * m : m, r_senc);
            enc = enc_row[byte];
          }
          const uint2 codes = convert16<SR>(f, enc, Nu14FromWords{rnd});
          if (FULL || (col_ok && 4 * i < rows_left)) *reinterpret_cast<uint2*>(r_out + (int64_t)(4 * i) * r_pitch) = codes;
          if (kNibbleTranspose)  // row r, bytes [8 cb, 8 cb + 8): byte k = columns (2k, 2k + 1) of the chunk
            *reinterpret_cast<uint2*>(smem + QuantSmem::kRand + (rl + 4 * i) * 64 + cb * 8) =
                (FULL || (col_ok && 4 * i < rows_left)) ? codes : make_uint2(0u, 0u);
          sf_row[sf_row_pos + i * sf_row_step] = (uint8_t)byte;
        }
      }
      // Phase 2 of a warp reads only what the same warp staged in phase 1 (its own 16 rows of the tile, their random
      // bytes, its 16x16 scales), so the warps need not wait for each other here
      __syncwarp();

      // ---------------------------------------------------------------- phase 2 ----
      if (HAS_COL) {
        const int q = warp;  // 16-row group inside the tile
#pragma unroll
        for (int it = 0; it < 2; ++it) {
          const int cp = lane + 32 * it;  // column pair: tile columns 2cp, 2cp+1
          if (kNibbleTranspose) {
            // byte [row][cp] of the staged row-wise codes = (column 2cp in the low nibble, 2cp + 1 in the high one)
            uint32_t w[4];
#pragma unroll
            for (int m = 0; m < 4; ++m) {
              uint32_t b[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) b[j] = smem[QuantSmem::kRand + (q * 16 + 4 * m + j) * 64 + cp];
              w[m] = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
            }
            auto gather = [](uint32_t x) {  // four nibbles, one per byte -> 16 bits
              const uint32_t t = (x | (x >> 4)) & 0x00FF00FFu;
              return (t | (t >> 8)) & 0xFFFFu;
            };
            uint32_t lo[4], hi[4];
#pragma unroll
            for (int m = 0; m < 4; ++m) {
              lo[m] = gather(w[m] & 0x0F0F0F0Fu);
              hi[m] = gather((w[m] >> 4) & 0x0F0F0F0Fu);
            }
            const uint2 codes0 = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
            const uint2 codes1 = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
            const uint32_t byte = smem[QuantSmem::kBlkByte + q * 8 + (cp >> 3)];
            *reinterpret_cast<uint4*>(col_codes + col_codes_st + it * 4096) =
                make_uint4(codes0.x, codes0.y, codes1.x, codes1.y);
            sf_col[sf_col_pos + it * sf_col_it] = (uint8_t)byte;
            sf_col[sf_col_pos + it * sf_col_it + sf_col_odd] = (uint8_t)byte;
            continue;
          }
          float f0[16], f1[16];
          const uint8_t* tp = tile_buf + q * 16 * 256 + cp * 4;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            uint32_t word = *reinterpret_cast<const uint32_t*>(tp + j * 256);
            if (RHT_COL) word ^= (sign2 << (15 - j)) & 0x80008000u;
            f0[j] = bf16_lo(word);
            f1[j] = bf16_hi(word);
          }
          if (RHT_COL) {  // values are 4 * y from here on
            float2 v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = make_float2(f0[j], f1[j]);
            fwht16_pairs(v);  // both columns in one pass of packed adds
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              f0[j] = v[j].x;
              f1[j] = v[j].y;
            }
          }
          uint32_t byte0, byte1;
          float enc0, enc1;
          if (BLOCK2D) {
            enc0 = enc1 = reinterpret_cast<const float*>(smem + QuantSmem::kBlkEnc)[q * 8 + (cp >> 3)];
            byte0 = byte1 = smem[QuantSmem::kBlkByte + q * 8 + (cp >> 3)];
          } else {
            const float m0 = amax16_3(f0), m1 = amax16_3(f1);
            byte0 = block_scale_byte(RHT_COL ? 0.25f * m0 : m0, c_senc);
            byte1 = block_scale_byte(RHT_COL ? 0.25f * m1 : m1, c_senc);
            enc0 = enc_col[byte0];
            enc1 = enc_col[byte1];
          }
          uint2 codes0, codes1;
          if (SR) {
            // low / high byte of ntwo[j] = 255 - draw of source element (row 16q + j, column 2cp / 2cp + 1)
            uint32_t ntwo[16];
            const uint8_t* rp = smem + QuantSmem::kRand + q * 16 * 128 + cp * 2;
#pragma unroll
            for (int j = 0; j < 16; ++j) ntwo[j] = *reinterpret_cast<const uint16_t*>(rp + j * 128);
            convert16x2_sr(f0, f1, enc0, enc1, ntwo, codes0, codes1);
          } else {
            const uint32_t none[4] = {0u, 0u, 0u, 0u};
            codes0 = convert16<false>(f0, enc0, Nu14FromWords{none});
            codes1 = convert16<false>(f1, enc1, Nu14FromWords{none});
          }
          // staging: both columns' eight bytes in one 16-byte unit (conflict-free: eight consecutive column pairs hit
          // eight different units of a 128-byte line)
          *reinterpret_cast<uint4*>(col_codes + col_codes_st + it * 4096) =
              make_uint4(codes0.x, codes0.y, codes1.x, codes1.y);
          sf_col[sf_col_pos + it * sf_col_it] = (uint8_t)byte0;
          sf_col[sf_col_pos + it * sf_col_it + sf_col_odd] = (uint8_t)byte1;
        }
      }
    };
    if (full_tile)
      phases_1_2(std::true_type{});
    else
      phases_1_2(std::false_type{});
    __syncthreads();
    if (*abort_flag) break;  // a wait expired (the word is read after the barrier: the same for every thread)
    if (threadIdx.x == 0 && j + 2 < n_jobs) issue_next(j + 2);  // every warp is done with this buffer

    // ------------------------------------------------------------------ phase 3 ----
    if (HAS_COL) {
      // a thread takes column pair cp and the 16-row groups (2m, 2m + 1): 16 bytes = 32 rows of each of its two columns
      const int64_t pitch = a.rows >> 1;  // bytes per row of the transposed copy
      const bool vec16 = (a.rows & 31) == 0;
      const int cp = threadIdx.x >> 2, m = threadIdx.x & 3;
      const uint8_t* unit = col_codes + cp * 128 + ((((2 * m) ^ cp) & 7) << 4);
      const uint4 g0 = *reinterpret_cast<const uint4*>(unit);  // group 2m: (first column, second column) x 8 bytes
      const uint4 g1 = *reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>((uintptr_t)unit ^ 16));
      const int64_t rr = row0 + 32 * m;
#pragma unroll
      for (int odd = 0; odd < 2; ++odd) {
        const int c = 2 * cp + odd;
        if (col0 + c >= a.cols) continue;
        const uint4 v = odd ? make_uint4(g0.z, g0.w, g1.z, g1.w) : make_uint4(g0.x, g0.y, g1.x, g1.y);
        uint8_t* dst = a.c_codes + (col0 + c) * pitch + (row0 >> 1) + m * 16;
        if (rr + 16 < a.rows && vec16) {
          *reinterpret_cast<uint4*>(dst) = v;
        } else {
          if (rr < a.rows) *reinterpret_cast<uint2*>(dst) = make_uint2(v.x, v.y);
          if (rr + 16 < a.rows) *reinterpret_cast<uint2*>(dst + 8) = make_uint2(v.z, v.w);
        }
      }
    }
    // scale bytes
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      if (which == 0 && !HAS_ROW) continue;
      if (which == 1 && !HAS_COL) continue;
      const uint8_t* src = which == 0 ? sf_row : sf_col;
      uint8_t* dst = which == 0 ? a.r_scales : a.c_scales;
      const int swz = which == 0 ? a.r_swz : a.c_swz;
      // the copy's row / block coordinates of this tile
      const int64_t R0 = which == 0 ? row0 : col0, K0 = which == 0 ? (col0 >> 4) : (row0 >> 4);
      const int64_t Rn = which == 0 ? a.rows : a.cols, n_kb = which == 0 ? n_cb : n_rb;
      if (swz) {
        if (threadIdx.x < 64) {
          const int atom = threadIdx.x >> 5;
          if (K0 + atom * 4 < n_kb) {
            const int64_t off = ((R0 >> 7) * (n_kb >> 2) + (K0 >> 2) + atom) * 512 + (threadIdx.x & 31) * 16;
            *reinterpret_cast<uint4*>(dst + off) = *reinterpret_cast<const uint4*>(src + threadIdx.x * 16);
          }
        }
      } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int idx = threadIdx.x * 4 + k;
          const int r = idx >> 3, kb = idx & 7;
          if (R0 + r < Rn && K0 + kb < n_kb) dst[(R0 + r) * n_kb + K0 + kb] = src[idx];
        }
      }
    }
    ++k;  // on to the CTA's next own tile
    tr -= step_r;
    tc -= step_c;
    if (tc < 0) {
      tc += a.tiles_c;
      --tr;
    }
  }
  if (j < n_jobs) {
    // left early: jobs j and j + 1 may still be in flight; give each one more bounded wait so that no copy lands
    // in shared memory after the CTA has gone
    if (threadIdx.x == 0)
      for (int i = j; i < j + 2 && i < n_jobs; ++i) {
        const unsigned long long t0 = globaltimer_ns();
        while (!mbar_try(bar0 + 8 * (i & 1), (uint32_t)(i >> 1) & 1u) && globaltimer_ns() - t0 < kWaitLimitNs) {
        }
      }
    return;  // no maximum is published by a CTA that gave up
  }
  if (SIDE) {
    float* red = reinterpret_cast<float*>(smem + QuantSmem::kBlkEnc);  // free in 1 x 16 mode
    const float m = warp_max(fmaxf(bf16_lo(side_acc), bf16_hi(side_acc)));
    __syncthreads();
    if (lane == 0) red[warp] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) t = fmaxf(t, red[w]);
      const uint32_t bits = __float_as_uint(t);  // non-negative floats order like their bit patterns
      if (a.side_out0) atomicMax(reinterpret_cast<unsigned int*>(a.side_out0), bits);
      if (a.side_out1) atomicMax(reinterpret_cast<unsigned int*>(a.side_out1), bits);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Test aids
// ---------------------------------------------------------------------------------------------
__global__ void dequantize_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                                  const float* __restrict__ global, int64_t rows, int64_t cols, int swz,
                                  int mx, int per_row, float* __restrict__ out) {
  const int64_t n = rows * cols;
  const float s_dec_t = global[1];
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / cols, c = i % cols;
    const uint32_t byte = codes[r * (cols >> 1) + (c >> 1)];
    const uint32_t code = (c & 1) ? (byte >> 4) : (byte & 15u);
    const float mags[8] = {0.f, 0.5f, 1.f, 1.5f, 2.f, 3.f, 4.f, 6.f};
    float m = mags[code & 7u];
    if (code & 8u) m = -m;
    const int sh = mx ? 5 : 4;  // block length 32 (UE8M0 scale) or 16 (E4M3 scale)
    const int64_t so = swz ? sf_swizzled_offset(r, c >> sh, cols >> sh) : (r * (cols >> sh) + (c >> sh));
    uint16_t sb = scales[so];
    float sf;
    if (mx) {
      sf = sb == 0 ? __uint_as_float(0x00400000u) : __uint_as_float((uint32_t)sb << 23);  // 2^(byte - 127)
    } else {
      uint32_t h2;
      asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(sb));
      sf = __half2float(__ushort_as_half((unsigned short)(h2 & 0xffffu)));
    }
    out[i] = __fmul_rn(__fmul_rn(m, sf), per_row ? global[2 * r + 1] : s_dec_t);
  }
}

__global__ void rht16_kernel(const uint16_t* __restrict__ x, int64_t rows, int64_t cols, int64_t ld,
                             int colwise, uint32_t mask, float* __restrict__ out) {
  // one thread per chunk of the requested copy
  const int64_t R = colwise ? cols : rows, C = colwise ? rows : cols;
  const int64_t n_chunks = R * (C >> 4);
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n_chunks;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / (C >> 4), kb = i % (C >> 4);
    float f[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int64_t sr = colwise ? (kb * 16 + j) : r, sc = colwise ? r : (kb * 16 + j);
      uint32_t bits = (uint32_t)x[sr * ld + sc] << 16;
      if ((mask >> j) & 1u) bits ^= 0x80000000u;
      f[j] = __uint_as_float(bits);
    }
    fwht16(f);
#pragma unroll
    for (int j = 0; j < 16; ++j) out[r * C + kb * 16 + j] = f[j] * 0.25f;
  }
}

// codes[i] = stochastic rounding of v[i] with the draw u[i], through the very conversion the quantizer uses
__global__ void e2m1_sr_kernel(const float* __restrict__ v, const uint8_t* __restrict__ u, int64_t n,
                               uint8_t* __restrict__ codes) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    // the element sits in the low slot on even i and in the high slot on odd i, the other slot holds a decoy
    const float w = __fmul_rz(v[i], kSrTowardsZero), decoy = __fmul_rz(-v[i] * 0.75f, kSrTowardsZero);
    const uint32_t nu = 255u - u[i], nd = (uint32_t)(i * 37) & 255u;
    const uint32_t d = (i & 1) ? e2m1x2_sr(decoy, w, (nu << 24) | (nd << 16) | 0x8080u)
                               : e2m1x2_sr(w, decoy, (nd << 24) | (nu << 16) | 0x8080u);
    codes[i] = (uint8_t)((i & 1) ? (d >> 8) & 15u : d & 15u);
  }
}

// ---------------------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------------------
template <bool PLAIN, bool RR, bool RC>
static cudaError_t launch_amax_t(const QuantArgs& a, float* plain0, float* plain1, float* rot_row,
                                 float* rot_col, cudaStream_t s) {
  const int tiles_c = (int)((a.cols + 255) / 256);
  const int64_t tiles = ((a.rows + 127) / 128) * tiles_c;
  amax_kernel<PLAIN, RR, RC><<<(unsigned)tiles, 256, 0, s>>>(a.x, a.rows, a.cols, a.ld, a.sign_mask, tiles_c,
                                                            plain0, plain1, rot_row, rot_col);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_amax(const QuantArgs& a, bool has_row, bool has_col, bool rht_row, bool rht_col,
                        cudaStream_t s) {
  cudaError_t e;
  if (has_row && (e = cudaMemsetAsync(a.r_global, 0, sizeof(float), s)) != cudaSuccess) return e;
  if (has_col && (e = cudaMemsetAsync(a.c_global, 0, sizeof(float), s)) != cudaSuccess) return e;
  const bool rr = has_row && rht_row, rc = has_col && rht_col;
  float* plain0 = (has_row && !rht_row) ? a.r_global : nullptr;
  float* plain1 = (has_col && !rht_col) ? a.c_global : nullptr;
  const bool plain = plain0 || plain1;
  float* rot_row = rr ? a.r_global : nullptr;
  float* rot_col = rc ? a.c_global : nullptr;
  if (rc && !rr) {  // tensor-core transform for the transposed copy
    const int tiles_c = (int)((a.cols + 255) / 256);
    const unsigned tiles = (unsigned)(((a.rows + 127) / 128) * tiles_c);
    if (plain)
      amax_rot_col_kernel<true><<<tiles, 256, 0, s>>>(a.x, a.rows, a.cols, a.ld, a.sign_mask, tiles_c, plain0, plain1,
                                                      rot_col, 16, 0.25f);
    else
      amax_rot_col_kernel<false><<<tiles, 256, 0, s>>>(a.x, a.rows, a.cols, a.ld, a.sign_mask, tiles_c, plain0,
                                                       plain1, rot_col, 16, 0.25f);
    count_launch();
    return cudaGetLastError();
  }
#define NVFP4_AMAX(P, R, C) \
  if (plain == P && rr == R && rc == C) return launch_amax_t<P, R, C>(a, plain0, plain1, rot_row, rot_col, s);
  NVFP4_AMAX(true, false, false)
  NVFP4_AMAX(true, false, true)
  NVFP4_AMAX(true, true, false)
  NVFP4_AMAX(false, true, true)
  NVFP4_AMAX(false, false, true)
  NVFP4_AMAX(false, true, false)
#undef NVFP4_AMAX
  return cudaErrorInvalidValue;
}

// Pass 1 of the transposed copy with a d x d transform (d = 2, 4, 8), and the plain amax of the row-wise copy
// beside it: the tensor-core kernel above with a block-diagonal matrix.  sign_mask: the d sign bits repeated to 16.
cudaError_t launch_amax_rot_col_small(const QuantArgs& a, bool has_row, uint32_t mask16, int d, float norm,
                                      cudaStream_t s) {
  cudaError_t e;
  if (has_row && (e = cudaMemsetAsync(a.r_global, 0, sizeof(float), s)) != cudaSuccess) return e;
  if ((e = cudaMemsetAsync(a.c_global, 0, sizeof(float), s)) != cudaSuccess) return e;
  const int tiles_c = (int)((a.cols + 255) / 256);
  const unsigned tiles = (unsigned)(((a.rows + 127) / 128) * tiles_c);
  if (has_row)
    amax_rot_col_kernel<true><<<tiles, 256, 0, s>>>(a.x, a.rows, a.cols, a.ld, mask16, tiles_c, a.r_global, nullptr,
                                                    a.c_global, d, norm);
  else
    amax_rot_col_kernel<false><<<tiles, 256, 0, s>>>(a.x, a.rows, a.cols, a.ld, mask16, tiles_c, nullptr, nullptr,
                                                     a.c_global, d, norm);
  count_launch();
  return cudaGetLastError();
}

template <bool HR, bool HC, bool B2, bool RR, bool RC, bool SR, bool SIDE = false>
static cudaError_t launch_quant_t(const QuantArgs& a_in, cudaStream_t s, const SideAmax* side = nullptr) {
  auto kern = quantize_kernel<HR, HC, B2, RR, RC, SR, SIDE>;
  QuantArgs a = a_in;
  constexpr bool kRowCodes = B2 && HR && HC;
  constexpr int smem = QuantSmem::bytes(SR && HC && !kRowCodes, kRowCodes);
  // the source as a 2-D tensor map: boxes of 128 x 128 bf16 (256-byte rows, no swizzle), zero fill outside
  CUtensorMap map;
  if (!make_map_2d(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.x, (uint64_t)a.cols, (uint64_t)a.rows,
                   (uint64_t)a.ld * 2, 128, 128, false))
    return cudaErrorInvalidValue;
  CUtensorMap side_map = map;
  int64_t side_tiles = 0;
  if (SIDE) {
    if (!side || !make_map_2d(&side_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, side->x, (uint64_t)side->cols,
                              (uint64_t)side->rows, (uint64_t)side->ld * 2, 128, 128, false))
      return cudaErrorInvalidValue;
    a.side_tiles_r = (int)((side->rows + 127) / 128);
    a.side_tiles_c = (int)((side->cols + 127) / 128);
    a.side_out0 = side->out0;
    a.side_out1 = side->out1;
    side_tiles = (int64_t)a.side_tiles_r * a.side_tiles_c;
    if (side_tiles > 0x7fffffff) return cudaErrorInvalidValue;
  }
  // per call site (template instantiation) and device: the dynamic shared-memory limit, and how many CTAs the device
  // keeps resident (the persistent grid)
  static std::atomic<uint64_t> configured{0};
  static std::atomic<int> resident[64] = {};
  int dev;
  if (device_needs_config(configured, &dev)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int sms = 0, per_sm = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev < 0 ? 0 : dev)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 256, smem)) != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) resident[dev].store(sms * (per_sm > 0 ? per_sm : 1), std::memory_order_relaxed);
    device_configured(configured, dev);
  }
  const int slots = (dev >= 0 && dev < 64) ? resident[dev].load(std::memory_order_relaxed) : 0;
  const int64_t own = (int64_t)a.tiles_r * a.tiles_c, tiles = own > side_tiles ? own : side_tiles;
  const int64_t grid = (slots > 0 && tiles > slots) ? slots : tiles;
  const cudaError_t e = launch_kernel(kern, dim3((unsigned)grid), dim3(256), smem, s, a.chained != 0, map, side_map, a);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t zero_side_amax(const SideAmax& side, cudaStream_t s) {
  cudaError_t e;
  if (side.out0 && (e = cudaMemsetAsync(side.out0, 0, sizeof(float), s)) != cudaSuccess) return e;
  if (side.out1 && (e = cudaMemsetAsync(side.out1, 0, sizeof(float), s)) != cudaSuccess) return e;
  return cudaSuccess;
}

cudaError_t launch_quantize_with_amax_of(const QuantArgs& a, bool has_col, const SideAmax& side, cudaStream_t s) {
  return has_col ? launch_quant_t<true, true, false, false, true, false, true>(a, s, &side)
                 : launch_quant_t<true, false, false, false, false, false, true>(a, s, &side);
}

cudaError_t launch_quantize(const QuantArgs& a, bool has_row, bool has_col, bool block2d, bool rht_row,
                            bool rht_col, bool sr, cudaStream_t s) {
  rht_row = rht_row && has_row;
  rht_col = rht_col && has_col;
#define NVFP4_Q(HR, HC, B2, RR, RC, SRV)                                                           \
  if (has_row == HR && has_col == HC && block2d == B2 && rht_row == RR && rht_col == RC && sr == SRV) \
    return launch_quant_t<HR, HC, B2, RR, RC, SRV>(a, s);
#define NVFP4_Q_COPIES(B2, RR, RC, SRV)      \
  NVFP4_Q(true, false, B2, RR, false, SRV)   \
  NVFP4_Q(false, true, B2, false, RC, SRV)   \
  NVFP4_Q(true, true, B2, RR, RC, SRV)
  NVFP4_Q_COPIES(true, false, false, false)
  NVFP4_Q_COPIES(true, false, false, true)
  NVFP4_Q_COPIES(false, false, false, false)
  NVFP4_Q_COPIES(false, false, false, true)
  NVFP4_Q_COPIES(false, false, true, false)
  NVFP4_Q_COPIES(false, false, true, true)
  NVFP4_Q_COPIES(false, true, false, false)
  NVFP4_Q_COPIES(false, true, false, true)
  NVFP4_Q_COPIES(false, true, true, false)
  NVFP4_Q_COPIES(false, true, true, true)
#undef NVFP4_Q_COPIES
#undef NVFP4_Q
  return cudaErrorInvalidValue;
}

cudaError_t launch_dequantize(const nvfp4_tensor& t, float* out, cudaStream_t s) {
  dequantize_kernel<<<1184, 256, 0, s>>>(t.codes, t.scales, t.global, t.rows, t.cols,
                                         t.sf_layout == NVFP4_SF_SWIZZLED, t.format == NVFP4_FORMAT_MXFP4,
                                         t.format == NVFP4_FORMAT_NVFP4_ROWSCALE, out);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_rht16(const void* x, int64_t rows, int64_t cols, int64_t ld, int colwise, uint32_t mask,
                         float* out, cudaStream_t s) {
  rht16_kernel<<<1184, 256, 0, s>>>(static_cast<const uint16_t*>(x), rows, cols, ld, colwise, mask, out);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_e2m1_sr(const float* v, const uint8_t* u, int64_t n, uint8_t* codes, cudaStream_t s) {
  e2m1_sr_kernel<<<1184, 256, 0, s>>>(v, u, n, codes);
  count_launch();
  return cudaGetLastError();
}

}  // namespace nvfp4
