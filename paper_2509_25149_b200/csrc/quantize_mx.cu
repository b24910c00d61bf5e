// MXFP4 quantizer for sm_100a: the format the paper compares NVFP4 against (Section 2, Section 5, Appendix B.4).
// E2M1 elements, one UE8M0 (power-of-two) scale per 32 elements, the decode scale amax_b / 6 rounded UP to a power
// of two so that no value saturates, no tensor-level scale: ONE pass over the tensor produces both copies.
// The recipe options are those of Section 4 at this format's block size: 1x32 blocks for activations and gradients,
// 32x32 blocks for weights, a 32-point random Hadamard transform on the transposed (weight-gradient) copy, stochastic
// rounding with the same Philox draws as the NVFP4 kernel.
#include "async_ptx.cuh"
#include "quantize.h"
#include "quantize_common.cuh"

namespace nvfp4 {

// UE8M0 byte and the exact encode scale 2^(127 - byte) of a block with the given amax (>= 0).
// amax = m * 2^E with m in [1, 2): the smallest e with 6 * 2^e >= amax is E - 2 if m <= 1.5, else E - 1;
// byte = e + 127 = (exponent field) - 2 (+ 1), clamped at 0 (zero and tiny blocks).
__device__ __forceinline__ void mx_scales(float amax, uint32_t& byte, float& enc) {
  const uint32_t bits = __float_as_uint(amax);
  int b = (int)(bits >> 23) - 2 + ((bits & 0x7fffffu) > 0x400000u ? 1 : 0);
  b = b < 0 ? 0 : b;
  byte = (uint32_t)b;
  enc = __uint_as_float((uint32_t)(254 - b) << 23);  // b <= 253 for finite amax
}

// 32-point butterfly on pairs (.x / .y = two adjacent columns); the caller applies 1 / sqrt(32)
__device__ __forceinline__ void fwht32_pairs(float2 v[32]) {
#pragma unroll
  for (int h = 1; h < 32; h <<= 1) {
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      if ((i & h) == 0) {
        const float2 p = v[i], q = v[i | h];
        v[i] = add2(p, q);
        v[i | h] = sub2(p, q);
      }
    }
  }
}

struct MxSmem {
  static constexpr int kTile = 0;                   // 128 rows x 256 B of bf16
  static constexpr int kColCodes = 32768;           // 128 columns x 64 B
  static constexpr int kSfRow = kColCodes + 8192;   // one 512-byte atom: 128 rows x 4 blocks of 32
  static constexpr int kSfCol = kSfRow + 512;
  static constexpr int kBlk = kSfCol + 512;         // 32x32 mode: amax of (warp's 16 rows) x (4 column blocks)
  static constexpr int kRand = kBlk + 128;          // 128 rows x 128 B (stochastic rounding only), chunk cb of row r
                                                    // at slot cb ^ ((r >> 2) & 7)
  static constexpr int kBytesNoRand = kRand;
  static constexpr int kBytesRand = kRand + 16384;
};

constexpr float kInvSqrt32 = 0.176776695296636893f;  // fl(1 / sqrt(32))

// One CTA (256 threads) per 128 x 128 tile of the source.
//   phase 1  each thread owns four 1x16 chunks (32-byte loads); a 1x32 block is the two chunks of an even / odd lane
//            pair; the row-wise copy is produced from registers, the raw tile (and the random bytes) are staged;
//   phase 2  each thread owns 32 rows x 2 columns of the staged tile and produces the transposed copy;
//   phase 3  staged codes and scale bytes leave with 16-byte stores.
template <bool HAS_ROW, bool HAS_COL, bool BLOCK2D, bool RHT_COL, bool SR>
__global__ void __launch_bounds__(256, RHT_COL ? 2 : 3) quantize_mx_kernel(const QuantArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = (int)blockIdx.x;
  griddep_launch_dependents();  // the GEMM of a composed call may set itself up while the last CTAs run
  const int64_t row0 = (int64_t)(tile / a.tiles_c) * 128;
  const int64_t col0 = (int64_t)(tile % a.tiles_c) * 128;
  const int64_t n_cb = a.cols >> 4;  // 16-chunks per source row (index of the random draws)

  // ------------------------------------------------------------------ phase 1 ----
  const int cb = lane & 7;  // 16-chunk column inside the tile
  uint32_t raw[4][8];
  bool ok[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = warp * 16 + i * 4 + (lane >> 3);
    ok[i] = (row0 + r < a.rows) && (col0 + cb * 16 < a.cols);
    if (ok[i]) {
      ldg256_stream(a.x + (row0 + r) * a.ld + col0 + cb * 16, raw[i]);
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) raw[i][k] = 0u;
    }
  }
  if (HAS_COL) {
    const int first = (lane >> 2) & 1;  // halves in lane-dependent order: a quarter warp covers all banks
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = warp * 16 + i * 4 + (lane >> 3);
      uint8_t* dst = smem + MxSmem::kTile + r * 256 + cb * 32;
      const uint4 h0 = make_uint4(raw[i][0], raw[i][1], raw[i][2], raw[i][3]);
      const uint4 h1 = make_uint4(raw[i][4], raw[i][5], raw[i][6], raw[i][7]);
      if (first) {
        *reinterpret_cast<uint4*>(dst + 16) = h1;
        *reinterpret_cast<uint4*>(dst) = h0;
      } else {
        *reinterpret_cast<uint4*>(dst) = h0;
        *reinterpret_cast<uint4*>(dst + 16) = h1;
      }
    }
  }

  // amax of the 1x32 block each chunk belongs to (the chunk of the neighbouring lane completes it)
  float am[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint32_t acc = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) acc = absmax_bf16x2(acc, raw[i][k]);
    const float own = fmaxf(bf16_lo(acc), bf16_hi(acc));
    am[i] = fmaxf(own, __shfl_xor_sync(0xffffffffu, own, 1));
  }
  float* blk = reinterpret_cast<float*>(smem + MxSmem::kBlk);
  if (BLOCK2D) {
    // 32x32 blocks: the warp's 16 rows first, then the neighbouring warp's 16 rows through shared memory
    float m = fmaxf(fmaxf(am[0], am[1]), fmaxf(am[2], am[3]));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 8));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 16));
    if (lane < 8 && !(lane & 1)) blk[warp * 4 + (cb >> 1)] = m;
    __syncthreads();
    m = fmaxf(blk[warp * 4 + (cb >> 1)], blk[(warp ^ 1) * 4 + (cb >> 1)]);
#pragma unroll
    for (int i = 0; i < 4; ++i) am[i] = m;
  }

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = warp * 16 + i * 4 + (lane >> 3);
    uint32_t rnd[4] = {0u, 0u, 0u, 0u};
    if (SR) {
      const uint64_t g = (uint64_t)(row0 + r) * (uint64_t)n_cb + (uint64_t)((col0 >> 4) + cb);
      uint4 q = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), a.off_lo, a.off_hi, a.rk);
      rnd[0] = q.x; rnd[1] = q.y; rnd[2] = q.z; rnd[3] = q.w;
      if (HAS_COL) {
        uint4 qc = q;
        if (a.off_hi_col != a.off_hi)
          qc = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), a.off_lo, a.off_hi_col, a.rk);
        *reinterpret_cast<uint4*>(smem + MxSmem::kRand + r * 128 + ((cb ^ ((r >> 2) & 7)) << 4)) = qc;
      }
    }
    if (HAS_ROW) {
      float f[16];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        f[2 * k] = bf16_lo(raw[i][k]);
        f[2 * k + 1] = bf16_hi(raw[i][k]);
      }
      uint32_t byte;
      float enc;
      mx_scales(am[i], byte, enc);
      const uint2 codes = convert16<SR>(f, enc, Nu14FromWords{rnd});
      if (ok[i])
        *reinterpret_cast<uint2*>(a.r_codes + (row0 + r) * (a.cols >> 1) + ((col0 + cb * 16) >> 1)) = codes;
      if (!(cb & 1)) {
        const int pos = a.r_swz ? ((r & 31) * 16 + (r >> 5) * 4 + (cb >> 1)) : (r * 4 + (cb >> 1));
        smem[MxSmem::kSfRow + pos] = (uint8_t)byte;
      }
    }
  }
  __syncthreads();

  // ------------------------------------------------------------------ phase 2 ----
  if (HAS_COL) {
    const int q32 = threadIdx.x >> 6;  // 32-row group inside the tile
    const int cp = threadIdx.x & 63;   // column pair: tile columns 2cp, 2cp + 1
    float2 v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      uint32_t word = *reinterpret_cast<const uint32_t*>(smem + MxSmem::kTile + (q32 * 32 + j) * 256 + cp * 4);
      if (RHT_COL) word ^= sign_pair(a.sign_mask, j, j);
      v[j] = make_float2(bf16_lo(word), bf16_hi(word));
    }
    if (RHT_COL) {
      fwht32_pairs(v);
      // y = fl(sum * fl(1 / sqrt(32))): Section 5, transform size 32
      const float2 c2 = make_float2(kInvSqrt32, kInvSqrt32);
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = mul2(v[j], c2);
    }
    float a0 = 0.f, a1 = 0.f;
    if (BLOCK2D) {
      a0 = a1 = fmaxf(blk[(2 * q32) * 4 + (cp >> 4)], blk[(2 * q32 + 1) * 4 + (cp >> 4)]);
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        a0 = fmaxf(a0, fabsf(v[j].x));
        a1 = fmaxf(a1, fabsf(v[j].y));
      }
    }
    uint32_t byte0, byte1;
    float enc0, enc1;
    mx_scales(a0, byte0, enc0);
    mx_scales(a1, byte1, enc1);
    uint4 out0, out1;  // 32 nibbles of column 2cp / 2cp + 1
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float f0[16], f1[16];
      uint32_t two[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        f0[j] = v[16 * h + j].x;
        f1[j] = v[16 * h + j].y;
        two[j] = 0u;
        if (SR) {
          // low / high byte = draw of source element (row 32 q32 + 16 h + j, column 2cp / 2cp + 1)
          const int r = q32 * 32 + 16 * h + j;
          two[j] = *reinterpret_cast<const uint16_t*>(smem + MxSmem::kRand + r * 128 +
                                                      (((cp >> 3) ^ ((r >> 2) & 7)) << 4) + (cp & 7) * 2);
        }
      }
      const uint2 c0 = convert16<SR>(f0, enc0, Nu14FromPairs<0>{two});
      const uint2 c1 = convert16<SR>(f1, enc1, Nu14FromPairs<1>{two});
      if (h == 0) {
        out0.x = c0.x; out0.y = c0.y; out1.x = c1.x; out1.y = c1.y;
      } else {
        out0.z = c0.x; out0.w = c0.y; out1.z = c1.x; out1.w = c1.y;
      }
    }
    // staging as in the NVFP4 kernel: column c holds eight 8-byte units (16 rows each), unit u stored at
    // (u ^ (c >> 1)) & 7.  The two units of this thread (2 q32, 2 q32 + 1) stay adjacent, swapped when the XOR is
    // odd; the column written first alternates with the XOR so that a quarter warp covers all banks.
    const int x = cp & 7;
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      const int odd = s ^ (x & 1);
      const int c = 2 * cp + odd;
      uint4 val = odd ? out1 : out0;
      if (x & 1) val = make_uint4(val.z, val.w, val.x, val.y);
      *reinterpret_cast<uint4*>(smem + MxSmem::kColCodes + c * 64 + ((((2 * q32) ^ x) & 6) << 3)) = val;
      const uint32_t byte = odd ? byte1 : byte0;
      const int pos = a.c_swz ? ((c & 31) * 16 + (c >> 5) * 4 + q32) : (c * 4 + q32);
      smem[MxSmem::kSfCol + pos] = (uint8_t)byte;
    }
  }
  __syncthreads();

  // ------------------------------------------------------------------ phase 3 ----
  if (HAS_COL) {
    const int64_t pitch = a.rows >> 1;  // bytes per row of the transposed copy
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int unit = threadIdx.x + 256 * k;
      const int c = unit >> 2, m = unit & 3;  // column, 32-row group
      if (col0 + c >= a.cols) continue;
      const int x = (c >> 1) & 7;
      uint4 val = *reinterpret_cast<const uint4*>(smem + MxSmem::kColCodes + c * 64 + ((((2 * m) ^ x) & 6) << 3));
      if (x & 1) val = make_uint4(val.z, val.w, val.x, val.y);
      if (row0 + 32 * m < a.rows)  // rows % 32 == 0: a 32-row group is inside or outside
        *reinterpret_cast<uint4*>(a.c_codes + (col0 + c) * pitch + (row0 >> 1) + m * 16) = val;
    }
  }
#pragma unroll
  for (int which = 0; which < 2; ++which) {
    if (which == 0 && !HAS_ROW) continue;
    if (which == 1 && !HAS_COL) continue;
    const uint8_t* src = smem + (which == 0 ? MxSmem::kSfRow : MxSmem::kSfCol);
    uint8_t* dst = which == 0 ? a.r_scales : a.c_scales;
    const int swz = which == 0 ? a.r_swz : a.c_swz;
    const int64_t R0 = which == 0 ? row0 : col0, K0 = which == 0 ? (col0 >> 5) : (row0 >> 5);
    const int64_t Rn = which == 0 ? a.rows : a.cols, n_kb = which == 0 ? (a.cols >> 5) : (a.rows >> 5);
    if (swz) {
      if (threadIdx.x < 32) {  // one 512-byte atom per tile and copy
        const int64_t off = ((R0 >> 7) * (n_kb >> 2) + (K0 >> 2)) * 512 + threadIdx.x * 16;
        *reinterpret_cast<uint4*>(dst + off) = *reinterpret_cast<const uint4*>(src + threadIdx.x * 16);
      }
    } else {
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int idx = threadIdx.x * 2 + k;
        const int r = idx >> 2, kb = idx & 3;
        if (R0 + r < Rn && K0 + kb < n_kb) dst[(R0 + r) * n_kb + K0 + kb] = src[idx];
      }
    }
  }
  // no tensor-level scale in this format: the copies' global words read {0, 1} so that the GEMM epilogue's
  // product of decode scales is 1
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (HAS_ROW) { a.r_global[0] = 0.f; a.r_global[1] = 1.f; }
    if (HAS_COL) { a.c_global[0] = 0.f; a.c_global[1] = 1.f; }
  }
}

template <bool HR, bool HC, bool B2, bool RC, bool SR>
static cudaError_t launch_mx_t(const QuantArgs& a, cudaStream_t s) {
  auto kern = quantize_mx_kernel<HR, HC, B2, RC, SR>;
  const int smem = (SR && HC) ? MxSmem::kBytesRand : MxSmem::kBytesNoRand;
  static std::atomic<uint64_t> configured{0};  // per call site (template instantiation) and device
  int dev;
  if (device_needs_config(configured, &dev)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, MxSmem::kBytesRand);
    if (e != cudaSuccess) return e;
    device_configured(configured, dev);
  }
  kern<<<(unsigned)((int64_t)a.tiles_r * a.tiles_c), 256, smem, s>>>(a);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_quantize_mx(const QuantArgs& a, bool has_row, bool has_col, bool block2d, bool rht_col, bool sr,
                               cudaStream_t s) {
  rht_col = rht_col && has_col;
#define NVFP4_MXQ(HR, HC, B2, RC, SRV)                                                        \
  if (has_row == HR && has_col == HC && block2d == B2 && rht_col == RC && sr == SRV)         \
    return launch_mx_t<HR, HC, B2, RC, SRV>(a, s);
#define NVFP4_MXQ_COPIES(B2, RC, SRV) \
  NVFP4_MXQ(true, false, B2, false, SRV) \
  NVFP4_MXQ(false, true, B2, RC, SRV)   \
  NVFP4_MXQ(true, true, B2, RC, SRV)
  NVFP4_MXQ_COPIES(true, false, false)
  NVFP4_MXQ_COPIES(true, false, true)
  NVFP4_MXQ_COPIES(false, false, false)
  NVFP4_MXQ_COPIES(false, false, true)
  NVFP4_MXQ_COPIES(false, true, false)
  NVFP4_MXQ_COPIES(false, true, true)
#undef NVFP4_MXQ_COPIES
#undef NVFP4_MXQ
  return cudaErrorInvalidValue;
}

}  // namespace nvfp4
