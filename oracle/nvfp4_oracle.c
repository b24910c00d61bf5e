/*
 * NVFP4 CPU oracle -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, step-by-step restatement of the NVFP4 quantization procedure
 * (paper Appendix B, Eq. 1-5), the tiled random Hadamard transform (Appendix C),
 * stochastic rounding (Section 4.4) and the block-scaled GEMM (Eq. 5 plus the
 * sentence after it); at the end, the same for MXFP4, the comparison format
 * (Section 2, Section 5, Appendix B.4).  It shares no code, table or constant generator with the
 * CUDA path.  Only tests, the smoke check and the CPU-baseline legs of the
 * benchmark may build or call it.
 *
 * Arithmetic conventions (the paper prints formulas, not an operation order):
 *   - "fl()" below is one IEEE binary32 operation; this file must be compiled
 *     with -ffp-contract=off and without -ffast-math so that every float
 *     expression is exactly one rounding, denormals are kept.
 *   - the Hadamard sum and every "reference" quantity (dequantize, GEMM) are
 *     evaluated in binary64.
 *
 * Pins: every function here is checked by the CPU test-suite against values the
 * paper prints, closed forms, brute force or library routines; no function is
 * left "parity unpinned".
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_EXPORT __attribute__((visibility("default")))

/* ------------------------------------------------------------------------- */
/* Number formats (Section 2)                                                 */
/* ------------------------------------------------------------------------- */

/* bf16 is the upper half of a binary32; widening is exact. */
ORC_EXPORT float orc_bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* E2M1 magnitudes for the 3 low bits (exponent 2 bits, mantissa 1 bit), the
 * set printed in Section 2: 0, 0.5, 1, 1.5, 2, 3, 4, 6.  Bit 3 is the sign. */
static const float kE2M1[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

ORC_EXPORT float orc_e2m1_decode(uint8_t code) {
  float m = kE2M1[code & 7];
  return (code & 8) ? -m : m;
}

/* E4M3 (finite-only variant: bias 7, subnormals, largest finite 448 = 0x7E,
 * 0x7F is NaN).  Decoded from its definition, not from a table. */
ORC_EXPORT float orc_e4m3_decode(uint8_t byte) {
  int e = (byte >> 3) & 15;
  int m = byte & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  if (e == 0)
    v = ldexp((double)m / 8.0, -6); /* subnormal: m/8 * 2^(1-bias) */
  else
    v = ldexp(1.0 + (double)m / 8.0, e - 7);
  return (float)((byte & 0x80) ? -v : v);
}

/* Round a non-negative binary32 to the nearest of the 127 finite non-negative
 * E4M3 values, ties to the even byte (= even mantissa), saturating at 448
 * (Appendix B.2: round-to-nearest-even for the decode scale; Appendix B.1:
 * 448 is the largest magnitude).  Brute force over all candidates. */
ORC_EXPORT uint8_t orc_e4m3_encode_rne(float t) {
  if (!(t > 0.0f)) return 0; /* zero (negative never occurs: scales are >= 0) */
  double x = (double)t;
  int best = 0;
  double best_err = fabs(x - 0.0);
  for (int b = 1; b <= 0x7E; ++b) {
    double err = fabs(x - (double)orc_e4m3_decode((uint8_t)b));
    if (err < best_err || (err == best_err && (b & 1) == 0)) {
      best = b;
      best_err = err;
    }
  }
  return (uint8_t)best;
}

/* q(.) of Eq. 4 with round-to-nearest-even (Section 4: weights and
 * activations).  Saturates at +-6; ties go to the code whose mantissa bit is
 * 0; the sign bit of the input is kept, also for zeros. */
ORC_EXPORT uint8_t orc_e2m1_encode_rne(float v) {
  uint8_t sign = signbit(v) ? 8 : 0;
  double a = fabs((double)v);
  if (a > 6.0) a = 6.0;
  int best = 0;
  double best_err = a;
  for (int c = 1; c < 8; ++c) {
    double err = fabs(a - (double)kE2M1[c]);
    if (err < best_err || (err == best_err && (c & 1) == 0)) {
      best = c;
      best_err = err;
    }
  }
  return (uint8_t)(sign | best);
}

/* q(.) with stochastic rounding (Section 4.4): the result is one of the two
 * representable neighbours lo <= a < hi, and the upper one is taken with
 * probability equal to the fractional position of a between them.  The draw is
 * an 8-bit uniform u; round up iff u + 0.5 < 256 * frac (so exact grid points
 * never move, and P(up) is within 1/512 of frac). */
ORC_EXPORT uint8_t orc_e2m1_encode_sr(float v, uint8_t u) {
  uint8_t sign = signbit(v) ? 8 : 0;
  float a = fabsf(v);
  if (!(a < 6.0f)) return (uint8_t)(sign | 7);
  int lo = 0;
  while (lo < 7 && kE2M1[lo + 1] <= a) ++lo; /* kE2M1[lo] <= a < kE2M1[lo+1] */
  float step = kE2M1[lo + 1] - kE2M1[lo];
  float frac = (a - kE2M1[lo]) / step; /* exact: power-of-two step */
  int up = ((float)u + 0.5f) < 256.0f * frac;
  return (uint8_t)(sign | (lo + up));
}

/* The same, element by element over arrays (a loop around the scalar routine, for sweeps in tests). */
ORC_EXPORT void orc_e2m1_encode_sr_many(const float* v, const uint8_t* u, int64_t n, uint8_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = orc_e2m1_encode_sr(v[i], u[i]);
}

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 counter-based generator (Salmon et al., SC'11).              */
/* The paper leaves the random source open; the draw is keyed by              */
/* (seed; index of the source element), see orc_sr_draw().                    */
/* ------------------------------------------------------------------------- */
ORC_EXPORT void orc_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2],
                                  uint32_t out[4]) {
  uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
  uint32_t k0 = key_in[0], k1 = key_in[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) {
      k0 += 0x9E3779B9u;
      k1 += 0xBB67AE85u;
    }
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 8-bit draw of the element at row-major position e of the source tensor:
 * one Philox call per 16 consecutive positions; counter = (e>>4 as 64 bit,
 * sr_offset as 64 bit), key = seed; byte (e & 15) of the 16 output bytes,
 * little-endian inside each word. */
ORC_EXPORT uint8_t orc_sr_draw(uint64_t seed, uint64_t sr_offset, uint64_t e) {
  uint64_t g = e >> 4;
  uint32_t ctr[4] = {(uint32_t)g, (uint32_t)(g >> 32), (uint32_t)sr_offset,
                     (uint32_t)(sr_offset >> 32)};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t r[4];
  orc_philox4x32_10(ctr, key, r);
  unsigned byte = (unsigned)(e & 15);
  return (uint8_t)(r[byte >> 2] >> (8 * (byte & 3)));
}

/* ------------------------------------------------------------------------- */
/* Random Hadamard transform, d = 16 (Appendix C; Section 4.2)                */
/* ------------------------------------------------------------------------- */

/* Entry (j,k) of the +-1 Sylvester matrix H_2 (x) H_2 (x) H_2 (x) H_2 with
 * H_2 = [[1,1],[1,-1]]: the sign is the parity of the bits j and k share. */
ORC_EXPORT int orc_hadamard16_entry(int j, int k) {
  int p = j & k, parity = 0;
  while (p) {
    parity ^= p & 1;
    p >>= 1;
  }
  return parity ? -1 : 1;
}

/* y = x * (S * H_16): y_k = (1/4) * sum_j s_j x_j h(j,k), where bit j of
 * sign_mask set means s_j = -1 (S multiplies the input element, i.e. flips
 * rows of H).  Accumulated in binary64, rounded once to binary32. */
ORC_EXPORT void orc_rht16(const float x[16], uint16_t sign_mask, float y[16]) {
  for (int k = 0; k < 16; ++k) {
    double acc = 0.0;
    for (int j = 0; j < 16; ++j) {
      double s = ((sign_mask >> j) & 1) ? -1.0 : 1.0;
      acc += s * (double)x[j] * (double)orc_hadamard16_entry(j, k);
    }
    y[k] = (float)(0.25 * acc);
  }
}

/* Other transform sizes (Appendix E.4.2 compares d = 2, 4, 16 and 128): the
 * Sylvester matrix of order d = 2^m has the same entry rule (parity of the bits
 * j and k share), the normalisation is 1/sqrt(d), and the sign vector has d
 * entries: bit (j & 31) of sign_words[j >> 5].  y_k = (1/sqrt d) sum_j s_j x_j
 * h(j,k), accumulated and normalised in binary64, rounded once to binary32.
 * Returns -1 unless d is a power of two in [2, 128]. */
ORC_EXPORT int orc_rht_d(const float* x, int d, const uint32_t* sign_words, float* y) {
  if (d < 2 || d > 128 || (d & (d - 1))) return -1;
  const double norm = sqrt((double)d);
  for (int k = 0; k < d; ++k) {
    double acc = 0.0;
    for (int j = 0; j < d; ++j) {
      double s = ((sign_words[j >> 5] >> (j & 31)) & 1u) ? -1.0 : 1.0;
      acc += s * (double)x[j] * (double)orc_hadamard16_entry(j, k);
    }
    y[k] = (float)(acc / norm);
  }
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Two-level scaling (Appendix B.1, B.2)                                      */
/* ------------------------------------------------------------------------- */

/* Eq. 1: s_enc = 6*448/amax, s_dec = 1/s_enc, both binary32.  A zero tensor
 * gets s_enc = 1; an overflowing quotient is clamped to FLT_MAX. */
ORC_EXPORT void orc_global_scale(float amax, float* s_enc, float* s_dec) {
  float e;
  if (amax == 0.0f) {
    e = 1.0f;
  } else {
    e = 2688.0f / amax;
    if (e > FLT_MAX) e = FLT_MAX;
  }
  *s_enc = e;
  *s_dec = 1.0f / e;
}

/* Eq. 2-3: stored block scale = e4m3( fl( fl(amax_b / 6) * s_enc ) ). */
ORC_EXPORT uint8_t orc_block_scale_byte(float amax_b, float s_enc) {
  float s_dec_b = amax_b / 6.0f;
  float t = s_dec_b * s_enc;
  return orc_e4m3_encode_rne(t);
}

/* Text after Eq. 3: s_enc_b = 1 / (fp32(stored scale) * s_dec); a zero scale
 * byte encodes the whole block as zeros; overflow clamps to FLT_MAX. */
ORC_EXPORT float orc_block_encode_scale(uint8_t scale_byte, float s_dec) {
  if (scale_byte == 0) return 0.0f;
  float d = orc_e4m3_decode(scale_byte) * s_dec;
  float r = 1.0f / d;
  if (r > FLT_MAX) r = FLT_MAX;
  return r;
}

/* Offset of scale byte (row r, 16-block kb) in the layout the block-scaled
 * tensor-core instruction consumes: 512-byte atoms covering 128 rows x 4
 * blocks; n_kb = blocks per row (a multiple of 4). */
ORC_EXPORT int64_t orc_sf_swizzled_offset(int64_t r, int64_t kb, int64_t n_kb) {
  int64_t atom = (r / 128) * (n_kb / 4) + kb / 4;
  return atom * 512 + (r % 32) * 16 + ((r % 128) / 32) * 4 + kb % 4;
}

/* ------------------------------------------------------------------------- */
/* Quantize one copy of a tensor (Appendix B; Sections 4.2-4.4)               */
/* ------------------------------------------------------------------------- */

/*
 * x_bf16    : source tensor, src_rows x src_cols, row-major, leading dim ld
 * colwise   : 0 = the copy is the tensor itself (blocks along src columns),
 *             1 = the copy is the transpose (blocks along src rows)
 * block_rows: 1 = 1x16 blocks along the copy's columns; 16 = 16x16 blocks
 * rht       : apply x*(S*H_16) to every aligned 16-chunk of every row of the
 *             copy before any amax is taken (scales live in the rotated space)
 * rounding  : 0 = round-to-nearest-even, 1 = stochastic (draws keyed by the
 *             source position the value is stored at)
 * amax_override >= 0: use it instead of the computed tensor amax (used by the
 *             comparison protocol under RHT, where a last-bit difference in
 *             amax must not be smeared over every block, and when a slab of
 *             rows of a larger tensor is quantized on its own)
 * sr_row0, sr_cols, sr_col0: the tensor is the block of rows [sr_row0, sr_row0 +
 *             src_rows) and columns [sr_col0, sr_col0 + src_cols) of a larger
 *             source with sr_cols columns (sr_cols = 0: it is the whole source);
 *             only the stochastic-rounding draw index depends on it
 * outputs   : codes [R][C/2] (even column in the low nibble), scales [R][C/16]
 *             linear, global = {amax, s_dec}, y_out (nullable) = the values
 *             that were quantized, [R][C] floats.   R x C = shape of the copy.
 * returns 0, or -1 when the copy's contraction length is not a multiple of 16
 * (or its row count not a multiple of block_rows).
 */
static int quantize_source(const uint16_t* x_bf16, const float* x_f32, int64_t src_rows, int64_t src_cols,
                           int64_t ld, int colwise, int block_rows, int rht, uint16_t sign_mask,
                           int rht_dim, const uint32_t* sign_words,
                           int rounding, uint64_t seed, uint64_t sr_offset,
                           float amax_override, int64_t sr_row0, int64_t sr_cols, int64_t sr_col0,
                           uint8_t* codes, uint8_t* scales, float* global, float* y_out) {
  const int64_t R = colwise ? src_cols : src_rows;
  const int64_t C = colwise ? src_rows : src_cols;
  if ((block_rows != 1 && block_rows != 16) || C % 16 || R % block_rows) return -1;
  if (rht && rht_dim != 16 && (rht_dim < 2 || rht_dim > 128 || (rht_dim & (rht_dim - 1)) || C % rht_dim)) return -1;
  float* y = (float*)malloc(sizeof(float) * (size_t)(R * C));
  if (!y) return -2;

  /* the copy, explicitly formed (transposed for a column-wise copy) */
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < R; ++r)
    for (int64_t c = 0; c < C; ++c) {
      int64_t sr = colwise ? c : r, sc = colwise ? r : c;
      y[r * C + c] = x_f32 ? x_f32[sr * ld + sc] : orc_bf16_to_f32(x_bf16[sr * ld + sc]);
    }

  /* Appendix C: rotate every aligned chunk of 16 along the contraction dim */
  if (rht && rht_dim == 16) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
      for (int64_t c0 = 0; c0 < C; c0 += 16) {
        float t[16];
        orc_rht16(&y[r * C + c0], sign_mask, t);
        memcpy(&y[r * C + c0], t, sizeof t);
      }
  } else if (rht) { /* Appendix E.4.2: every aligned chunk of rht_dim elements instead */
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
      for (int64_t c0 = 0; c0 < C; c0 += rht_dim) {
        float t[128];
        orc_rht_d(&y[r * C + c0], rht_dim, sign_words, t);
        memcpy(&y[r * C + c0], t, sizeof(float) * (size_t)rht_dim);
      }
  }

  /* Appendix B.1: tensor amax (in the rotated space when rht) and Eq. 1 */
  float amax = 0.0f;
  for (int64_t i = 0; i < R * C; ++i) {
    float a = fabsf(y[i]);
    if (a > amax) amax = a;
  }
  if (amax_override >= 0.0f) amax = amax_override;
  float s_enc, s_dec;
  orc_global_scale(amax, &s_enc, &s_dec);
  global[0] = amax;
  global[1] = s_dec;

  const int64_t nkb = C / 16;
  /* Appendix B.2: block scales (one per 1x16 chunk, or one per 16x16 tile
   * replicated to its 16 chunks, Section 4.3) */
#pragma omp parallel for schedule(static)
  for (int64_t rb = 0; rb < R / block_rows; ++rb)
    for (int64_t kb = 0; kb < nkb; ++kb) {
      float amax_b = 0.0f;
      for (int64_t i = 0; i < block_rows; ++i)
        for (int64_t j = 0; j < 16; ++j) {
          float a = fabsf(y[(rb * block_rows + i) * C + kb * 16 + j]);
          if (a > amax_b) amax_b = a;
        }
      uint8_t sb = orc_block_scale_byte(amax_b, s_enc);
      for (int64_t i = 0; i < block_rows; ++i) scales[(rb * block_rows + i) * nkb + kb] = sb;
    }

  /* Appendix B.3, Eq. 4: scale, convert, pack */
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < R; ++r)
    for (int64_t kb = 0; kb < nkb; ++kb) {
      const float s_enc_b = orc_block_encode_scale(scales[r * nkb + kb], s_dec);
      uint8_t code[16];
      for (int64_t j = 0; j < 16; ++j) {
        int64_t c = kb * 16 + j;
        float v = y[r * C + c] * s_enc_b;
        if (rounding == 0) {
          code[j] = orc_e2m1_encode_rne(v);
        } else {
          int64_t sr = colwise ? c : r, sc = colwise ? r : c;
          uint64_t e = (uint64_t)(sr + sr_row0) * (uint64_t)(sr_cols ? sr_cols : src_cols) + (uint64_t)(sc + sr_col0);
          code[j] = orc_e2m1_encode_sr(v, orc_sr_draw(seed, sr_offset, e));
        }
      }
      for (int64_t j = 0; j < 16; j += 2)
        codes[r * (C / 2) + (kb * 16 + j) / 2] = (uint8_t)(code[j] | (code[j + 1] << 4));
    }

  if (y_out) memcpy(y_out, y, sizeof(float) * (size_t)(R * C));
  free(y);
  return 0;
}

ORC_EXPORT int orc_quantize(const uint16_t* x_bf16, int64_t src_rows, int64_t src_cols, int64_t ld,
                            int colwise, int block_rows, int rht, uint16_t sign_mask,
                            int rounding, uint64_t seed, uint64_t sr_offset,
                            float amax_override, int64_t sr_row0, int64_t sr_cols, int64_t sr_col0,
                            uint8_t* codes, uint8_t* scales, float* global, float* y_out) {
  return quantize_source(x_bf16, NULL, src_rows, src_cols, ld, colwise, block_rows, rht, sign_mask, 16, NULL,
                         rounding, seed, sr_offset, amax_override, sr_row0, sr_cols, sr_col0, codes, scales, global, y_out);
}

/* The same procedure with a transform of another size (Appendix E.4.2): every aligned chunk of rht_dim elements
 * along the contraction dimension is rotated (several per 16-block for rht_dim < 16, one per eight blocks for 128);
 * blocks, scales and rounding are unchanged.  sign_words: rht_dim sign bits. */
ORC_EXPORT int orc_quantize_rht(const uint16_t* x_bf16, int64_t src_rows, int64_t src_cols, int64_t ld,
                                int colwise, int rht_dim, const uint32_t* sign_words,
                                int rounding, uint64_t seed, uint64_t sr_offset,
                                float amax_override, int64_t sr_row0, int64_t sr_cols, int64_t sr_col0,
                                uint8_t* codes, uint8_t* scales, float* global, float* y_out) {
  return quantize_source(x_bf16, NULL, src_rows, src_cols, ld, colwise, 1, 1, (uint16_t)sign_words[0], rht_dim,
                         sign_words, rounding, seed, sr_offset, amax_override, sr_row0, sr_cols, sr_col0, codes,
                         scales, global, y_out);
}

/* The same procedure from a binary32 source (Appendix B names FP32 as well as BF16 as the precision converted from): only step one,
 * reading the element, differs. */
ORC_EXPORT int orc_quantize_f32(const float* x_f32, int64_t src_rows, int64_t src_cols, int64_t ld,
                                int colwise, int block_rows, int rht, uint16_t sign_mask,
                                int rounding, uint64_t seed, uint64_t sr_offset,
                                float amax_override, int64_t sr_row0, int64_t sr_cols, int64_t sr_col0,
                                uint8_t* codes, uint8_t* scales, float* global, float* y_out) {
  return quantize_source(NULL, x_f32, src_rows, src_cols, ld, colwise, block_rows, rht, sign_mask, 16, NULL,
                         rounding, seed, sr_offset, amax_override, sr_row0, sr_cols, sr_col0, codes, scales, global, y_out);
}

/* Decode: x^ = (+-magnitude) * fp32(block scale) * s_dec, in binary64 (exact:
 * 2 + 4 + 24 significant bits).  scales are in the linear layout. */
ORC_EXPORT void orc_dequantize(const uint8_t* codes, const uint8_t* scales, const float* global,
                               int64_t R, int64_t C, double* out) {
  const double s_dec = (double)global[1];
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < R; ++r)
    for (int64_t c = 0; c < C; ++c) {
      uint8_t byte = codes[r * (C / 2) + c / 2];
      uint8_t code = (c & 1) ? (byte >> 4) : (byte & 15);
      double sb = (double)orc_e4m3_decode(scales[r * (C / 16) + c / 16]);
      out[r * C + c] = (double)orc_e2m1_decode(code) * sb * s_dec;
    }
}

/* Same decode but leaving the per-tensor scale out: code * block scale. */
ORC_EXPORT void orc_dequantize_local(const uint8_t* codes, const uint8_t* scales, int64_t R,
                                     int64_t C, double* out) {
  float unit[2] = {0.0f, 1.0f};
  orc_dequantize(codes, scales, unit, R, C, out);
}

/* ------------------------------------------------------------------------- */
/* GEMM reference (Eq. 5 and the sentence after it): the exact product of the */
/* decoded operands, D[i][j] = sum_k A[i][k] * B[j][k], binary64, naive.      */
/* T[i][j] = sum_k |A[i][k]| |B[j][k]| is the scale of the error tolerance.   */
/* ------------------------------------------------------------------------- */
ORC_EXPORT void orc_gemm_tn(const double* A, const double* B, int64_t M, int64_t N, int64_t K,
                            double* D, double* T) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i)
    for (int64_t j = 0; j < N; ++j) {
      double acc = 0.0, mag = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        double p = A[i * K + k] * B[j * K + k];
        acc += p;
        mag += fabs(p);
      }
      D[i * N + j] = acc;
      if (T) T[i * N + j] = mag;
    }
}

/* Eq. 5 written out literally: per 16-block partial dot product of the codes,
 * times the two block scales, summed over blocks, then the two global decode
 * scales applied once on the result.  Used to check that the "exact product of
 * decoded operands" above is the same quantity the paper describes. */
ORC_EXPORT void orc_gemm_blockscaled(const uint8_t* a_codes, const uint8_t* a_scales,
                                     const float* a_global, const uint8_t* b_codes,
                                     const uint8_t* b_scales, const float* b_global, int64_t M,
                                     int64_t N, int64_t K, double* D) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i)
    for (int64_t j = 0; j < N; ++j) {
      double acc = 0.0;
      for (int64_t kb = 0; kb < K / 16; ++kb) {
        double part = 0.0;
        for (int64_t k = kb * 16; k < kb * 16 + 16; ++k) {
          uint8_t ab = a_codes[i * (K / 2) + k / 2], bb = b_codes[j * (K / 2) + k / 2];
          double av = orc_e2m1_decode((k & 1) ? (ab >> 4) : (ab & 15));
          double bv = orc_e2m1_decode((k & 1) ? (bb >> 4) : (bb & 15));
          part += av * bv;
        }
        acc += (double)orc_e4m3_decode(a_scales[i * (K / 16) + kb]) *
               (double)orc_e4m3_decode(b_scales[j * (K / 16) + kb]) * part;
      }
      D[i * N + j] = acc * (double)a_global[1] * (double)b_global[1];
    }
}

/* ------------------------------------------------------------------------- */
/* MXFP4, the comparison format (Section 2, Section 5, Appendix B.4):         */
/* E2M1 elements, one UE8M0 (power-of-two) scale per 32 contiguous elements,  */
/* no tensor-level scale.                                                     */
/* ------------------------------------------------------------------------- */

/* UE8M0: byte b encodes 2^(b - 127), b = 0..254 (0xFF is NaN, never produced). */
ORC_EXPORT float orc_ue8m0_decode(uint8_t b) { return ldexpf(1.0f, (int)b - 127); }

/* Appendix B.4: the decode scale amax_b / 6 is rounded UP to a power of two so
 * that the scaled block never exceeds 6: the smallest e with 6 * 2^e >= amax_b,
 * found by search.  A zero block gets the smallest scale (byte 0); e is clamped
 * to what the byte can hold. */
ORC_EXPORT uint8_t orc_mx_block_scale_byte(float amax_b) {
  if (amax_b == 0.0f) return 0;
  int e = -160;
  while (ldexp(6.0, e) < (double)amax_b) ++e;
  int b = e + 127;
  if (b < 0) b = 0;
  if (b > 254) b = 254;
  return (uint8_t)b;
}

/* encode scale = 1 / decode scale = 2^(127 - b), exact */
ORC_EXPORT float orc_mx_block_encode_scale(uint8_t b) { return ldexpf(1.0f, 127 - (int)b); }

/* +-1 Sylvester matrix of order 32 = H_2 (x) H_16 */
ORC_EXPORT int orc_hadamard32_entry(int j, int k) {
  int top = ((j >> 4) & (k >> 4) & 1) ? -1 : 1;
  return top * orc_hadamard16_entry(j & 15, k & 15);
}

/* Section 5: transform size d = 32 for MXFP4, aligned with its block size.
 * y_k = (1/sqrt(32)) * sum_j s_j x_j h(j,k); the whole expression is evaluated
 * in binary64 and rounded once to binary32. */
ORC_EXPORT void orc_rht32(const float x[32], uint32_t sign_mask, float y[32]) {
  const double norm = 1.0 / sqrt(32.0);
  for (int k = 0; k < 32; ++k) {
    double acc = 0.0;
    for (int j = 0; j < 32; ++j) {
      double s = ((sign_mask >> j) & 1u) ? -1.0 : 1.0;
      acc += s * (double)x[j] * (double)orc_hadamard32_entry(j, k);
    }
    y[k] = (float)(norm * acc);
  }
}

/*
 * MXFP4 quantization of one copy; arguments as orc_quantize, except:
 * block_rows: 1 = 1x32 blocks along the copy's columns; 32 = 32x32 blocks
 *             (the 2D weight scaling of Section 4.3 at this format's block size)
 * rht       : x * (S * H_32) on every aligned 32-chunk
 * outputs   : codes [R][C/2], scales [R][C/32] UE8M0 bytes (linear layout),
 *             y_out (nullable).  There is no tensor-level scale.
 * returns -1 when C is not a multiple of 32 (or R not of block_rows).
 */
ORC_EXPORT int orc_quantize_mx(const uint16_t* x_bf16, int64_t src_rows, int64_t src_cols, int64_t ld,
                               int colwise, int block_rows, int rht, uint32_t sign_mask, int rounding,
                               uint64_t seed, uint64_t sr_offset, int64_t sr_row0, int64_t sr_cols,
                               int64_t sr_col0, uint8_t* codes, uint8_t* scales, float* y_out) {
  const int64_t R = colwise ? src_cols : src_rows;
  const int64_t C = colwise ? src_rows : src_cols;
  if ((block_rows != 1 && block_rows != 32) || C % 32 || R % block_rows) return -1;
  float* y = (float*)malloc(sizeof(float) * (size_t)(R * C));
  if (!y) return -2;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < R; ++r)
    for (int64_t c = 0; c < C; ++c) {
      int64_t sr = colwise ? c : r, sc = colwise ? r : c;
      y[r * C + c] = orc_bf16_to_f32(x_bf16[sr * ld + sc]);
    }
  if (rht) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
      for (int64_t c0 = 0; c0 < C; c0 += 32) {
        float t[32];
        orc_rht32(&y[r * C + c0], sign_mask, t);
        memcpy(&y[r * C + c0], t, sizeof t);
      }
  }
  const int64_t nkb = C / 32;
#pragma omp parallel for schedule(static)
  for (int64_t rb = 0; rb < R / block_rows; ++rb)
    for (int64_t kb = 0; kb < nkb; ++kb) {
      float amax_b = 0.0f;
      for (int64_t i = 0; i < block_rows; ++i)
        for (int64_t j = 0; j < 32; ++j) {
          float a = fabsf(y[(rb * block_rows + i) * C + kb * 32 + j]);
          if (a > amax_b) amax_b = a;
        }
      uint8_t sb = orc_mx_block_scale_byte(amax_b);
      for (int64_t i = 0; i < block_rows; ++i) scales[(rb * block_rows + i) * nkb + kb] = sb;
    }
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < R; ++r)
    for (int64_t kb = 0; kb < nkb; ++kb) {
      const float s_enc_b = orc_mx_block_encode_scale(scales[r * nkb + kb]);
      uint8_t code[32];
      for (int64_t j = 0; j < 32; ++j) {
        int64_t c = kb * 32 + j;
        float v = y[r * C + c] * s_enc_b;
        if (rounding == 0) {
          code[j] = orc_e2m1_encode_rne(v);
        } else {
          int64_t sr = colwise ? c : r, sc = colwise ? r : c;
          uint64_t e = (uint64_t)(sr + sr_row0) * (uint64_t)(sr_cols ? sr_cols : src_cols) + (uint64_t)(sc + sr_col0);
          code[j] = orc_e2m1_encode_sr(v, orc_sr_draw(seed, sr_offset, e));
        }
      }
      for (int64_t j = 0; j < 32; j += 2)
        codes[r * (C / 2) + (kb * 32 + j) / 2] = (uint8_t)(code[j] | (code[j + 1] << 4));
    }
  if (y_out) memcpy(y_out, y, sizeof(float) * (size_t)(R * C));
  free(y);
  return 0;
}

/* Decode: x^ = (+-magnitude) * 2^(scale byte - 127), exact in binary64. */
ORC_EXPORT void orc_dequantize_mx(const uint8_t* codes, const uint8_t* scales, int64_t R, int64_t C,
                                  double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < R; ++r)
    for (int64_t c = 0; c < C; ++c) {
      uint8_t byte = codes[r * (C / 2) + c / 2];
      uint8_t code = (c & 1) ? (byte >> 4) : (byte & 15);
      out[r * C + c] = (double)orc_e2m1_decode(code) * ldexp(1.0, (int)scales[r * (C / 32) + c / 32] - 127);
    }
}
