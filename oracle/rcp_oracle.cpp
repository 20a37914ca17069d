// rcp_oracle.cpp -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// Plain, slow, single-threaded CPU oracle for the decode-time W2A4 hot path of RCP
// (Rotate, Clip, Partition; arXiv 2502.15779):
//   * block-Hadamard rotation of the activation (Appendix A.2, definition of the
//     normalized Hadamard matrix H_n = H'_n / sqrt(n), Sylvester recursion),
//   * per-token symmetric absmax int4 quantization and nibble packing (Section 4.4
//     "Fast GEMV via Latency Hiding": X_q is 1 x C/2 INT8 holding two INT4 each, scale is
//     one FP16 scalar; Table "Quantization configurations": activations symmetric,
//     per-token),
//   * 2-bit weight-code packing (Section 4.4: W_q packed sub-byte along the input channel),
//   * the look-up-table GEMV  O = s * X_q * LUT[W_q]  (Section 4.4, Eq. "deqgrid": the
//     four-entry dequantization grid W^_0..W^_3 per quantization unit).
//
// Only tests, the smoke check and the benchmark's CPU-baseline leg may call this file.
// It shares no code, header, table or helper with the CUDA library, and the CUDA library
// never calls it. No SIMD intrinsics, no threads, no blocking or reordering beyond what the
// definitions state.
//
// Pins (all in tests marked "not gpu"): H H^T = I and FWHT == explicit Sylvester matrix
// product; library fp16 conversion; hand-computed rounding cases; brute-force 8x8 and
// 16x32 GEMV; exact integer equality of the per-code-sum form and the direct form;
// LUT lookup of unpacked codes == dequantized weight matrix; affine/constant LUT special
// cases reducing to a plain integer GEMV. Group-wise LUT form: one group == the per-row form;
// equal grids in every group == the per-row form; brute force; exact integer equality with
// its direct form; dense matrix product with the group-wise dequantized weights. Export of the
// partitioning quantizer: hand-computed fixture, the uniform initial point == the textbook
// asymmetric 2-bit quantizer, the range ends and bin centres the paper states, monotone codes,
// the sum form of the dequantizer == LUT lookup.
// Weight-only variant: equals the W2A4 oracle when the activations are integers times a power of
// two; affine grid == plain matrix product; brute force; the fixed-point digits reproduce the
// activations (exactly for elements within 2^-11 of the token's maximum, to half a unit otherwise)
// and a hand-written case. Per-code sums of 8-bit planes: equal to the W2A4 oracle's S on int4 planes, a
// pure-Python loop, sum_c S_c == sum_k a_k.
// 3-bit weights: packing round trip and hand-written words; GEMV by a pure-Python loop; per-code form ==
// direct form as exact integers; sum_c S_c == sum_k q_k; a grid with equal levels for codes c and c + 4
// == the W2A4 oracle on the low two bits; planted index mistakes. NF3 export: hand-worked unit, zero-centred
// symmetric case == nearest level of the table scaled by the absmax, levels at the range ends and the centre.
// fp16 output y: the paper prints no worked numeric GEMV example, so y is pinned only by the
// mathematical identities above, not by a printed value.
#include <cstdint>
#include <cstring>
#include <cmath>
#include <cstdlib>

extern "C" {

// ---------------------------------------------------------------------------------------
// IEEE binary16 <-> binary32, written at the bit level (round-to-nearest-even, subnormals,
// infinities and NaN handled). No compiler half type is used.
// ---------------------------------------------------------------------------------------
float orc_f16_to_f32(uint16_t h) {
  uint32_t sign = (uint32_t)(h >> 15) & 1u;
  uint32_t exp = (uint32_t)(h >> 10) & 0x1Fu;
  uint32_t man = (uint32_t)h & 0x3FFu;
  uint32_t out;
  if (exp == 0) {
    if (man == 0) {
      out = sign << 31;
    } else {
      // subnormal: value = man * 2^-24; normalise
      int e = -1;
      do { man <<= 1; e++; } while ((man & 0x400u) == 0);
      man &= 0x3FFu;
      out = (sign << 31) | ((uint32_t)(127 - 15 - e) << 23) | (man << 13);
    }
  } else if (exp == 31) {
    out = (sign << 31) | 0x7F800000u | (man << 13);
  } else {
    out = (sign << 31) | ((exp - 15 + 127) << 23) | (man << 13);
  }
  float f;
  std::memcpy(&f, &out, 4);
  return f;
}

uint16_t orc_f32_to_f16(float f) {
  uint32_t x;
  std::memcpy(&x, &f, 4);
  uint32_t sign = (x >> 16) & 0x8000u;
  uint32_t exp = (x >> 23) & 0xFFu;
  uint32_t man = x & 0x7FFFFFu;
  if (exp == 255) {  // inf / nan
    return (uint16_t)(sign | 0x7C00u | (man ? (0x200u | (man >> 13)) : 0u));
  }
  int e = (int)exp - 127 + 15;  // biased half exponent
  if (e >= 31) return (uint16_t)(sign | 0x7C00u);  // overflow -> inf
  if (e <= 0) {
    // result is subnormal or zero: value = 1.man * 2^(e-15), unit 2^-24
    if (e < -10) return (uint16_t)sign;  // below half of the smallest subnormal
    uint32_t m = man | 0x800000u;         // 24-bit significand
    int shift = 14 - e;                   // bits to drop (14..24)
    uint32_t q = m >> shift;
    uint32_t rem = m & ((1u << shift) - 1u);
    uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (q & 1u))) q++;
    return (uint16_t)(sign | q);  // a carry into bit 10 yields the smallest normal: correct
  }
  uint32_t q = man >> 13;
  uint32_t rem = man & 0x1FFFu;
  uint32_t h = (uint32_t)e << 10 | q;
  if (rem > 0x1000u || (rem == 0x1000u && (q & 1u))) h++;  // carry may bump exponent; inf if needed
  return (uint16_t)(sign | h);
}

// ---------------------------------------------------------------------------------------
// Appendix A.2: unnormalised Hadamard matrix by the Sylvester recursion
//   H'_1 = [1],  H'_{2n} = [[H'_n, H'_n], [H'_n, -H'_n]],   H_n = H'_n / sqrt(n).
// Written out as a dense matrix (row-major n x n doubles) for the identity checks.
// ---------------------------------------------------------------------------------------
int orc_hadamard_matrix(int n, double* H) {
  if (n < 1 || (n & (n - 1))) return -1;
  H[0] = 1.0;
  for (int m = 1; m < n; m *= 2) {
    // grow the m x m block in the top-left corner (stride n) to 2m x 2m
    for (int i = 0; i < m; i++)
      for (int j = 0; j < m; j++) {
        double v = H[(size_t)i * n + j];
        H[(size_t)i * n + (j + m)] = v;
        H[(size_t)(i + m) * n + j] = v;
        H[(size_t)(i + m) * n + (j + m)] = -v;
      }
  }
  double c = 1.0 / std::sqrt((double)n);
  for (size_t i = 0; i < (size_t)n * n; i++) H[i] *= c;
  return 0;
}

// Exact block rotation in double: y = blockdiag(H_B,...,H_B) x  by the dense definition
// (O(K*B) work). Every fp16 is a multiple of 2^-24 with magnitude < 2^16, so the +-1 sums are
// exact in double for B <= 8192; only the final division by sqrt(B) rounds.
int orc_rotate_exact_f64(const uint16_t* x_f16, int K, int B, double* y) {
  if (B <= 1) { for (int k = 0; k < K; k++) y[k] = (double)orc_f16_to_f32(x_f16[k]); return 0; }
  if ((B & (B - 1)) || K % B) return -1;
  double c = std::sqrt((double)B);
  for (int b0 = 0; b0 < K; b0 += B) {
    for (int i = 0; i < B; i++) {
      double acc = 0.0;
      for (int j = 0; j < B; j++) {
        // entry (i,j) of H'_B in Sylvester (natural) order is (-1)^{popcount(i & j)}
        int p = __builtin_popcount((unsigned)(i & j)) & 1;
        double xv = (double)orc_f16_to_f32(x_f16[b0 + j]);
        acc += p ? -xv : xv;
      }
      y[b0 + i] = acc / c;
    }
  }
  return 0;
}

// ---------------------------------------------------------------------------------------
// Rotation as the quantizer performs it: fp32 fast Walsh-Hadamard butterflies with ascending
// strides (each add/sub one fp32 round-to-nearest operation), then one fp32 multiply by
// (float)(1/sqrt(B)). This fixes the rounding order so that the int4 decision below is
// reproducible bit for bit (the paper's latency table lists an FP32 Hadamard variant; the
// butterfly order is this build's reading, the paper gives none).
// ---------------------------------------------------------------------------------------
static void fwht_f32(float* v, int B) {
  for (int h = 1; h < B; h *= 2) {
    for (int i = 0; i < B; i++) {
      if ((i & h) == 0) {
        float u = v[i];
        float w = v[i + h];
        v[i] = u + w;
        v[i + h] = u - w;
      }
    }
  }
  float c = (float)(1.0 / std::sqrt((double)B));
  for (int i = 0; i < B; i++) v[i] = v[i] * c;
}

int orc_rotate_f32(const uint16_t* x_f16, int K, int B, float* v) {
  for (int k = 0; k < K; k++) v[k] = orc_f16_to_f32(x_f16[k]);
  if (B <= 1) return 0;
  if ((B & (B - 1)) || K % B) return -1;
  for (int b0 = 0; b0 < K; b0 += B) fwht_f32(v + b0, B);
  return 0;
}

// round half to even of a finite float, as an int
static int rint_half_even(float r) {
  double d = (double)r;  // exact
  double fl = std::floor(d);
  double diff = d - fl;  // exact for |d| < 2^52
  long long n = (long long)fl;
  if (diff > 0.5) n += 1;
  else if (diff == 0.5 && (n & 1)) n += 1;
  return (int)n;
}

// ---------------------------------------------------------------------------------------
// Per-token symmetric int4 quantization (Section 4.4; Table "Quantization configurations").
//   v      = rotated token (fp32, above)
//   amax   = max_k |v_k| over the whole token
//   s32    = (amax * clip_ratio) / 7        (fp32 multiply, then fp32 IEEE division)
//   s16    = fp16(s32)  -- the FP16 scalar the paper stores; s = (float)s16 is what divides
//   q_k    = clamp(round_half_even(v_k / s), -8, 7)      (fp32 IEEE division)
//   xq[j]  = (q_{2j} & 0xF) | ((q_{2j+1} & 0xF) << 4)    -- low nibble = even index
// s == 0 (all-zero token, or scale underflow) gives q = 0 everywhere and scale 0.
// Compile with -ffp-contract=off and without fast-math: every operation is one IEEE fp32 op.
// q_out (optional, int8 [M][K]) and v_out (optional, float [M][K]) expose intermediates.
// Returns 0, or -1 on a bad shape, -2 on a non-finite input.
// ---------------------------------------------------------------------------------------
int orc_quantize_act(const uint16_t* x_f16, int M, int K, int had_block, float clip_ratio,
                     uint8_t* xq, uint16_t* scale_f16, int8_t* q_out, float* v_out) {
  if (M < 1 || K < 2 || (K & 1)) return -1;
  int B = had_block <= 1 ? 1 : had_block;
  if ((B & (B - 1)) || K % B) return -1;
  float* v = (float*)std::malloc(sizeof(float) * (size_t)K);
  int8_t* q = (int8_t*)std::malloc((size_t)K);
  for (int m = 0; m < M; m++) {
    const uint16_t* xm = x_f16 + (size_t)m * K;
    for (int k = 0; k < K; k++) {
      float f = orc_f16_to_f32(xm[k]);
      if (!(f - f == 0.0f)) { std::free(v); std::free(q); return -2; }
    }
    orc_rotate_f32(xm, K, B, v);
    float amax = 0.0f;
    for (int k = 0; k < K; k++) { float a = std::fabs(v[k]); if (a > amax) amax = a; }
    float num = amax * clip_ratio;
    float s32 = num / 7.0f;
    uint16_t s16 = orc_f32_to_f16(s32);
    float s = orc_f16_to_f32(s16);
    for (int k = 0; k < K; k++) {
      int qi = 0;
      if (s != 0.0f) {
        float r = v[k] / s;  // s = +inf (scale overflowed fp16) gives r = 0
        qi = rint_half_even(r);
        if (qi < -8) qi = -8;
        if (qi > 7) qi = 7;
      }
      q[k] = (int8_t)qi;
    }
    for (int j = 0; j < K / 2; j++)
      xq[(size_t)m * (K / 2) + j] = (uint8_t)((q[2 * j] & 0xF) | ((q[2 * j + 1] & 0xF) << 4));
    scale_f16[m] = s16;
    if (q_out) std::memcpy(q_out + (size_t)m * K, q, (size_t)K);
    if (v_out) std::memcpy(v_out + (size_t)m * K, v, sizeof(float) * (size_t)K);
  }
  std::free(v);
  std::free(q);
  return 0;
}

// Decode packed int4 pairs the way Appendix A.7 ("Online Dequantization") describes:
// high element by an arithmetic right shift of the signed byte by 4; low element by a left
// shift by 4 (sign bit of the low nibble to the MSB) then an arithmetic right shift by 4.
void orc_unpack_act(const uint8_t* xq, size_t nbytes, int8_t* q) {
  for (size_t j = 0; j < nbytes; j++) {
    int8_t b = (int8_t)xq[j];
    int8_t hi = (int8_t)(b >> 4);
    int8_t lo = (int8_t)((int8_t)(b << 4) >> 4);
    q[2 * j] = lo;
    q[2 * j + 1] = hi;
  }
}

// ---------------------------------------------------------------------------------------
// Weight-code packing: 16 two-bit codes per 32-bit word along the input channel K,
// code 16w+j in bits [2j, 2j+1] (least-significant first). Returns -3 if a code exceeds 3.
// ---------------------------------------------------------------------------------------
int orc_pack_weights(const uint8_t* codes, int N, int K, uint32_t* words) {
  if (N < 1 || K < 16 || K % 16) return -1;
  for (size_t i = 0; i < (size_t)N * K; i++) if (codes[i] > 3) return -3;
  for (int n = 0; n < N; n++)
    for (int w = 0; w < K / 16; w++) {
      uint32_t acc = 0;
      for (int j = 0; j < 16; j++) acc += (uint32_t)codes[(size_t)n * K + 16 * w + j] << (2 * j);
      words[(size_t)n * (K / 16) + w] = acc;
    }
  return 0;
}

// Independent unpack (division/modulo, not the pack routine's shifts).
void orc_unpack_weights(const uint32_t* words, int N, int K, uint8_t* codes) {
  for (int n = 0; n < N; n++)
    for (int k = 0; k < K; k++) {
      uint32_t w = words[(size_t)n * (K / 16) + k / 16];
      uint32_t div = 1;
      for (int t = 0; t < k % 16; t++) div *= 4;
      codes[(size_t)n * K + k] = (uint8_t)((w / div) % 4);
    }
}

// ---------------------------------------------------------------------------------------
// LUT GEMV (Section 4.4). For token m and output row n:
//   S_c[m][n] = sum over k with code[n][k] == c of q[m][k]            (exact integers)
//   y_ref     = s_m * sum_c LUT[n][c] * S_c                          (double)
//   tol       = 2e-3 * ( s_m * sum_c |LUT[n][c]| * |S_c| ) + 1e-5
// Outputs: S int32 [M][N][4] (may be NULL), y_ref double [M][N], tol double [M][N] (may be
// NULL). Returns 0; -1 bad shape; -4 if an S_c does not fit int32.
// ---------------------------------------------------------------------------------------
int orc_gemv_w2a4(const uint32_t* words, const uint16_t* lut_f16, const uint8_t* xq,
                  const uint16_t* scale_f16, int M, int N, int K,
                  int32_t* S, double* y_ref, double* tol) {
  if (M < 1 || N < 1 || K < 16 || K % 16) return -1;
  uint8_t* codes = (uint8_t*)std::malloc((size_t)K);
  int8_t* q = (int8_t*)std::malloc((size_t)M * K);
  orc_unpack_act(xq, (size_t)M * (K / 2), q);
  int rc = 0;
  for (int n = 0; n < N; n++) {
    orc_unpack_weights(words + (size_t)n * (K / 16), 1, K, codes);
    double L[4];
    for (int c = 0; c < 4; c++) L[c] = (double)orc_f16_to_f32(lut_f16[(size_t)n * 4 + c]);
    for (int m = 0; m < M; m++) {
      long long Sc[4] = {0, 0, 0, 0};
      for (int k = 0; k < K; k++) Sc[codes[k]] += (long long)q[(size_t)m * K + k];
      double s = (double)orc_f16_to_f32(scale_f16[m]);
      double acc = 0.0, mag = 0.0;
      for (int c = 0; c < 4; c++) {
        if (Sc[c] > 2147483647LL || Sc[c] < -2147483648LL) rc = -4;
        if (S) S[((size_t)m * N + n) * 4 + c] = (int32_t)Sc[c];
        acc += L[c] * (double)Sc[c];
        mag += std::fabs(L[c]) * std::fabs((double)Sc[c]);
      }
      y_ref[(size_t)m * N + n] = s * acc;
      if (tol) tol[(size_t)m * N + n] = 2e-3 * (s * mag) + 1e-5;
    }
  }
  std::free(codes);
  std::free(q);
  return rc;
}

// Direct form of the same product: y = s_m * sum_k LUT[n][code[n][k]] * q[m][k], the sum
// taken over k in order, in double. Also returns the exact integer value of the sum with
// every fp16 level scaled by 2^24 (each level is then an integer below 2^41 in magnitude, and
// the K-term sum stays below 2^60): acc_int[m][n] = sum_k Lint[code]*q.
int orc_gemv_direct(const uint32_t* words, const uint16_t* lut_f16, const uint8_t* xq,
                    const uint16_t* scale_f16, int M, int N, int K,
                    double* y_direct, long long* acc_int) {
  if (M < 1 || N < 1 || K < 16 || K % 16) return -1;
  uint8_t* codes = (uint8_t*)std::malloc((size_t)N * K);
  int8_t* q = (int8_t*)std::malloc((size_t)M * K);
  orc_unpack_weights(words, N, K, codes);
  orc_unpack_act(xq, (size_t)M * (K / 2), q);
  for (int n = 0; n < N; n++) {
    double L[4];
    long long Li[4];
    for (int c = 0; c < 4; c++) {
      L[c] = (double)orc_f16_to_f32(lut_f16[(size_t)n * 4 + c]);
      Li[c] = (long long)std::ldexp(L[c], 24);  // exact: fp16 values are multiples of 2^-24
    }
    for (int m = 0; m < M; m++) {
      double acc = 0.0;
      long long ai = 0;
      for (int k = 0; k < K; k++) {
        int c = codes[(size_t)n * K + k];
        int qq = q[(size_t)m * K + k];
        acc += L[c] * (double)qq;
        ai += Li[c] * (long long)qq;
      }
      y_direct[(size_t)m * N + n] = (double)orc_f16_to_f32(scale_f16[m]) * acc;
      if (acc_int) acc_int[(size_t)m * N + n] = ai;
    }
  }
  std::free(codes);
  std::free(q);
  return 0;
}

// Same exact integer, from the per-code sums: sum_c Lint[c] * S_c.
void orc_percode_int(const uint16_t* lut_f16, const int32_t* S, int M, int N, long long* acc_int) {
  for (int m = 0; m < M; m++)
    for (int n = 0; n < N; n++) {
      long long ai = 0;
      for (int c = 0; c < 4; c++) {
        long long Li = (long long)std::ldexp((double)orc_f16_to_f32(lut_f16[(size_t)n * 4 + c]), 24);
        ai += Li * (long long)S[((size_t)m * N + n) * 4 + c];
      }
      acc_int[(size_t)m * N + n] = ai;
    }
}

// Dequantized weight matrix (Eq. "deqgrid"): W^[n][k] = LUT[n][code[n][k]], as double.
void orc_dequant_weights(const uint32_t* words, const uint16_t* lut_f16, int N, int K, double* W) {
  uint8_t* codes = (uint8_t*)std::malloc((size_t)K);
  for (int n = 0; n < N; n++) {
    orc_unpack_weights(words + (size_t)n * (K / 16), 1, K, codes);
    for (int k = 0; k < K; k++)
      W[(size_t)n * K + k] = (double)orc_f16_to_f32(lut_f16[(size_t)n * 4 + codes[k]]);
  }
  std::free(codes);
}

// ---------------------------------------------------------------------------------------
// Group-wise LUT GEMV. Section 4.4 gives the dequantization grid the shape H x (N*4) with N
// groups per input channel row, and Appendix A.3 sets C = N*G with group size G (128 in the
// table of quantization configurations): weight k of row n takes its four levels from group
// k / G. For token m, row n, group j:
//   S_c[m][n][j] = sum over k in [jG, (j+1)G) with code[n][k] == c of q[m][k]   (exact integers)
//   y_ref        = s_m * sum_j sum_c LUT[n][j][c] * S_c[m][n][j]                 (double)
//   tol          = 2e-3 * ( s_m * sum_j sum_c |LUT[n][j][c]| * |S_c[m][n][j]| ) + 1e-5
// lut_f16 is [N][K/G][4]. Outputs: S int32 [M][N][K/G][4] (may be NULL), y_ref [M][N], tol
// [M][N] (may be NULL). Returns 0; -1 bad shape (G must divide K).
// ---------------------------------------------------------------------------------------
int orc_gemv_w2a4_grouped(const uint32_t* words, const uint16_t* lut_f16, const uint8_t* xq,
                          const uint16_t* scale_f16, int M, int N, int K, int G,
                          int32_t* S, double* y_ref, double* tol) {
  if (M < 1 || N < 1 || K < 16 || K % 16 || G < 1 || K % G) return -1;
  const int NG = K / G;
  uint8_t* codes = (uint8_t*)std::malloc((size_t)K);
  int8_t* q = (int8_t*)std::malloc((size_t)M * K);
  orc_unpack_act(xq, (size_t)M * (K / 2), q);
  for (int n = 0; n < N; n++) {
    orc_unpack_weights(words + (size_t)n * (K / 16), 1, K, codes);
    for (int m = 0; m < M; m++) {
      double s = (double)orc_f16_to_f32(scale_f16[m]);
      double acc = 0.0, mag = 0.0;
      for (int j = 0; j < NG; j++) {
        long long Sc[4] = {0, 0, 0, 0};
        for (int k = j * G; k < (j + 1) * G; k++) Sc[codes[k]] += (long long)q[(size_t)m * K + k];
        for (int c = 0; c < 4; c++) {
          double L = (double)orc_f16_to_f32(lut_f16[((size_t)n * NG + j) * 4 + c]);
          if (S) S[(((size_t)m * N + n) * NG + j) * 4 + c] = (int32_t)Sc[c];
          acc += L * (double)Sc[c];
          mag += std::fabs(L) * std::fabs((double)Sc[c]);
        }
      }
      y_ref[(size_t)m * N + n] = s * acc;
      if (tol) tol[(size_t)m * N + n] = 2e-3 * (s * mag) + 1e-5;
    }
  }
  std::free(codes);
  std::free(q);
  return 0;
}

// Direct form with a grid per group: y = s_m * sum_k LUT[n][k / G][code[n][k]] * q[m][k], in
// double, and the same sum as an exact integer with every level scaled by 2^24.
int orc_gemv_direct_grouped(const uint32_t* words, const uint16_t* lut_f16, const uint8_t* xq,
                            const uint16_t* scale_f16, int M, int N, int K, int G,
                            double* y_direct, long long* acc_int) {
  if (M < 1 || N < 1 || K < 16 || K % 16 || G < 1 || K % G) return -1;
  const int NG = K / G;
  uint8_t* codes = (uint8_t*)std::malloc((size_t)K);
  int8_t* q = (int8_t*)std::malloc((size_t)M * K);
  orc_unpack_act(xq, (size_t)M * (K / 2), q);
  for (int n = 0; n < N; n++) {
    orc_unpack_weights(words + (size_t)n * (K / 16), 1, K, codes);
    for (int m = 0; m < M; m++) {
      double acc = 0.0;
      long long ai = 0;
      for (int k = 0; k < K; k++) {
        double L = (double)orc_f16_to_f32(lut_f16[((size_t)n * NG + k / G) * 4 + codes[k]]);
        int qq = q[(size_t)m * K + k];
        acc += L * (double)qq;
        ai += (long long)std::ldexp(L, 24) * (long long)qq;
      }
      y_direct[(size_t)m * N + n] = (double)orc_f16_to_f32(scale_f16[m]) * acc;
      if (acc_int) acc_int[(size_t)m * N + n] = ai;
    }
  }
  std::free(codes);
  std::free(q);
  return 0;
}

// The same exact integer from the per-group per-code sums: sum_j sum_c Lint[n][j][c] * S_c[m][n][j].
void orc_percode_int_grouped(const uint16_t* lut_f16, const int32_t* S, int M, int N, int NG, long long* acc_int) {
  for (int m = 0; m < M; m++)
    for (int n = 0; n < N; n++) {
      long long ai = 0;
      for (int j = 0; j < NG; j++)
        for (int c = 0; c < 4; c++) {
          long long Li = (long long)std::ldexp((double)orc_f16_to_f32(lut_f16[((size_t)n * NG + j) * 4 + c]), 24);
          ai += Li * (long long)S[(((size_t)m * N + n) * NG + j) * 4 + c];
        }
      acc_int[(size_t)m * N + n] = ai;
    }
}

// ---------------------------------------------------------------------------------------
// Learnable direct partitioning, export of a trained layer to the kernel's inputs (Section 4.3,
// Eqs. "partition", the grid t_i, "quant", "dequantgrid" and Section 4.4 Eq. "deqgrid"; clipping
// range from Section 4.2). One quantization unit = G consecutive weights of a row. Per unit, in
// fp32 with one rounding per operation (the precision the export kernel works in):
//   lo = sb * min(W_r), hi = sg * max(W_r), h = hi - lo      (sb, sg: the sigmoids of beta, gamma)
//   W_rc = clip(W_r, lo, hi)
//   p1 = s1, p2 = (1 - p1) s2, p3 = (1 - p1)(1 - s2)         (s1, s2: the sigmoids of s_1, s_2)
//   t1 = p1 / 2, t2 = t1 + (p1 + p2) / 2, t3 = t2 + (p2 + p3) / 2
//   code = u(x - t1) + u(x - t2) + u(x - t3), x = (W_rc - lo) / h, u(z) = 1 for z >= 0 else 0
//   w0 = 0, w1 = (t1 + t2) / 2, w2 = (t2 + t3) / 2, w3 = 1;  LUT_i = fp16(lo + h w_i)
// Readings: the normalized weight is taken relative to the range minimum (Eq. "quant" prints W/h,
// Eq. "dequant" offsets the levels by the minimum: only the offset form puts the thresholds
// inside the range); the step function counts z = 0 as reached; a unit with h <= 0 gets code 0
// everywhere and four levels equal to lo. The sigmoids are inputs (the caller evaluates them),
// so that both sides work from identical fp32 numbers.
// Inputs: w_f16 [N][K], sb, sg, s1, s2 float [N][K/G]. Outputs: codes u8 [N][K], lut fp16 bits
// [N][K/G][4]. Returns 0, -1 bad shape.
// ---------------------------------------------------------------------------------------
int orc_ldp_export(const uint16_t* w_f16, const float* sb, const float* sg, const float* s1, const float* s2,
                   int N, int K, int G, uint8_t* codes, uint16_t* lut_f16) {
  if (N < 1 || K < 1 || G < 1 || K % G) return -1;
  const int NG = K / G;
  for (int n = 0; n < N; n++)
    for (int j = 0; j < NG; j++) {
      const uint16_t* w = w_f16 + (size_t)n * K + (size_t)j * G;
      const size_t u = (size_t)n * NG + j;
      float wmin = orc_f16_to_f32(w[0]), wmax = wmin;
      for (int k = 1; k < G; k++) {
        float v = orc_f16_to_f32(w[k]);
        if (v < wmin) wmin = v;
        if (v > wmax) wmax = v;
      }
      volatile float lo = sb[u] * wmin;
      volatile float hi = sg[u] * wmax;
      volatile float h = hi - lo;
      volatile float p1 = s1[u];
      volatile float rest = 1.0f - p1;
      volatile float p2 = rest * s2[u];
      volatile float one_m = 1.0f - s2[u];
      volatile float p3 = rest * one_m;
      volatile float t1 = p1 / 2.0f;
      volatile float p12 = p1 + p2;
      volatile float h12 = p12 / 2.0f;
      volatile float t2 = t1 + h12;
      volatile float p23 = p2 + p3;
      volatile float h23 = p23 / 2.0f;
      volatile float t3 = t2 + h23;
      volatile float s12 = t1 + t2;
      volatile float w1 = s12 / 2.0f;
      volatile float s23 = t2 + t3;
      volatile float w2 = s23 / 2.0f;
      const float lv[4] = {0.0f, w1, w2, 1.0f};
      const bool ok = h > 0.0f;
      for (int c = 0; c < 4; c++) {
        volatile float prod = h * lv[c];
        volatile float level = lo + prod;
        lut_f16[u * 4 + c] = orc_f32_to_f16(ok ? (float)level : (float)lo);
      }
      for (int k = 0; k < G; k++) {
        int code = 0;
        if (ok) {
          float v = orc_f16_to_f32(w[k]);
          if (v < lo) v = lo;
          if (v > hi) v = hi;
          volatile float d = v - lo;
          volatile float x = d / h;
          code = (x >= t1) + (x >= t2) + (x >= t3);
        }
        codes[(size_t)n * K + (size_t)j * G + k] = (uint8_t)code;
      }
    }
  return 0;
}

// ---------------------------------------------------------------------------------------
// 3-bit weights (Section 4.3, paragraph "Application of LDP on NF3 format"; Table "memory", W3
// column). The same look-up-table GEMV with eight levels per quantization unit instead of four.
//
// Packing. A code c in 0..7 is split into its low two bits, stored exactly like a 2-bit code
// (words2 [N][K/16], code 16w+j in bits [2j, 2j+1]), and its top bit, stored in a bit plane of
// its own: words1 [N][K/32], where word v covers the codes 32v .. 32v+31 and holds the top bit
// of code 32v + i in bit 2i and of code 32v + 16 + i in bit 2i+1 (i = 0..15). Three bits per
// code in all. (The paper prints no W3 layout; this one is this implementation's.)
// ---------------------------------------------------------------------------------------
int orc_pack_weights3(const uint8_t* codes, int N, int K, uint32_t* words2, uint32_t* words1) {
  if (N < 1 || K < 32 || K % 32) return -1;
  for (int n = 0; n < N; n++) {
    for (int w = 0; w < K / 16; w++) {
      uint32_t word = 0;
      for (int j = 0; j < 16; j++) {
        const uint8_t c = codes[(size_t)n * K + 16 * w + j];
        if (c > 7) return -4;
        word |= (uint32_t)(c & 3u) << (2 * j);
      }
      words2[(size_t)n * (K / 16) + w] = word;
    }
    for (int v = 0; v < K / 32; v++) {
      uint32_t word = 0;
      for (int i = 0; i < 16; i++) {
        word |= (uint32_t)((codes[(size_t)n * K + 32 * v + i] >> 2) & 1u) << (2 * i);
        word |= (uint32_t)((codes[(size_t)n * K + 32 * v + 16 + i] >> 2) & 1u) << (2 * i + 1);
      }
      words1[(size_t)n * (K / 32) + v] = word;
    }
  }
  return 0;
}

// Inverse of the packing, written independently of it: code k of a row from its two words.
void orc_unpack_weights3(const uint32_t* words2, const uint32_t* words1, int N, int K, uint8_t* codes) {
  for (int n = 0; n < N; n++)
    for (int k = 0; k < K; k++) {
      const uint32_t lo2 = (words2[(size_t)n * (K / 16) + k / 16] >> (2 * (k % 16))) & 3u;
      const int r = k % 32;                                  // place inside the 32 codes of a plane word
      const int bit = (r < 16) ? 2 * r : 2 * (r - 16) + 1;
      const uint32_t top = (words1[(size_t)n * (K / 32) + k / 32] >> bit) & 1u;
      codes[(size_t)n * K + k] = (uint8_t)(lo2 | (top << 2));
    }
}

// W3A4 look-up-table GEMV, one eight-entry grid per group of G weights of a row (G = K: one per row).
//   S_c[m][n][j] = sum over k in group j with code[n][k] == c of q[m][k]          (exact integers)
//   y_ref        = s_m * sum_j sum_c LUT[n][j][c] * S_c[m][n][j]                   (double)
//   tol          = 2e-3 * ( s_m * sum_j sum_c |LUT[n][j][c]| * |S_c| ) + 1e-5
// S int32 [M][N][K/G][8] (may be NULL). Returns 0; -1 bad shape.
int orc_gemv_w3a4(const uint32_t* words2, const uint32_t* words1, const uint16_t* lut_f16, const uint8_t* xq,
                  const uint16_t* scale_f16, int M, int N, int K, int G, int32_t* S, double* y_ref, double* tol) {
  if (M < 1 || N < 1 || K < 32 || K % 32 || G < 1 || K % G) return -1;
  const int NG = K / G;
  uint8_t* codes = (uint8_t*)std::malloc((size_t)K);
  int8_t* q = (int8_t*)std::malloc((size_t)M * K);
  orc_unpack_act(xq, (size_t)M * (K / 2), q);
  for (int n = 0; n < N; n++) {
    orc_unpack_weights3(words2 + (size_t)n * (K / 16), words1 + (size_t)n * (K / 32), 1, K, codes);
    for (int m = 0; m < M; m++) {
      const double s = (double)orc_f16_to_f32(scale_f16[m]);
      double acc = 0.0, mag = 0.0;
      for (int j = 0; j < NG; j++) {
        long long Sc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int k = j * G; k < (j + 1) * G; k++) Sc[codes[k]] += (long long)q[(size_t)m * K + k];
        for (int c = 0; c < 8; c++) {
          const double L = (double)orc_f16_to_f32(lut_f16[((size_t)n * NG + j) * 8 + c]);
          if (S) S[(((size_t)m * N + n) * NG + j) * 8 + c] = (int32_t)Sc[c];
          acc += L * (double)Sc[c];
          mag += std::fabs(L) * std::fabs((double)Sc[c]);
        }
      }
      y_ref[(size_t)m * N + n] = s * acc;
      if (tol) tol[(size_t)m * N + n] = 2e-3 * (s * mag) + 1e-5;
    }
  }
  std::free(codes);
  std::free(q);
  return 0;
}

// Direct form of the same product with every fp16 level scaled by 2^24 (exact integers):
// acc_int[m][n] = sum_k Lint[n][k / G][code[n][k]] * q[m][k]. For the check that the per-code form
// and the direct form are the same number.
int orc_gemv_w3a4_direct_int(const uint32_t* words2, const uint32_t* words1, const uint16_t* lut_f16,
                             const uint8_t* xq, int M, int N, int K, int G, long long* acc_int) {
  if (M < 1 || N < 1 || K < 32 || K % 32 || G < 1 || K % G) return -1;
  const int NG = K / G;
  uint8_t* codes = (uint8_t*)std::malloc((size_t)K);
  int8_t* q = (int8_t*)std::malloc((size_t)M * K);
  orc_unpack_act(xq, (size_t)M * (K / 2), q);
  for (int n = 0; n < N; n++) {
    orc_unpack_weights3(words2 + (size_t)n * (K / 16), words1 + (size_t)n * (K / 32), 1, K, codes);
    for (int m = 0; m < M; m++) {
      long long acc = 0;
      for (int k = 0; k < K; k++) {
        const double L = (double)orc_f16_to_f32(lut_f16[((size_t)n * NG + k / G) * 8 + codes[k]]);
        acc += (long long)std::ldexp(L, 24) * (long long)q[(size_t)m * K + k];
      }
      acc_int[(size_t)m * N + n] = acc;
    }
  }
  std::free(codes);
  std::free(q);
  return 0;
}

// Export of a 3-bit layer (paragraph "Application of LDP on NF3 format", Eq. "nf3scales", Eq. "nf3").
// Per quantization unit (G consecutive weights of a row), fp32 arithmetic, one rounding per operation:
//   lo = sigma(beta) min(W), hi = sigma(gamma) max(W), h = hi - lo, W clipped to [lo, hi]
//   c  = lo + h sigma(s_1)                       the learnable centre
//   s_neg = |c - lo|,  s_pos = |hi - c|          Eq. "nf3scales"
//   v  = (W - c) / s_pos if W > c, else (W - c) / s_neg            in [-1, 1]
//   code = index of the level of the format nearest to v, searched among the levels of v's side
//   level_i = c + T_i * (s_pos if T_i > 0 else s_neg), rounded to fp16
// The format is a table T of eight ascending normalized levels with T[zero_index] == 0 (three bits:
// the asymmetric normal-float format has three negative levels, zero, four positive ones, its end levels
// -1 and 1). Readings: Eq. "nf3" prints a round-to-nearest of the normalized weight and the text says the
// result is multiplied by the scale and offset by c, so "rounding" is to the nearest representable level
// of the format, not to an integer; the paper takes the level values from the format's own publication
// and prints none, so the table is an argument here; a weight exactly between two levels takes the lower
// one; a weight equal to c belongs to the negative side ("otherwise"); h <= 0 gives code zero_index and
// eight levels equal to lo. Sigmoids are inputs, as for the 2-bit export.
// codes u8 [N][K], lut fp16 bits [N][K/G][8]. Returns 0; -1 bad shape; -2 bad table.
int orc_nf3_export(const uint16_t* w_f16, const float* sb, const float* sg, const float* s1, const float* table,
                   int zero_index, int N, int K, int G, uint8_t* codes, uint16_t* lut_f16) {
  if (N < 1 || K < 1 || G < 1 || K % G) return -1;
  if (zero_index < 0 || zero_index > 7 || table[zero_index] != 0.0f) return -2;
  for (int i = 1; i < 8; i++) if (!(table[i] > table[i - 1])) return -2;
  const int NG = K / G;
  for (int n = 0; n < N; n++)
    for (int j = 0; j < NG; j++) {
      const uint16_t* w = w_f16 + (size_t)n * K + (size_t)j * G;
      const size_t u = (size_t)n * NG + j;
      float wmin = orc_f16_to_f32(w[0]), wmax = wmin;
      for (int k = 1; k < G; k++) {
        float v = orc_f16_to_f32(w[k]);
        if (v < wmin) wmin = v;
        if (v > wmax) wmax = v;
      }
      volatile float lo = sb[u] * wmin;
      volatile float hi = sg[u] * wmax;
      volatile float h = hi - lo;
      volatile float off = h * s1[u];
      volatile float c = lo + off;
      volatile float dn = c - lo;
      volatile float dp = hi - c;
      const float s_neg = std::fabs((float)dn), s_pos = std::fabs((float)dp);
      const bool ok = h > 0.0f;
      for (int i = 0; i < 8; i++) {
        volatile float prod = table[i] * (i > zero_index ? s_pos : s_neg);
        volatile float level = c + prod;
        lut_f16[u * 8 + i] = orc_f32_to_f16(ok ? (float)level : (float)lo);
      }
      for (int k = 0; k < G; k++) {
        int code = zero_index;
        if (ok) {
          float v = orc_f16_to_f32(w[k]);
          if (v < lo) v = lo;
          if (v > hi) v = hi;
          volatile float d = v - c;
          const bool pos = v > c;
          const float sc = pos ? s_pos : s_neg;
          if (sc > 0.0f) {
            volatile float x = d / sc;
            const int first = pos ? zero_index : 0, last = pos ? 7 : zero_index;
            code = first;
            float best = std::fabs((float)x - table[first]);
            for (int i = first + 1; i <= last; i++) {
              volatile float diff = (float)x - table[i];
              const float dist = std::fabs((float)diff);
              if (dist < best) { best = dist; code = i; }   // strict: a tie keeps the lower level
            }
          }
        }
        codes[(size_t)n * K + (size_t)j * G + k] = (uint8_t)code;
      }
    }
  return 0;
}

// ---------------------------------------------------------------------------------------
// Weight-only variant (Section 5, "W2-only setting", Table "W2_inference": the GEMV with the
// 2-bit codes and the dequantization grid of Section 4.4 but activations left in 16-bit floating
// point). The plain definition, in double, the sum over k taken in order:
//   y[m][n]    = sum_k LUT[n][code[n][k]] * x[m][k]
//   labsx[m][n] = sum_k |LUT[n][code[n][k]]| * |x[m][k]|     (magnitude the tolerance refers to)
//   labs[n]    = sum_k |LUT[n][code[n][k]]|
// x is fp16 [M][K]. Returns 0; -1 bad shape.
// ---------------------------------------------------------------------------------------
int orc_gemv_w2a16(const uint32_t* words, const uint16_t* lut_f16, const uint16_t* x_f16, int M, int N, int K,
                   double* y, double* labsx, double* labs) {
  if (M < 1 || N < 1 || K < 16 || K % 16) return -1;
  uint8_t* codes = (uint8_t*)std::malloc((size_t)K);
  for (int n = 0; n < N; n++) {
    orc_unpack_weights(words + (size_t)n * (K / 16), 1, K, codes);
    double L[4];
    for (int c = 0; c < 4; c++) L[c] = (double)orc_f16_to_f32(lut_f16[(size_t)n * 4 + c]);
    double la = 0.0;
    for (int k = 0; k < K; k++) la += std::fabs(L[codes[k]]);
    if (labs) labs[n] = la;
    for (int m = 0; m < M; m++) {
      double acc = 0.0, mag = 0.0;
      for (int k = 0; k < K; k++) {
        const double xv = (double)orc_f16_to_f32(x_f16[(size_t)m * K + k]);
        acc += L[codes[k]] * xv;
        mag += std::fabs(L[codes[k]]) * std::fabs(xv);
      }
      y[(size_t)m * N + n] = acc;
      if (labsx) labsx[(size_t)m * N + n] = mag;
    }
  }
  std::free(codes);
  return 0;
}

// Per-code sums of signed 8-bit activation planes (Section 4.4: the accumulation respects the grid, one
// sum per code). For plane j (a row of K signed bytes) and output row n:
//   S[j][n][c] = sum over k with code[n][k] == c of a[j][k]
// The weight-only form feeds the GEMV kernels the four digit planes of a token; this is what their
// integer sums must equal. a int8 [C][K], S int32 [C][N][4]. Returns 0; -1 bad shape.
int orc_percode_sums_i8(const uint32_t* words, const int8_t* a, int C, int N, int K, int32_t* S) {
  if (C < 1 || N < 1 || K < 16 || K % 16) return -1;
  uint8_t* codes = (uint8_t*)std::malloc((size_t)K);
  for (int n = 0; n < N; n++) {
    orc_unpack_weights(words + (size_t)n * (K / 16), 1, K, codes);
    for (int j = 0; j < C; j++) {
      long long Sc[4] = {0, 0, 0, 0};
      for (int k = 0; k < K; k++) Sc[codes[k]] += (long long)a[(size_t)j * K + k];
      for (int c = 0; c < 4; c++) S[((size_t)j * N + n) * 4 + c] = (int32_t)Sc[c];
    }
  }
  std::free(codes);
  return 0;
}

// Block fixed point of a token of fp16 activations, as base-64 digits (an encoding chosen by this
// implementation of the weight-only variant, not by the paper: it lets 16-bit activations run
// through exact 8-bit integer dot products). Per token m, with E = floor(log2(max_k |x[m][k]|))
// (E = 0 for an all-zero token):
//   X[k]   = round-half-even( x[m][k] * 2^(21 - E) )              an integer, |X| < 2^22
//   X[k]   = sum_{d=0..3} 64^d * q_d[k],  q_0..q_2 in [-32, 31] taken least significant first,
//            q_3 what remains (within [-16, 16])
//   unit_d = 2^(E - 21) * 64^d
// digits int8 [M][4][K] (digit-major per token), unit double [M][4]. Returns 0; -1 bad shape;
// -2 if an activation is not finite.
int orc_split_act16(const uint16_t* x_f16, int M, int K, int8_t* digits, double* unit) {
  if (M < 1 || K < 1) return -1;
  for (int m = 0; m < M; m++) {
    double amax = 0.0;
    for (int k = 0; k < K; k++) {
      const double v = std::fabs((double)orc_f16_to_f32(x_f16[(size_t)m * K + k]));
      if (!(v <= 65504.0)) return -2;
      if (v > amax) amax = v;
    }
    int E = 0;
    if (amax > 0.0) {
      int e2 = 0;
      (void)std::frexp(amax, &e2);   // amax = f * 2^e2 with f in [0.5, 1)
      E = e2 - 1;
    }
    for (int d = 0; d < 4; d++) unit[(size_t)m * 4 + d] = std::ldexp(1.0, E - 21 + 6 * d);
    for (int k = 0; k < K; k++) {
      const double v = (double)orc_f16_to_f32(x_f16[(size_t)m * K + k]);
      long long X = (long long)std::nearbyint(std::ldexp(v, 21 - E));   // default rounding mode: half to even
      for (int d = 0; d < 4; d++) {
        long long q;
        if (d < 3) {
          q = ((X + 32) % 64 + 64) % 64 - 32;   // the residue of X in [-32, 31]
          X = (X - q) / 64;
        } else {
          q = X;
        }
        digits[((size_t)m * 4 + d) * K + k] = (int8_t)q;
      }
    }
  }
  return 0;
}

}  // extern "C"
