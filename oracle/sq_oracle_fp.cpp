// CPU oracle for the floating-point variant of the SQ-format hot path.  TEST INFRASTRUCTURE ONLY
// (see sq_oracle.cpp: same rules -- never linked into or called from the product path).
//
// Section 3.1 defines the format for floating-point precisions as well as integer ones, and the
// appendix "FP Quantization Results" reports h_high = FP8, h_low = FP4.  This file applies that
// pair to the path the integer oracle covers: activations in SQ-format (sparse FP8 E4M3 entries,
// dense FP4 E2M1 elsewhere) times FP4 per-output-channel weights.
//
// Number formats (OCP 8-bit / 4-bit floating point):
//   E2M1  4 bits: sign, 2 exponent bits (bias 1), 1 mantissa bit; magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6
//   E4M3  8 bits: sign, 4 exponent bits (bias 7), 3 mantissa bits; no infinities, largest finite 448,
//         smallest subnormal 2^-9; the two all-ones-mantissa codes of the top exponent are NaN
// Rounding: to the nearest representable value, ties to the neighbour with an even code (even
// mantissa), magnitudes beyond the largest finite value saturate to it.  Written as a search over
// the table of representable values so that it can be read off this definition.
//
// Readings (the paper fixes none of this for activations):
//   * per-token scales on ONE grid, as in the integer oracle: s_hi = amax / 256 (the row maximum
//     maps to 256, not to 448, so that every dense value times its power-of-two shift is still an
//     E4M3 number), s_lo = s_hi * 2^e with e = the smallest shift in 0..6 that brings the largest
//     unselected magnitude to at most 6;
//   * the product the GEMM computes is defined on the MERGED operand a8[m,j] = E4M3(dense * 2^e) at
//     dense places (exact) and the sparse entry at selected ones, times the weights' E2M1 values,
//     summed exactly (every product is a multiple of 2^-10 and the sum stays below 2^29: exact in
//     fp64), rounded once to fp32, then scaled: ref32 = ((float)acc * s_hi[m]) * s_w[n];
//   * weights: s_w = wmax / 6, code = E2M1(w * (6 / wmax)), per output channel.
// Parity status: every function is pinned by tests/test_oracle_fp_pins.py (enumerated tables,
// a library conversion for E4M3, exact rationals, brute force); none is "parity unpinned".
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

inline float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}
inline uint16_t f32_to_bf16(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

// value of a magnitude code (sign bit stripped)
double e2m1_mag(unsigned c) {  // c in 0..7: exponent c >> 1, mantissa c & 1
  const unsigned e = c >> 1, m = c & 1u;
  return e == 0 ? 0.5 * m : std::ldexp(1.0 + 0.5 * m, (int)e - 1);
}
double e4m3_mag(unsigned c) {  // c in 0..0x7E: exponent c >> 3, mantissa c & 7
  const unsigned e = c >> 3, m = c & 7u;
  return e == 0 ? std::ldexp((double)m, -9) : std::ldexp(1.0 + m / 8.0, (int)e - 7);
}

// nearest magnitude code among 0..max_code (values ascending with the code), ties to the even code
template <typename F>
unsigned round_mag(double a, unsigned max_code, F value) {
  if (a >= value(max_code)) return max_code;  // saturate
  unsigned lo = 0;
  while (value(lo + 1) <= a) ++lo;            // value(lo) <= a < value(lo + 1)
  const double dlo = a - value(lo), dhi = value(lo + 1) - a;
  if (dlo < dhi) return lo;
  if (dhi < dlo) return lo + 1;
  return (lo & 1u) ? lo + 1 : lo;
}
unsigned e2m1_round(double v) {
  const unsigned s = std::signbit(v) ? 8u : 0u;
  return s | round_mag(std::fabs(v), 7u, e2m1_mag);
}
unsigned e4m3_round(double v) {
  const unsigned s = std::signbit(v) ? 0x80u : 0u;
  return s | round_mag(std::fabs(v), 0x7Eu, e4m3_mag);
}
double e2m1_value(unsigned code) { return (code & 8u) ? -e2m1_mag(code & 7u) : e2m1_mag(code & 7u); }
double e4m3_value(unsigned code) { return (code & 0x80u) ? -e4m3_mag(code & 0x7Fu) : e4m3_mag(code & 0x7Fu); }

template <typename T>
void topk_bank(const T* score, int b, int k, uint8_t* out_sorted) {
  std::vector<char> taken(b, 0);
  for (int pick = 0; pick < k; ++pick) {
    int best = -1;
    for (int j = 0; j < b; ++j) {
      if (taken[j]) continue;
      if (best < 0 || score[j] > score[best]) best = j;
    }
    taken[best] = 1;
  }
  int n = 0;
  for (int j = 0; j < b; ++j)
    if (taken[j]) out_sorted[n++] = (uint8_t)j;
}

}  // namespace

extern "C" {

// Tables of representable values (for the pins): e2m1[16], e4m3[256] (NaN codes hold NaN).
void sqo_fp_tables(double* e2m1, double* e4m3) {
  for (unsigned c = 0; c < 16; ++c) e2m1[c] = e2m1_value(c);
  for (unsigned c = 0; c < 256; ++c) e4m3[c] = (c & 0x7Fu) == 0x7Fu ? NAN : e4m3_value(c);
}
// kind 0: E2M1, 1: E4M3.
void sqo_fp_round(int kind, const double* in, long n, uint8_t* out) {
  for (long i = 0; i < n; ++i) out[i] = (uint8_t)(kind == 0 ? e2m1_round(in[i]) : e4m3_round(in[i]));
}

// Per-output-channel FP4 weights.
//   wmax = max_j |W[n,j]|; c = 6.0f / wmax, s_w = wmax / 6.0f (fp32 divisions); zero channel: codes 0, s_w 0
//   code[n,j] = E2M1(W[n,j] * c) on the exact product; wq4[n, j/2]: element 2*(j/2) low nibble, next one high
//   w8[n,j] = the same value as an E4M3 code (every E2M1 value is an E4M3 value)
void sqo_fp_pack_weights(const uint16_t* W, long N, long K, uint8_t* wq4, float* s_w, uint8_t* w8 /*or NULL*/) {
#pragma omp parallel for schedule(static)
  for (long n = 0; n < N; ++n) {
    float wmax = 0.f;
    for (long j = 0; j < K; ++j) wmax = std::fmax(wmax, std::fabs(bf16_to_f32(W[n * K + j])));
    const float c = wmax > 0.f ? 6.0f / wmax : 0.f;
    s_w[n] = wmax > 0.f ? wmax / 6.0f : 0.f;
    std::vector<unsigned> q(K);
    for (long j = 0; j < K; ++j) q[j] = wmax > 0.f ? e2m1_round((double)bf16_to_f32(W[n * K + j]) * (double)c) : 0u;
    for (long j = 0; j < K; ++j) q[j] = (q[j] & 7u) ? q[j] : 0u;  // a rounded-to-zero value is +0
    for (long j = 0; j < K; j += 2) wq4[n * (K / 2) + j / 2] = (uint8_t)(q[j] | (q[j + 1] << 4));
    if (w8)
      for (long j = 0; j < K; ++j) w8[n * K + j] = (uint8_t)e4m3_round(e2m1_value(q[j]));
  }
}

// Activation encode, one token row at a time (positions == NULL: per bank the k largest |a_j|,
// ties to the smaller index; else the given static positions).
//   amax == 0: every code 0, shift 0, scales 0.  Otherwise
//   inv = 256.0f / amax, s_hi = amax / 256.0f (fp32 divisions)
//   j in S:     vals = E4M3(a_j * inv)                          (|a_j * inv| <= 256)
//   rmax = max over j not in S of |a_j|;  e = min{e in 0..6 : rmax * inv * 2^-e <= 6};  s_lo = s_hi * 2^e
//   j not in S: dense = E2M1(a_j * inv * 2^-e); dense code 0 at selected places
//   a8[m,j] = E4M3(value(dense) * 2^e) (exact) at dense places, vals at selected ones
void sqo_fp_encode(int b, int k, const uint16_t* X, long M, long K, const uint8_t* positions, uint8_t* dq4,
                   uint8_t* vals, uint8_t* idx /*NULL if static*/, float* s_hi, float* s_lo, uint8_t* shift,
                   uint8_t* a8 /*[M,K] or NULL*/) {
  const long G = K / b;
#pragma omp parallel for schedule(static)
  for (long m = 0; m < M; ++m) {
    std::vector<float> a(K), mag(K);
    std::vector<char> inS(K, 0);
    std::vector<uint8_t> sel(G * k);
    float amax = 0.f;
    for (long j = 0; j < K; ++j) {
      a[j] = bf16_to_f32(X[m * K + j]);
      mag[j] = std::fabs(a[j]);
      if (mag[j] > amax) amax = mag[j];
    }
    for (long g = 0; g < G; ++g) {
      if (positions)
        for (int i = 0; i < k; ++i) sel[g * k + i] = positions[g * k + i];
      else
        topk_bank(&mag[g * b], b, k, &sel[g * k]);
      for (int i = 0; i < k; ++i) inS[g * b + sel[g * k + i]] = 1;
    }
    float rmax = 0.f;
    for (long j = 0; j < K; ++j)
      if (!inS[j] && mag[j] > rmax) rmax = mag[j];
    int e = 0;
    float inv = 0.f, sh = 0.f;
    if (amax > 0.f) {
      inv = 256.0f / amax;
      sh = amax / 256.0f;
      e = 6;
      for (int t = 0; t <= 6; ++t)
        if ((double)rmax * (double)std::ldexp(inv, -t) <= 6.0) { e = t; break; }
    }
    s_hi[m] = sh;
    s_lo[m] = std::ldexp(sh, e);
    shift[m] = (uint8_t)e;
    const float inv_lo = std::ldexp(inv, -e);
    std::vector<unsigned> dense(K, 0u);
    for (long j = 0; j < K; ++j)
      if (!inS[j] && amax > 0.f) {
        dense[j] = e2m1_round((double)a[j] * (double)inv_lo);
        if ((dense[j] & 7u) == 0) dense[j] = 0;  // a rounded-to-zero value is +0
      }
    for (long j = 0; j < K; j += 2) dq4[m * (K / 2) + j / 2] = (uint8_t)(dense[j] | (dense[j + 1] << 4));
    if (a8)
      for (long j = 0; j < K; ++j) a8[m * K + j] = (uint8_t)e4m3_round(std::ldexp(e2m1_value(dense[j]), e));
    for (long g = 0; g < G; ++g)
      for (int i = 0; i < k; ++i) {
        const long j = g * b + sel[g * k + i];
        unsigned q = amax > 0.f ? e4m3_round((double)a[j] * (double)inv) : 0u;
        if ((q & 0x7Fu) == 0) q = 0;
        vals[(m * G + g) * k + i] = (uint8_t)q;
        if (idx) idx[(m * G + g) * k + i] = sel[g * k + i];
        if (a8) a8[m * K + j] = (uint8_t)q;
      }
  }
}

// GEMM + dequant epilogue on the merged operand.
//   acc[m,n]   = sum_j value_e4m3(a8[m,j]) * value_e2m1(wq4[n,j])     exact (fp64), rounded once to fp32
//   ref32[m,n] = (acc * s_hi[m]) * s_w[n];  out = bf16_rne(ref32)
// abs_out (or NULL): sum_j |a8| * |w| in the same units, the quantity the accumulation-order
// tolerance of the GPU comparison is stated in.
void sqo_fp_gemm(const uint8_t* a8, const float* s_hi, const uint8_t* wq4, const float* s_w, long M, long N, long K,
                 const long* rows, long n_rows, const long* cols, long n_cols, float* acc_out, float* abs_out,
                 float* ref32_out, uint16_t* out_bf16) {
  const long R = rows ? n_rows : M, C = cols ? n_cols : N;
#pragma omp parallel for schedule(static)
  for (long r = 0; r < R; ++r) {
    const long m = rows ? rows[r] : r;
    std::vector<double> av(K);
    for (long j = 0; j < K; ++j) av[j] = e4m3_value(a8[m * K + j]);
    for (long c = 0; c < C; ++c) {
      const long n = cols ? cols[c] : c;
      double acc = 0.0, sabs = 0.0;
      for (long j = 0; j < K; ++j) {
        const unsigned byte = wq4[n * (K / 2) + j / 2];
        const double w = e2m1_value((j & 1) ? (byte >> 4) : (byte & 0xFu));
        acc += av[j] * w;
        sabs += std::fabs(av[j] * w);
      }
      const float acc32 = (float)acc;
      const float ref = (acc32 * s_hi[m]) * s_w[n];
      if (acc_out) acc_out[r * C + c] = acc32;
      if (abs_out) abs_out[r * C + c] = (float)sabs;
      if (ref32_out) ref32_out[r * C + c] = ref;
      if (out_bf16) out_bf16[r * C + c] = f32_to_bf16(ref);
    }
  }
}

// Decode (inverse of Eq. 1): s_hi * value(vals) at selected places, s_lo * value(dense) elsewhere.
void sqo_fp_decode(int b, int k, const uint8_t* dq4, const uint8_t* vals, const uint8_t* idx, const uint8_t* positions,
                   const float* s_hi, const float* s_lo, long M, long K, float* out_f32, uint16_t* out_bf16) {
  const long G = K / b;
#pragma omp parallel for schedule(static)
  for (long m = 0; m < M; ++m) {
    std::vector<float> x(K);
    for (long j = 0; j < K; ++j) {
      const unsigned byte = dq4[m * (K / 2) + j / 2];
      x[j] = s_lo[m] * (float)e2m1_value((j & 1) ? (byte >> 4) : (byte & 0xFu));
    }
    for (long g = 0; g < G; ++g)
      for (int i = 0; i < k; ++i) {
        const int local = idx ? idx[(m * G + g) * k + i] : positions[g * k + i];
        x[g * b + local] = s_hi[m] * (float)e4m3_value(vals[(m * G + g) * k + i]);
      }
    for (long j = 0; j < K; ++j) {
      if (out_f32) out_f32[m * K + j] = x[j];
      if (out_bf16) out_bf16[m * K + j] = f32_to_bf16(x[j]);
    }
  }
}

}  // extern "C"
