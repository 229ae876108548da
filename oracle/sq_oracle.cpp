// CPU oracle for the SQ-format hot path.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, obviously-correct implementation of what the path computes:
// static position selection, weight packing, activation encoding, the hybrid
// integer GEMM with its dequantising epilogue, and decoding.  It exists so the
// CUDA kernels can be compared against something written straight from the
// paper; it shares no code, header, table or helper with the CUDA library and
// must never be linked into or called from the product path.  Only the test
// suite, the smoke check and the benchmark's CPU-baseline leg may use it.
//
// What each function follows (SQ-format paper, arXiv 2512.05409):
//   * format tuple, banks of size b, fixed count k = (1-s)*b of high-precision
//     entries per bank: Section 3.1, Eq. 1;
//   * symmetric integer codes that leave the most negative code unused
//     (INT4 in [-7,7], INT8 in [-127,127]): Section 3.2.1;
//   * dynamic activation split = per token, per bank Top-K of |activation|:
//     Section 3.2.2 and Section 3.3;
//   * static activation split = per bank top (1-s) of I_j = |A_j * sum_i W_ij|:
//     Section 3.2.2, Algorithm 2;
//   * hybrid GEMM = dense low-precision product + sparse high-precision
//     product into one result: Section 1 and Section 3.3 (Fig. 2b);
//   * independent-scale variant: separate scales for the high- and the
//     low-precision part, Algorithm 1 (S_high, S_low).
// Points on which the paper is silent (scale granularity, tie-breaks, rounding
// mode, ...) follow the readings listed in the repository's design notes; every
// one of them is restated next to the code that implements it.
//
// Parity status: every function below is pinned by the CPU tests (brute force,
// closed forms, special cases that reduce to textbook quantisers); none is
// "parity unpinned".
//
// No blocking, fusion or reordering: loops run in the order the definition
// states.  OpenMP only splits independent rows/channels across cores.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

#if defined(_OPENMP)
#include <omp.h>
#endif

namespace {

inline float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

// fp32 -> bf16, round to nearest even (finite inputs).
inline uint16_t f32_to_bf16(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return (uint16_t)(u >> 16);
}

// Round-half-to-even of the EXACT real product a*c.  a carries at most 8
// significant bits (it came from bf16) and c at most 24, so the double product
// is exact and nearbyint() in the default rounding mode is the single rounding.
inline long rne_prod(float a, float c) { return (long)std::nearbyint((double)a * (double)c); }

inline long clampl(long v, long lo, long hi) { return v < lo ? lo : (v > hi ? hi : v); }

inline int nibble_to_int(unsigned nib) { return (nib & 8u) ? (int)nib - 16 : (int)nib; }

// The k indices of a bank with the largest score under the total order
// "larger score first; equal score -> smaller index first", returned ascending.
// Written as k passes of "take the best not yet taken" so it can be read off
// the definition.
template <typename T>
void topk_bank(const T* score, int b, int k, uint8_t* out_sorted) {
  std::vector<char> taken(b, 0);
  for (int pick = 0; pick < k; ++pick) {
    int best = -1;
    for (int j = 0; j < b; ++j) {
      if (taken[j]) continue;
      if (best < 0 || score[j] > score[best]) best = j;  // strict > keeps the smaller index on ties
    }
    taken[best] = 1;
  }
  int n = 0;
  for (int j = 0; j < b; ++j)
    if (taken[j]) out_sorted[n++] = (uint8_t)j;
}

}  // namespace

extern "C" {

int sqo_num_threads(void) {
#if defined(_OPENMP)
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Equivalent bits per element (Section 4.1, "Notation").
//   on_weights != 0: x = (1-s)*h_high + h_low      (W(SQx)Ay)
//   on_weights == 0: y = (1-s)*h_high + s*h_low    (WxA(SQy))
double sqo_equivalent_bits(double h_high, double h_low, double s, int on_weights) {
  return on_weights ? (1.0 - s) * h_high + h_low : (1.0 - s) * h_high + s * h_low;
}

// Static positions (Algorithm 2).  calib: bf16 [T,K]; W: bf16 [N,K] or NULL.
//   Abar_j = (sum_t |calib[t,j]|) / T        sequential in t, fp64
//   r_j    = sum_n W[n,j]                    sequential in n, fp64 (1 if W == NULL)
//   I_j    = |Abar_j * r_j|
//   per bank: the k channels with the largest I_j (ties -> smaller j), ascending.
// Readings: "average activation" is the mean magnitude; the weight sum is the
// signed sum over output channels as printed; smoothing is the identity.
void sqo_calib_positions(int b, int k, const uint16_t* calib, long T, long K,
                         const uint16_t* W, long N, uint8_t* positions /*[K/b,k]*/,
                         double* importance_out /*[K] or NULL*/) {
  std::vector<double> I(K);
#pragma omp parallel for schedule(static)
  for (long j = 0; j < K; ++j) {
    double sum = 0.0;
    for (long t = 0; t < T; ++t) sum += std::fabs((double)bf16_to_f32(calib[t * K + j]));
    double abar = sum / (double)T;
    double r = 1.0;
    if (W) {
      r = 0.0;
      for (long n = 0; n < N; ++n) r += (double)bf16_to_f32(W[n * K + j]);
    }
    I[j] = std::fabs(abar * r);
  }
  const long G = K / b;
  for (long g = 0; g < G; ++g) topk_bank(&I[g * b], b, k, positions + g * k);
  if (importance_out) std::memcpy(importance_out, I.data(), sizeof(double) * K);
}

// Per-output-channel symmetric INT4 weights (Section 3.2.1 range; per-channel
// scale = the "classic quantization" of the other operand, Section 3.2).
//   wmax = max_j |W[n,j]|; c = 7.0f / wmax (fp32 division); s_w = wmax / 7.0f
//   wq   = clamp(RNE(W[n,j] * c), -7, 7); zero channel -> codes 0, s_w = 0
//   wq4[n, j/2]: element 2*(j/2) in the low nibble, the next one in the high
//   nibble, two's complement; colsum[n] = sum_j wq
//   static only: w_sparse[n, g*k+i] = wq[n, g*b + positions[g][i]]: the codes of the selected
//   input channels gathered bank by bank, which is all Algorithm 2's "reorder" line states.
void sqo_pack_weights(int b, int k, const uint16_t* W, long N, long K, const uint8_t* positions,
                      uint8_t* wq4, float* s_w, int32_t* colsum, int8_t* w_sparse /*or NULL*/,
                      int8_t* wq_plain /*[N,K] or NULL*/) {
  const long G = K / b;
#pragma omp parallel for schedule(static)
  for (long n = 0; n < N; ++n) {
    float wmax = 0.f;
    for (long j = 0; j < K; ++j) wmax = std::fmax(wmax, std::fabs(bf16_to_f32(W[n * K + j])));
    std::vector<int> q(K, 0);
    float c = 0.f;
    if (wmax > 0.f) {
      c = 7.0f / wmax;
      s_w[n] = wmax / 7.0f;
    } else {
      s_w[n] = 0.f;
    }
    long sum = 0;
    for (long j = 0; j < K; ++j) {
      if (wmax > 0.f) q[j] = (int)clampl(rne_prod(bf16_to_f32(W[n * K + j]), c), -7, 7);
      sum += q[j];
      if (wq_plain) wq_plain[n * K + j] = (int8_t)q[j];
    }
    colsum[n] = (int32_t)sum;
    for (long j = 0; j < K; j += 2)
      wq4[n * (K / 2) + j / 2] = (uint8_t)((q[j] & 0xF) | ((q[j + 1] & 0xF) << 4));
    if (positions && w_sparse)
      for (long g = 0; g < G; ++g)
        for (int i = 0; i < k; ++i)
          w_sparse[n * G * k + g * k + i] = (int8_t)q[g * b + positions[g * k + i]];
  }
}

// Activation encode, one token row at a time.  positions == NULL -> dynamic.
//  1. mag_j = |a_j|, amax = max_j mag_j                              (a_j = fp32(X[m,j]))
//  2. S = per bank the k largest mag (ties -> smaller j)   [dynamic, Sections 3.2.2/3.3]
//       or positions[g]                                    [static, Algorithm 2]
//  3. rmax = max_{j not in S} mag_j (0 if none)
//  4. amax == 0 -> all codes 0, e = 0, s_hi = s_lo = 0;
//     else inv = 127.0f/amax, s_hi = amax/127.0f   (both IEEE fp32 divisions)
//  5. RNE(p) = round-half-even of the exact product
//  6. e = min{e in 0..4 : RNE(rmax * ldexpf(inv,-e)) <= 7}, 4 if none; s_lo = ldexpf(s_hi, e)
//  7. j in S:     q_hi = clamp(RNE(a_j * inv), -127, 127); dense nibble = 0
//  8. j not in S: q_lo = clamp(RNE(a_j * ldexpf(inv,-e)), -7, 7)
//  9. dq4[m, j/2]: even element low nibble, odd element high nibble, two's complement;
//     vals[m,g,0..k), idx[m,g,0..k) ascending bank-local index; s_hi[m], s_lo[m], shift[m] = e.
// Readings: per-token scales on one common integer grid (the dense grid is the
// sparse grid coarsened by 2^e) so that the hybrid GEMM has a single int32
// accumulator and one dequantising epilogue; the scale is taken from the whole
// row in both modes.
void sqo_encode(int b, int k, const uint16_t* X, long M, long K, const uint8_t* positions,
                uint8_t* dq4, int8_t* vals, uint8_t* idx /*NULL if static*/, float* s_hi,
                float* s_lo, uint8_t* shift) {
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
    float inv = 0.f, sh = 0.f, sl = 0.f;
    if (amax > 0.f) {
      inv = 127.0f / amax;
      sh = amax / 127.0f;
      e = 4;
      for (int t = 0; t <= 4; ++t)
        if (rne_prod(rmax, std::ldexp(inv, -t)) <= 7) { e = t; break; }
      sl = std::ldexp(sh, e);
    }
    s_hi[m] = sh;
    s_lo[m] = sl;
    shift[m] = (uint8_t)e;
    const float inv_lo = std::ldexp(inv, -e);

    std::vector<int> qlo(K, 0);
    for (long j = 0; j < K; ++j)
      if (!inS[j] && amax > 0.f) qlo[j] = (int)clampl(rne_prod(a[j], inv_lo), -7, 7);
    for (long j = 0; j < K; j += 2)
      dq4[m * (K / 2) + j / 2] = (uint8_t)((qlo[j] & 0xF) | ((qlo[j + 1] & 0xF) << 4));
    for (long g = 0; g < G; ++g)
      for (int i = 0; i < k; ++i) {
        long j = g * b + sel[g * k + i];
        int q = amax > 0.f ? (int)clampl(rne_prod(a[j], inv), -127, 127) : 0;
        vals[(m * G + g) * k + i] = (int8_t)q;
        if (idx) idx[(m * G + g) * k + i] = sel[g * k + i];
      }
  }
}

// Merged integer activation row: a8[j] = (q_lo[j] << e) + [j in S] q_hi[j].
static void merged_row(int b, int k, long K, long m, const uint8_t* dq4, const int8_t* vals,
                       const uint8_t* idx, const uint8_t* positions, const uint8_t* shift,
                       std::vector<int>& a8) {
  const long G = K / b;
  const int e = shift[m];
  for (long j = 0; j < K; ++j) {
    unsigned byte = dq4[m * (K / 2) + j / 2];
    unsigned nib = (j & 1) ? (byte >> 4) : (byte & 0xF);
    a8[j] = nibble_to_int(nib) * (1 << e);
  }
  for (long g = 0; g < G; ++g)
    for (int i = 0; i < k; ++i) {
      int local = idx ? idx[(m * G + g) * k + i] : positions[g * k + i];
      a8[g * b + local] += vals[(m * G + g) * k + i];
    }
}

// Hybrid GEMM + dequant epilogue (Section 3.3).
//   acc[m,n]   = sum_j ((q_lo[m,j] << e[m]) + [j in S_m] q_hi[m,j]) * wq[n,j]      (int32)
//   ref32[m,n] = ((float)acc * s_hi[m]) * s_w[n]
//   out[m,n]   = bf16_rne(ref32)
// rows / cols (may be NULL = all) select which outputs to compute; outputs are
// written densely as [n_rows, n_cols].  Returns 0, or 1 if any accumulator
// would not fit in int32 (checked against a 64-bit accumulation).
int sqo_gemm(int b, int k, const uint8_t* dq4, const int8_t* vals, const uint8_t* idx,
             const uint8_t* positions, const float* s_hi, const uint8_t* shift, const uint8_t* wq4,
             const float* s_w, long M, long N, long K, const long* rows, long n_rows,
             const long* cols, long n_cols, int32_t* acc_out, float* ref32_out, uint16_t* out_bf16) {
  const long R = rows ? n_rows : M;
  const long C = cols ? n_cols : N;
  int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
  for (long r = 0; r < R; ++r) {
    const long m = rows ? rows[r] : r;
    std::vector<int> a8(K);
    merged_row(b, k, K, m, dq4, vals, idx, positions, shift, a8);
    for (long c = 0; c < C; ++c) {
      const long n = cols ? cols[c] : c;
      long long acc = 0;
      for (long j = 0; j < K; ++j) {
        unsigned byte = wq4[n * (K / 2) + j / 2];
        unsigned nib = (j & 1) ? (byte >> 4) : (byte & 0xF);
        acc += (long long)a8[j] * nibble_to_int(nib);
      }
      if (acc > INT32_MAX || acc < INT32_MIN) overflow |= 1;
      const int32_t acc32 = (int32_t)acc;
      const float ref = ((float)acc32 * s_hi[m]) * s_w[n];
      if (acc_out) acc_out[r * C + c] = acc32;
      if (ref32_out) ref32_out[r * C + c] = ref;
      if (out_bf16) out_bf16[r * C + c] = f32_to_bf16(ref);
    }
  }
  return overflow;
}

// ---------------------------------------------------------------------------
// Independent-scale variant for static positions.  Algorithm 1 quantises the
// high- and the low-precision part of a bank split with separate scales S_high
// and S_low; here that rule is applied to the statically split activations of
// Algorithm 2 (per token row, like the tied-scale encode above):
//  1. S = positions[g] for every bank g                      (Algorithm 2)
//  2. smax = max_{j in S} |a_j|,  rmax = max_{j not in S} |a_j|
//  3. smax > 0: inv_hi = 127.0f/smax, s_hi = smax/127.0f (fp32 divisions); else both 0
//     rmax > 0: inv_lo = 7.0f/rmax,   s_lo = rmax/7.0f;                     else both 0
//  4. j in S:     q_hi = clamp(RNE(a_j * inv_hi), -127, 127); dense nibble = 0
//     j not in S: q_lo = clamp(RNE(a_j * inv_lo), -7, 7)
//  5. same packing as sqo_encode; no idx (static), no shift (written as 0).
void sqo_encode_indep(int b, int k, const uint16_t* X, long M, long K, const uint8_t* positions,
                      uint8_t* dq4, int8_t* vals, float* s_hi, float* s_lo, uint8_t* shift) {
  const long G = K / b;
#pragma omp parallel for schedule(static)
  for (long m = 0; m < M; ++m) {
    std::vector<float> a(K);
    std::vector<char> inS(K, 0);
    for (long j = 0; j < K; ++j) a[j] = bf16_to_f32(X[m * K + j]);
    for (long g = 0; g < G; ++g)
      for (int i = 0; i < k; ++i) inS[g * b + positions[g * k + i]] = 1;
    float smax = 0.f, rmax = 0.f;
    for (long j = 0; j < K; ++j) {
      const float mag = std::fabs(a[j]);
      if (inS[j]) {
        if (mag > smax) smax = mag;
      } else {
        if (mag > rmax) rmax = mag;
      }
    }
    const float inv_hi = smax > 0.f ? 127.0f / smax : 0.f;
    const float inv_lo = rmax > 0.f ? 7.0f / rmax : 0.f;
    s_hi[m] = smax > 0.f ? smax / 127.0f : 0.f;
    s_lo[m] = rmax > 0.f ? rmax / 7.0f : 0.f;
    shift[m] = 0;
    std::vector<int> qlo(K, 0);
    for (long j = 0; j < K; ++j)
      if (!inS[j]) qlo[j] = (int)clampl(rne_prod(a[j], inv_lo), -7, 7);
    for (long j = 0; j < K; j += 2)
      dq4[m * (K / 2) + j / 2] = (uint8_t)((qlo[j] & 0xF) | ((qlo[j + 1] & 0xF) << 4));
    for (long g = 0; g < G; ++g)
      for (int i = 0; i < k; ++i) {
        const long j = g * b + positions[g * k + i];
        vals[(m * G + g) * k + i] = (int8_t)clampl(rne_prod(a[j], inv_hi), -127, 127);
      }
  }
}

// Hybrid GEMM with independent scales: the two products keep their own int32
// accumulator and meet in fp32 (Section 3.3's two streams; scales per Algorithm 1).
//   acc_lo[m,n] = sum_j            q_lo[m,j] * wq[n,j]       (q_lo is 0 at the positions)
//   acc_hi[m,n] = sum_{j in S}     q_hi[m,j] * wq[n,j]
//   ref32[m,n]  = fmaf((float)acc_hi, s_hi[m], (float)acc_lo * s_lo[m]) * s_w[n]
//   out[m,n]    = bf16_rne(ref32)
// Returns 0, or 1 if an accumulator would not fit in int32.
int sqo_gemm_indep(int b, int k, const uint8_t* dq4, const int8_t* vals, const uint8_t* positions,
                   const float* s_hi, const float* s_lo, const uint8_t* wq4, const float* s_w, long M,
                   long N, long K, const long* rows, long n_rows, const long* cols, long n_cols,
                   int32_t* acc_lo_out, int32_t* acc_hi_out, float* ref32_out, uint16_t* out_bf16) {
  const long R = rows ? n_rows : M;
  const long C = cols ? n_cols : N;
  const long G = K / b;
  int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
  for (long r = 0; r < R; ++r) {
    const long m = rows ? rows[r] : r;
    for (long c = 0; c < C; ++c) {
      const long n = cols ? cols[c] : c;
      long long lo = 0, hi = 0;
      for (long j = 0; j < K; ++j) {
        unsigned ab = dq4[m * (K / 2) + j / 2], wb = wq4[n * (K / 2) + j / 2];
        int qa = nibble_to_int((j & 1) ? (ab >> 4) : (ab & 0xF));
        int qw = nibble_to_int((j & 1) ? (wb >> 4) : (wb & 0xF));
        lo += (long long)qa * qw;
      }
      for (long g = 0; g < G; ++g)
        for (int i = 0; i < k; ++i) {
          const long j = g * b + positions[g * k + i];
          unsigned wb = wq4[n * (K / 2) + j / 2];
          int qw = nibble_to_int((j & 1) ? (wb >> 4) : (wb & 0xF));
          hi += (long long)vals[(m * G + g) * k + i] * qw;
        }
      if (lo > INT32_MAX || lo < INT32_MIN || hi > INT32_MAX || hi < INT32_MIN) overflow |= 1;
      const float ref = std::fmaf((float)(int32_t)hi, s_hi[m], (float)(int32_t)lo * s_lo[m]) * s_w[n];
      if (acc_lo_out) acc_lo_out[r * C + c] = (int32_t)lo;
      if (acc_hi_out) acc_hi_out[r * C + c] = (int32_t)hi;
      if (ref32_out) ref32_out[r * C + c] = ref;
      if (out_bf16) out_bf16[r * C + c] = f32_to_bf16(ref);
    }
  }
  return overflow;
}

// Decode (inverse of Eq. 1): x^[m,j] = s_hi*q_hi at sparse positions,
// s_lo*q_lo elsewhere, in fp32, then bf16 RNE.
void sqo_decode(int b, int k, const uint8_t* dq4, const int8_t* vals, const uint8_t* idx,
                const uint8_t* positions, const float* s_hi, const float* s_lo, long M, long K,
                float* out_f32 /*or NULL*/, uint16_t* out_bf16 /*or NULL*/) {
  const long G = K / b;
#pragma omp parallel for schedule(static)
  for (long m = 0; m < M; ++m) {
    std::vector<float> x(K);
    for (long j = 0; j < K; ++j) {
      unsigned byte = dq4[m * (K / 2) + j / 2];
      unsigned nib = (j & 1) ? (byte >> 4) : (byte & 0xF);
      x[j] = s_lo[m] * (float)nibble_to_int(nib);
    }
    for (long g = 0; g < G; ++g)
      for (int i = 0; i < k; ++i) {
        int local = idx ? idx[(m * G + g) * k + i] : positions[g * k + i];
        x[g * b + local] = s_hi[m] * (float)vals[(m * G + g) * k + i];
      }
    for (long j = 0; j < K; ++j) {
      if (out_f32) out_f32[m * K + j] = x[j];
      if (out_bf16) out_bf16[m * K + j] = f32_to_bf16(x[j]);
    }
  }
}

}  // extern "C"
