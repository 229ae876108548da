// CPU oracle for SQ-format on WEIGHTS (format part of Algorithm 1).  TEST INFRASTRUCTURE ONLY
// (see sq_oracle.cpp: same rules -- never linked into or called from the product path).
//
// Algorithm 1 ("SQ-format on Weights") picks, per bank of b consecutive input channels of an
// output channel, the (1-s)*b = k most important weights for the high precision and quantises
// the two parts separately (S_high, S_low).  Section 3.2.1 and the weight-matrix figure give the
// storage: the low-precision array keeps its shape and holds, at a high-precision place, the
// code the symmetric low-precision range leaves unused (v_mask), so the mask is implicit; the
// high-precision values are stored compactly, k per bank, in position order.
// What is NOT reproduced: the importance scores themselves (smoothing and a Hessian of real
// calibration data): they are an INPUT here, I[n,j] >= 0.
//
// Readings:
//   * h_high = INT8 in [-127,127], h_low = INT4 in [-7,7]; v_mask = the 4-bit pattern 1000 (-8);
//   * scales per output channel (the granularity of the other weight formats of this library):
//     S_high[n] = (largest selected |w|) / 127, S_low[n] = (largest other |w|) / 7, 0 for an empty
//     or all-zero part; codes = RNE of the exact product with the reciprocal scale, as elsewhere;
//   * ties in I go to the smaller index; the compact values of a bank are in ascending position;
//   * the decode-shaped product uses per-token symmetric INT8 activations (s_x = amax/127) and
//     joins the two integer sums in fp32:
//       out = bf16( fmaf((float)acc_hi, S_high[n], (float)acc_lo * S_low[n]) * s_x[m] ).
// Parity status: pinned by tests/test_oracle_w_pins.py (brute-force selection, exact rationals,
// the storage closed form, reconstruction bounds, fp64 brute-force product); nothing unpinned.
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
inline long rne_prod(float a, float c) { return (long)std::nearbyint((double)a * (double)c); }
inline long clampl(long v, long lo, long hi) { return v < lo ? lo : (v > hi ? hi : v); }
constexpr unsigned kVMask = 8u;  // 0b1000
}  // namespace

extern "C" {

// W bf16 [N,K], I float [N,K] -> wq4 u8 [N,K/2] (v_mask at selected places), w_hi i8 [N,G,k],
// s_high, s_low f32 [N].
void sqo_w_encode(int b, int k, const uint16_t* W, const float* I, long N, long K, uint8_t* wq4, int8_t* w_hi,
                  float* s_high, float* s_low) {
  const long G = K / b;
#pragma omp parallel for schedule(static)
  for (long n = 0; n < N; ++n) {
    std::vector<char> inS(K, 0);
    for (long g = 0; g < G; ++g) {  // k passes of "take the most important not yet taken"
      for (int pick = 0; pick < k; ++pick) {
        long best = -1;
        for (long j = g * b; j < (g + 1) * b; ++j) {
          if (inS[j]) continue;
          if (best < 0 || I[n * K + j] > I[n * K + best]) best = j;  // strict >: ties keep the smaller index
        }
        inS[best] = 1;
      }
    }
    float hmax = 0.f, lmax = 0.f;
    for (long j = 0; j < K; ++j) {
      const float mag = std::fabs(bf16_to_f32(W[n * K + j]));
      if (inS[j]) hmax = std::fmax(hmax, mag);
      else lmax = std::fmax(lmax, mag);
    }
    const float inv_hi = hmax > 0.f ? 127.0f / hmax : 0.f, inv_lo = lmax > 0.f ? 7.0f / lmax : 0.f;
    s_high[n] = hmax > 0.f ? hmax / 127.0f : 0.f;
    s_low[n] = lmax > 0.f ? lmax / 7.0f : 0.f;
    std::vector<unsigned> nib(K);
    for (long g = 0; g < G; ++g) {
      int slot = 0;
      for (long j = g * b; j < (g + 1) * b; ++j) {
        const float w = bf16_to_f32(W[n * K + j]);
        if (inS[j]) {
          nib[j] = kVMask;
          w_hi[(n * G + g) * k + slot++] = (int8_t)clampl(rne_prod(w, inv_hi), -127, 127);
        } else {
          nib[j] = (unsigned)clampl(rne_prod(w, inv_lo), -7, 7) & 0xFu;
        }
      }
    }
    for (long j = 0; j < K; j += 2) wq4[n * (K / 2) + j / 2] = (uint8_t)(nib[j] | (nib[j + 1] << 4));
  }
}

// w^[n,j] = S_high * next compact value at a v_mask place, S_low * code elsewhere (fp32).
void sqo_w_decode(int b, int k, const uint8_t* wq4, const int8_t* w_hi, const float* s_high, const float* s_low, long N,
                  long K, float* out) {
  const long G = K / b;
#pragma omp parallel for schedule(static)
  for (long n = 0; n < N; ++n)
    for (long g = 0; g < G; ++g) {
      int slot = 0;
      for (long j = g * b; j < (g + 1) * b; ++j) {
        const unsigned byte = wq4[n * (K / 2) + j / 2];
        const unsigned nb = (j & 1) ? (byte >> 4) : (byte & 0xFu);
        if (nb == kVMask) out[n * K + j] = s_high[n] * (float)w_hi[(n * G + g) * k + slot++];
        else out[n * K + j] = s_low[n] * (float)((nb & 8u) ? (int)nb - 16 : (int)nb);
      }
    }
}

// Per-token symmetric INT8 activations: s_x = amax / 127, xq = clamp(RNE(x * (127 / amax)), -127, 127).
void sqo_act_quant8(const uint16_t* X, long M, long K, int8_t* xq, float* s_x) {
  for (long m = 0; m < M; ++m) {
    float amax = 0.f;
    for (long j = 0; j < K; ++j) amax = std::fmax(amax, std::fabs(bf16_to_f32(X[m * K + j])));
    const float inv = amax > 0.f ? 127.0f / amax : 0.f;
    s_x[m] = amax > 0.f ? amax / 127.0f : 0.f;
    for (long j = 0; j < K; ++j) xq[m * K + j] = (int8_t)clampl(rne_prod(bf16_to_f32(X[m * K + j]), inv), -127, 127);
  }
}

// Two integer sums per output, joined in fp32 (see the header).
void sqo_w_gemm(int b, int k, const int8_t* xq, const float* s_x, const uint8_t* wq4, const int8_t* w_hi,
                const float* s_high, const float* s_low, long M, long N, long K, int32_t* acc_lo_out, int32_t* acc_hi_out,
                float* ref32_out, uint16_t* out_bf16) {
  const long G = K / b;
#pragma omp parallel for schedule(static)
  for (long n = 0; n < N; ++n)
    for (long m = 0; m < M; ++m) {
      long long lo = 0, hi = 0;
      for (long g = 0; g < G; ++g) {
        int slot = 0;
        for (long j = g * b; j < (g + 1) * b; ++j) {
          const unsigned byte = wq4[n * (K / 2) + j / 2];
          const unsigned nb = (j & 1) ? (byte >> 4) : (byte & 0xFu);
          if (nb == kVMask) hi += (long long)xq[m * K + j] * w_hi[(n * G + g) * k + slot++];
          else lo += (long long)xq[m * K + j] * ((nb & 8u) ? (int)nb - 16 : (int)nb);
        }
      }
      const float ref = std::fmaf((float)(int32_t)hi, s_high[n], (float)(int32_t)lo * s_low[n]) * s_x[m];
      if (acc_lo_out) acc_lo_out[m * N + n] = (int32_t)lo;
      if (acc_hi_out) acc_hi_out[m * N + n] = (int32_t)hi;
      if (ref32_out) ref32_out[m * N + n] = ref;
      if (out_bf16) out_bf16[m * N + n] = f32_to_bf16(ref);
    }
}

}  // extern "C"
