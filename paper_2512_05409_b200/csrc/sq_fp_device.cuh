// Device helpers of the floating-point variant (sparse FP8 E4M3 + dense FP4 E2M1) shared by its
// own kernels (sq_fp.cu) and by the static-position encode kernel (sq_encode.cu): the codes of
// the format's roundings in single precision.
#pragma once
#include "sq_device.cuh"

namespace sq {

// E4M3 byte of an E2M1 code's value times 2^e (exact: e <= 6 keeps it at or below 384).
__device__ __forceinline__ uint32_t e4m3_of_e2m1(uint32_t code, int e) {
  const uint32_t t = code & 7u;
  if (t == 0) return 0;
  // t = 1 -> 0.5 = 2^-1; t >= 2: exponent (t >> 1) - 1, mantissa bit t & 1
  const uint32_t mag = t == 1 ? (uint32_t)((6 + e) << 3) : ((uint32_t)((t >> 1) + 6 + e) << 3) | ((t & 1u) << 2);
  return mag | ((code & 8u) << 4);
}

// The same codes without double precision, for the encoder's per-element work: the code of the
// magnitude |a| * c (a bf16, c fp32 > 0) in a format with `mb` mantissa bits and smallest normal
// exponent emin.  The spacing of the format's grid at that magnitude is 2^(ex - mb), ex = the
// (clamped) exponent; one FMA with the constant 1.5 * 2^(ex - mb + 23) rounds the EXACT product to
// that grid, half-even, and leaves the integer n = round(|a| c / spacing) in its low mantissa
// bits; code = ((ex - emin) << mb) + n as in round_code.  ex is read off the rounded product: it
// differs from the exact product's exponent only when that lies within 2^-24 of a power of two from
// below, where both grids round to the power of two itself.
template <int MB, int EMIN, uint32_t MAXC>
__device__ __forceinline__ uint32_t round_code32(float a_abs, float c) {
  const int ex = max((int)(__float_as_uint(a_abs * c) >> 23) - 127, EMIN);
  const uint32_t magic = ((uint32_t)(ex - MB + 23 + 127) << 23) | 0x00400000u;
  const uint32_t n = __float_as_uint(__fmaf_rn(a_abs, c, __uint_as_float(magic))) - magic;
  return min(((uint32_t)(ex - EMIN) << MB) + n, MAXC);
}
// a: bf16 bit pattern (finite); c > 0.
__device__ __forceinline__ uint32_t e2m1_of32(uint32_t a_bits, float c) {
  const uint32_t code = round_code32<1, 0, 7u>(__uint_as_float((a_bits & 0x7FFFu) << 16), c);
  return code == 0 ? 0u : (code | ((a_bits >> 12) & 8u));
}
__device__ __forceinline__ uint32_t e4m3_of32(uint32_t a_bits, float c) {
  const uint32_t code = round_code32<3, -6, 0x7Eu>(__uint_as_float((a_bits & 0x7FFFu) << 16), c);
  return code == 0 ? 0u : (code | ((a_bits >> 8) & 0x80u));
}

}  // namespace sq
