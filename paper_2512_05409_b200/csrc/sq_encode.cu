// Activation encode (bf16 -> SQ-format) and decode (SQ-format -> bf16).
//
// Encode is one pass over HBM: 2 B read and 0.5 + 2k/b B (dynamic) or 0.5 + k/b B (static)
// written per element.  The scale of a row is its maximum, so a row must be seen in full
// before anything can be quantised: a GROUP of 1-16 warps owns one token row at a time,
// staged in shared memory by one bulk asynchronous copy; the host picks the group size
// that keeps the most warps resident (16 per block, 8 for b = 128), so that the rows other
// groups have in flight hide the copy latency.  Groups synchronise on their own named
// barrier, never block-wide.
//
//   phase 1  (dynamic) each lane owns whole banks.  The k-th largest magnitude of a bank is
//            found with a sorting network on packed bf16x2 magnitudes (two columns at once;
//            sorted runs of k merged with truncation), then one compare pass builds the
//            selection mask; equal magnitudes at the threshold are resolved towards the lower
//            index.  The largest UNSELECTED magnitude of the row, which fixes the shift, is not
//            tracked element by element: the network yields per bank an upper bound (the k-th
//            largest) and a lower bound (the largest loser of the last merge) for free, and
//            only a row whose two bounds give different shifts is swept once more (its
//            selected places are zero by then) for the exact value.
//            (static) the given positions are copied out and zeroed in the staged row.
//   reduce   row maximum and the two bounds over the group -> inv, s_hi, shift e, s_lo
//            The kernel is bound by the integer/logic pipe (16 lanes per cycle and scheduler
//            for min/max, logic, compares, selects), so whatever integer work can be written
//            as a multiply-add (magnitudes, picking the k positions out of the mask, nibble
//            packing) is issued on the multiply-add pipe instead.
//   phase 2  selected values -> INT8 in ascending position (and their indices), zeroed in
//            the staged row; then the whole row -> INT4, eight codes per 32-bit word, in a
//            coalesced sweep (the zeroed places give the zero nibbles the format asks for).
//
// Formats outside the fast kernels' set (k not a power of two, k/b other than 1/2 .. 1/16 for
// dynamic positions) take a plain one-block-per-row kernel that ranks every element.
#include <cstdio>
#include <cstdlib>
#include "sq_device.cuh"
#include "sq_fp_device.cuh"
#include "sq_host.h"

namespace sq {

namespace {

__device__ __forceinline__ uint32_t block_max_u32(uint32_t v, uint32_t* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();  // scratch may still be read from a previous reduction
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  uint32_t r = 0;
  for (int q = 0; q < (int)(blockDim.x >> 5); ++q) r = max(r, scratch[q]);
  return r;
}

// packed bf16x2 helpers on raw 32-bit registers (magnitudes: non-negative, finite)
__device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t min2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t ge2_mask(uint32_t a, uint32_t b) {  // 0xFFFF per half where a >= b
  uint32_t d;
  asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t swap_halves(uint32_t a) { return __byte_perm(a, a, 0x1032); }
__device__ __forceinline__ uint32_t abs2(uint32_t a) {  // compiles to a packed multiply-add pipe instruction
  uint32_t d;
  asm("abs.bf16x2 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// The dynamic kernel is bound by the integer/logic pipe (min/max, logic, compares, selects,
// shifts: 16 lanes per cycle and scheduler) while the multiply-add pipe has room, so integer
// work that can be written as d = a * m + c is issued as a multiply-add.  The multipliers come
// from kernel parameters: as immediates the compiler would turn the instruction back into an
// add or a shift on the busy pipe.
struct MulK {
  uint32_t neg1, two, k32, k256, k65536, k16m, k16, one;
};
__device__ __forceinline__ uint32_t imad(uint32_t a, uint32_t m, uint32_t c) {
  uint32_t d;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(m), "r"(c));
  return d;
}

// compare-exchange of packed magnitudes, larger first
__device__ __forceinline__ void ce(uint32_t& a, uint32_t& b) {
  const uint32_t hi = max2(a, b), lo = min2(a, b);
  a = hi;
  b = lo;
}

// Batcher's odd-even merge sort of r[LO..LO+N), descending, both bf16 columns at once.
// Written as compile-time recursion so that every index is a constant and the array stays
// in registers whatever N is.
template <int I, int END, int STEP, int R>
__device__ __forceinline__ void ce_run(uint32_t* r) {  // ce(i, i+R) for i = I, I+STEP, ... < END
  if constexpr (I < END) {
    ce(r[I], r[I + R]);
    ce_run<I + STEP, END, STEP, R>(r);
  }
}
template <int LO, int HI, int R>  // HI inclusive
__device__ __forceinline__ void oe_merge(uint32_t* r) {
  constexpr int STEP = R * 2;
  if constexpr (STEP < HI - LO) {
    oe_merge<LO, HI, STEP>(r);
    oe_merge<LO + R, HI, STEP>(r);
    ce_run<LO + R, HI - R, STEP, R>(r);
  } else {
    ce(r[LO], r[LO + R]);
  }
}
template <int LO, int HI>  // HI inclusive
__device__ __forceinline__ void oe_sort(uint32_t* r) {
  if constexpr (HI - LO >= 1) {
    constexpr int MID = LO + (HI - LO) / 2;
    oe_sort<LO, MID>(r);
    oe_sort<MID + 1, HI>(r);
    oe_merge<LO, HI, 1>(r);
  }
}
template <int N>
__device__ __forceinline__ void sort_desc(uint32_t* r) {
  oe_sort<0, N - 1>(r);
}

// r[0..N) bitonic -> sorted descending (compile-time recursion, see above).
template <int N, int S, int I>
__device__ __forceinline__ void bitonic_stage(uint32_t* r) {
  if constexpr (I < N) {
    if constexpr ((I & S) == 0) ce(r[I], r[I + S]);
    bitonic_stage<N, S, I + 1>(r);
  }
}
template <int N, int S>
__device__ __forceinline__ void bitonic_stages(uint32_t* r) {
  if constexpr (S >= 1) {
    bitonic_stage<N, S, 0>(r);
    bitonic_stages<N, S / 2>(r);
  }
}
template <int N>
__device__ __forceinline__ void bitonic_merge_desc(uint32_t* r) {
  bitonic_stages<N, N / 2>(r);
}

// bits 0..15 of x -> even bit positions, bits 16..31 -> odd bit positions.
__device__ __forceinline__ uint32_t spread16(uint32_t x) {
  x &= 0xFFFFu;
  x = (x | (x << 8)) & 0x00FF00FFu;
  x = (x | (x << 4)) & 0x0F0F0F0Fu;
  x = (x | (x << 2)) & 0x33333333u;
  x = (x | (x << 1)) & 0x55555555u;
  return x;
}
__device__ __forceinline__ uint32_t interleave_halves(uint32_t x) { return spread16(x) | (spread16(x >> 16) << 1); }

// Eight fp32 values holding integers in their low mantissa bits (magic-number rounding)
// -> eight two's-complement nibbles, element i in nibble i.
// `ev` / `od` receive the codes of the even / odd elements as four two's-complement bytes each.
__device__ __forceinline__ uint32_t pack_nibbles(const float (&r)[8], uint32_t& ev, uint32_t& od) {
  const uint32_t u0 = __float_as_uint(r[0]), u1 = __float_as_uint(r[1]), u2 = __float_as_uint(r[2]),
                 u3 = __float_as_uint(r[3]), u4 = __float_as_uint(r[4]), u5 = __float_as_uint(r[5]),
                 u6 = __float_as_uint(r[6]), u7 = __float_as_uint(r[7]);
  ev = __byte_perm(__byte_perm(u0, u2, 0x0040), __byte_perm(u4, u6, 0x0040), 0x5410);
  od = __byte_perm(__byte_perm(u1, u3, 0x0040), __byte_perm(u5, u7, 0x0040), 0x5410);
  return (ev & 0x0F0F0F0Fu) | ((od << 4) & 0xF0F0F0F0u);
}
__device__ __forceinline__ uint32_t pack_nibbles(const float (&r)[8]) {
  uint32_t ev, od;
  return pack_nibbles(r, ev, od);
}

// The same packing for codes that carry an offset of 8 (u = q + 8 in 1..15, produced by adding
// kMagic + 8 in the rounding FMA): the eight float bit patterns 0x4B400000 + u are summed with
// weights 16^i by integer multiply-adds (no carries between nibbles since u fits four bits), the
// constant part is taken off and the offset undone by flipping bit 3 of every nibble.  Seven
// multiply-adds on the multiply-add pipe instead of nine byte-permute/logic operations on the
// integer pipe, which is the one this kernel is bound by.
__device__ __forceinline__ uint32_t mad16(uint32_t hi, uint32_t mul, uint32_t lo) {
  uint32_t d;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(hi), "r"(mul), "r"(lo));
  return d;
}
__device__ __forceinline__ uint32_t pack_nibbles_off8(const float (&r)[8]) {
  const uint32_t t01 = mad16(__float_as_uint(r[1]), 16u, __float_as_uint(r[0]));
  const uint32_t t23 = mad16(__float_as_uint(r[3]), 16u, __float_as_uint(r[2]));
  const uint32_t t45 = mad16(__float_as_uint(r[5]), 16u, __float_as_uint(r[4]));
  const uint32_t t67 = mad16(__float_as_uint(r[7]), 16u, __float_as_uint(r[6]));
  const uint32_t t03 = mad16(t23, 256u, t01), t47 = mad16(t67, 256u, t45);
  return (mad16(t47, 65536u, t03) - 0x3F400000u) ^ 0x88888888u;  // 0x3F400000 = 0x4B400000 * 0x11111111 mod 2^32
}

// Row scales from the two maxima (bf16 magnitude bit patterns).
struct RowScale {
  float inv, inv_lo, s_hi, s_lo;
  int e;
  bool clamp;  // some dense code may exceed 7 before clamping (only possible when e == 4)
};
__device__ __forceinline__ RowScale row_scale(uint32_t amax_bits, uint32_t rmax_bits) {
  RowScale rs;
  const float amax = bf16_bits_to_f32(amax_bits), rmax = bf16_bits_to_f32(rmax_bits);
  rs.inv = amax > 0.f ? __fdiv_rn(127.0f, amax) : 0.f;
  rs.s_hi = amax > 0.f ? __fdiv_rn(amax, 127.0f) : 0.f;
  int e = 0;
  if (amax > 0.f) {
    e = 4;
#pragma unroll
    for (int t = 4; t >= 0; --t) {
      if (rne_prod(rmax, rs.inv * (1.0f / (float)(1 << t))) <= 7) e = t;  // ends on the smallest fitting t
    }
  }
  rs.e = e;
  rs.inv_lo = rs.inv * (1.0f / (float)(1 << e));
  rs.s_lo = rs.s_hi * (float)(1 << e);
  rs.clamp = rne_prod(rmax, rs.inv_lo) > 7;
  return rs;
}

// The same scales computed by a whole warp at once (every lane returns all of them): the two
// divisions run side by side on even and odd lanes, and the five candidate shifts are tried by
// five lanes and picked with a ballot, instead of one lane walking through all of it.
__device__ __forceinline__ RowScale row_scale_warp(uint32_t amax_bits, uint32_t rmax_bits, int lane) {
  RowScale rs;
  const float amax = bf16_bits_to_f32(amax_bits), rmax = bf16_bits_to_f32(rmax_bits);
  const bool odd = lane & 1;
  const float quot = __fdiv_rn(odd ? amax : 127.0f, odd ? 127.0f : amax);
  const bool nz = amax > 0.f;
  rs.inv = nz ? __shfl_sync(0xffffffffu, quot, 0) : 0.f;
  rs.s_hi = nz ? __shfl_sync(0xffffffffu, quot, 1) : 0.f;
  const int t = lane < 4 ? lane : 4;
  const bool fits = rne_prod(rmax, rs.inv * __int_as_float((127 - t) << 23)) <= 7;
  const uint32_t fit_mask = __ballot_sync(0xffffffffu, fits) & 0x1Fu;
  rs.e = !nz ? 0 : (fit_mask ? __ffs((int)fit_mask) - 1 : 4);
  rs.inv_lo = rs.inv * __int_as_float((127 - rs.e) << 23);
  rs.s_lo = rs.s_hi * (float)(1 << rs.e);
  rs.clamp = rne_prod(rmax, rs.inv_lo) > 7;
  return rs;
}

// Independent scales (Algorithm 1's S_high / S_low on a static split): each part is scaled by
// its own maximum; no shift, and no dense code can pass 7.
__device__ __forceinline__ RowScale row_scale_indep(uint32_t smax_bits, uint32_t rmax_bits) {
  RowScale rs;
  const float smax = bf16_bits_to_f32(smax_bits), rmax = bf16_bits_to_f32(rmax_bits);
  rs.inv = smax > 0.f ? __fdiv_rn(127.0f, smax) : 0.f;
  rs.s_hi = smax > 0.f ? __fdiv_rn(smax, 127.0f) : 0.f;
  rs.inv_lo = rmax > 0.f ? __fdiv_rn(7.0f, rmax) : 0.f;
  rs.s_lo = rmax > 0.f ? __fdiv_rn(rmax, 7.0f) : 0.f;
  rs.e = 0;
  rs.clamp = false;
  return rs;
}

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}

// Eight bf16 (four packed words) times c, rounded half-even to integers held in the low
// mantissa bits (magic-number rounding); two FMAs per instruction on the packed fp32 pipe,
// each half rounding like fmaf.
template <bool OFF8 = false>
__device__ __forceinline__ void quant8(const uint4& v, float c, float (&r)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  constexpr float kM = OFF8 ? kMagic + 8.0f : kMagic;
  const float2 cc = make_float2(c, c), mm = make_float2(kM, kM);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float2 a = make_float2(__uint_as_float(w[q] << 16), __uint_as_float(w[q] & 0xFFFF0000u));
    const float2 d = __ffma2_rn(a, cc, mm);
    r[2 * q] = d.x;
    r[2 * q + 1] = d.y;
  }
}

// The coalesced INT4 sweep over a staged row (selected places already zeroed): lane l of the
// group takes 16-byte chunks l, l + gsize, ... and writes one 32-bit word per chunk.
__device__ __forceinline__ void dense_sweep(const uint16_t* row, int K, const RowScale& rs, uint8_t* dq4_row, int lane,
                                            int gsize) {
  const float c = rs.inv_lo;
  const uint4* src = reinterpret_cast<const uint4*>(row) + lane;
  uint32_t* dst = reinterpret_cast<uint32_t*>(dq4_row) + lane;
  const int iters = (K / 8 - lane + gsize - 1) / gsize;
  if (!rs.clamp) {
#pragma unroll 2
    for (int i = 0; i < iters; ++i, src += gsize, dst += gsize) {
      float r[8];
      quant8<true>(*src, c, r);
      *dst = pack_nibbles_off8(r);
    }
  } else {
    // Codes beyond +-7 are possible: limit the inputs instead of the codes, two elements per
    // instruction.  xl = the bf16 at or just below 7 / c still rounds to code 7, anything
    // larger in magnitude would round to 7 or more, anything smaller is untouched.
    const uint32_t xl = __float_as_uint(__fdiv_rd(7.0f, c)) >> 16;
    const uint32_t hi2 = xl | (xl << 16), lo2 = hi2 | 0x80008000u;
#pragma unroll 2
    for (int i = 0; i < iters; ++i, src += gsize, dst += gsize) {
      uint4 v = *src;
      v.x = max2(min2(v.x, hi2), lo2);
      v.y = max2(min2(v.y, hi2), lo2);
      v.z = max2(min2(v.z, hi2), lo2);
      v.w = max2(min2(v.w, hi2), lo2);
      float r[8];
      quant8<true>(v, c, r);
      *dst = pack_nibbles_off8(r);
    }
  }
}

// ---- floating-point variant (sparse E4M3 + dense E2M1; the selection is the integer path's)
// Scales from the row maximum and the largest unselected magnitude (bf16 bit patterns): the row
// maximum maps to 256; the dense grid is coarser by the smallest power of two (up to 2^6) that
// brings the largest unselected magnitude to at most 6.
__device__ __forceinline__ int fp_shift_of(float inv, float rmax, bool nonzero) {
  int e = 0;
  if (nonzero) {
    e = 6;
#pragma unroll
    for (int t = 6; t >= 0; --t)
      if ((double)rmax * (double)(inv * __int_as_float((127 - t) << 23)) <= 6.0) e = t;  // ends on the smallest fitting t
  }
  return e;
}
__device__ __forceinline__ RowScale row_scale_fp(uint32_t amax_bits, uint32_t rmax_bits) {
  RowScale rs;
  const float amax = bf16_bits_to_f32(amax_bits), rmax = bf16_bits_to_f32(rmax_bits);
  rs.inv = amax > 0.f ? __fdiv_rn(256.0f, amax) : 0.f;
  rs.s_hi = amax > 0.f ? __fdiv_rn(amax, 256.0f) : 0.f;
  rs.e = fp_shift_of(rs.inv, rmax, amax > 0.f);
  rs.s_lo = rs.s_hi * (float)(1 << rs.e);
  rs.inv_lo = rs.inv * __int_as_float((127 - rs.e) << 23);
  rs.clamp = false;  // the code construction saturates by itself
  return rs;
}
// The dense E2M1 code of a magnitude is a step function of the bf16 input: seven thresholds per
// row decide it.  Threshold i = the smallest bf16 magnitude a whose exact product a * c reaches the
// midpoint between the (i-1)-th and the i-th grid value (0, 0.5, 1, 1.5, 2, 3, 4, 6) -- reaches it
// or passes it, whichever the tie rule (to the even code) asks for.  One fused multiply-add
// a * c - midpoint has the exact difference's sign, so the candidate from the quotient is checked
// exactly.  Lane i (0..6) computes threshold i + 1; every lane gets all seven, each in both
// halves of a register.  With c = 0 no magnitude reaches any threshold (a NaN pattern).
struct FpSteps {
  uint32_t t[7];          // thresholds 1..7, duplicated into both halves
  uint32_t lut_lo, lut_hi;  // E4M3 bytes of the eight magnitudes times 2^e
};
__device__ __forceinline__ FpSteps fp_steps(float c, int e, int lane) {
  const int i = min(lane, 6);
  const float mid = i == 0 ? 0.25f : i == 1 ? 0.75f : i == 2 ? 1.25f : i == 3 ? 1.75f : i == 4 ? 2.5f : i == 5 ? 3.5f : 5.0f;
  const bool strict = (i & 1) == 0;  // a tie goes to the even code: codes 0, 2, 4, 6 keep it
  uint32_t thr = 0x7FFFu;
  if (c > 0.f) {
    const uint32_t a0 = __float_as_uint(__fdiv_rn(mid, c)) >> 16;  // the quotient cut to bf16: at or just below the threshold
    auto reaches = [&](uint32_t a) {
      const float d = __fmaf_rn(__uint_as_float(a << 16), c, -mid);
      return strict ? d > 0.f : d >= 0.f;
    };
    thr = reaches(a0) ? a0 : (reaches(a0 + 1u) ? a0 + 1u : a0 + 2u);
    thr = min(thr, 0x7F80u);
  }
  FpSteps st;
#pragma unroll
  for (int j = 0; j < 7; ++j) st.t[j] = __shfl_sync(0xffffffffu, thr, j) * 0x10001u;
  uint32_t lo = 0, hi = 0;
#pragma unroll
  for (int n = 0; n < 4; ++n) {
    lo |= e4m3_of_e2m1((uint32_t)n, e) << (8 * n);
    hi |= e4m3_of_e2m1((uint32_t)(n + 4), e) << (8 * n);
  }
  st.lut_lo = lo;
  st.lut_hi = hi;
  return st;
}
// Two bf16 inputs (one word) -> their E2M1 codes in bits 0-3 and 16-19: three compares walk the
// thresholds as a binary tree, a fourth tells zero codes (which carry no sign) from the rest.
__device__ __forceinline__ uint32_t fp_codes2(uint32_t w, const FpSteps& st) {
  const uint32_t mag = w & 0x7FFF7FFFu;
  const uint32_t g2 = ge2_mask(mag, st.t[3]);                                   // code >= 4
  const uint32_t ta = (g2 & st.t[5]) | (~g2 & st.t[1]);
  const uint32_t g1 = ge2_mask(mag, ta);                                        // next bit
  const uint32_t hi = (g1 & st.t[6]) | (~g1 & st.t[4]), lo = (g1 & st.t[2]) | (~g1 & st.t[0]);
  const uint32_t tb = (g2 & hi) | (~g2 & lo);
  const uint32_t g0 = ge2_mask(mag, tb);                                        // last bit
  const uint32_t nz = ge2_mask(mag, st.t[0]);
  return (g2 & 0x00040004u) | (g1 & 0x00020002u) | (g0 & 0x00010001u) | ((w >> 12) & 0x00080008u & nz);
}
__device__ __forceinline__ uint32_t prmt_u32(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
// Eight codes (one nibble each, element i in nibble i) -> the eight E4M3 bytes of code * 2^e: the
// magnitudes through the row's byte table, the signs moved from bit 3 of a nibble to bit 7 of
// its byte.
__device__ __forceinline__ uint2 fp_bytes8(uint32_t nib, const FpSteps& st) {
  const uint32_t mags = nib & 0x77777777u, sg = nib & 0x88888888u;
  uint2 by;
  by.x = prmt_u32(st.lut_lo, st.lut_hi, mags) | prmt_u32((sg << 4) & 0x8080u, 0u, 0x4140u) | prmt_u32(sg & 0x8080u, 0u, 0x1404u);
  const uint32_t sh = sg >> 16;
  by.y = prmt_u32(st.lut_lo, st.lut_hi, mags >> 16) | prmt_u32((sh << 4) & 0x8080u, 0u, 0x4140u) | prmt_u32(sh & 0x8080u, 0u, 0x1404u);
  return by;
}

// A selected place of the staged row carries its E4M3 byte in a NaN pattern (exponent field all
// ones, which no finite input has; the byte's sign in the sign bit, its other seven bits,
// complemented, in the mantissa: the byte's low seven bits never reach 0x7F, so the mantissa is
// never zero and the pattern never an infinity).  Every threshold compare of fp_codes2 is false
// for a NaN, so such a place gets code 0 by itself, and the dense pass finds the merged operand's
// byte in the pattern.
__device__ __forceinline__ uint32_t fp_marker(uint32_t q) { return ((q & 0x80u) << 8) | 0x7F80u | ((q & 0x7Fu) ^ 0x7Fu); }
__device__ __forceinline__ uint32_t nan2_mask(uint32_t a) {  // 0xFFFF per half that holds a NaN
  uint32_t d;
  asm("set.nan.u32.bf16x2 %0, %1, %1;" : "=r"(d) : "r"(a));
  return d;
}
// The bytes carried by the markers among four staged elements (two words), zero elsewhere.
__device__ __forceinline__ uint32_t fp_marker_bytes4(uint32_t w0, uint32_t w1) {
  const uint32_t lo4 = prmt_u32(w0, w1, 0x6420u), hi4 = prmt_u32(w0, w1, 0x7531u);  // low / high bytes of the four
  const uint32_t mk4 = prmt_u32(nan2_mask(w0), nan2_mask(w1), 0x6420u);
  return (((lo4 ^ 0x7F7F7F7Fu) & 0x7F7F7F7Fu) | (hi4 & 0x80808080u)) & mk4;
}
// The dense pass over a staged row: E2M1 codes (eight nibbles per word; a selected place has code
// 0) and the merged operand's E4M3 bytes in element order.
__device__ __forceinline__ void dense_sweep_fp(const uint16_t* row, int K, const RowScale& rs, uint8_t* dq4_row, uint8_t* a8_row,
                                               int lane, int gsize) {
  const FpSteps st = fp_steps(rs.inv_lo, rs.e, lane & 31);
  const uint4* src = reinterpret_cast<const uint4*>(row) + lane;
  uint32_t* dst = reinterpret_cast<uint32_t*>(dq4_row) + lane;
  uint2* adst = reinterpret_cast<uint2*>(a8_row) + lane;
  const int iters = (K / 8 - lane + gsize - 1) / gsize;
#pragma unroll 2
  for (int i = 0; i < iters; ++i, src += gsize, dst += gsize, adst += gsize) {
    const uint4 v = *src;
    const uint32_t c0 = fp_codes2(v.x, st), c1 = fp_codes2(v.y, st), c2 = fp_codes2(v.z, st), c3 = fp_codes2(v.w, st);
    const uint32_t nib = ((c0 | (c0 >> 12)) & 0xFFu) | (((c1 | (c1 >> 12)) & 0xFFu) << 8) | (((c2 | (c2 >> 12)) & 0xFFu) << 16) |
                         ((c3 | (c3 >> 12)) << 24);
    const uint2 by = fp_bytes8(nib, st);
    *dst = nib;
    *adst = make_uint2(by.x | fp_marker_bytes4(v.x, v.y), by.y | fp_marker_bytes4(v.z, v.w));
  }
}

struct EncodeParams {
  const uint16_t* X;
  const uint8_t* positions;
  uint8_t* dq4;
  int8_t* vals;
  uint8_t* idx;
  float* s_hi;
  float* s_lo;
  uint8_t* shift;
  uint8_t* a8;        // merged 8-bit operand [M, K] (static register kernel, tied scales), or nullptr
  int* status;
  int64_t M;
  int K, k, b;
  int nbuf;           // row buffers per group (1 or 2)
  int rw;             // warps per row group
  int group_stride;   // bytes of shared memory per group
  MulK mk;            // -1, 2, 32, 2^8, 2^16, 2^24 (see MulK)
  const uint16_t* gamma;  // fused normalisation (ring kernel, NORM): its weights [K], else nullptr
  float eps;
};

// A packed pair of the fused normalisation (w and g: two bf16 per word): bf16(bf16(x * r) * gamma),
// the first product in fp32, the second exact before its rounding; both roundings to nearest even.
__device__ __forceinline__ uint32_t norm2(uint32_t w, float r, uint32_t g) {
  const float lo = __fmul_rn(__uint_as_float(w << 16), r), hi = __fmul_rn(__uint_as_float(w & 0xFFFF0000u), r);
  uint32_t t, y;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(t) : "f"(hi), "f"(lo));
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(y) : "r"(t), "r"(g));
  return y;
}
// A packed pair normalised as above, their squares added to the fp64 sum `acc` on the way in
// (the widened values serve both).
__device__ __forceinline__ void sq2_add(uint32_t w, double& acc) {
  const double lo = (double)__uint_as_float(w << 16), hi = (double)__uint_as_float(w & 0xFFFF0000u);
  acc = fma(lo, lo, acc);
  acc = fma(hi, hi, acc);
}

__device__ __forceinline__ void group_sync(int rw, int grp) {
  if (rw == 1) __syncwarp();
  else asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(rw * 32) : "memory");
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// Row-group kernel.  B = bank size; KK = k for dynamic positions (a power of two), 0 for static.
template <int B, int KK, bool FP = false, bool NORM = false>
__global__ void __launch_bounds__(B == 128 ? 256 : 512) encode_rows_kernel(const EncodeParams p) {
  extern __shared__ __align__(128) uint8_t smem_enc[];
  constexpr bool kStatic = (KK == 0);
  constexpr int NP = B / 2;          // packed registers per bank
  constexpr int NCH = B / 8;         // 16-byte chunks per bank
  constexpr int NM = (B + 63) / 64;  // 64-bit mask words per bank
  const int warp = threadIdx.x >> 5;
  const int rw = p.rw, grp = warp / rw;
  const int lane = (warp % rw) * 32 + (threadIdx.x & 31);  // lane within the row group
  const int gsize = rw * 32;
  const int ngroups = (blockDim.x >> 5) / rw;
  const int K = p.K, G = K / B, k = kStatic ? p.k : KK;
  const int GK = G * k;
  const int nbuf = p.nbuf;
  const MulK mk = p.mk;

  // shared memory: [static only: table of selected element offsets, uint16 [GK]] then per group
  // [nbuf rows][stash of selected raw values, uint16 [GK]][4 mbarriers][4 x 16 exchange words]
  // A successor that was launched with permission to start early may do so now: what it does before
  // its own wait for this kernel (the few-token product fetches its first weight tiles) runs beside
  // the encode.  (This kernel itself starts only when its predecessor has completed.)
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const size_t table_bytes = kStatic ? (((size_t)GK * 2 + 127) & ~(size_t)127) : 0;
  uint16_t* jt = reinterpret_cast<uint16_t*>(smem_enc);
  uint8_t* wbase = smem_enc + table_bytes + (size_t)grp * p.group_stride;
  uint16_t* stash = reinterpret_cast<uint16_t*>(wbase + (size_t)nbuf * K * 2);
  // (floating-point variant: the stash is followed by the selected places' element offsets)
  const size_t stash_half = ((size_t)GK * 2 + 15) & ~(size_t)15;
  const size_t stash_bytes = stash_half * (FP ? 2 : 1);
  uint16_t* spos = reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(stash) + stash_half);
  const uint32_t bar0 = smem_u32(reinterpret_cast<uint8_t*>(stash) + stash_bytes);
  uint32_t* exch = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(stash) + stash_bytes + 32);
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;

  if (threadIdx.x == 0) abort_flag_s = 0;
  if (lane == 0) {
    for (int i = 0; i < 4; ++i) mbar_init(bar0 + 8 * i, 1);
    fence_mbar_init();
  }
  if constexpr (kStatic) {
    // element offset inside a row of every selected position, in the order vals are stored
    for (int t = threadIdx.x; t < GK; t += blockDim.x) jt[t] = (uint16_t)((t / k) * B + p.positions[t]);
  }
  __syncthreads();

  const int64_t gw = (int64_t)blockIdx.x * ngroups + grp;
  const int64_t wstride = (int64_t)gridDim.x * ngroups;
  const uint32_t row_bytes = (uint32_t)K * 2;

  // Ring of nbuf row buffers: the row processed in iteration `it` sits in buffer it % nbuf and
  // rows up to nbuf - 1 iterations ahead are already on their way (with one buffer the next
  // row is requested only after the current one is done).
  const int ahead = nbuf > 1 ? nbuf - 1 : 1;
  if (lane == 0) {
    for (int i = 0; i < ahead; ++i) {
      const int64_t mi = gw + (int64_t)i * wstride;
      if (mi < p.M && (nbuf > 1 || i == 0))
        bulk_copy_g2s(smem_u32(wbase + (size_t)i * row_bytes), p.X + mi * K, row_bytes, bar0 + 8 * i);
    }
  }

  uint32_t cur = 0, parity = 0;
  for (int64_t m = gw; m < p.M; m += wstride) {
    uint16_t* row = reinterpret_cast<uint16_t*>(wbase + (size_t)cur * row_bytes);
    if (nbuf > 1 && lane == 0) {
      // the buffer released at the end of the previous iteration takes the row `ahead` steps on
      const int64_t mn = m + (int64_t)ahead * wstride;
      const uint32_t nb = cur == 0 ? (uint32_t)nbuf - 1 : cur - 1;
      if (mn < p.M) bulk_copy_g2s(smem_u32(wbase + (size_t)nb * row_bytes), p.X + mn * K, row_bytes, bar0 + 8 * nb);
    }
    if (!mbar_wait_park(bar0 + 8 * cur, parity, abort_flag)) break;
    // the row this group takes next is asked into L2 now, so that the copy issued when this row
    // is done (the buffer is single) finds it there
    if (nbuf == 1 && lane == 0 && m + wstride < p.M)
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p.X + (m + wstride) * K), "r"(row_bytes) : "memory");

    if constexpr (NORM) {
      // Fused normalisation: the staged row is replaced by bf16(bf16(x * r) * gamma), r from the
      // row's mean of squares in fp64 (every square exact; four chains per lane), before anything
      // else looks at it -- the rest of the kernel then encodes the normalised row.
      uint4* rc = reinterpret_cast<uint4*>(row);
      double s4[4] = {0.0, 0.0, 0.0, 0.0};
      for (int c = lane; c < K / 8; c += gsize) {
        const uint4 v = rc[c];
        sq2_add(v.x, s4[0]);
        sq2_add(v.y, s4[1]);
        sq2_add(v.z, s4[2]);
        sq2_add(v.w, s4[3]);
      }
      double ss = (s4[0] + s4[1]) + (s4[2] + s4[3]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      if (rw > 1) {
        uint32_t* exn = exch + 64;  // 2 x 16 words of their own
        if ((threadIdx.x & 31) == 0) {
          exn[warp % rw] = (uint32_t)__double2loint(ss);
          exn[16 + warp % rw] = (uint32_t)__double2hiint(ss);
        }
        group_sync(rw, grp);
        ss = 0.0;
        for (int w = 0; w < rw; ++w) ss += __hiloint2double((int)exn[16 + w], (int)exn[w]);
      }
      const float rn = (float)(1.0 / sqrt(ss / (double)K + (double)p.eps));
      const uint4* gc = reinterpret_cast<const uint4*>(p.gamma);
      for (int c = lane; c < K / 8; c += gsize) {
        uint4 v = rc[c];
        const uint4 g = __ldg(gc + c);
        v.x = norm2(v.x, rn, g.x);
        v.y = norm2(v.y, rn, g.y);
        v.z = norm2(v.z, rn, g.z);
        v.w = norm2(v.w, rn, g.w);
        rc[c] = v;
      }
      group_sync(rw, grp);  // the banks a lane reads below were written by other lanes
    }

    // lane_rmax: static positions: the largest unselected magnitude.  Dynamic positions: an UPPER
    // bound of it (the largest k-th magnitude of any bank), with lane_rlow a LOWER bound (see below).
    uint32_t lane_amax = 0, lane_rmax = 0, lane_rlow = 0;
    if constexpr (!kStatic) {
      // ------------------------------------------------------------ phase 1: selection
      // conflict-free chunk rotation: consecutive lanes start on different 16-byte bank groups
      const int rot = (B == 32) ? ((lane >> 1) & (NCH - 1)) : (lane & (NCH - 1));
      for (int g = lane; g < G; g += gsize) {
        uint16_t* bank = row + g * B;
        // k-th largest magnitude: sorted runs of KK per column, merged with truncation
        uint32_t x[NP], s[NP];
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const uint4 v = *reinterpret_cast<const uint4*>(bank + ((c + rot) & (NCH - 1)) * 8);
          x[4 * c] = abs2(v.x);
          x[4 * c + 1] = abs2(v.y);
          x[4 * c + 2] = abs2(v.z);
          x[4 * c + 3] = abs2(v.w);
        }
#pragma unroll
        for (int i = 0; i < NP; ++i) s[i] = x[i];
#pragma unroll
        for (int grp2 = 0; grp2 < NP / KK; ++grp2) sort_desc<KK>(s + grp2 * KK);
#pragma unroll
        for (int span = KK; span < NP; span *= 2) {
#pragma unroll
          for (int a = 0; a + span < NP; a += 2 * span) {
#pragma unroll
            for (int i = 0; i < KK; ++i) s[a + i] = max2(s[a + i], s[a + span + KK - 1 - i]);
            bitonic_merge_desc<KK>(s + a);
          }
        }
        // s[0..KK): per column the KK largest, descending.  Pairing entry i of one column with
        // entry KK-1-i of the other splits those 2*KK values into their KK largest (the larger of
        // each pair) and the rest (the smaller of each pair): T = the smallest of the former is the
        // bank's k-th largest magnitude (with multiplicity), and the largest of the latter is a
        // LOWER bound of the bank's (k+1)-th largest, i.e. of its largest unselected magnitude.
        // (Both halves of a register hold a pair, so half of the entries cover all pairs.)
        constexpr int HP = KK >= 2 ? KK / 2 : 1;
        uint32_t dmin, lmax;
        {
          uint32_t d[HP], l[HP];
#pragma unroll
          for (int i = 0; i < HP; ++i) {
            const uint32_t o = swap_halves(s[KK - 1 - i]);
            d[i] = max2(s[i], o);
            l[i] = min2(s[i], o);
          }
#pragma unroll
          for (int w = HP / 2; w >= 1; w /= 2) {
#pragma unroll
            for (int i = 0; i < w; ++i) {
              d[i] = min2(d[i], d[i + w]);
              l[i] = max2(l[i], l[i + w]);
            }
          }
          dmin = min(d[0] & 0xFFFFu, d[0] >> 16);
          lmax = max(l[0] & 0xFFFFu, l[0] >> 16);
        }
        const uint32_t T = dmin;  // k-th largest magnitude of the bank (with multiplicity)
        const uint32_t bank_max = max(s[0] & 0xFFFFu, s[0] >> 16);
        lane_amax = max(lane_amax, bank_max);

        // compare pass: one flag per element reaching T.  Register q of a 16-element group holds
        // elements 2q and 2q+1; its flags go to bits 2q and 17+2q of the group's word, so that
        // (word | word >> 16) has the group's 16 flags in element order in its low half.
        const uint32_t T2 = T * 0x10001u;
        uint32_t acc[NP / 8];
#pragma unroll
        for (int w = 0; w < NP / 8; ++w) acc[w] = 0;
#pragma unroll
        for (int q = 0; q < NP; ++q) acc[q / 8] |= ge2_mask(x[q], T2) & (0x00020001u << (2 * (q % 8)));
        uint64_t sel[NM];
#pragma unroll
        for (int w = 0; w < NM; ++w) sel[w] = 0;
#pragma unroll
        for (int w = 0; w < NP / 16; ++w) {
          const uint32_t f0 = acc[2 * w] | (acc[2 * w] >> 16), f1 = acc[2 * w + 1] | (acc[2 * w + 1] >> 16);
          sel[w / 2] |= (uint64_t)__byte_perm(f0, f1, 0x5410) << (32 * (w & 1));
        }
        // slot order -> element order: slot c holds chunk (c + rot) mod NCH
        if (B == 128) {
          const int sh = 8 * rot;  // 0..120
          uint64_t lo = sel[0], hi = sel[NM - 1];
          if (sh >= 64) {
            const uint64_t t = lo;
            lo = hi;
            hi = t;
          }
          const int r = sh & 63;
          if (r) {
            const uint64_t nlo = (lo << r) | (hi >> (64 - r)), nhi = (hi << r) | (lo >> (64 - r));
            lo = nlo;
            hi = nhi;
          }
          sel[0] = lo;
          sel[NM - 1] = hi;
        } else if (B == 64) {
          const int r = 8 * rot;
          if (r) sel[0] = (sel[0] << r) | (sel[0] >> (64 - r));
        } else {
          const uint32_t v = (uint32_t)sel[0];
          sel[0] = (uint64_t)__funnelshift_l(v, v, 8 * rot);
        }
        int cnt = 0;
#pragma unroll
        for (int w = 0; w < NM; ++w) cnt += __popcll(sel[w]);
        uint32_t rest_low = lmax;
        if (cnt > KK) {
          // more than k elements reach T: drop the equal ones with the largest indices; the
          // largest unselected magnitude of this bank is then T itself
          rest_low = T;
          int excess = cnt - KK;
#pragma unroll
          for (int w = NM - 1; w >= 0; --w) {
            uint64_t scan = sel[w];
            while (excess > 0 && scan != 0) {
              const int pos = 63 - __clzll((long long)scan);
              scan &= ~(1ull << pos);
              if ((uint32_t)(bank[64 * w + pos] & 0x7FFFu) == T) {
                sel[w] &= ~(1ull << pos);
                --excess;
              }
            }
          }
        }
        lane_rmax = max(lane_rmax, T);
        lane_rlow = max(lane_rlow, rest_low);

        // the k selected elements in ascending position: raw values to the stash, zero in the
        // staged row, positions to global memory (they do not depend on the scale)
        uint32_t iout[(KK + 3) / 4];
#pragma unroll
        for (int w = 0; w < (KK + 3) / 4; ++w) iout[w] = 0;
        uint32_t m0 = (uint32_t)sel[0], m1 = (uint32_t)(sel[0] >> 32), m2 = 0, m3 = 0;
        if (NM == 2) {
          m2 = (uint32_t)sel[NM - 1];
          m3 = (uint32_t)(sel[NM - 1] >> 32);
        }
        uint16_t* sg = stash + g * KK;
        // positions first (bit arithmetic only), then all loads, then all stores: the loads of
        // the k raw values are then in flight together instead of each waiting behind the
        // previous element's stores
        uint32_t pos[KK];
#pragma unroll
        for (int i = 0; i < KK; ++i) {
          // lowest set bit of the (up to 128-bit) mask, then clear it.  Which word it sits in is
          // a 0/1 flag per word (min(word, 1)); selecting the word, adding its base and writing the
          // remainder back are multiply-adds by those flags, not compares and selects.
          uint32_t word, rest_bits;
          if (B == 32) {
            word = m0;
            pos[i] = (uint32_t)(__ffs((int)word) - 1);
            m0 = word & (word - 1u);
          } else if (B == 64) {
            const uint32_t n0 = min(m0, 1u), z0 = imad(n0, mk.neg1, 1u);   // m0 != 0, m0 == 0
            word = imad(z0, m1, m0);                                       // m0 == 0 ? m1 : m0
            pos[i] = imad(z0, mk.k32, (uint32_t)(__ffs((int)word) - 1));
            rest_bits = word & (word - 1u);
            m0 = imad(n0, rest_bits, 0u);                                  // stays 0 once empty
            m1 = imad(z0, rest_bits, imad(n0, m1, 0u));
          } else {
            const bool z0 = m0 == 0;
            word = z0 ? m1 : m0;
            uint32_t base = z0 ? 32u : 0u;
            const bool z1 = (m0 | m1) == 0;
            const bool z2 = z1 && m2 == 0;
            word = z1 ? (z2 ? m3 : m2) : word;
            base = z1 ? (z2 ? 96u : 64u) : base;
            pos[i] = base + (uint32_t)(__ffs((int)word) - 1);
            rest_bits = word & (word - 1u);
            m0 = base == 0 ? rest_bits : m0;
            m1 = base == 32 ? rest_bits : m1;
            m2 = base == 64 ? rest_bits : m2;
            m3 = base == 96 ? rest_bits : m3;
          }
          // position byte i of the bank's index list
          iout[i / 4] = (i % 4) == 0 ? pos[i]
                                     : imad(pos[i], (i % 4) == 1 ? mk.k256 : ((i % 4) == 2 ? mk.k65536 : mk.k16m), iout[i / 4]);
        }
        if constexpr (FP) {
          uint16_t* sp = spos + g * KK;
          const uint32_t e0 = (uint32_t)(g * B);
          if (KK >= 8) {
#pragma unroll
            for (int i = 0; i < KK; i += 8)
              *reinterpret_cast<uint4*>(sp + i) =
                  make_uint4((e0 + pos[i]) | ((e0 + pos[i + 1]) << 16), (e0 + pos[i + 2]) | ((e0 + pos[i + 3]) << 16),
                             (e0 + pos[i + 4]) | ((e0 + pos[i + 5]) << 16), (e0 + pos[i + 6]) | ((e0 + pos[i + 7]) << 16));
          } else {
#pragma unroll
            for (int i = 0; i < KK; ++i) sp[i] = (uint16_t)(e0 + pos[i]);
          }
        }
        uint32_t raw[KK];
        const uint32_t bank_s = smem_u32(bank);
#pragma unroll
        for (int i = 0; i < KK; ++i) {
          const uint32_t addr = imad(pos[i], mk.two, bank_s);
          asm volatile("ld.shared.u16 %0, [%1];" : "=r"(raw[i]) : "r"(addr));
          pos[i] = addr;
        }
#pragma unroll
        for (int i = 0; i < KK; ++i) asm volatile("st.shared.u16 [%0], %1;" ::"r"(pos[i]), "h"((uint16_t)0) : "memory");
        if (KK >= 8) {
#pragma unroll
          for (int i = 0; i < KK; i += 8)
            *reinterpret_cast<uint4*>(sg + i) = make_uint4(raw[i] | (raw[i + 1] << 16), raw[i + 2] | (raw[i + 3] << 16),
                                                           raw[i + 4] | (raw[i + 5] << 16), raw[i + 6] | (raw[i + 7] << 16));
        } else if (KK == 4) {
          *reinterpret_cast<uint2*>(sg) = make_uint2(raw[0] | (raw[1] << 16), raw[2] | (raw[3] << 16));
        } else if (KK == 2) {
          *reinterpret_cast<uint32_t*>(sg) = raw[0] | (raw[1] << 16);
        } else {
          sg[0] = (uint16_t)raw[0];
        }
        uint8_t* idst = p.idx + ((size_t)m * G + g) * KK;
        if (KK >= 16) {
#pragma unroll
          for (int w = 0; w < KK / 16; ++w)
            reinterpret_cast<uint4*>(idst)[w] = make_uint4(iout[4 * w], iout[4 * w + 1], iout[4 * w + 2], iout[4 * w + 3]);
        } else if (KK == 8) {
          *reinterpret_cast<uint2*>(idst) = make_uint2(iout[0], iout[1]);
        } else if (KK == 4) {
          *reinterpret_cast<uint32_t*>(idst) = iout[0];
        } else if (KK == 2) {
          *reinterpret_cast<uint16_t*>(idst) = (uint16_t)iout[0];
        } else {
          *idst = (uint8_t)iout[0];
        }
      }
    } else {
      // ------------------------------------------------------------ phase 1 (static): stash and zero
#pragma unroll 4
      for (int t = lane; t < GK; t += gsize) {
        const int j = jt[t];
        const uint16_t v = row[j];
        stash[t] = v;
        row[j] = 0;
        lane_amax = max(lane_amax, (uint32_t)(v & 0x7FFFu));
      }
      group_sync(rw, grp);
      const uint4* src = reinterpret_cast<const uint4*>(row) + lane;
      const int iters = (K / 8 - lane + gsize - 1) / gsize;
#pragma unroll 4
      for (int i = 0; i < iters; ++i, src += gsize) {
        const uint4 v = *src;
        const uint32_t mx = max2(max2(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu), max2(v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu));
        lane_rmax = max(lane_rmax, max(mx & 0xFFFFu, mx >> 16));
      }
      lane_amax = max(lane_amax, lane_rmax);
    }

    uint32_t amax_bits = __reduce_max_sync(0xffffffffu, lane_amax);
    uint32_t rmax_bits = __reduce_max_sync(0xffffffffu, lane_rmax);
    uint32_t rlow_bits = kStatic ? 0u : __reduce_max_sync(0xffffffffu, lane_rlow);
    if (rw > 1) {
      if ((threadIdx.x & 31) == 0) {
        exch[warp % rw] = amax_bits;
        exch[16 + warp % rw] = rmax_bits;
        if (!kStatic) exch[32 + warp % rw] = rlow_bits;
      }
      group_sync(rw, grp);  // also: every stash entry of the row is written
      amax_bits = rmax_bits = rlow_bits = 0;
      for (int w = 0; w < rw; ++w) {
        amax_bits = max(amax_bits, exch[w]);
        rmax_bits = max(rmax_bits, exch[16 + w]);
        if (!kStatic) rlow_bits = max(rlow_bits, exch[32 + w]);
      }
    } else {
      __syncwarp();
    }
    RowScale rs = FP ? row_scale_fp(amax_bits, rmax_bits) : row_scale_warp(amax_bits, rmax_bits, threadIdx.x & 31);
    if constexpr (!kStatic) {
      // The shift was computed from an upper bound of the largest unselected magnitude.  It is the
      // true one unless the lower bound would still fit one shift less; only then (the same for
      // the whole group) the row, whose selected places are zero by now, is swept for the exact
      // maximum.  (A clamp flag set by the upper bound alone only costs time.)
      const bool exact =
          FP ? fp_shift_of(rs.inv, bf16_bits_to_f32(rlow_bits), rs.inv > 0.f) < rs.e
             : rs.e > 0 && rne_prod(bf16_bits_to_f32(rlow_bits), rs.inv * __int_as_float((127 - (rs.e - 1)) << 23)) <= 7;
      if (exact) {
        const uint4* src = reinterpret_cast<const uint4*>(row) + lane;
        const int iters = (K / 8 - lane + gsize - 1) / gsize;
        uint32_t mx = 0;
#pragma unroll 4
        for (int i = 0; i < iters; ++i, src += gsize) {
          const uint4 v = *src;
          mx = max2(mx, max2(max2(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu), max2(v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu)));
        }
        uint32_t rx = __reduce_max_sync(0xffffffffu, max(mx & 0xFFFFu, mx >> 16));
        if (rw > 1) {
          if ((threadIdx.x & 31) == 0) exch[48 + warp % rw] = rx;
          group_sync(rw, grp);
          rx = 0;
          for (int w = 0; w < rw; ++w) rx = max(rx, exch[48 + w]);
        }
        rs = FP ? row_scale_fp(amax_bits, rx) : row_scale_warp(amax_bits, rx, threadIdx.x & 31);
      }
    }
    if (lane == 0) {
      p.s_hi[m] = rs.s_hi;
      p.s_lo[m] = rs.s_lo;
      p.shift[m] = (uint8_t)rs.e;
    }

    // -------------------------------------------------------------- phase 2a: sparse component
    if constexpr (FP) {
      // E4M3 bytes of the selected values; their places in the staged row (zero until now) get
      // the marker that carries the byte
      uint8_t* vdst = reinterpret_cast<uint8_t*>(p.vals) + (size_t)m * GK;
      for (int t = lane; t < GK; t += gsize) {
        const uint32_t q = e4m3_of32(stash[t], rs.inv);
        vdst[t] = (uint8_t)q;
        row[spos[t]] = (uint16_t)fp_marker(q);
      }
      group_sync(rw, grp);
      dense_sweep_fp(row, K, rs, p.dq4 + (size_t)m * (K / 2), p.a8 + (size_t)m * K, lane, gsize);
    } else {
      int8_t* vdst = p.vals + (size_t)m * GK;
      if ((GK & 3) == 0) {
        for (int t4 = lane * 4; t4 < GK; t4 += gsize * 4) {
          const uint2 sv = *reinterpret_cast<const uint2*>(stash + t4);
          const uint32_t w[2] = {sv.x, sv.y};
          uint32_t o = 0;
#pragma unroll
          for (int q = 0; q < 2; ++q) {  // |a * inv| <= 127 by construction: no clamp
            const uint32_t q0 = __float_as_uint(__fmaf_rn(__uint_as_float(w[q] << 16), rs.inv, kMagic)) & 0xFFu;
            const uint32_t q1 = __float_as_uint(__fmaf_rn(__uint_as_float(w[q] & 0xFFFF0000u), rs.inv, kMagic)) & 0xFFu;
            o |= (q0 << (16 * q)) | (q1 << (16 * q + 8));
          }
          *reinterpret_cast<uint32_t*>(vdst + t4) = o;
        }
      } else {
        for (int t = lane; t < GK; t += gsize)
          vdst[t] = (int8_t)(__float_as_uint(__fmaf_rn(bf16_bits_to_f32(stash[t]), rs.inv, kMagic)) & 0xFFu);
      }
    }

    // -------------------------------------------------------------- phase 2b: dense component
    // (the group barrier above also ordered the zeroing of the selected places before this sweep)
    if constexpr (!FP) dense_sweep(row, K, rs, p.dq4 + (size_t)m * (K / 2), lane, gsize);

    // the row buffer is about to be refilled by the async proxy: order this group's generic
    // accesses before it
    fence_proxy_async_smem();
    group_sync(rw, grp);
    if (nbuf == 1 && m + wstride < p.M && lane == 0)
      bulk_copy_g2s(smem_u32(wbase), p.X + (m + wstride) * K, row_bytes, bar0);
    if (++cur == (uint32_t)nbuf) {
      cur = 0;
      parity ^= 1u;
    }
  }
  if (*abort_flag && lane == 0) atomicExch(p.status, (int)SQ_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------
// Static positions, row held in registers.  A row is split over `rw` warps; each warp keeps its
// slice of NCL * 256 elements in NCL 16-byte register quads per lane (lane l owns chunks l,
// l + 32, ...: every load and every INT4 store is one fully coalesced warp access) and nothing
// of the row is staged in shared memory.  What the positions imply is the same for every row,
// so it is tabulated once per block: per element a half-word magnitude mask (0x7FFF, or 0 at a
// selected place) and the element offset of every selected place.  Per row:
//   load; in the same breath fetch the selected values a second time (asynchronous 4-byte
//   copies into shared memory) -> maxima of all and of the unselected magnitudes -> scales
//   -> INT8 codes of the selected values, INT4 codes straight from the registers (selected
//   places were cleared there while taking the maxima).
// The kernel is bound by instruction issue, which is why the masks are tables.
// On request (tied scales) the row's merged 8-bit operand for the product is written as well:
// the dense codes are at hand as bytes while they are packed, so it costs two shifts, two
// logic operations and two stores per eight elements, plus one byte store per selected place
// -- instead of a second kernel that reads the codes back and expands them.
template <int NCL, int NT, bool INDEP>
__global__ void __launch_bounds__(NT, 1) encode_static_regs_kernel(const EncodeParams p) {
  extern __shared__ __align__(128) uint8_t smem_enc[];
  const int K = p.K, k = p.k;
  const int GK = (K / p.b) * k;
  const int rw = p.rw;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = warp / rw, slice = warp % rw;
  const int glane = slice * 32 + lane, gsize = rw * 32;
  const int ngroups = (NT / 32) / rw;
  constexpr int S8 = NCL * 32;  // 16-byte chunks per warp slice

  // shared memory: [magnitude masks, uint16 [K]] [selected offsets, uint16 [GK]] then per group [gathered words, uint32 [GK]] and, after all
  // of those, 32 exchange words per group
  const size_t jt_bytes = ((size_t)GK * 2 + 15) & ~(size_t)15;
  const size_t stash_bytes = ((size_t)GK * 4 + 15) & ~(size_t)15;
  uint16_t* hmask = reinterpret_cast<uint16_t*>(smem_enc);
  uint16_t* jt = hmask + K;
  uint32_t* stash = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(jt) + jt_bytes + stash_bytes * grp);
  uint32_t* exch = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(jt) + jt_bytes + stash_bytes * ngroups) + grp * 32;
  // With the merged operand asked for: per group an image of a row's selected places in the order
  // the dense loop walks (chunk by chunk, [4 even | 4 odd] bytes): INT8 code ^ 0x80 there, 0x80
  // everywhere else (written once); and, once per block, where in the image each place lies.
  uint8_t* img = reinterpret_cast<uint8_t*>(jt) + jt_bytes + (stash_bytes + 128) * ngroups + (size_t)K * grp;
  uint16_t* jimg = reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(jt) + jt_bytes + (stash_bytes + 128 + (size_t)K) * ngroups);
  const bool want_a8 = !INDEP && p.a8 != nullptr;
  const uint32_t stash_s = smem_u32(stash);

  for (int i = threadIdx.x; i < K / 2; i += NT) reinterpret_cast<uint32_t*>(hmask)[i] = 0x7FFF7FFFu;
  __syncthreads();
  for (int t = threadIdx.x; t < GK; t += NT) {
    const int j = (t / k) * p.b + p.positions[t];
    jt[t] = (uint16_t)j;
    hmask[j] = 0;
    if (want_a8) jimg[t] = (uint16_t)((j & ~7) | ((j & 1) << 2) | ((j & 7) >> 1));
  }
  if (want_a8)
    for (int i = threadIdx.x; i < (K / 4) * ngroups; i += NT)
      reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(jt) + jt_bytes + (stash_bytes + 128) * ngroups)[i] = 0x80808080u;
  __syncthreads();

  const int64_t gw = (int64_t)blockIdx.x * ngroups + grp;
  const int64_t wstride = (int64_t)gridDim.x * ngroups;
  for (int64_t m = gw; m < p.M; m += wstride) {
    const uint16_t* xrow = p.X + m * K;
    const uint4* src = reinterpret_cast<const uint4*>(xrow) + slice * S8 + lane;
    uint4 v[NCL];
#pragma unroll
    for (int c = 0; c < NCL; ++c) v[c] = __ldg(src + c * 32);
    // The selected values come a second time, as the aligned 32-bit words that hold them,
    // by asynchronous copies straight into shared memory: all in flight together with the
    // row itself, no registers held.
#pragma unroll 4
    for (int t = glane; t < GK; t += gsize) {
      const uint32_t j = jt[t];
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(stash_s + 4u * (uint32_t)t), "l"(xrow + (j & ~1u))
                   : "memory");
    }

    const uint4* mk = reinterpret_cast<const uint4*>(hmask) + slice * S8 + lane;
    uint32_t r2 = 0, a2 = 0;
#pragma unroll
    for (int c = 0; c < NCL; ++c) {
      const uint4 q = mk[c * 32];
      // all magnitudes (tied scales), or only the selected ones (independent scales)
      if (INDEP)
        a2 = max2(a2, max2(max2(v[c].x & ~q.x & 0x7FFF7FFFu, v[c].y & ~q.y & 0x7FFF7FFFu),
                           max2(v[c].z & ~q.z & 0x7FFF7FFFu, v[c].w & ~q.w & 0x7FFF7FFFu)));
      else
        a2 = max2(a2, max2(max2(v[c].x & 0x7FFF7FFFu, v[c].y & 0x7FFF7FFFu),
                           max2(v[c].z & 0x7FFF7FFFu, v[c].w & 0x7FFF7FFFu)));
      r2 = max2(r2, max2(max2(v[c].x & q.x, v[c].y & q.y), max2(v[c].z & q.z, v[c].w & q.w)));
      // selected places become (signed) zeros: their codes must not reach the packing below
      v[c].x &= q.x | 0x80008000u;
      v[c].y &= q.y | 0x80008000u;
      v[c].z &= q.z | 0x80008000u;
      v[c].w &= q.w | 0x80008000u;
    }
    const uint32_t lane_rmax = max(r2 & 0xFFFFu, r2 >> 16);

    const uint32_t lane_amax = max(a2 & 0xFFFFu, a2 >> 16);  // selected places included
    asm volatile("cp.async.wait_all;" ::: "memory");

    uint32_t amax_bits = __reduce_max_sync(0xffffffffu, lane_amax);
    uint32_t rmax_bits = __reduce_max_sync(0xffffffffu, lane_rmax);
    if (rw > 1) {
      if (lane == 0) {
        exch[slice] = amax_bits;
        exch[16 + slice] = rmax_bits;
      }
      group_sync(rw, grp);  // also: every gathered word of the row is in the stash
      amax_bits = rmax_bits = 0;
      for (int w = 0; w < rw; ++w) {
        amax_bits = max(amax_bits, exch[w]);
        rmax_bits = max(rmax_bits, exch[16 + w]);
      }
    } else {
      __syncwarp();
    }
    const RowScale rs = INDEP ? row_scale_indep(amax_bits, rmax_bits) : row_scale_warp(amax_bits, rmax_bits, lane);
    if (glane == 0) {
      p.s_hi[m] = rs.s_hi;
      p.s_lo[m] = rs.s_lo;
      p.shift[m] = (uint8_t)rs.e;
    }

    // sparse component: INT8 codes of the gathered values (|a * inv| <= 127 by construction)
    {
      int8_t* vdst = p.vals + (size_t)m * GK;
      if ((GK & 3) == 0) {
        for (int t4 = glane * 4; t4 < GK; t4 += gsize * 4) {
          const uint4 sw = *reinterpret_cast<const uint4*>(stash + t4);
          const uint2 jj = *reinterpret_cast<const uint2*>(jt + t4);
          const uint32_t w[4] = {sw.x, sw.y, sw.z, sw.w};
          const uint32_t odd[4] = {jj.x & 1u, (jj.x >> 16) & 1u, jj.y & 1u, (jj.y >> 16) & 1u};
          uint32_t o = 0;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t a = odd[q] ? (w[q] & 0xFFFF0000u) : (w[q] << 16);
            o |= (__float_as_uint(__fmaf_rn(__uint_as_float(a), rs.inv, kMagic)) & 0xFFu) << (8 * q);
          }
          *reinterpret_cast<uint32_t*>(vdst + t4) = o;
          if (want_a8) {
            const uint2 ji = *reinterpret_cast<const uint2*>(jimg + t4);
            const uint32_t ox = o ^ 0x80808080u;
            img[ji.x & 0xFFFFu] = (uint8_t)ox;
            img[ji.x >> 16] = (uint8_t)(ox >> 8);
            img[ji.y & 0xFFFFu] = (uint8_t)(ox >> 16);
            img[ji.y >> 16] = (uint8_t)(ox >> 24);
          }
        }
      } else {
        for (int t = glane; t < GK; t += gsize) {
          const uint32_t a = (jt[t] & 1u) ? (stash[t] & 0xFFFF0000u) : (stash[t] << 16);
          const uint32_t o = __float_as_uint(__fmaf_rn(__uint_as_float(a), rs.inv, kMagic)) & 0xFFu;
          vdst[t] = (int8_t)o;
          if (want_a8) img[jimg[t]] = (uint8_t)(o ^ 0x80u);
        }
      }
    }

    // dense component: INT4 codes of the registers, one 32-bit word per chunk
    uint32_t* dst = reinterpret_cast<uint32_t*>(p.dq4 + (size_t)m * (K / 2)) + slice * S8 + lane;
    const float cq = rs.inv_lo;
    if (rs.clamp) {
      // Codes beyond +-7 are possible: limit the inputs instead of the codes, two elements per
      // instruction.  xl = the bf16 at or just below 7 / cq still rounds to code 7, anything
      // larger in magnitude would round to 7 or more, anything smaller is untouched.
      const uint32_t xl = __float_as_uint(__fdiv_rd(7.0f, cq)) >> 16;
      const uint32_t hi2 = xl | (xl << 16), lo2 = hi2 | 0x80008000u;
#pragma unroll
      for (int c = 0; c < NCL; ++c) {
        v[c].x = max2(min2(v[c].x, hi2), lo2);
        v[c].y = max2(min2(v[c].y, hi2), lo2);
        v[c].z = max2(min2(v[c].z, hi2), lo2);
        v[c].w = max2(min2(v[c].w, hi2), lo2);
      }
    }
    if (want_a8) {
      // The merged operand of the same row, in the product's K order ([16 even | 16 odd] bytes per
      // 32 elements): byte = code * 2^e + 128 for a dense element -- the codes are at hand as bytes
      // -- and INT8 code + 128 at a selected place, where the dense code is 0 and the image has it.
      // chunk c of this lane: elements 8 * wi .. 8 * wi + 7 with wi = slice * S8 + c * 32 + lane, i.e.
      // block wi / 4 = (slice * S8 + lane) / 4 + 8 * c, quarter lane % 4
      uint32_t* aw = reinterpret_cast<uint32_t*>(p.a8 + (size_t)m * K) + ((slice * S8 + lane) >> 2) * 8 + (lane & 3);
      const uint2* iw = reinterpret_cast<const uint2*>(img) + slice * S8 + lane;
      const uint32_t e = (uint32_t)rs.e;
      const uint32_t keep = 0x01010101u * ((0xFFu << e) & 0xFFu);
      group_sync(rw, grp);  // the image holds this row's codes
#pragma unroll
      for (int c = 0; c < NCL; ++c) {
        float r[8];
        uint32_t ev, od;
        quant8(v[c], cq, r);
        dst[c * 32] = pack_nibbles(r, ev, od);
        const uint2 im = iw[c * 32];
        aw[c * 64] = ((ev << e) & keep) ^ im.x;
        aw[c * 64 + 4] = ((od << e) & keep) ^ im.y;
      }
      group_sync(rw, grp);  // the stash, the image and the exchange words are reused by the next row
      continue;
    }
#pragma unroll
    for (int c = 0; c < NCL; ++c) {
      float r[8];
      quant8(v[c], cq, r);
      dst[c * 32] = pack_nibbles(r);
    }
    group_sync(rw, grp);  // the stash and the exchange words are reused by the next row
  }
}

// ------------------------------------------------------------------------------------------------
// Static positions, rows streamed through shared memory.  The register kernel above asks for a
// row only when its warps are ready for it, so the load's latency is hidden by other groups alone
// and the selected values have to be fetched a second time from L1/L2.  Here every group of `rw`
// warps owns a row slot that one bulk asynchronous copy fills (the slot is asked to take its next
// row the moment its row's selected values have been quantised, about half-way through the
// row's work, so the copy's latency is covered by the rest of it), and the selected values are
// plain shared-memory reads of the staged row.  A lane still keeps its NCL 16-byte chunks in
// registers between the maximum pass and the quantising pass, so the row is read from shared
// memory once.  The arithmetic that can be written as a multiply-add (magnitudes, the low half's
// bf16 -> fp32 move, nibble and byte packing) is issued on the multiply-add pipe.  A block owns
// every gridDim.x-th row and its groups draw the next one from a shared counter.
// Measured on 8192 x 8192: every row after a group's first takes ~3.7 us, which over the GPU is
// the memory's full rate; what a launch of this size loses is its start (tables, the first round
// of rows arriving) and its end (the last row's work with nothing left to fetch).
//   wait for the slot -> chunks to registers, selected places cleared, maximum of the rest;
//   maximum of the selected values (read through the offset table) -> group exchange -> scales
//   -> INT8 codes of the selected values (and, on request, their bytes in the per-group image of
//   the merged operand) -> slot released and refilled -> INT4 codes (and merged bytes) straight
//   from the registers.
// MASK8: the per-element magnitude masks are kept as bytes and widened on the fly (long rows,
// where a half-word table would not leave room for the slots).
template <int NCL, int NT, bool INDEP, bool MASK8, bool FP = false, bool NORM = false>
__global__ void __launch_bounds__(NT, 1) encode_static_ring_kernel(const EncodeParams p) {
  extern __shared__ __align__(128) uint8_t smem_enc[];
  const int K = p.K, k = p.k;
  const int GK = (K / p.b) * k;
  const int rw = p.rw;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = warp / rw, slice = warp % rw;
  const int glane = slice * 32 + lane, gsize = rw * 32;
  const int ngroups = (NT / 32) / rw;
  constexpr int S8 = NCL * 32;  // 16-byte chunks per warp slice
  const bool want_a8 = !INDEP && p.a8 != nullptr;
  const MulK mk = p.mk;

  // shared memory: [magnitude masks: uint16 [K], or uint8 [K]] [selected offsets, uint16 [GK]]
  // [their places in the image, uint16 [GK] (merged operand only)] then per group
  // [row slot][image, K bytes (merged operand only)][2 x 32 exchange words][2 next-row words][mbarrier]
  const size_t mask_bytes = MASK8 ? (size_t)K : (size_t)K * 2;
  const size_t jt_bytes = ((size_t)GK * 2 + 15) & ~(size_t)15;
  const size_t row_bytes = (size_t)K * 2;
  uint8_t* hmask = smem_enc;
  uint16_t* jt = reinterpret_cast<uint16_t*>(smem_enc + mask_bytes);
  uint16_t* jimg = reinterpret_cast<uint16_t*>(smem_enc + mask_bytes + jt_bytes);
  // (fused normalisation: its weights [K] and the weights at the selected places [GK] follow the tables)
  uint16_t* gam = reinterpret_cast<uint16_t*>(smem_enc + mask_bytes + jt_bytes * (want_a8 ? 2 : 1));
  uint16_t* gjt = gam + K;
  uint8_t* gbase = smem_enc + mask_bytes + jt_bytes * (want_a8 ? 2 : 1) + (NORM ? row_bytes + jt_bytes : 0) +
                   (size_t)grp * p.group_stride;
  uint8_t* img = gbase + row_bytes;
  uint32_t* exch = reinterpret_cast<uint32_t*>(img + (want_a8 ? (size_t)K : 0));
  volatile int* nexti = reinterpret_cast<volatile int*>(exch + 64);
  const uint32_t bar0 = smem_u32(exch + 66);
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;

  // A block owns the rows blockIdx.x + i * gridDim.x; its groups take the next i from a shared
  // counter whenever they have released their slot, so that no group idles while rows are left.
  __shared__ int next_row_s;
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    next_row_s = ngroups;
    // a successor launched with permission to start early (the few-token product: it fetches only
    // weight tiles until this kernel has completed) may do so now
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  // The first rows are asked for as early as possible, but after the positions: issued before
  // them, the grid's first 19 MB of rows would keep the tables waiting.  So every thread first
  // issues the loads of (up to PQ of) its positions, the block meets, and then the rows go out
  // while the tables are built.  The rows of the second round are asked into L2 at once: memory
  // keeps streaming while the first round is being worked on.
  constexpr int PQ = 4;
  int pj[PQ];
#pragma unroll
  for (int i = 0; i < PQ; ++i) {
    const int t = threadIdx.x + i * NT;
    pj[i] = t < GK ? (int)p.positions[t] : 0;
  }
  int64_t m = (int64_t)blockIdx.x + (int64_t)grp * gridDim.x;
  const uint8_t* slot = gbase;
  const uint16_t* srow = reinterpret_cast<const uint16_t*>(slot);
  if (glane == 0) {
    mbar_init(bar0, 1);
    fence_mbar_init();
  }
  __syncthreads();
  if (glane == 0 && m < p.M) {
    bulk_copy_g2s(smem_u32(slot), p.X + m * K, (uint32_t)row_bytes, bar0);
    const int64_t m2 = m + (int64_t)ngroups * gridDim.x;
    if (m2 < p.M) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p.X + m2 * K), "r"((uint32_t)row_bytes) : "memory");
  }
  if (MASK8) {
    for (int i = threadIdx.x; i < K / 4; i += NT) reinterpret_cast<uint32_t*>(hmask)[i] = 0xFFFFFFFFu;
  } else {
    for (int i = threadIdx.x; i < K / 2; i += NT) reinterpret_cast<uint32_t*>(hmask)[i] = 0x7FFF7FFFu;
  }
  if (want_a8)
    for (int i = glane; i < K / 4; i += gsize) reinterpret_cast<uint32_t*>(img)[i] = 0u;
  if (NORM)
    for (int i = threadIdx.x; i < K / 8; i += NT) reinterpret_cast<uint4*>(gam)[i] = reinterpret_cast<const uint4*>(p.gamma)[i];
  __syncthreads();
  for (int t = threadIdx.x, i = 0; t < GK; t += NT, ++i) {
    int pos = 0;
    if (i < PQ) {
#pragma unroll
      for (int u = 0; u < PQ; ++u)
        if (u == i) pos = pj[u];
    } else {
      pos = p.positions[t];
    }
    const int j = (t / k) * p.b + pos;
    jt[t] = (uint16_t)j;
    if (MASK8) hmask[j] = 0;
    else reinterpret_cast<uint16_t*>(hmask)[j] = 0;
    if (want_a8) jimg[t] = FP ? (uint16_t)j : (uint16_t)((j & ~7) | ((j & 1) << 2) | ((j & 7) >> 1));
    if (NORM) gjt[t] = gam[j];
  }
  __syncthreads();

  const int nquads = GK / 4;
  uint32_t parity = 0, flip = 0;
  while (m < p.M) {
    const bool landed = __all_sync(0xffffffffu, mbar_wait_park(bar0, parity, abort_flag));
    parity ^= 1u;

    uint4 v[NCL];
    uint32_t r2 = 0, smax = 0;
    float rn = 0.f;  // fused normalisation: 1 / sqrt(mean of squares + eps)
    if (landed) {
      const uint4* src = reinterpret_cast<const uint4*>(slot) + slice * S8 + lane;
#pragma unroll
      for (int c = 0; c < NCL; ++c) v[c] = src[c * 32];
    }
    if constexpr (NORM) {
      // The row's mean of squares in fp64 (every square exact), across the group; then the chunks in
      // the registers are replaced by the normalised values (the slot keeps the raw row: the few
      // selected values read from it below are normalised one by one).
      double ss = 0.0;
      if (landed) {
        double s4[4] = {0.0, 0.0, 0.0, 0.0};  // four chains: a lane's 8 * NCL additions must not wait for one another
#pragma unroll
        for (int c = 0; c < NCL; ++c) {
          sq2_add(v[c].x, s4[0]);
          sq2_add(v[c].y, s4[1]);
          sq2_add(v[c].z, s4[2]);
          sq2_add(v[c].w, s4[3]);
        }
        ss = (s4[0] + s4[1]) + (s4[2] + s4[3]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      if (rw > 1) {
        uint32_t* ex = exch + flip * 32;
        if (lane == 0) {
          ex[8 + slice] = (uint32_t)__double2loint(ss);
          ex[24 + slice] = (uint32_t)__double2hiint(ss);
        }
        group_sync(rw, grp);
        ss = 0.0;
        for (int w = 0; w < rw; ++w) ss += __hiloint2double((int)ex[24 + w], (int)ex[8 + w]);
      }
      rn = (float)(1.0 / sqrt(ss / (double)K + (double)p.eps));
      if (landed) {
        const uint4* gsrc = reinterpret_cast<const uint4*>(gam) + slice * S8 + lane;
#pragma unroll
        for (int c = 0; c < NCL; ++c) {
          const uint4 g = gsrc[c * 32];
          v[c].x = norm2(v[c].x, rn, g.x);
          v[c].y = norm2(v[c].y, rn, g.y);
          v[c].z = norm2(v[c].z, rn, g.z);
          v[c].w = norm2(v[c].w, rn, g.w);
        }
      }
    }
    if (landed) {
      // selected places become (signed) zeros; the maximum of what is left
#pragma unroll
      for (int c = 0; c < NCL; ++c) {
        uint4 q;
        if (MASK8) {
          const uint2 q8 = reinterpret_cast<const uint2*>(hmask)[slice * S8 + c * 32 + lane];
          q.x = __byte_perm(q8.x, 0, 0x1100) | 0x80008000u;
          q.y = __byte_perm(q8.x, 0, 0x3322) | 0x80008000u;
          q.z = __byte_perm(q8.y, 0, 0x1100) | 0x80008000u;
          q.w = __byte_perm(q8.y, 0, 0x3322) | 0x80008000u;
          v[c].x &= q.x;
          v[c].y &= q.y;
          v[c].z &= q.z;
          v[c].w &= q.w;
        } else {
          q = reinterpret_cast<const uint4*>(hmask)[slice * S8 + c * 32 + lane];
          v[c].x &= q.x | 0x80008000u;
          v[c].y &= q.y | 0x80008000u;
          v[c].z &= q.z | 0x80008000u;
          v[c].w &= q.w | 0x80008000u;
        }
        r2 = max2(r2, max2(max2(abs2(v[c].x), abs2(v[c].y)), max2(abs2(v[c].z), abs2(v[c].w))));
      }
      // largest selected magnitude, through the offset table
      for (int q4 = glane; q4 < nquads; q4 += gsize) {
        const uint2 jj = *reinterpret_cast<const uint2*>(jt + 4 * q4);
        uint32_t a = srow[jj.x & 0xFFFFu], b = srow[jj.x >> 16], c = srow[jj.y & 0xFFFFu], d = srow[jj.y >> 16];
        if constexpr (NORM) {  // two at a time, as the registers' words
          const uint2 gg = *reinterpret_cast<const uint2*>(gjt + 4 * q4);
          const uint32_t y01 = norm2(a | (b << 16), rn, gg.x), y23 = norm2(c | (d << 16), rn, gg.y);
          a = y01 & 0xFFFFu;
          b = y01 >> 16;
          c = y23 & 0xFFFFu;
          d = y23 >> 16;
        }
        smax = max(max(smax, a & 0x7FFFu), max(max(b & 0x7FFFu, c & 0x7FFFu), d & 0x7FFFu));
      }
    }
    uint32_t rmax_bits = __reduce_max_sync(0xffffffffu, max(r2 & 0xFFFFu, r2 >> 16));
    uint32_t smax_bits = __reduce_max_sync(0xffffffffu, smax);
    if (!landed) smax_bits = 0xFFFFFFFFu;  // tells the whole group to stop together
    if (rw > 1) {
      uint32_t* ex = exch + flip * 32;
      if (lane == 0) {
        ex[slice] = smax_bits;
        ex[16 + slice] = rmax_bits;
      }
      group_sync(rw, grp);
      smax_bits = rmax_bits = 0;
      for (int w = 0; w < rw; ++w) {
        smax_bits = max(smax_bits, ex[w]);
        rmax_bits = max(rmax_bits, ex[16 + w]);
      }
    }
    if (smax_bits == 0xFFFFFFFFu) break;
    const uint32_t amax_bits = INDEP ? smax_bits : max(smax_bits, rmax_bits);
    RowScale rs;
    if constexpr (FP) {
      // floating-point variant: the row maximum maps to 256, the dense grid is coarser by the
      // smallest power of two (up to 2^6) that brings the largest unselected magnitude to at most 6
      const float amax = bf16_bits_to_f32(amax_bits), rmax = bf16_bits_to_f32(rmax_bits);
      rs.inv = amax > 0.f ? __fdiv_rn(256.0f, amax) : 0.f;
      rs.s_hi = amax > 0.f ? __fdiv_rn(amax, 256.0f) : 0.f;
      int e = 0;
      if (amax > 0.f) {
        e = 6;
#pragma unroll
        for (int t = 6; t >= 0; --t)
          if ((double)rmax * (double)(rs.inv * __int_as_float((127 - t) << 23)) <= 6.0) e = t;  // ends on the smallest fitting t
      }
      rs.e = e;
      rs.s_lo = rs.s_hi * (float)(1 << e);
      rs.inv_lo = rs.inv * __int_as_float((127 - e) << 23);
      rs.clamp = false;  // the code construction saturates by itself
    } else {
      rs = INDEP ? row_scale_indep(amax_bits, rmax_bits) : row_scale_warp(amax_bits, rmax_bits, lane);
    }
    if (glane == 0) {
      p.s_hi[m] = rs.s_hi;
      p.s_lo[m] = rs.s_lo;
      p.shift[m] = (uint8_t)rs.e;
    }

    // sparse component: INT8 codes of the selected values, four per lane and step
    {
      int8_t* vdst = p.vals + (size_t)m * GK;
#pragma unroll 2
      for (int q4 = glane; q4 < nquads; q4 += gsize) {
        const uint2 jj = *reinterpret_cast<const uint2*>(jt + 4 * q4);
        uint32_t w[4] = {srow[jj.x & 0xFFFFu], srow[jj.x >> 16], srow[jj.y & 0xFFFFu], srow[jj.y >> 16]};
        if constexpr (NORM) {
          const uint2 gg = *reinterpret_cast<const uint2*>(gjt + 4 * q4);
          const uint32_t y01 = norm2(w[0] | (w[1] << 16), rn, gg.x), y23 = norm2(w[2] | (w[3] << 16), rn, gg.y);
          w[0] = y01 & 0xFFFFu;
          w[1] = y01 >> 16;
          w[2] = y23 & 0xFFFFu;
          w[3] = y23 >> 16;
        }
        uint32_t o = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if constexpr (FP) o |= e4m3_of32(w[q], rs.inv) << (8 * q);
          else o |= (__float_as_uint(__fmaf_rn(__uint_as_float(w[q] << 16), rs.inv, kMagic)) & 0xFFu) << (8 * q);
        }
        *reinterpret_cast<uint32_t*>(vdst + 4 * q4) = o;
        if (want_a8) {
          const uint2 ji = *reinterpret_cast<const uint2*>(jimg + 4 * q4);
          img[ji.x & 0xFFFFu] = (uint8_t)o;
          img[ji.x >> 16] = (uint8_t)(o >> 8);
          img[ji.y & 0xFFFFu] = (uint8_t)(o >> 16);
          img[ji.y >> 16] = (uint8_t)(o >> 24);
        }
      }
    }
    // every lane of the group is done with the slot (and the image holds this row's codes); the
    // slot is refilled by the async proxy: order this group's generic accesses before it
    if (glane == 0) nexti[flip] = atomicAdd(&next_row_s, 1);
    fence_proxy_async_smem();
    group_sync(rw, grp);
    const int64_t m_this = m;
    m = (int64_t)blockIdx.x + (int64_t)nexti[flip] * gridDim.x;
    flip ^= 1u;
    if (glane == 0 && m < p.M) bulk_copy_g2s(smem_u32(slot), p.X + m * K, (uint32_t)row_bytes, bar0);

    // dense component: INT4 codes of the registers, one 32-bit word per chunk
    uint32_t* dst = reinterpret_cast<uint32_t*>(p.dq4 + (size_t)m_this * (K / 2)) + slice * S8 + lane;
    const float cq = rs.inv_lo;
    if (rs.clamp) {
      // Codes beyond +-7 are possible: limit the inputs instead of the codes (see dense_sweep)
      const uint32_t xl = __float_as_uint(__fdiv_rd(7.0f, cq)) >> 16;
      const uint32_t hi2 = xl | (xl << 16), lo2 = hi2 | 0x80008000u;
#pragma unroll
      for (int c = 0; c < NCL; ++c) {
        v[c].x = max2(min2(v[c].x, hi2), lo2);
        v[c].y = max2(min2(v[c].y, hi2), lo2);
        v[c].z = max2(min2(v[c].z, hi2), lo2);
        v[c].w = max2(min2(v[c].w, hi2), lo2);
      }
    }
    const float2 cc = make_float2(cq, cq), mm = make_float2(kMagic + 8.0f, kMagic + 8.0f);
    if constexpr (FP) {
      // E2M1 codes of the registers, eight nibbles per word, and (on request) the merged operand:
      // the E4M3 byte of code * 2^e in element order, the selected places' bytes from the image.
      // Codes by the row's seven thresholds, bytes by the row's table (see fp_steps).
      uint2* aw = want_a8 ? reinterpret_cast<uint2*>(p.a8 + (size_t)m_this * K) + slice * S8 + lane : nullptr;
      const uint2* iw = reinterpret_cast<const uint2*>(img) + slice * S8 + lane;
      const FpSteps st = fp_steps(cq, rs.e, lane);
#pragma unroll
      for (int c = 0; c < NCL; ++c) {
        const uint32_t c0 = fp_codes2(v[c].x, st), c1 = fp_codes2(v[c].y, st), c2 = fp_codes2(v[c].z, st), c3 = fp_codes2(v[c].w, st);
        const uint32_t nib = ((c0 | (c0 >> 12)) & 0xFFu) | (((c1 | (c1 >> 12)) & 0xFFu) << 8) | (((c2 | (c2 >> 12)) & 0xFFu) << 16) |
                             ((c3 | (c3 >> 12)) << 24);
        dst[c * 32] = nib;
        if (want_a8) {
          const uint2 by = fp_bytes8(nib, st), im = iw[c * 32];
          aw[c * 32] = make_uint2(by.x | im.x, by.y | im.y);
        }
      }
    } else if (want_a8) {
      // Codes carry an offset of 8 (u = code + 8 in 1..15 in the low bits of 0x4B400000 + u).
      // The four even and the four odd ones are summed into bytes by multiply-adds; their
      // constant parts come off in the last step of each use:
      //   dq4 word  = (ev + 16 * od - 0x3F400000) ^ 0x88888888
      //   merged    = ev * 2^e + [0x80808080 - (0x08080808 + 0x8B400000) * 2^e]   (code * 2^e + 128
      //               per byte, no carries: u * 2^e <= 240), XOR the image's bytes (0 where nothing
      //               is selected, the INT8 code at a selected place, whose dense byte is 0x80)
      uint32_t* aw = reinterpret_cast<uint32_t*>(p.a8 + (size_t)m_this * K) + ((slice * S8 + lane) >> 2) * 8 + (lane & 3);
      const uint2* iw = reinterpret_cast<const uint2*>(img) + slice * S8 + lane;
      const uint32_t pw = 1u << rs.e;
      const uint32_t ce = 0x80808080u - (0x08080808u + 0x8B400000u) * pw;
#pragma unroll
      for (int c = 0; c < NCL; ++c) {
        const uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
        uint32_t u[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float2 a = make_float2(__uint_as_float(imad(w[q], mk.k65536, 0u)), __uint_as_float(w[q] & 0xFFFF0000u));
          const float2 d = __ffma2_rn(a, cc, mm);
          u[2 * q] = __float_as_uint(d.x);
          u[2 * q + 1] = __float_as_uint(d.y);
        }
        const uint32_t ev = imad(imad(u[6], mk.k256, u[4]), mk.k65536, imad(u[2], mk.k256, u[0]));
        const uint32_t od = imad(imad(u[7], mk.k256, u[5]), mk.k65536, imad(u[3], mk.k256, u[1]));
        const uint2 im = iw[c * 32];
        dst[c * 32] = imad(imad(od, mk.k16, ev), mk.one, 0u - 0x3F400000u) ^ 0x88888888u;
        aw[c * 64] = imad(ev, pw, ce) ^ im.x;
        aw[c * 64 + 4] = imad(od, pw, ce) ^ im.y;
      }
    } else {
#pragma unroll
      for (int c = 0; c < NCL; ++c) {
        const uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
        uint32_t u[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float2 a = make_float2(__uint_as_float(imad(w[q], mk.k65536, 0u)), __uint_as_float(w[q] & 0xFFFF0000u));
          const float2 d = __ffma2_rn(a, cc, mm);
          u[2 * q] = __float_as_uint(d.x);
          u[2 * q + 1] = __float_as_uint(d.y);
        }
        const uint32_t t03 = imad(imad(u[3], mk.k16, u[2]), mk.k256, imad(u[1], mk.k16, u[0]));
        const uint32_t t47 = imad(imad(u[7], mk.k16, u[6]), mk.k256, imad(u[5], mk.k16, u[4]));
        dst[c * 32] = imad(imad(t47, mk.k65536, t03), mk.one, 0u - 0x3F400000u) ^ 0x88888888u;
      }
    }
  }
  if (*abort_flag && glane == 0) atomicExch(p.status, (int)SQ_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------
// Plain kernel for any (b, k): one block per token row, the row staged in shared memory.
//   phase 1  load the row, row maximum -> inv = 127/amax, s_hi = amax/127
//   phase 2  positions: dynamic = rank every element of a bank by (magnitude, then lower
//            index) and keep ranks < k; static = the given positions.  Selected elements
//            are quantised to INT8, written in ascending position with ballot/popc slots,
//            and zeroed in the staged row.
//   phase 3  maximum of what is left -> shift e, s_lo
//   phase 4  INT4 codes of the staged row (zeros at the selected places), 8 per 32-bit word
template <int B>
__global__ void __launch_bounds__(256) encode_generic_kernel(int k, bool is_static, bool indep, const uint16_t* __restrict__ X, int64_t K,
                                                             const uint8_t* __restrict__ positions,
                                                             uint8_t* __restrict__ dq4, int8_t* __restrict__ vals,
                                                             uint8_t* __restrict__ idx, float* __restrict__ s_hi,
                                                             float* __restrict__ s_lo, uint8_t* __restrict__ shift) {
  extern __shared__ __align__(16) uint16_t srow[];
  __shared__ uint32_t scratch[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t m = blockIdx.x;
  const int64_t G = K / B;
  const uint16_t* xrow = X + m * K;

  uint32_t mx = 0;
  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8) {
    const uint4 v = ldg_nc_v4(xrow + i);
    *reinterpret_cast<uint4*>(srow + i) = v;
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      mx = max(mx, w[q] & 0x7FFFu);
      mx = max(mx, (w[q] >> 16) & 0x7FFFu);
    }
  }
  uint32_t amax_bits = block_max_u32(mx, scratch);  // barrier inside: row staged
  if (indep) {
    // independent scales (static positions only): the INT8 grid spans the selected values alone
    uint32_t sx = 0;
    for (int64_t t = tid; t < G * k; t += 256) sx = max(sx, (uint32_t)srow[(t / k) * B + positions[t]] & 0x7FFFu);
    amax_bits = block_max_u32(sx, scratch);
  }
  const float amax = bf16_bits_to_f32(amax_bits);
  const float inv = amax > 0.f ? __fdiv_rn(127.0f, amax) : 0.f;

  if (is_static) {
    const int64_t GK = G * k;
    for (int64_t t = tid; t < GK; t += 256) {
      const int64_t g = t / k;
      const int64_t j = g * B + positions[t];
      const int q = min(127, max(-127, rne_prod(bf16_bits_to_f32(srow[j]), inv)));
      vals[m * GK + t] = (int8_t)q;
      srow[j] = 0;
    }
  } else {
    constexpr int EPL = B / 32;  // elements per lane
    for (int64_t g = warp; g < G; g += 8) {
      uint32_t key[EPL];
      uint32_t raw[EPL];
#pragma unroll
      for (int t = 0; t < EPL; ++t) {
        const int j = lane + 32 * t;
        raw[t] = srow[g * B + j];
        key[t] = ((raw[t] & 0x7FFFu) << 7) | (uint32_t)(127 - j);  // unique: magnitude, then lower index
      }
      int rank[EPL];
#pragma unroll
      for (int t = 0; t < EPL; ++t) rank[t] = 0;
#pragma unroll
      for (int u = 0; u < EPL; ++u) {
        for (int l = 0; l < 32; ++l) {
          const uint32_t other = __shfl_sync(0xffffffffu, key[u], l);
#pragma unroll
          for (int t = 0; t < EPL; ++t) rank[t] += (other > key[t]) ? 1 : 0;
        }
      }
      int before = 0;
#pragma unroll
      for (int t = 0; t < EPL; ++t) {
        const bool sel = rank[t] < k;
        const uint32_t mask = __ballot_sync(0xffffffffu, sel);
        if (sel) {
          const int slot = before + __popc(mask & ((1u << lane) - 1u));
          const int j = lane + 32 * t;
          const int q = min(127, max(-127, rne_prod(bf16_bits_to_f32(raw[t]), inv)));
          vals[(m * G + g) * k + slot] = (int8_t)q;
          idx[(m * G + g) * k + slot] = (uint8_t)j;
          srow[g * B + j] = 0;
        }
        before += __popc(mask);
      }
    }
  }
  __syncthreads();

  uint32_t rm = 0;
  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(srow + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      rm = max(rm, w[q] & 0x7FFFu);
      rm = max(rm, (w[q] >> 16) & 0x7FFFu);
    }
  }
  const uint32_t rmax_bits = block_max_u32(rm, scratch);
  const RowScale rs = indep ? row_scale_indep(amax_bits, rmax_bits) : row_scale(amax_bits, rmax_bits);
  if (tid == 0) {
    s_hi[m] = rs.s_hi;
    s_lo[m] = rs.s_lo;
    shift[m] = (uint8_t)rs.e;
  }
  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(srow + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t word = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      int q0 = rne_prod(bf16_bits_to_f32(w[q] & 0xFFFFu), rs.inv_lo);
      int q1 = rne_prod(bf16_bits_to_f32(w[q] >> 16), rs.inv_lo);
      q0 = min(7, max(-7, q0));
      q1 = min(7, max(-7, q1));
      word |= (uint32_t)(q0 & 0xF) << (8 * q);
      word |= (uint32_t)(q1 & 0xF) << (8 * q + 4);
    }
    *reinterpret_cast<uint32_t*>(dq4 + m * (K / 2) + i / 2) = word;
  }
}

// One block per row: dense INT4 part first, then the k entries per bank overwrite
// their places (they hold a zero nibble in the dense part).
__global__ void __launch_bounds__(256) decode_kernel(int b, int k, const uint8_t* __restrict__ dq4,
                                                     const int8_t* __restrict__ vals,
                                                     const uint8_t* __restrict__ idx,
                                                     const uint8_t* __restrict__ positions,
                                                     const float* __restrict__ s_hi,
                                                     const float* __restrict__ s_lo, int64_t K,
                                                     uint16_t* __restrict__ out) {
  // The row is put together in shared memory (dense values, then the sparse entries over the
  // zeros at their places) and leaves in coalesced 16-byte stores: the sparse entries as 2-byte
  // stores to global memory, one row at a time, had held the kernel at 2.9 TB/s.
  extern __shared__ __align__(16) uint16_t drow[];
  __shared__ uint32_t pair_tab[256];  // the two bf16 values of every possible byte of codes, for this row's scale
  const int tid = threadIdx.x;
  const int64_t m = blockIdx.x;
  const int64_t G = K / b, GK = G * k;
  const int8_t* vrow = vals + m * GK;
  const uint8_t* irow = idx != nullptr ? idx + m * GK : positions;
  const bool words = (GK & 3) == 0 && ((reinterpret_cast<uintptr_t>(vrow) | reinterpret_cast<uintptr_t>(irow)) & 3) == 0;
  // every global read of this thread's first pass is issued before anything waits for one of them:
  // a block pays one memory latency, not three in a row
  const float sl = s_lo[m], sh = s_hi[m];
  const int64_t i0 = (int64_t)tid * 32, t0 = (int64_t)tid * 4;
  uint4 c0 = make_uint4(0, 0, 0, 0);
  uint32_t vw0 = 0, iw0 = 0;
  if (i0 < K) c0 = *reinterpret_cast<const uint4*>(dq4 + m * (K / 2) + i0 / 2);
  if (words && t0 < GK) {
    vw0 = *reinterpret_cast<const uint32_t*>(vrow + t0);
    iw0 = *reinterpret_cast<const uint32_t*>(irow + t0);
  }
  {
    const int n0 = ((int)((uint32_t)tid << 28)) >> 28, n1 = ((int)((uint32_t)tid << 24)) >> 28;  // sign-extended nibbles
    pair_tab[tid] = f32_to_bf16_bits(sl * (float)n0) | (f32_to_bf16_bits(sl * (float)n1) << 16);
  }
  __syncthreads();
  for (int64_t i = i0; i < K; i += 256 * 32) {  // 16 bytes of codes -> 32 values
    const uint4 c = i == i0 ? c0 : *reinterpret_cast<const uint4*>(dq4 + m * (K / 2) + i / 2);
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int q = 0; q < 4; ++q)
      *reinterpret_cast<uint4*>(drow + i + 8 * q) = make_uint4(pair_tab[w[q] & 0xFFu], pair_tab[(w[q] >> 8) & 0xFFu],
                                                             pair_tab[(w[q] >> 16) & 0xFFu], pair_tab[w[q] >> 24]);
  }
  __syncthreads();
  if (words) {
    for (int64_t t4 = t0; t4 < GK; t4 += 256 * 4) {  // four entries per pair of 4-byte reads
      const uint32_t vw = t4 == t0 ? vw0 : *reinterpret_cast<const uint32_t*>(vrow + t4);
      const uint32_t iw = t4 == t0 ? iw0 : *reinterpret_cast<const uint32_t*>(irow + t4);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int64_t t = t4 + q;
        const int v = (int)(int8_t)((vw >> (8 * q)) & 0xFFu);
        drow[(t / k) * b + ((iw >> (8 * q)) & 0xFFu)] = (uint16_t)f32_to_bf16_bits(sh * (float)v);
      }
    }
  } else {
    for (int64_t t = tid; t < GK; t += 256)
      drow[(t / k) * b + irow[t]] = (uint16_t)f32_to_bf16_bits(sh * (float)vrow[t]);
  }
  __syncthreads();
  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8)
    *reinterpret_cast<uint4*>(out + m * K + i) = *reinterpret_cast<const uint4*>(drow + i);
}

namespace {

// The current device and its SM count (asked once per device: the encode of a few decode tokens
// is bound by the host's launch path).
static cudaError_t device_and_sms(int* dev, int* sms) {
  static std::atomic<int> cached[64];
  cudaError_t err = cudaGetDevice(dev);
  if (err != cudaSuccess) return err;
  if (*dev < 0 || *dev >= 64) return cudaErrorInvalidDevice;
  int n = cached[*dev].load(std::memory_order_acquire);
  if (n == 0) {
    err = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, *dev);
    if (err != cudaSuccess) return err;
    cached[*dev].store(n, std::memory_order_release);
  }
  *sms = n;
  return cudaSuccess;
}
// Raises a kernel's dynamic shared memory limit when a launch needs more than any before it
// (the limit only ever grows, so a concurrent launch that needs less is never cut short).
#define SQ_ENSURE_SMEM(KERNEL_, DEV_, BYTES_)                                                            \
  do {                                                                                                   \
    static std::atomic<size_t> limit_[64];                                                               \
    if ((BYTES_) > limit_[DEV_].load(std::memory_order_acquire)) {                                       \
      std::lock_guard<std::mutex> lock_(setup_mutex());                                                  \
      if ((BYTES_) > limit_[DEV_].load(std::memory_order_relaxed)) {                                     \
        err = cudaFuncSetAttribute(KERNEL_, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(BYTES_)); \
        if (err != cudaSuccess) return err;                                                              \
        limit_[DEV_].store((BYTES_), std::memory_order_release);                                         \
      }                                                                                                  \
    }                                                                                                    \
  } while (0)

template <int B, int KK, bool FP = false, bool NORM = false>
cudaError_t launch_rows(const EncodeParams& base, cudaStream_t st) {
  EncodeParams p = base;
  const int K = p.K, G = K / B, k = (KK == 0) ? p.k : KK;
  constexpr int kMaxWarps = (B == 128) ? 8 : 16;
  const size_t side = ((((size_t)G * k * 2) + 15) & ~(size_t)15) * (FP ? 2 : 1);  // stash of selected raw values (and their places)
  const size_t table = (KK == 0) ? ((((size_t)G * k * 2) + 127) & ~(size_t)127) : 0;  // static offset table
  const size_t budget = 224 * 1024 - table;
  const size_t row = (size_t)K * 2;
  const size_t extra = side + 32 + 256 + 128 + 128;  // side buffer, four mbarriers, exchange words (+ the normalisation's), rounding
  // Rows are single-buffered: with 16 resident warps the rows other groups have in flight
  // hide the copy latency, and a second buffer would only cost warps.  Pick the group size
  // that keeps the most warps resident, preferring smaller groups (less per-row overhead per
  // element) on a tie.
  int rw = kMaxWarps, nbuf = 1, best = 0;
  for (int cand = 1; cand <= kMaxWarps; cand *= 2) {
    const size_t per = ((row + extra) + 127) & ~(size_t)127;
    if (per > budget) break;
    int groups = (int)(budget / per);
    if (groups > kMaxWarps / cand) groups = kMaxWarps / cand;
    if (groups > 15) groups = 15;  // named barrier ids 1..15
    if (groups * cand > best) {
      best = groups * cand;
      rw = cand;
    }
  }
  int dev = 0, sms = 0;
  cudaError_t err = device_and_sms(&dev, &sms);
  if (err != cudaSuccess) return err;
  // Few rows (decode, short prompts): latency, not throughput, is what counts.  As many warps per
  // row as still give every row a group of its own in ONE wave of blocks, and every lane at least
  // two 16-byte chunks (K = 4096, 16 tokens: 5.6 instead of 7.2 us; K = 14336: 5.9 instead of 9.8).
  for (int cand = kMaxWarps; cand > rw; cand /= 2) {
    if ((size_t)cand * 64 > (size_t)K / 8) continue;
    const int groups = kMaxWarps / cand;
    if ((p.M + groups - 1) / groups <= sms) {
      rw = cand;
      break;
    }
  }
  const size_t per_group = (((size_t)nbuf * row + extra) + 127) & ~(size_t)127;
  if (per_group > 224 * 1024) return cudaErrorNotSupported;
  int ngroups = kMaxWarps / rw;
  {
    const size_t fit = (224 * 1024 - table) / ((((size_t)nbuf * row + extra) + 127) & ~(size_t)127);
    if ((size_t)ngroups > fit) ngroups = (int)fit;
    if (ngroups < 1) ngroups = 1;
  }
  p.nbuf = nbuf;
  p.rw = rw;
  p.group_stride = (int)per_group;
  const size_t smem = table + per_group * ngroups;
  if (smem > 227 * 1024) return cudaErrorNotSupported;  // long rows with many selected places: the plain kernel

  SQ_ENSURE_SMEM((encode_rows_kernel<B, KK, FP, NORM>), dev, smem);
  int64_t blocks = (p.M + ngroups - 1) / ngroups;
  if (blocks > sms) blocks = sms;
  encode_rows_kernel<B, KK, FP, NORM><<<(unsigned)blocks, ngroups * rw * 32, smem, st>>>(p);
  return cudaGetLastError();
}

// Register-resident static kernel: usable when a row splits into 1, 2, 4 or 8 warp slices of
// NCL * 256 elements with NCL one of the instantiated sizes, and its tables fit in shared memory.
template <int NCL, int NT, bool INDEP>
cudaError_t launch_static_regs_as(EncodeParams p, int rw, cudaStream_t st) {
  const int GK = (p.K / p.b) * p.k;
  const int ngroups = (NT / 32) / rw;
  const size_t jt_bytes = ((size_t)GK * 2 + 15) & ~(size_t)15;
  const size_t stash_bytes = ((size_t)GK * 4 + 15) & ~(size_t)15;
  const size_t img_bytes = p.a8 != nullptr ? (size_t)p.K : 0;  // per group: the image of the selected places
  const size_t smem = (size_t)p.K * 2 + jt_bytes + (stash_bytes + 128 + img_bytes) * ngroups + (p.a8 != nullptr ? jt_bytes : 0);
  if (smem > 200 * 1024) return cudaErrorNotSupported;
  p.rw = rw;
  int dev = 0, sms = 0;
  cudaError_t err = device_and_sms(&dev, &sms);
  if (err != cudaSuccess) return err;
  SQ_ENSURE_SMEM((encode_static_regs_kernel<NCL, NT, INDEP>), dev, smem);
  int64_t blocks = (p.M + ngroups - 1) / ngroups;
  if (blocks > sms) blocks = sms;
  encode_static_regs_kernel<NCL, NT, INDEP><<<(unsigned)blocks, NT, smem, st>>>(p);
  return cudaGetLastError();
}

// Ring kernel: `rw` warps per row, 16 / rw groups per block, one slot per group.
template <int NCL, bool INDEP, bool MASK8, bool FP = false, bool NORM = false>
cudaError_t launch_static_ring_as(EncodeParams p, int rw, cudaStream_t st) {
  constexpr int NT = 512;
  const int GK = (p.K / p.b) * p.k;
  const int ngroups = (NT / 32) / rw;
  const bool a8 = !INDEP && p.a8 != nullptr;
  const size_t mask_bytes = MASK8 ? (size_t)p.K : (size_t)p.K * 2;
  const size_t jt_bytes = ((size_t)GK * 2 + 15) & ~(size_t)15;
  const size_t per_group = ((size_t)p.K * 2 + (a8 ? (size_t)p.K : 0) + 256 + 16 + 127) & ~(size_t)127;
  const size_t smem = mask_bytes + jt_bytes * (a8 ? 2 : 1) + (NORM ? (size_t)p.K * 2 + jt_bytes : 0) + per_group * ngroups;
  if (smem > 226 * 1024) return cudaErrorNotSupported;
  p.rw = rw;
  p.group_stride = (int)per_group;
  int dev = 0, sms = 0;
  cudaError_t err = device_and_sms(&dev, &sms);
  if (err != cudaSuccess) return err;
  SQ_ENSURE_SMEM((encode_static_ring_kernel<NCL, NT, INDEP, MASK8, FP, NORM>), dev, smem);
  const int64_t blocks = p.M < sms ? p.M : sms;
  encode_static_ring_kernel<NCL, NT, INDEP, MASK8, FP, NORM><<<(unsigned)blocks, NT, smem, st>>>(p);
  return cudaGetLastError();
}

// Picks the ring kernel's shape: the fewest warps per row whose slice is an instantiated size
// (the per-row work that does not shrink with the slice -- scales, barriers -- is then spread over
// the most elements, and the most rows are in flight); half-word masks if the tables and slots
// fit, else byte masks.
template <bool INDEP, bool FP = false, bool NORM = false>
cudaError_t launch_static_ring(const EncodeParams& p, cudaStream_t st) {
  if (p.K % 256 != 0 || p.K > 65535 || (reinterpret_cast<uintptr_t>(p.X) & 15) != 0) return cudaErrorNotSupported;
  for (int mask8 = 0; mask8 < 2; ++mask8) {
    for (int rw = 1; rw <= 8; rw *= 2) {
      if ((p.K / 256) % rw != 0) continue;
      const int ncl = p.K / 256 / rw;
      cudaError_t err = cudaErrorNotSupported;
#define SQ_RING(NCL_)                                                                   \
  if (ncl == NCL_)                                                                      \
    err = mask8 ? launch_static_ring_as<NCL_, INDEP, true, FP, NORM>(p, rw, st)         \
                : launch_static_ring_as<NCL_, INDEP, false, FP, NORM>(p, rw, st);
      SQ_RING(8) SQ_RING(12) SQ_RING(14) SQ_RING(16)
#undef SQ_RING
      if (err != cudaErrorNotSupported) return err;
    }
  }
  return cudaErrorNotSupported;
}

// cudaErrorNotSupported = this shape is left to the shared-memory kernel.  Slices of at most
// 16 chunks per lane keep 16 warps resident (measured faster than fewer warps holding more).
template <bool INDEP>
cudaError_t launch_static_regs(const EncodeParams& p, cudaStream_t st) {
  if (p.K % 256 != 0 || p.K > 65535) return cudaErrorNotSupported;
  for (int rw = 1; rw <= 8; rw *= 2) {
    if ((p.K / 256) % rw != 0) continue;
    switch (p.K / 256 / rw) {
      case 8: return launch_static_regs_as<8, 512, INDEP>(p, rw, st);
      case 12: return launch_static_regs_as<12, 512, INDEP>(p, rw, st);
      case 14: return launch_static_regs_as<14, 512, INDEP>(p, rw, st);
      case 16: return launch_static_regs_as<16, 512, INDEP>(p, rw, st);
      default: break;
    }
  }
  return cudaErrorNotSupported;
}

template <int B>
cudaError_t launch_generic(int k, bool is_static, bool indep, const uint16_t* X, int64_t M, int64_t K,
                           const uint8_t* positions, const sq_encoded& out, cudaStream_t st) {
  const size_t smem = (size_t)K * 2;
  int dev = 0, sms = 0;
  cudaError_t err = device_and_sms(&dev, &sms);
  if (err != cudaSuccess) return err;
  SQ_ENSURE_SMEM((encode_generic_kernel<B>), dev, smem);
  encode_generic_kernel<B><<<(unsigned)M, 256, smem, st>>>(k, is_static, indep, X, K, positions, out.dq4, out.vals, out.idx,
                                                          out.s_hi, out.s_lo, out.shift);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_encode(int b, int k, bool is_static, bool indep, const uint16_t* X, int64_t M, int64_t K,
                          const uint8_t* positions, const sq_encoded& out, int* status, cudaStream_t st,
                          uint8_t* a8, bool* a8_written) {
  EncodeParams p;
  if (a8_written != nullptr) *a8_written = false;
  p.a8 = nullptr;
  p.X = X;
  p.positions = positions;
  p.dq4 = out.dq4;
  p.vals = out.vals;
  p.idx = out.idx;
  p.s_hi = out.s_hi;
  p.s_lo = out.s_lo;
  p.shift = out.shift;
  p.status = status;
  p.M = M;
  p.K = (int)K;
  p.k = k;
  p.b = b;
  p.nbuf = 1;
  p.rw = 1;
  p.group_stride = 0;
  p.mk = MulK{0xFFFFFFFFu, 2u, 32u, 256u, 65536u, 1u << 24, 16u, 1u};
  p.gamma = nullptr;
  p.eps = 0.f;
  if (is_static && indep) {
    // independent scales: the register kernel, or the plain one for row lengths it does not take
    cudaError_t err = launch_static_ring<true>(p, st);
    if (err != cudaErrorNotSupported) return err;
    err = launch_static_regs<true>(p, st);
    if (err != cudaErrorNotSupported) return err;
    if (b == 32) return launch_generic<32>(k, true, true, X, M, K, positions, out, st);
    if (b == 64) return launch_generic<64>(k, true, true, X, M, K, positions, out, st);
    return launch_generic<128>(k, true, true, X, M, K, positions, out, st);
  }
  if (is_static) {
    p.a8 = a8;  // only the ring and register kernels write the merged operand
    cudaError_t err = std::getenv("SQ_ENCODE_RING_OFF") ? cudaErrorNotSupported : launch_static_ring<false>(p, st);
    if (err == cudaSuccess && a8 != nullptr && a8_written != nullptr) *a8_written = true;
    if (err != cudaErrorNotSupported) return err;
    err = launch_static_regs<false>(p, st);
    if (err == cudaSuccess && a8 != nullptr && a8_written != nullptr) *a8_written = true;
    if (err != cudaErrorNotSupported) return err;
    p.a8 = nullptr;
    err = b == 32 ? launch_rows<32, 0>(p, st) : (b == 64 ? launch_rows<64, 0>(p, st) : launch_rows<128, 0>(p, st));
    if (err != cudaErrorNotSupported) return err;
    // a row, its offset table and its stash together exceed shared memory: one block per row
    if (b == 32) return launch_generic<32>(k, true, false, X, M, K, positions, out, st);
    if (b == 64) return launch_generic<64>(k, true, false, X, M, K, positions, out, st);
    return launch_generic<128>(k, true, false, X, M, K, positions, out, st);
  }
  // dynamic fast kernels: k/b in {1/16, 1/8, 1/4, 1/2}
#define SQ_DYN(BB, KK_)                                       \
  if (b == BB && k == KK_) {                                  \
    const cudaError_t err = launch_rows<BB, KK_>(p, st);      \
    if (err != cudaErrorNotSupported) return err;             \
  }
  SQ_DYN(32, 2) SQ_DYN(32, 4) SQ_DYN(32, 8) SQ_DYN(32, 16)
  SQ_DYN(64, 4) SQ_DYN(64, 8) SQ_DYN(64, 16) SQ_DYN(64, 32)
  SQ_DYN(128, 8) SQ_DYN(128, 16) SQ_DYN(128, 32) SQ_DYN(128, 64)
#undef SQ_DYN
  if (b == 32) return launch_generic<32>(k, false, false, X, M, K, positions, out, st);
  if (b == 64) return launch_generic<64>(k, false, false, X, M, K, positions, out, st);
  return launch_generic<128>(k, false, false, X, M, K, positions, out, st);
}

// Floating-point variant, static positions: the ring kernel with that format's roundings.
// cudaErrorNotSupported = this shape is left to the variant's own one-block-per-row kernel.
cudaError_t launch_fp_encode_static_ring(int b, int k, const uint16_t* X, int64_t M, int64_t K, const uint8_t* positions,
                                         const sq_encoded& out, uint8_t* a8, int* status, cudaStream_t st) {
  if (positions == nullptr || M < 1) return cudaErrorNotSupported;
  EncodeParams p;
  p.a8 = a8;
  p.X = X;
  p.positions = positions;
  p.dq4 = out.dq4;
  p.vals = out.vals;
  p.idx = out.idx;
  p.s_hi = out.s_hi;
  p.s_lo = out.s_lo;
  p.shift = out.shift;
  p.status = status;
  p.M = M;
  p.K = (int)K;
  p.k = k;
  p.b = b;
  p.nbuf = 1;
  p.rw = 1;
  p.group_stride = 0;
  p.mk = MulK{0xFFFFFFFFu, 2u, 32u, 256u, 65536u, 1u << 24, 16u, 1u};
  p.gamma = nullptr;
  p.eps = 0.f;
  return launch_static_ring<false, true>(p, st);
}

// Root-mean-square normalisation fused into the static-position encode (tied scales): the ring
// kernel normalises a row in its registers before it encodes it.  cudaErrorNotSupported = a row
// length the ring kernel does not take, or one whose slots, tables and weights exceed shared memory.
cudaError_t launch_rmsnorm_encode(int b, int k, bool fp, const uint16_t* X, const uint16_t* gamma, float eps, int64_t M,
                                  int64_t K, const uint8_t* positions, const sq_encoded& out, uint8_t* a8, int* status,
                                  cudaStream_t st) {
  if (M < 1) return cudaErrorNotSupported;
  EncodeParams p;
  p.a8 = a8;
  p.X = X;
  p.positions = positions;
  p.dq4 = out.dq4;
  p.vals = out.vals;
  p.idx = out.idx;
  p.s_hi = out.s_hi;
  p.s_lo = out.s_lo;
  p.shift = out.shift;
  p.status = status;
  p.M = M;
  p.K = (int)K;
  p.k = k;
  p.b = b;
  p.nbuf = 1;
  p.rw = 1;
  p.group_stride = 0;
  p.mk = MulK{0xFFFFFFFFu, 2u, 32u, 256u, 65536u, 1u << 24, 16u, 1u};
  p.gamma = gamma;
  p.eps = eps;
  if (positions == nullptr) {
    // dynamic positions (integer variant, the row-group kernel's ratios): the staged row is
    // normalised in shared memory before the selection; the merged operand is not this kernel's
    if (fp) return cudaErrorNotSupported;
    p.a8 = nullptr;
#define SQ_DYN_NORM(BB, KK_) \
  if (b == BB && k == KK_) return launch_rows<BB, KK_, false, true>(p, st);
    SQ_DYN_NORM(32, 2) SQ_DYN_NORM(32, 4) SQ_DYN_NORM(32, 8) SQ_DYN_NORM(32, 16)
    SQ_DYN_NORM(64, 4) SQ_DYN_NORM(64, 8) SQ_DYN_NORM(64, 16) SQ_DYN_NORM(64, 32)
    SQ_DYN_NORM(128, 8) SQ_DYN_NORM(128, 16) SQ_DYN_NORM(128, 32) SQ_DYN_NORM(128, 64)
#undef SQ_DYN_NORM
    return cudaErrorNotSupported;
  }
  if (fp) return launch_static_ring<false, true, true>(p, st);  // the floating-point variant's codes and scales
  return launch_static_ring<false, false, true>(p, st);
}

// Floating-point variant, dynamic positions: the row-group kernel's selection with that format's
// scales and roundings.  cudaErrorNotSupported = left to the variant's own kernel.
cudaError_t launch_fp_encode_dynamic_rows(int b, int k, const uint16_t* X, int64_t M, int64_t K, const sq_encoded& out,
                                          uint8_t* a8, int* status, cudaStream_t st) {
  if (M < 1 || a8 == nullptr) return cudaErrorNotSupported;
  EncodeParams p;
  p.a8 = a8;
  p.X = X;
  p.positions = nullptr;
  p.dq4 = out.dq4;
  p.vals = out.vals;
  p.idx = out.idx;
  p.s_hi = out.s_hi;
  p.s_lo = out.s_lo;
  p.shift = out.shift;
  p.status = status;
  p.M = M;
  p.K = (int)K;
  p.k = k;
  p.b = b;
  p.nbuf = 1;
  p.rw = 1;
  p.group_stride = 0;
  p.mk = MulK{0xFFFFFFFFu, 2u, 32u, 256u, 65536u, 1u << 24, 16u, 1u};
  p.gamma = nullptr;
  p.eps = 0.f;
#define SQ_DYN_FP(BB, KK_) \
  if (b == BB && k == KK_) return launch_rows<BB, KK_, true>(p, st);
  SQ_DYN_FP(32, 4) SQ_DYN_FP(64, 8) SQ_DYN_FP(128, 16) SQ_DYN_FP(64, 4) SQ_DYN_FP(128, 8) SQ_DYN_FP(32, 8) SQ_DYN_FP(64, 16) SQ_DYN_FP(128, 32)
#undef SQ_DYN_FP
  return cudaErrorNotSupported;
}

cudaError_t launch_decode(int b, int k, const sq_encoded& A, const uint8_t* positions, int64_t M,
                          int64_t K, uint16_t* out, cudaStream_t st) {
  const size_t smem = (size_t)K * 2;
  int dev = 0, sms = 0;
  cudaError_t err = device_and_sms(&dev, &sms);
  if (err != cudaSuccess) return err;
  SQ_ENSURE_SMEM(decode_kernel, dev, smem);
  decode_kernel<<<(unsigned)M, 256, smem, st>>>(b, k, A.dq4, A.vals, A.idx, positions, A.s_hi, A.s_lo, K, out);
  return cudaGetLastError();
}

}  // namespace sq
