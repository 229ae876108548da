// Floating-point variant of the SQ-format hot path: sparse FP8 (E4M3) entries + dense FP4 (E2M1)
// elsewhere for the activations, FP4 per-output-channel weights (Section 3.1 defines the format
// for floating-point precisions; the appendix "FP Quantization Results" uses this pair).
//
// sm_100's tensor cores take these types natively (tcgen05.mma.kind::f8f6f4, fp32 accumulation in
// tensor memory), so unlike the INT4 path nothing has to be widened on chip.  The two parts of an
// activation row live on one grid (s_lo = s_hi * 2^e), and a dense E2M1 value times 2^e is an E4M3
// number, so the encoder also writes the MERGED operand a8[m,j] (one E4M3 byte per element: the
// dense value times 2^e, or the sparse entry at a selected place) and the GEMM is one stream of
// FP8 x FP8 MMAs into one accumulator, fed by TMA alone:
//     acc[m,n] = sum_j value(a8[m,j]) * value(w8[n,j]);  out = bf16((acc * s_hi[m]) * s_w[n])
// (w8: the weights' E2M1 values as E4M3 bytes, written by the packer next to the packed codes).
//
// Roundings are those of the format definition: nearest representable value of the EXACT product
// a * scale (a bf16, scale fp32: exact in fp64), ties to the even code, saturating.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <string.h>

#include "sq_device.cuh"
#include "sq_fp_device.cuh"
#include "sq_host.h"

namespace sq {

namespace {

// Code of the magnitude v >= 0 in a small floating-point format with `mb` mantissa bits whose
// smallest normal exponent is emin: v is scaled (exactly) so that one unit is the spacing at its
// exponent, rounded half-even to an integer n, and code = (exponent field << mb) + n, where the
// implicit one inside n bumps the exponent field and a round-up to the next power of two carries
// by itself.  Below the smallest normal the spacing stays that of emin (subnormals).
__device__ __forceinline__ uint32_t round_code(double v, int mb, int emin, uint32_t max_code) {
  if (!(v > 0.0)) return 0;
  int e = ((__double2hiint(v) >> 20) & 0x7FF) - 1023;
  e = max(e, emin);
  const uint32_t n = (uint32_t)__double2int_rn(scalbn(v, mb - e));
  const uint32_t code = ((uint32_t)(e - emin) << mb) + n;
  return min(code, max_code);
}
__device__ __forceinline__ uint32_t e2m1_of(double p) {  // sign in bit 3; a value that rounds to zero is +0
  const uint32_t c = round_code(fabs(p), 1, 0, 7u);
  return c == 0 ? 0u : (c | (p < 0.0 ? 8u : 0u));
}
__device__ __forceinline__ uint32_t block_max(uint32_t v, uint32_t* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  uint32_t r = 0;
  for (int q = 0; q < (int)(blockDim.x >> 5); ++q) r = max(r, scratch[q]);
  return r;
}

}  // namespace

// One block per output channel: wmax, then codes = E2M1(w * (6 / wmax)) packed two per byte and the
// same values as E4M3 bytes.
__global__ void __launch_bounds__(256) fp_pack_weights_kernel(const uint16_t* __restrict__ W, int64_t K,
                                                              uint8_t* __restrict__ wq4, float* __restrict__ s_w,
                                                              uint8_t* __restrict__ w8) {
  __shared__ uint32_t scratch[8];
  const int tid = threadIdx.x;
  const int64_t n = blockIdx.x;
  const uint16_t* row = W + n * K;
  uint32_t mx = 0;
  for (int64_t j = tid; j < K; j += 256) mx = max(mx, (uint32_t)(row[j] & 0x7FFFu));
  const float wmax = bf16_bits_to_f32(block_max(mx, scratch));
  const float c = wmax > 0.f ? __fdiv_rn(6.0f, wmax) : 0.f;
  if (tid == 0) s_w[n] = wmax > 0.f ? __fdiv_rn(wmax, 6.0f) : 0.f;
  for (int64_t j2 = tid; j2 < K / 2; j2 += 256) {
    const uint32_t q0 = e2m1_of((double)bf16_bits_to_f32(row[2 * j2]) * (double)c);
    const uint32_t q1 = e2m1_of((double)bf16_bits_to_f32(row[2 * j2 + 1]) * (double)c);
    wq4[n * (K / 2) + j2] = (uint8_t)(q0 | (q1 << 4));
    *reinterpret_cast<uint16_t*>(w8 + n * K + 2 * j2) = (uint16_t)(e4m3_of_e2m1(q0, 0) | (e4m3_of_e2m1(q1, 0) << 8));
  }
}

// Plain encoder for the formats and row lengths the integer path's fast kernels do not take (those
// kernels, templated on the format, encode the rest: sq_encode.cu).  One block per token row, the
// row staged in shared memory.  Dynamic positions: a warp per bank finds the k-th largest
// magnitude by a bitwise search on warp-wide counts; codes by single-precision magic-number
// rounding; a selected place is marked in the staged row by a non-finite pattern that carries its
// byte, so the dense pass writes whole words of nibbles and of the merged operand.
template <int B>
__global__ void __launch_bounds__(256) fp_encode_kernel(int k, const uint16_t* __restrict__ X, int64_t K,
                                                        const uint8_t* __restrict__ positions, uint8_t* __restrict__ dq4,
                                                        uint8_t* __restrict__ vals, uint8_t* __restrict__ idx,
                                                        float* __restrict__ s_hi, float* __restrict__ s_lo,
                                                        uint8_t* __restrict__ shift, uint8_t* __restrict__ a8) {
  extern __shared__ __align__(16) uint16_t srow[];
  __shared__ uint32_t scratch[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t m = blockIdx.x, G = K / B;
  const uint16_t* xrow = X + m * K;
  uint32_t mx = 0;
  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8) {
    const uint4 v = ldg_nc_v4(xrow + i);
    *reinterpret_cast<uint4*>(srow + i) = v;
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) mx = max(mx, max(w[q] & 0x7FFFu, (w[q] >> 16) & 0x7FFFu));
  }
  const float amax = bf16_bits_to_f32(block_max(mx, scratch));  // barrier inside: row staged
  const float inv = amax > 0.f ? __fdiv_rn(256.0f, amax) : 0.f;
  const float sh = amax > 0.f ? __fdiv_rn(amax, 256.0f) : 0.f;
  uint8_t* arow = a8 + m * K;

  // sparse entries: E4M3 of a * inv, in ascending position.  Their places in the staged row are
  // overwritten with a marker that carries the byte: exponent field all ones (no finite input has
  // it), the byte's sign in the sign bit, its other seven bits in the mantissa -- the dense pass
  // recognises the place and finds the merged operand's byte there.
  auto marker = [](uint32_t q) -> uint16_t { return (uint16_t)(((q & 0x80u) << 8) | 0x7F80u | (q & 0x7Fu)); };
  if (positions != nullptr) {
    for (int64_t t = tid; t < G * k; t += 256) {
      const int64_t j = (t / k) * B + positions[t];
      const uint32_t q = e4m3_of32(srow[j], inv);
      vals[m * G * k + t] = (uint8_t)q;
      srow[j] = marker(q);
    }
  } else {
    constexpr int EPL = B / 32;
    for (int64_t g = warp; g < G; g += 8) {
      uint32_t mag[EPL], raw[EPL];
#pragma unroll
      for (int t = 0; t < EPL; ++t) {
        raw[t] = srow[g * B + lane + 32 * t];
        mag[t] = raw[t] & 0x7FFFu;
      }
      // T = the k-th largest magnitude of the bank (with multiplicity): the largest T with at least
      // k magnitudes >= T, built bit by bit from warp-wide counts.  Everything above T is selected;
      // of the elements equal to T the lowest indices fill what is left.  (Several banks in flight
      // per warp were measured no faster: the kernel is bound by instruction count, not latency.)
      uint32_t T = 0;
      for (int bit = 14; bit >= 0; --bit) {
        const uint32_t cand = T | (1u << bit);
        int c = 0;
#pragma unroll
        for (int t = 0; t < EPL; ++t) c += mag[t] >= cand ? 1 : 0;
        if (__reduce_add_sync(0xffffffffu, c) >= k) T = cand;
      }
      int above = 0;
#pragma unroll
      for (int t = 0; t < EPL; ++t) above += mag[t] > T ? 1 : 0;
      const int need = k - __reduce_add_sync(0xffffffffu, above);
      int before_eq = 0, before = 0;
#pragma unroll
      for (int t = 0; t < EPL; ++t) {  // index order: t = 0 holds elements 0..31, lanes ascending
        const bool eq = mag[t] == T;
        const uint32_t m_eq = __ballot_sync(0xffffffffu, eq);
        const bool sel = mag[t] > T || (eq && before_eq + __popc(m_eq & ((1u << lane) - 1u)) < need);
        before_eq += __popc(m_eq);
        const uint32_t mask = __ballot_sync(0xffffffffu, sel);
        if (sel) {
          const int slot = before + __popc(mask & ((1u << lane) - 1u));
          const int j = lane + 32 * t;
          const uint32_t q = e4m3_of32(raw[t], inv);
          vals[(m * G + g) * k + slot] = (uint8_t)q;
          idx[(m * G + g) * k + slot] = (uint8_t)j;
          srow[g * B + j] = marker(q);
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
      const uint32_t lo = w[q] & 0x7FFFu, hi = (w[q] >> 16) & 0x7FFFu;
      if (lo < 0x7F80u) rm = max(rm, lo);  // (a marker's magnitude bits are at least 0x7F80)
      if (hi < 0x7F80u) rm = max(rm, hi);
    }
  }
  const float rmax = bf16_bits_to_f32(block_max(rm, scratch));
  int e = 0;
  if (amax > 0.f) {
    e = 6;
    for (int t = 6; t >= 0; --t)
      if ((double)rmax * (double)(inv * __int_as_float((127 - t) << 23)) <= 6.0) e = t;  // ends on the smallest fitting t
  }
  if (tid == 0) {
    s_hi[m] = sh;
    s_lo[m] = sh * (float)(1 << e);
    shift[m] = (uint8_t)e;
  }
  // dense codes, eight elements per thread and step: one 32-bit word of nibbles and eight bytes of
  // the merged operand
  const float inv_lo = inv * __int_as_float((127 - e) << 23);
  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(srow + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t nib = 0, by[2] = {0, 0};
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const uint32_t h = (w[q >> 1] >> (16 * (q & 1))) & 0xFFFFu;
      uint32_t code = 0, byte;
      if ((h & 0x7F80u) == 0x7F80u) {
        byte = ((h >> 8) & 0x80u) | (h & 0x7Fu);
      } else {
        code = e2m1_of32(h, inv_lo);
        byte = e4m3_of_e2m1(code, e);
      }
      nib |= code << (4 * q);
      by[q >> 2] |= byte << (8 * (q & 3));
    }
    *reinterpret_cast<uint32_t*>(dq4 + m * (K / 2) + i / 2) = nib;
    *reinterpret_cast<uint2*>(arow + i) = make_uint2(by[0], by[1]);
  }
}

__device__ __forceinline__ float e2m1_value_f(uint32_t c) {
  const uint32_t t = c & 7u;
  const float mag = t < 2 ? 0.5f * (float)t : __int_as_float((int)(((t >> 1) + 126) << 23) | (int)((t & 1u) << 22));
  return (c & 8u) ? -mag : mag;
}
__device__ __forceinline__ float e4m3_value_f(uint32_t c) {
  const uint32_t e = (c >> 3) & 15u, mt = c & 7u;
  const float mag = e == 0 ? (float)mt * 0.001953125f : __int_as_float((int)((e + 120) << 23) | (int)(mt << 20));
  return (c & 0x80u) ? -mag : mag;
}

__global__ void __launch_bounds__(256) fp_decode_kernel(int b, int k, const uint8_t* __restrict__ dq4,
                                                        const uint8_t* __restrict__ vals, const uint8_t* __restrict__ idx,
                                                        const uint8_t* __restrict__ positions, const float* __restrict__ s_hi,
                                                        const float* __restrict__ s_lo, int64_t K, uint16_t* __restrict__ out) {
  const int tid = threadIdx.x;
  const int64_t m = blockIdx.x;
  const float sl = s_lo[m], shh = s_hi[m];
  for (int64_t i = tid; i < K / 2; i += 256) {
    const uint32_t byte = dq4[m * (K / 2) + i];
    out[m * K + 2 * i] = (uint16_t)f32_to_bf16_bits(sl * e2m1_value_f(byte & 0xFu));
    out[m * K + 2 * i + 1] = (uint16_t)f32_to_bf16_bits(sl * e2m1_value_f(byte >> 4));
  }
  __syncthreads();
  const int64_t G = K / b, GK = G * k;
  for (int64_t t = tid; t < GK; t += 256) {
    const int local = idx != nullptr ? idx[m * GK + t] : positions[t];
    out[m * K + (t / k) * b + local] = (uint16_t)f32_to_bf16_bits(shh * e4m3_value_f(vals[m * GK + t]));
  }
}

// ------------------------------------------------------------------------------------------------
// GEMM: persistent, one CTA per SM, K steps of 128, everything fed by TMA.
//   warp 0      one thread: TMA loads of this CTA's A (a8) and B (w8) tiles of a step into a ring
//               (128-byte swizzle: the layout the tensor core reads), both on one mbarrier
//   warp 1      one thread (of the leader CTA): four tcgen05.mma.kind::f8f6f4 (K = 32 each) per
//               step, fp32 accumulation in tensor memory; two accumulators (all 512 columns), so
//               the epilogue of a tile overlaps the main loop of the next
//   warps 2-5   epilogue: tcgen05.ld, (acc * s_hi[m]) * s_w[n], bf16, 16-byte stores
// PAIR = 1 (at most 128 rows): tiles of 128 rows x 256 output channels per CTA.  Its shared memory
// is the bound: per K = 32 instruction 12 KB arrive by TMA and 12 KB are read by the tensor core in
// the 128 cycles the instruction takes, 192 of the 128 bytes per cycle there are (measured: the
// tensor pipe 69 % busy).
// PAIR = 2 (more rows): two CTAs of a cluster share a tile of 256 rows x 256 channels through
// tcgen05.mma.cta_group::2.  Each holds its own 128 rows of A and HALF of the weight tile, which
// both tensor cores read from both shared memories: 8 KB in and 8 KB out per instruction and CTA.
// Only the leader issues; the peer's idle MMA warp reports each of its landed stages to the
// leader's "full" barrier; completions are multicast to both CTAs' "empty" and "accumulator
// ready" barriers; both epilogues hand the accumulators back on the leader's barrier.
// Concurrent CTAs work on neighbouring row tiles of the same 256 channels, so a weight tile is
// fetched from HBM once and then served by L2.
namespace {

constexpr int FBM = 128, FBN = 256, FBK = 128;
template <int PAIR>
struct FGeo {
  // 128-byte blocks of K per stage.  A pair's stage is 8 instructions: with 4, waiting for the
  // stage's barrier, issuing and committing take longer than the 0.28 us of tensor work they start.
  static constexpr int KB = PAIR == 2 ? 2 : 1;
  static constexpr int NS = PAIR == 2 ? 3 : 4;
  static constexpr int kStageA = KB * FBM * FBK;             // this CTA's rows
  static constexpr int kStageB = KB * (FBN / PAIR) * FBK;    // this CTA's share of the output channels
  static constexpr int kSmem = NS * (kStageA + kStageB) + 256;
};
constexpr int kFThreads = 6 * 32;

struct FpGemmParams {
  const float* s_hi;
  const float* s_w;
  uint16_t* out;
  float* acc_out;
  int* status;
  int M, N, K;
};

__device__ __forceinline__ uint64_t fdesc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// D = f32 (1 at bit 4); A, B = E4M3 (format 0), K-major; N at bit 17, M (of the whole instruction:
// 128 per participating CTA) at bit 24.
__device__ __forceinline__ constexpr uint32_t f_idesc(int m) {
  return (1u << 4) | (0u << 7) | (0u << 10) | ((uint32_t)(FBN >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

template <int CG>
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  if (CG == 2)
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void f_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void f_tma_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// A wait of the leader on a barrier the peer also arrives on acquires at cluster scope.
template <int PAIR>
__device__ __forceinline__ bool f_wait_leader(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return PAIR == 2 ? mbar_wait_cluster(bar, parity, abort_flag) : mbar_wait(bar, parity, abort_flag);
}

}  // namespace

template <int PAIR>
__global__ void __launch_bounds__(kFThreads, 1)
    fp_gemm_kernel(const FpGemmParams p, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b) {
  using G = FGeo<PAIR>;
  constexpr int NS = G::NS, KB = G::KB, kStageA = G::kStageA, kStageB = G::kStageB;
  constexpr int TM = FBM * PAIR;  // rows of a tile
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  const bool misaligned = (smem_u32(smem_raw) & 1023u) != 0;  // the same in every CTA: nobody is left waiting
  if (misaligned) {
    if (threadIdx.x == 0) atomicExch(p.status, (int)SQ_ERR_CUDA);
    return;
  }
  uint8_t* sA = smem;
  uint8_t* sB = sA + NS * kStageA;
  uint8_t* sCtl = sB + NS * kStageB;
  const uint32_t bar_full = smem_u32(sCtl);          // NS
  const uint32_t bar_empty = bar_full + 8 * NS;      // NS
  const uint32_t bar_tfull = bar_empty + 8 * NS;     // 2: accumulator complete
  const uint32_t bar_tempty = bar_tfull + 16;        // 2: accumulator read out
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sCtl + 8 * (2 * NS + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sCtl + 8 * (2 * NS + 4) + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rank = PAIR == 2 ? (int)cluster_ctarank() : 0;
  const int cl = (int)blockIdx.x / PAIR, ncl = (int)gridDim.x / PAIR;  // this CTA (pair) among the CTAs (pairs)
  const int tiles_m = (p.M + TM - 1) / TM, tiles_n = (p.N + FBN - 1) / FBN;
  const int KBT = p.K / FBK;              // 128-byte blocks of K
  const int ntiles = tiles_m * tiles_n, KS = (KBT + KB - 1) / KB;

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      // leader of a pair: its own loads' arrival plus the peer's report
      mbar_init(bar_full + 8 * s, (PAIR == 2 && rank == 0) ? 2 : 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, PAIR * 4);  // one arrival per epilogue warp (of both CTAs, on the leader's)
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc<PAIR>(smem_u32(tmem_slot), 2 * FBN);
    tmem_relinquish<PAIR>();
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR == 2) cluster_sync_all();  // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = cl; t < ntiles && ok; t += ncl) {
        const int m0 = (t % tiles_m) * TM + rank * FBM, n0 = (t / tiles_m) * FBN + rank * (FBN / PAIR);
        for (int ks = 0; ks < KS && ok; ++ks, ++it) {
          const int s = it % NS;
          ok = mbar_wait(bar_empty + 8 * s, ((it / NS) & 1u) ^ 1u, abort_flag);
          if (!ok) break;
          const uint32_t bar = bar_full + 8 * s;
          const int nkb = min(KB, KBT - ks * KB);
          f_expect_tx(bar, (uint32_t)(nkb * (kStageA + kStageB) / KB));  // rows past M / N come back as zeros
          for (int kb = 0; kb < nkb; ++kb) {
            f_tma_2d(smem_u32(sA + s * kStageA + kb * (FBM * FBK)), &map_a, (ks * KB + kb) * FBK, m0, bar);
            f_tma_2d(smem_u32(sB + s * kStageB + kb * ((FBN / PAIR) * FBK)), &map_b, (ks * KB + kb) * FBK, n0, bar);
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = f_idesc(TM);
      uint32_t it = 0, tc = 0;
      bool ok = true;
      for (int t = cl; t < ntiles && ok; t += ncl, ++tc) {
        const uint32_t buf = tc & 1u;
        // the accumulator's previous tile was read out (by both CTAs)
        ok = f_wait_leader<PAIR>(bar_tempty + 8 * buf, ((tc >> 1) & 1u) ^ 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        for (int ks = 0; ks < KS && ok; ++ks, ++it) {
          const int s = it % NS;
          ok = f_wait_leader<PAIR>(bar_full + 8 * s, (it / NS) & 1u, abort_flag);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kb = 0; kb < KB; ++kb) {
            if (ks * KB + kb < KBT) {  // (the last stage of an odd number of 128-byte blocks is half full)
              const uint64_t da = fdesc(smem_u32(sA + s * kStageA + kb * (FBM * FBK)));
              const uint64_t db = fdesc(smem_u32(sB + s * kStageB + kb * ((FBN / PAIR) * FBK)));
#pragma unroll
              for (int kk = 0; kk < FBK / 32; ++kk)
                umma_f8<PAIR>(tmem + buf * FBN, da + 2 * kk, db + 2 * kk, idesc, (ks > 0 || kb > 0 || kk > 0) ? 1u : 0u);
            }
          }
          umma_commit<PAIR>(bar_empty + 8 * s);
        }
        if (ok) umma_commit<PAIR>(bar_tfull + 8 * buf);
      }
    } else if (lane == 0 && PAIR == 2) {
      // The leader's MMA thread cannot watch this CTA's barriers: report every landed stage, in
      // order, on the leader's "full" barrier.  (A stage is re-armed only after the leader has
      // used it, so no phase can pass unseen.)
      uint32_t it = 0;
      bool ok = true;
      for (int t = cl; t < ntiles && ok; t += ncl) {
        for (int ks = 0; ks < KS && ok; ++ks, ++it) {
          const int s = it % NS;
          ok = mbar_wait(bar_full + 8 * s, (it / NS) & 1u, abort_flag);
          if (ok) mbar_arrive_cta(bar_full + 8 * s, 0);
        }
      }
    }
    __syncwarp();
  } else {
    const int q = warp & 3;  // tensor-memory lane quarter this warp may read
    uint32_t tc = 0;
    for (int t = cl; t < ntiles; t += ncl, ++tc) {
      const uint32_t buf = tc & 1u;
      const int m0 = (t % tiles_m) * TM + rank * FBM, n0 = (t / tiles_m) * FBN;
      const int m = m0 + 32 * q + lane;
      const float sh = m < p.M ? __ldg(p.s_hi + m) : 0.f;
      if (!mbar_wait_idle(bar_tfull + 8 * buf, (tc >> 1) & 1u, abort_flag)) break;
      tc_fence_after();
      for (int c0 = 0; c0 < FBN; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * FBN + c0), v);
        tmem_ld_wait();
        if (m < p.M) {
#pragma unroll
          for (int c8 = 0; c8 < 32; c8 += 8) {
            const int n = n0 + c0 + c8;
            if (n < p.N) {  // N % 8 == 0: a group of 8 columns is all in or all out
              uint32_t o[4];
#pragma unroll
              for (int cc = 0; cc < 8; cc += 2) {
                const float f0 = (__uint_as_float(v[c8 + cc]) * sh) * __ldg(p.s_w + n + cc);
                const float f1 = (__uint_as_float(v[c8 + cc + 1]) * sh) * __ldg(p.s_w + n + cc + 1);
                o[cc >> 1] = pack_bf16x2(f0, f1);
              }
              *reinterpret_cast<uint4*>(p.out + (size_t)m * p.N + n) = make_uint4(o[0], o[1], o[2], o[3]);
              if (p.acc_out != nullptr) {
                uint4* dst = reinterpret_cast<uint4*>(p.acc_out + (size_t)m * p.N + n);
                dst[0] = make_uint4(v[c8], v[c8 + 1], v[c8 + 2], v[c8 + 3]);
                dst[1] = make_uint4(v[c8 + 4], v[c8 + 5], v[c8 + 6], v[c8 + 7]);
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR == 2) mbar_arrive_cta(bar_tempty + 8 * buf, 0);
        else mbar_arrive(bar_tempty + 8 * buf);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  // Neither CTA of a pair may leave (or free tensor memory) while the other can still arrive on
  // its barriers or have instructions reading its shared memory.
  if (PAIR == 2) cluster_sync_all();
  if (tid == 0 && *abort_flag) atomicExch(p.status, (int)SQ_ERR_TIMEOUT);
  if (warp == 1) tmem_dealloc<PAIR>(tmem, 2 * FBN);
}

// ------------------------------------------------------------------------------------------------

cudaError_t launch_fp_pack_weights(const uint16_t* W, int64_t N, int64_t K, uint8_t* wq4, float* s_w, uint8_t* w8,
                                   cudaStream_t st) {
  fp_pack_weights_kernel<<<(unsigned)N, 256, 0, st>>>(W, K, wq4, s_w, w8);
  return cudaGetLastError();
}

cudaError_t launch_fp_encode(int b, int k, const uint16_t* X, int64_t M, int64_t K, const uint8_t* positions,
                             const sq_encoded& out, uint8_t* a8, cudaStream_t st) {
  const size_t smem = (size_t)K * 2;
  uint8_t* vals = reinterpret_cast<uint8_t*>(out.vals);
#define SQ_FP_ENC(BB)                                                                                                \
  do {                                                                                                               \
    static std::atomic<size_t> limit[64];                                                                            \
    int dev = 0;                                                                                                     \
    cudaError_t err = cudaGetDevice(&dev);                                                                           \
    if (err != cudaSuccess) return err;                                                                              \
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;                                                         \
    if (smem > limit[dev].load(std::memory_order_acquire)) {                                                         \
      std::lock_guard<std::mutex> lock(setup_mutex());                                                               \
      err = cudaFuncSetAttribute(fp_encode_kernel<BB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);      \
      if (err != cudaSuccess) return err;                                                                            \
      limit[dev].store(smem, std::memory_order_release);                                                             \
    }                                                                                                                \
    fp_encode_kernel<BB><<<(unsigned)M, 256, smem, st>>>(k, X, K, positions, out.dq4, vals, out.idx, out.s_hi,       \
                                                         out.s_lo, out.shift, a8);                                   \
  } while (0)
  if (b == 32) SQ_FP_ENC(32);
  else if (b == 64) SQ_FP_ENC(64);
  else SQ_FP_ENC(128);
#undef SQ_FP_ENC
  return cudaGetLastError();
}

cudaError_t launch_fp_decode(int b, int k, const sq_encoded& A, const uint8_t* positions, int64_t M, int64_t K,
                             uint16_t* out, cudaStream_t st) {
  fp_decode_kernel<<<(unsigned)M, 256, 0, st>>>(b, k, A.dq4, reinterpret_cast<const uint8_t*>(A.vals), A.idx, positions,
                                               A.s_hi, A.s_lo, K, out);
  return cudaGetLastError();
}

// Measurement aid, as the integer path's: the rate at which the tensor core takes this variant's
// instruction (tcgen05.mma.kind::f8f6f4, E4M3 x E4M3, 128 x 256 x 32) on operands that stay in
// shared memory; no loads, no epilogue.
__global__ void __launch_bounds__(128, 1) fp8_peak_kernel(int iters, int* status) {
  extern __shared__ __align__(1024) uint8_t smem_pk[];  // A: 128 rows x 128 B | B: 256 rows x 128 B
  __shared__ uint64_t bar_s;
  __shared__ uint32_t tmem_slot_s;
  __shared__ int abort_s;
  const int tid = threadIdx.x, warp = tid >> 5;
  if ((smem_u32(smem_pk) & 1023u) != 0) {
    if (tid == 0) atomicExch(status, (int)SQ_ERR_CUDA);
    return;
  }
  // operands of mixed bits (small finite E4M3 values: the exponent's top bit stays clear)
  for (int i = tid; i < (FBM + FBN) * FBK / 16; i += 128) {
    const uint32_t h = (uint32_t)i * 2654435761u;
    reinterpret_cast<uint4*>(smem_pk)[i] = make_uint4(h & 0xBFBFBFBFu, (h * 2246822519u) & 0xBFBFBFBFu, (h ^ 0x9E3779B9u) & 0xBFBFBFBFu,
                                                      (~h * 3266489917u) & 0xBFBFBFBFu);
  }
  fence_proxy_async_smem();
  const uint32_t bar = smem_u32(&bar_s);
  if (tid == 0) {
    mbar_init(bar, 1);
    abort_s = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc<1>(smem_u32(&tmem_slot_s), 2 * FBN);
    tmem_relinquish<1>();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot_s;
  if (tid == 0) {
    const uint64_t da = fdesc(smem_u32(smem_pk)), db = fdesc(smem_u32(smem_pk + FBM * FBK));
    constexpr uint32_t idesc = f_idesc(FBM);
    uint32_t phase = 0;
    bool ok = true;
    for (int it = 0; it < iters && ok; ++it) {
#pragma unroll
      for (int kk = 0; kk < FBK / 32; ++kk) umma_f8<1>(tmem + (uint32_t)((it & 1) * FBN), da + 2 * kk, db + 2 * kk, idesc, 1u);
      if ((it & 63) == 63 || it == iters - 1) {  // a bounded wait every 256 instructions keeps the queue shallow
        umma_commit<1>(bar);
        ok = mbar_wait(bar, phase, &abort_s);
        phase ^= 1u;
      }
    }
    if (!ok) atomicExch(status, (int)SQ_ERR_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc<1>(tmem, 2 * FBN);
}

cudaError_t launch_fp8_peak_probe(int iters, double* ops, int* status, cudaStream_t st) {
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  const int smem = (FBM + FBN) * FBK;
  err = cudaFuncSetAttribute(fp8_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (err != cudaSuccess) return err;
  if (ops != nullptr) *ops = 2.0 * FBM * FBN * FBK * (double)iters * (double)sms;
  fp8_peak_kernel<<<(unsigned)sms, 128, smem, st>>>(iters, status);
  return cudaGetLastError();
}

cudaError_t launch_fp_gemm(const float* s_hi, const uint8_t* a8, const float* s_w, const uint8_t* w8, int64_t M, int64_t N,
                           int64_t K, uint16_t* out, float* acc_out, int* status, cudaStream_t st) {
  static std::atomic<int> sm_count_of[64];
  static std::atomic<bool> attr_set[64];
  static std::atomic<PFN_cuTensorMapEncodeTiled> encode_fn{nullptr};
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int sms = sm_count_of[dev].load(std::memory_order_acquire);
  if (sms == 0) {
    err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (err != cudaSuccess) return err;
    sm_count_of[dev].store(sms, std::memory_order_release);
  }
  PFN_cuTensorMapEncodeTiled encode = encode_fn.load(std::memory_order_acquire);
  if (encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (err != cudaSuccess) return err;
    if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
    encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
    encode_fn.store(encode, std::memory_order_release);
  }
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(setup_mutex());
    err = cudaFuncSetAttribute(fp_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, FGeo<1>::kSmem);
    if (err != cudaSuccess) return err;
    err = cudaFuncSetAttribute(fp_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, FGeo<2>::kSmem);
    if (err != cudaSuccess) return err;
    attr_set[dev].store(true, std::memory_order_release);
  }
  // CTA pairs from 129 rows on (a second CTA would have no rows below that)
  const int pair = M > FBM ? 2 : 1;
  CUtensorMap map_a, map_b;
  const cuuint32_t estr[2] = {1, 1};
  const cuuint64_t pitch[1] = {(cuuint64_t)K};
  const cuuint64_t dim_a[2] = {(cuuint64_t)K, (cuuint64_t)M}, dim_b[2] = {(cuuint64_t)K, (cuuint64_t)N};
  const cuuint32_t box_a[2] = {FBK, FBM}, box_b[2] = {FBK, (cuuint32_t)(FBN / pair)};
  if (encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(a8), dim_a, pitch, box_a, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  if (encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(w8), dim_b, pitch, box_b, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  FpGemmParams p;
  p.s_hi = s_hi;
  p.s_w = s_w;
  p.out = out;
  p.acc_out = acc_out;
  p.status = status;
  p.M = (int)M;
  p.N = (int)N;
  p.K = (int)K;
  const int64_t ntiles = ((M + FBM * pair - 1) / (FBM * pair)) * ((N + FBN - 1) / FBN);
  if (pair == 1) {
    const unsigned grid = (unsigned)(ntiles < sms ? ntiles : sms);
    fp_gemm_kernel<1><<<grid, kFThreads, FGeo<1>::kSmem, st>>>(p, map_a, map_b);
  } else {
    const int64_t slots = sms / 2;
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof(lc));
    cudaLaunchAttribute la[1];
    la[0].id = cudaLaunchAttributeClusterDimension;
    la[0].val.clusterDim.x = 2;
    la[0].val.clusterDim.y = 1;
    la[0].val.clusterDim.z = 1;
    lc.gridDim = dim3((unsigned)(2 * (ntiles < slots ? ntiles : slots)), 1, 1);
    lc.blockDim = dim3(kFThreads, 1, 1);
    lc.dynamicSmemBytes = FGeo<2>::kSmem;
    lc.stream = st;
    lc.attrs = la;
    lc.numAttrs = 1;
    err = cudaLaunchKernelEx(&lc, fp_gemm_kernel<2>, p, map_a, map_b);
    if (err != cudaSuccess) return err;
  }
  return cudaGetLastError();
}

}  // namespace sq
