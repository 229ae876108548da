// Hybrid SQ-format GEMM on the sm_100a tensor cores (tcgen05, kind::i8).
//
//   acc[m,n] = sum_j ( (dq4[m,j] << e[m]) + [j in S_m] vals[m,j] ) * code[n,j]
//   out[m,n] = bf16( ((float)acc * s_hi[m]) * s_w[n] )
//
// sm_100 has no INT4 MMA, so both operands are widened to 8 bits on chip.  The two
// components of the activation live on one integer grid (the dense one coarsened by
// 2^e), so they can be MERGED into a single 8-bit operand before the tensor core
// sees them: the dense nibbles are widened and shifted, then the k sparse INT8
// entries of every bank overwrite the (zero) places they belong to.  One MMA stream,
// one int32 accumulator in tensor memory, one epilogue.
//
// Operand encodings inside the kernel (chosen so the widening is a few logic ops on
// eight nibbles at a time, never a per-byte sign extension):
//   A is fed UNSIGNED with an offset of 128:  a_u = a + 128, a in [-127, 127].
//     dense:  nibble q in two's complement -> u = q ^ 8 = q + 8 in [1, 15];
//             a_u = u * 2^e + (128 - 8 * 2^e)      (no carries between bytes)
//     sparse: a_u = vals ^ 0x80
//   B is fed SIGNED as 16 * code: a nibble moved to the top of its byte.
//   Hence acc_internal = 16 * acc + 2048 * colsum[n]; the epilogue undoes both exactly.
//   |acc_internal| <= K * 255 * 112 < 2^31 for K <= 65536.
//
// K order inside a 32-element MMA block: eight nibbles come out of one 32-bit word as
// the four even elements and the four odd ones, so both operands store a block as
// [16 even elements | 16 odd elements].  The contraction does not care as long as A
// and B agree.
//
// Shared-memory operand layout: K-major, 128-byte rows (one K step = 128 elements),
// 128-byte swizzle (the 16-byte chunk index is XORed with row % 8), 8-row groups 1024
// bytes apart: the canonical layout a tcgen05 shared-memory descriptor describes.
#include "sq_device.cuh"
#include "sq_host.h"

namespace sq {

namespace {

constexpr int BM = 128;       // rows of A per CTA = TMEM lanes
constexpr int BK = 128;       // K elements per pipeline step = bytes per operand row
constexpr int kThreads = 256;

struct GemmParams {
  const uint8_t* dq4;
  const int8_t* vals;
  const uint8_t* idx;  // dynamic positions [M,G,k] or nullptr
  const uint8_t* pos;  // static positions [G,k] or nullptr
  const float* s_hi;
  const uint8_t* shift;
  const uint8_t* wq4;
  const float* s_w;
  const int32_t* colsum;
  uint16_t* out;
  int32_t* acc_out;
  int* status;
  int M, N, K, b, k;
};

// Shared-memory matrix descriptor: K-major, SWIZZLE_128B, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address
  d |= (uint64_t)1 << 16;                    // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset
  d |= (uint64_t)1 << 46;                    // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                    // SWIZZLE_128B
  return d;
}

// Instruction descriptor: D = s32, A = u8, B = s8, both K-major, M = 128, N = BN.
template <int BN>
__device__ __forceinline__ constexpr uint32_t make_idesc() {
  return (2u << 4)                      // D format: S32
         | (0u << 7)                    // A format: unsigned 8-bit
         | (1u << 10)                   // B format: signed 8-bit
         | ((uint32_t)(BN >> 3) << 17)  // N
         | ((uint32_t)(BM >> 4) << 24); // M
}

// Byte offset inside a [rows][128 B] swizzled tile of K-position p (0..127) of `row`.
__device__ __forceinline__ uint32_t swz(uint32_t row, uint32_t p) {
  return row * 128u + ((((p >> 4) ^ row) & 7u) << 4) + (p & 15u);
}

// K-position (within the 128 of a step) where element jj is stored: blocks of 32,
// even elements first.
__device__ __forceinline__ uint32_t kpos(uint32_t jj) {
  return (jj & ~31u) | ((jj & 1u) << 4) | ((jj & 31u) >> 1);
}

template <int BN, int NS>
struct Smem {
  static constexpr int kA = BM * BK;   // 16 KB
  static constexpr int kB = BN * BK;
  static constexpr int kBytes = NS * (kA + kB) + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

}  // namespace

template <int BN, int NS>
__global__ void __launch_bounds__(kThreads, 1) gemm_kernel(const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - smem_u32(smem_raw));
  uint8_t* sA = smem;                                  // NS x [128][128]
  uint8_t* sB = smem + NS * Smem<BN, NS>::kA;          // NS x [BN][128]
  uint8_t* sCtl = sB + NS * Smem<BN, NS>::kB;
  const uint32_t bar_empty = smem_u32(sCtl);           // NS x 8 B
  const uint32_t bar_done = bar_empty + 8 * NS;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sCtl + 8 * NS + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sCtl + 8 * NS + 16);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile_n = blockIdx.x * BN;
  const int tile_m = blockIdx.y * BM;
  const int KS = p.K / BK;
  const int Kh = p.K / 2;
  const int G = p.K / p.b;

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) mbar_init(bar_empty + 8 * s, 1);
    mbar_init(bar_done, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(tmem_slot), BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  constexpr uint32_t idesc = make_idesc<BN>();
  const int banks_per_step = BK / p.b;
  const int nb = banks_per_step * p.k;  // sparse entries per row per step
  bool ok = true;

  for (int ks = 0; ks < KS && ok; ++ks) {
    const int s = ks % NS;
    uint8_t* a_st = sA + s * Smem<BN, NS>::kA;
    uint8_t* b_st = sB + s * Smem<BN, NS>::kB;
    if (ks >= NS) {
      // the MMAs that read this stage NS steps ago must have finished
      const bool w = mbar_wait(bar_empty + 8 * s, (uint32_t)((ks / NS - 1) & 1), abort_flag);
      ok = __syncthreads_and(w);
      if (!ok) break;
    }
    // ---- widen A: 128 rows x 4 packed chunks of 16 B (32 nibbles) -> two 16 B chunks each
    for (int t = tid; t < BM * 4; t += kThreads) {
      const int row = t >> 2, c = t & 3;
      const int m = tile_m + row;
      uint4 w = make_uint4(0, 0, 0, 0);
      int e = 0;
      if (m < p.M) {
        w = ldg_nc_v4(p.dq4 + (size_t)m * Kh + (size_t)ks * 64 + c * 16);
        e = p.shift[m];
      }
      const uint32_t off = 0x01010101u * (uint32_t)(128 - (8 << e));
      const uint32_t in[4] = {w.x, w.y, w.z, w.w};
      uint32_t ev[4], od[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t u = in[q] ^ 0x88888888u;  // offset-binary nibbles
        ev[q] = ((u & 0x0F0F0F0Fu) << e) + off;
        od[q] = (((u >> 4) & 0x0F0F0F0Fu) << e) + off;
      }
      const uint32_t r7 = row & 7;
      *reinterpret_cast<uint4*>(a_st + row * 128 + (((2 * c) ^ r7) << 4)) = make_uint4(ev[0], ev[1], ev[2], ev[3]);
      *reinterpret_cast<uint4*>(a_st + row * 128 + (((2 * c + 1) ^ r7) << 4)) = make_uint4(od[0], od[1], od[2], od[3]);
    }
    // ---- widen B: BN rows x 4 packed chunks -> 16 * code
    for (int t = tid; t < BN * 4; t += kThreads) {
      const int row = t >> 2, c = t & 3;
      const int n = tile_n + row;
      uint4 w = make_uint4(0, 0, 0, 0);
      if (n < p.N) w = ldg_nc_v4(p.wq4 + (size_t)n * Kh + (size_t)ks * 64 + c * 16);
      const uint32_t in[4] = {w.x, w.y, w.z, w.w};
      uint32_t ev[4], od[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        ev[q] = (in[q] << 4) & 0xF0F0F0F0u;
        od[q] = in[q] & 0xF0F0F0F0u;
      }
      const uint32_t r7 = row & 7;
      *reinterpret_cast<uint4*>(b_st + row * 128 + (((2 * c) ^ r7) << 4)) = make_uint4(ev[0], ev[1], ev[2], ev[3]);
      *reinterpret_cast<uint4*>(b_st + row * 128 + (((2 * c + 1) ^ r7) << 4)) = make_uint4(od[0], od[1], od[2], od[3]);
    }
    __syncthreads();
    // ---- sparse INT8 entries overwrite their places in the widened A tile
    for (int t = tid; t < BM * nb; t += kThreads) {
      const int row = t / nb, i = t - row * nb;
      const int m = tile_m + row;
      if (m < p.M) {
        const int bank = i / p.k;
        const int g = ks * banks_per_step + bank;
        const size_t entry = ((size_t)m * G + g) * p.k + (i - bank * p.k);
        const int local = p.idx != nullptr ? p.idx[entry] : p.pos[(size_t)g * p.k + (i - bank * p.k)];
        const uint32_t jj = (uint32_t)(bank * p.b + local);
        a_st[swz((uint32_t)row, kpos(jj))] = (uint8_t)((uint8_t)p.vals[entry] ^ 0x80u);
      }
    }
    fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's async reads
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint64_t da = make_desc(smem_u32(a_st));
      const uint64_t db = make_desc(smem_u32(b_st));
#pragma unroll
      for (int kk = 0; kk < BK / 32; ++kk)  // 32 bytes of K per MMA: +2 in 16-byte address units
        umma_i8(tmem, da + 2 * kk, db + 2 * kk, idesc, (ks > 0 || kk > 0) ? 1u : 0u);
      umma_commit(bar_empty + 8 * s);
      if (ks == KS - 1) umma_commit(bar_done);
    }
  }

  if (ok) {
    const bool w = mbar_wait(bar_done, 0, abort_flag);
    ok = __syncthreads_and(w);
  }
  tc_fence_after();

  if (ok) {
    // ---- epilogue: warp w reads TMEM lanes 32*(w%4).., columns half (w/4)
    const int q = warp & 3, h = warp >> 2;
    const int m = tile_m + 32 * q + lane;
    const float sh = (m < p.M) ? p.s_hi[m] : 0.f;
    for (int c0 = h * (BN / 2); c0 < (h + 1) * (BN / 2); c0 += 32) {
      uint32_t v[32];
      tmem_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)c0, v);
      tmem_ld_wait();
      const int n0 = tile_n + c0;
      if (m < p.M && n0 < p.N) {
#pragma unroll
        for (int c8 = 0; c8 < 32; c8 += 8) {
          if (n0 + c8 < p.N) {  // N % 8 == 0: a group of 8 columns is all in or all out
            int acc[8];
            uint32_t o[4];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const int n = n0 + c8 + c;
              acc[c] = ((int)v[c8 + c] - 2048 * __ldg(p.colsum + n)) >> 4;
            }
#pragma unroll
            for (int c = 0; c < 8; c += 2) {
              const float f0 = ((float)acc[c] * sh) * __ldg(p.s_w + n0 + c8 + c);
              const float f1 = ((float)acc[c + 1] * sh) * __ldg(p.s_w + n0 + c8 + c + 1);
              o[c >> 1] = f32_to_bf16_bits(f0) | (f32_to_bf16_bits(f1) << 16);
            }
            *reinterpret_cast<uint4*>(p.out + (size_t)m * p.N + n0 + c8) = make_uint4(o[0], o[1], o[2], o[3]);
            if (p.acc_out != nullptr) {
              int4* dst = reinterpret_cast<int4*>(p.acc_out + (size_t)m * p.N + n0 + c8);
              dst[0] = make_int4(acc[0], acc[1], acc[2], acc[3]);
              dst[1] = make_int4(acc[4], acc[5], acc[6], acc[7]);
            }
          }
        }
      }
    }
  } else if (tid == 0) {
    atomicExch(p.status, (int)SQ_ERR_TIMEOUT);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, BN);
}

cudaError_t launch_gemm(int b, int k, const sq_encoded& A, const sq_weights& W,
                        const uint8_t* positions, int64_t M, int64_t N, int64_t K, uint16_t* out,
                        int32_t* acc_out, int* status, cudaStream_t st) {
  constexpr int BN = 256, NS = 4;
  GemmParams p;
  p.dq4 = A.dq4;
  p.vals = A.vals;
  p.idx = positions == nullptr ? A.idx : nullptr;
  p.pos = positions;
  p.s_hi = A.s_hi;
  p.shift = A.shift;
  p.wq4 = W.wq4;
  p.s_w = W.s_w;
  p.colsum = W.colsum;
  p.out = out;
  p.acc_out = acc_out;
  p.status = status;
  p.M = (int)M;
  p.N = (int)N;
  p.K = (int)K;
  p.b = b;
  p.k = k;
  const int smem = Smem<BN, NS>::kBytes;
  cudaError_t err = cudaFuncSetAttribute(gemm_kernel<BN, NS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM));
  gemm_kernel<BN, NS><<<grid, kThreads, smem, st>>>(p);
  return cudaGetLastError();
}

}  // namespace sq
