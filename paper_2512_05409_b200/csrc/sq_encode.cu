// Activation encode (bf16 -> SQ-format) and decode (SQ-format -> bf16).
#include "sq_device.cuh"
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

}  // namespace

// One block per token row; the row is staged in shared memory because the scale
// (row maximum) must be known before anything is quantised.
//   phase 1  load the row, row maximum -> inv = 127/amax, s_hi = amax/127
//   phase 2  positions: dynamic = rank every element of a bank by (magnitude, then lower
//            index) and keep ranks < k; static = the given positions.  Selected elements
//            are quantised to INT8, written in ascending position with ballot/popc slots,
//            and zeroed in the staged row.
//   phase 3  maximum of what is left -> shift e, s_lo
//   phase 4  INT4 codes of the staged row (zeros at the selected places), 8 per 32-bit word
template <int B>
__global__ void __launch_bounds__(256) encode_kernel(int k, bool is_static, const uint16_t* __restrict__ X, int64_t K,
                                                     const uint8_t* __restrict__ positions,
                                                     uint8_t* __restrict__ dq4, int8_t* __restrict__ vals,
                                                     uint8_t* __restrict__ idx, float* __restrict__ s_hi,
                                                     float* __restrict__ s_lo, uint8_t* __restrict__ shift) {
  extern __shared__ __align__(16) uint16_t srow[];
  __shared__ uint32_t scratch[8];
  __shared__ int sE;
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
  const float amax = bf16_bits_to_f32(block_max_u32(mx, scratch));  // barrier inside: row staged
  const float inv = amax > 0.f ? __fdiv_rn(127.0f, amax) : 0.f;
  const float sh = amax > 0.f ? __fdiv_rn(amax, 127.0f) : 0.f;

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
  const float rmax = bf16_bits_to_f32(block_max_u32(rm, scratch));
  if (tid == 0) {
    int e = 0;
    if (amax > 0.f) {
      e = 4;
      for (int t = 0; t <= 4; ++t) {
        if (rne_prod(rmax, inv * (1.0f / (float)(1 << t))) <= 7) {
          e = t;
          break;
        }
      }
    }
    sE = e;
    s_hi[m] = sh;
    s_lo[m] = sh * (float)(1 << e);
    shift[m] = (uint8_t)e;
  }
  __syncthreads();
  const float inv_lo = inv * (1.0f / (float)(1 << sE));

  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(srow + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t word = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      int q0 = rne_prod(bf16_bits_to_f32(w[q] & 0xFFFFu), inv_lo);
      int q1 = rne_prod(bf16_bits_to_f32(w[q] >> 16), inv_lo);
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
  const int tid = threadIdx.x;
  const int64_t m = blockIdx.x;
  const float sl = s_lo[m], sh = s_hi[m];
  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8) {
    const uint32_t word = *reinterpret_cast<const uint32_t*>(dq4 + m * (K / 2) + i / 2);
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int n0 = ((int)(word << (28 - 8 * q))) >> 28;  // sign-extended nibble 2q
      const int n1 = ((int)(word << (24 - 8 * q))) >> 28;  // nibble 2q+1
      o[q] = f32_to_bf16_bits(sl * (float)n0) | (f32_to_bf16_bits(sl * (float)n1) << 16);
    }
    *reinterpret_cast<uint4*>(out + m * K + i) = make_uint4(o[0], o[1], o[2], o[3]);
  }
  __syncthreads();
  const int64_t G = K / b, GK = G * k;
  for (int64_t t = tid; t < GK; t += 256) {
    const int64_t g = t / k;
    const int local = idx != nullptr ? idx[m * GK + t] : positions[t];
    out[m * K + g * b + local] = (uint16_t)f32_to_bf16_bits(sh * (float)vals[m * GK + t]);
  }
}

cudaError_t launch_encode(int b, int k, bool is_static, const uint16_t* X, int64_t M, int64_t K,
                          const uint8_t* positions, const sq_encoded& out, cudaStream_t st) {
  const size_t smem = (size_t)K * 2;
  cudaError_t err = cudaSuccess;
#define SQ_LAUNCH_ENCODE(BB)                                                                         \
  do {                                                                                               \
    err = cudaFuncSetAttribute(encode_kernel<BB>, cudaFuncAttributeMaxDynamicSharedMemorySize,       \
                               (int)smem);                                                           \
    if (err != cudaSuccess) return err;                                                              \
    encode_kernel<BB><<<(unsigned)M, 256, smem, st>>>(k, is_static, X, K, positions, out.dq4,        \
                                                      out.vals, out.idx, out.s_hi, out.s_lo,         \
                                                      out.shift);                                    \
  } while (0)
  if (b == 32) SQ_LAUNCH_ENCODE(32);
  else if (b == 64) SQ_LAUNCH_ENCODE(64);
  else SQ_LAUNCH_ENCODE(128);
#undef SQ_LAUNCH_ENCODE
  return cudaGetLastError();
}

cudaError_t launch_decode(int b, int k, const sq_encoded& A, const uint8_t* positions, int64_t M,
                          int64_t K, uint16_t* out, cudaStream_t st) {
  decode_kernel<<<(unsigned)M, 256, 0, st>>>(b, k, A.dq4, A.vals, A.idx, positions, A.s_hi, A.s_lo, K, out);
  return cudaGetLastError();
}

}  // namespace sq
