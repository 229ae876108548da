// SQ-format on WEIGHTS (format part of Algorithm 1; storage of Section 3.2.1 and the weight-matrix
// figure): per bank of b input channels of an output channel the k most important weights are
// kept as INT8, compactly and in position order, and the INT4 array holds the unused code 1000 at
// their places, so the mask is implicit; each part has its own per-channel scale.  The importance
// scores are an input (the paper derives them from smoothing and a Hessian of calibration data).
//
//   sqw_encode_kernel   one block per output channel: per-bank ranking by importance (ties to the
//                       smaller index), the two maxima, both codes, compact values by ballot/popc
//   sqw_act_kernel      per-token symmetric INT8 activations, written in the order the product
//                       kernel reads them ([4 even | 4 odd] elements per 8)
//   sqw_gemm_kernel     decode-shaped product for at most 4 tokens: bound by the weight stream.
//                       The mask differs from channel to channel, so the sparse part is a gather
//                       per output channel and runs on the general-purpose cores; with this few
//                       tokens so does the dense part (packed 4-way integer dot products).  A warp
//                       owns two output channels at a time, a lane whole banks (so the compact
//                       values of a bank are counted off locally); the activations sit in shared
//                       memory.  Two int32 sums per output, joined in fp32:
//                         out = bf16(fmaf(acc_hi, S_high[n], acc_lo * S_low[n]) * s_x[m])
#include "sq_device.cuh"
#include "sq_host.h"

namespace sq {

namespace {

__device__ __forceinline__ uint32_t wblock_max(uint32_t v, uint32_t* scratch) {
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

template <int B>
__global__ void __launch_bounds__(256) sqw_encode_kernel(int k, const uint16_t* __restrict__ W, const float* __restrict__ I,
                                                         int64_t K, uint8_t* __restrict__ wq4, int8_t* __restrict__ w_hi,
                                                         float* __restrict__ s_high, float* __restrict__ s_low) {
  extern __shared__ __align__(16) uint8_t smem_w[];
  uint16_t* srow = reinterpret_cast<uint16_t*>(smem_w);       // the channel's weights
  uint8_t* ssel = smem_w + K * 2;                             // 1 at a selected place
  __shared__ uint32_t scratch[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t n = blockIdx.x, G = K / B;
  constexpr int EPL = B / 32;
  for (int64_t j = tid; j < K; j += 256) srow[j] = W[n * K + j];
  // per-bank ranking: an element is selected when fewer than k elements of its bank beat it
  // (larger score, or equal score and smaller index)
  for (int64_t g = warp; g < G; g += 8) {
    float sc[EPL];
    int rank[EPL];
#pragma unroll
    for (int t = 0; t < EPL; ++t) {
      sc[t] = I[n * K + g * B + lane + 32 * t];
      rank[t] = 0;
    }
#pragma unroll
    for (int u = 0; u < EPL; ++u)
      for (int l = 0; l < 32; ++l) {
        const float other = __shfl_sync(0xffffffffu, sc[u], l);
        const int oj = l + 32 * u;
#pragma unroll
        for (int t = 0; t < EPL; ++t) rank[t] += (other > sc[t] || (other == sc[t] && oj < lane + 32 * t)) ? 1 : 0;
      }
#pragma unroll
    for (int t = 0; t < EPL; ++t) ssel[g * B + lane + 32 * t] = rank[t] < k ? 1 : 0;
  }
  __syncthreads();
  uint32_t hm = 0, lm = 0;
  for (int64_t j = tid; j < K; j += 256) {
    const uint32_t mag = srow[j] & 0x7FFFu;
    if (ssel[j]) hm = max(hm, mag);
    else lm = max(lm, mag);
  }
  const float hmax = bf16_bits_to_f32(wblock_max(hm, scratch)), lmax = bf16_bits_to_f32(wblock_max(lm, scratch));
  const float inv_hi = hmax > 0.f ? __fdiv_rn(127.0f, hmax) : 0.f, inv_lo = lmax > 0.f ? __fdiv_rn(7.0f, lmax) : 0.f;
  if (tid == 0) {
    s_high[n] = hmax > 0.f ? __fdiv_rn(hmax, 127.0f) : 0.f;
    s_low[n] = lmax > 0.f ? __fdiv_rn(lmax, 7.0f) : 0.f;
  }
  // INT4 array (the pattern 1000 at a selected place)
  for (int64_t j2 = tid; j2 < K / 2; j2 += 256) {
    uint32_t nb[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int64_t j = 2 * j2 + h;
      nb[h] = ssel[j] ? 8u : ((uint32_t)min(7, max(-7, rne_prod(bf16_bits_to_f32(srow[j]), inv_lo))) & 0xFu);
    }
    wq4[n * (K / 2) + j2] = (uint8_t)(nb[0] | (nb[1] << 4));
  }
  // compact INT8 values, in position order
  for (int64_t g = warp; g < G; g += 8) {
    int before = 0;
#pragma unroll
    for (int t = 0; t < EPL; ++t) {
      const int64_t j = g * B + lane + 32 * t;
      const bool sel = ssel[j] != 0;
      const uint32_t mask = __ballot_sync(0xffffffffu, sel);
      if (sel)
        w_hi[(n * G + g) * k + before + __popc(mask & ((1u << lane) - 1u))] =
            (int8_t)min(127, max(-127, rne_prod(bf16_bits_to_f32(srow[j]), inv_hi)));
      before += __popc(mask);
    }
  }
}

// One block per token: s_x = amax / 127, xq = clamp(RNE(x * 127 / amax)); element j of a group of 8 goes
// to byte (j & 1) * 4 + (j >> 1) of the group.
__global__ void __launch_bounds__(256) sqw_act_kernel(const uint16_t* __restrict__ X, int64_t K, int8_t* __restrict__ xq,
                                                      float* __restrict__ s_x) {
  __shared__ uint32_t scratch[8];
  const int tid = threadIdx.x;
  const int64_t m = blockIdx.x;
  uint32_t mx = 0;
  for (int64_t j = tid; j < K; j += 256) mx = max(mx, (uint32_t)(X[m * K + j] & 0x7FFFu));
  const float amax = bf16_bits_to_f32(wblock_max(mx, scratch));
  const float inv = amax > 0.f ? __fdiv_rn(127.0f, amax) : 0.f;
  if (tid == 0) s_x[m] = amax > 0.f ? __fdiv_rn(amax, 127.0f) : 0.f;
  for (int64_t j = tid; j < K; j += 256) {
    const int q = min(127, max(-127, rne_prod(bf16_bits_to_f32(X[m * K + j]), inv)));
    xq[m * K + (j & ~(int64_t)7) + (j & 1) * 4 + ((j & 7) >> 1)] = (int8_t)q;
  }
}

namespace {
// Byte `sel & 7` of the pair (lo, hi), sign-extended: selector nibbles 1-3 carry bit 3, which makes
// the permute replicate the chosen byte's sign bit.
__device__ __forceinline__ int pick_s8(uint32_t lo, uint32_t hi, uint32_t sel) {
  int d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(lo), "r"(hi), "r"(sel));
  return d;
}
constexpr int kWsqWarps = 8;
constexpr int kWsqCh = 2;  // output channels a warp works on at a time
}

// MT: tokens (1..4).  Shared memory: the reordered INT8 activations [MT][K].
//
// A lane owns whole banks, so it meets exactly k masked places per bank and channel and every lane
// of a warp runs the same number of steps.  Per bank and channel:
//   dense part   three operations per word mark the nibbles that hold 1000, one more turns them
//                into code 0, and the nibbles go as bytes 16 * code into packed 4-way dot products.
//   mask         five more operations per word squeeze the
//                eight marks into a byte (two shifts, one logic operation, one multiply whose
//                partial products do not overlap), and byte permutes string the bytes of four
//                words together: one bit per weight, in position order.
//   sparse part  k steps: lowest set bit -> place, the activation of that place from shared
//                memory, one multiply-add with the compact value (its slot is the step number, so
//                it is picked out of the registers with constant shifts).
template <int B, int MT>
__global__ void __launch_bounds__(kWsqWarps * 32, B == 128 ? 2 : 3) sqw_gemm_kernel(int k, const int8_t* __restrict__ xq,
                                                                     const float* __restrict__ s_x,
                                                                     const uint8_t* __restrict__ wq4,
                                                                     const int8_t* __restrict__ w_hi,
                                                                     const float* __restrict__ s_high,
                                                                     const float* __restrict__ s_low, int M, int N, int K,
                                                                     uint16_t* __restrict__ out, int32_t* __restrict__ acc_out) {
  extern __shared__ __align__(16) int8_t sx[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = K / B;
  constexpr int WPB = B / 8;   // 32-bit words of nibbles per bank
  constexpr int NM = B / 32;   // 32-bit mask registers per bank (one bit per weight)
  constexpr int KW = B / 8;    // 32-bit words of compact values per bank, at most (k <= B / 2)
  // Shared-memory image of the activations: bank by bank (the unit a lane owns), inside a bank
  // word by word (8 elements), inside a word token by token, so that one 16-byte read serves two
  // tokens; a bank is padded so that the lanes of a warp, which read the same word of 32
  // consecutive banks, fall on different memory banks.
  constexpr int kPad = MT == 1 ? 8 : 16;
  constexpr int kBankStride = B * MT + kPad;
  for (int i = tid; i < MT * (K / 16); i += kWsqWarps * 32) {
    const int m = i / (K / 16), c = i % (K / 16);
    const uint4 v = m < M ? __ldg(reinterpret_cast<const uint4*>(xq + (size_t)m * K) + c) : make_uint4(0, 0, 0, 0);
    const int j = 16 * c, g = j / B, w = (j % B) >> 3;  // elements j .. j + 15: words w and w + 1 of bank g
    int8_t* dst = sx + (size_t)g * kBankStride + w * (8 * MT) + m * 8;
    *reinterpret_cast<uint2*>(dst) = make_uint2(v.x, v.y);
    *reinterpret_cast<uint2*>(dst + 8 * MT) = make_uint2(v.z, v.w);
  }
  __syncthreads();
  const bool words_ok = (k & 3) == 0;  // the compact values of a bank start on a 32-bit boundary
  const int pairs = (N + kWsqCh - 1) / kWsqCh;
  for (int pr = blockIdx.x * kWsqWarps + warp; pr < pairs; pr += gridDim.x * kWsqWarps) {
    int lo[kWsqCh][MT], hi[kWsqCh][MT];
#pragma unroll
    for (int c = 0; c < kWsqCh; ++c)
#pragma unroll
      for (int m = 0; m < MT; ++m) lo[c][m] = hi[c][m] = 0;
    for (int g = lane; g < G; g += 32) {
      const int8_t* xb = sx + (size_t)g * kBankStride;  // the bank's activations, reused for both channels
      uint32_t words[kWsqCh][WPB], hv[kWsqCh][KW];
#pragma unroll
      for (int c = 0; c < kWsqCh; ++c) {
        const int n = min(pr * kWsqCh + c, N - 1);
        const uint4* wp = reinterpret_cast<const uint4*>(wq4 + (size_t)n * (K / 2) + g * (B / 2));
#pragma unroll
        for (int w4 = 0; w4 < WPB / 4; ++w4) {
          const uint4 v = __ldg(wp + w4);
          words[c][4 * w4] = v.x;
          words[c][4 * w4 + 1] = v.y;
          words[c][4 * w4 + 2] = v.z;
          words[c][4 * w4 + 3] = v.w;
        }
        const int8_t* hp = w_hi + ((size_t)n * G + g) * k;
        if (words_ok) {
#pragma unroll
          for (int q = 0; q < KW; ++q) hv[c][q] = 4 * q < k ? __ldg(reinterpret_cast<const uint32_t*>(hp) + q) : 0u;
        } else {
#pragma unroll
          for (int q = 0; q < KW; ++q) {
            uint32_t v = 0;
#pragma unroll
            for (int t = 0; t < 4; ++t)
              if (4 * q + t < k) v |= (uint32_t)(uint8_t)__ldg(hp + 4 * q + t) << (8 * t);
            hv[c][q] = v;
          }
        }
      }
      // dense part, word by word for both channels (the word's activations are read once), and the
      // one-bit-per-weight masks
      uint32_t mreg[kWsqCh][NM];
#pragma unroll
      for (int r = 0; r < NM; ++r) {
        uint32_t sq[kWsqCh][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int8_t* xw = xb + (4 * r + j) * (8 * MT);
          int xr[2 * MT];
          if constexpr (MT == 1) {
            const int2 xv = *reinterpret_cast<const int2*>(xw);
            xr[0] = xv.x;
            xr[1] = xv.y;
          } else {
#pragma unroll
            for (int m2 = 0; m2 < MT / 2; ++m2) {
              const int4 xv = *reinterpret_cast<const int4*>(xw + 16 * m2);
              xr[4 * m2] = xv.x;
              xr[4 * m2 + 1] = xv.y;
              xr[4 * m2 + 2] = xv.z;
              xr[4 * m2 + 3] = xv.w;
            }
          }
#pragma unroll
          for (int c = 0; c < kWsqCh; ++c) {
            const uint32_t word = words[c][4 * r + j];
            // nibbles holding 1000: bit 3 set and the three low bits clear -> a mark at bit 4i + 3;
            // flipping the marked bits turns the mask code into code 0
            const uint32_t t = (word & 0x77777777u) + 0x77777777u;
            const uint32_t f3 = word & ~t & 0x88888888u;
            const uint32_t clean = word ^ f3;
            const int ev = (int)((clean << 4) & 0xF0F0F0F0u), od = (int)(clean & 0xF0F0F0F0u);  // 16 * code, bytewise
#pragma unroll
            for (int m = 0; m < MT; ++m) lo[c][m] = __dp4a(ev, xr[2 * m], __dp4a(od, xr[2 * m + 1], lo[c][m]));
            // marks of a byte's two nibbles side by side, then the four pairs into the top byte
            const uint32_t y = ((f3 >> 3) | (f3 >> 6)) & 0x03030303u;
            sq[c][j] = y * 0x01041040u;
          }
        }
#pragma unroll
        for (int c = 0; c < kWsqCh; ++c)
          mreg[c][r] = __byte_perm(__byte_perm(sq[c][0], sq[c][1], 0x0073), __byte_perm(sq[c][2], sq[c][3], 0x0073), 0x5410);
      }
#pragma unroll
      for (int c = 0; c < kWsqCh; ++c) {
        // sparse part: the k masked places in position order
#pragma unroll
        for (int s = 0; s < B / 2; ++s) {
          if ((s & 3) == 0 && s >= k) break;  // (uniform: whole words of compact values are skipped at once)
          if (s < k) {
            uint32_t cur = mreg[c][0];
            int base = 0;
#pragma unroll
            for (int r = 1; r < NM; ++r)
              if (cur == 0u) {
                cur = mreg[c][r];
                base = 32 * r;
              }
            const int pl = base + __ffs((int)cur) - 1;
#pragma unroll
            for (int r = 0; r < NM; ++r)
              if (base == 32 * r) mreg[c][r] &= mreg[c][r] - 1u;
            const int v = (int)(hv[c][s >> 2] << (24 - 8 * (s & 3))) >> 24;
            const int8_t* xw = xb + (pl >> 3) * (8 * MT);
            const int rb = ((pl & 1) << 2) | ((pl & 7) >> 1);  // byte of the place inside its word
            if constexpr (MT == 1) {
              hi[c][0] += v * (int)xw[rb];
            } else {
              // both tokens of a 16-byte read; the byte is picked (and sign-extended) by a byte permute
              const uint32_t sel = (uint32_t)rb * 0x1111u + 0x8880u;
#pragma unroll
              for (int m2 = 0; m2 < MT / 2; ++m2) {
                const uint4 xv = *reinterpret_cast<const uint4*>(xw + 16 * m2);
                hi[c][2 * m2] += v * pick_s8(xv.x, xv.y, sel);
                hi[c][2 * m2 + 1] += v * pick_s8(xv.z, xv.w, sel);
              }
            }
          }
        }
      }
    }
#pragma unroll
    for (int c = 0; c < kWsqCh; ++c)
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        lo[c][m] = warp_sum(lo[c][m]);
        hi[c][m] = warp_sum(hi[c][m]);
      }
    if (lane == 0) {
#pragma unroll
      for (int c = 0; c < kWsqCh; ++c) {
        const int n = pr * kWsqCh + c;
        if (n < N) {
          const float sh = s_high[n], sl = s_low[n];
#pragma unroll
          for (int m = 0; m < MT; ++m)
            if (m < M) {
              const int a_lo = lo[c][m] >> 4;  // the dense codes were fed as 16 * code
              const float f = __fmul_rn(__fmaf_rn((float)hi[c][m], sh, __fmul_rn((float)a_lo, sl)), s_x[m]);
              out[(size_t)m * N + n] = (uint16_t)f32_to_bf16_bits(f);
              if (acc_out != nullptr) {
                acc_out[(size_t)m * N + n] = a_lo;
                acc_out[(size_t)M * N + (size_t)m * N + n] = hi[c][m];
              }
            }
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------

namespace {
template <typename KernelT>
cudaError_t ensure_smem(KernelT kernel, std::atomic<size_t>* limit, size_t smem) {
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (smem > limit[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(setup_mutex());
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    limit[dev].store(smem, std::memory_order_release);
  }
  return cudaSuccess;
}
}  // namespace

cudaError_t launch_wsq_encode(int b, int k, const uint16_t* W, const float* I, int64_t N, int64_t K, uint8_t* wq4,
                              int8_t* w_hi, float* s_high, float* s_low, cudaStream_t st) {
  const size_t smem = (size_t)K * 3;
  cudaError_t err;
#define SQ_WENC(BB)                                                                        \
  do {                                                                                     \
    static std::atomic<size_t> limit[64];                                                  \
    err = ensure_smem(sqw_encode_kernel<BB>, limit, smem);                                 \
    if (err != cudaSuccess) return err;                                                    \
    sqw_encode_kernel<BB><<<(unsigned)N, 256, smem, st>>>(k, W, I, K, wq4, w_hi, s_high, s_low); \
  } while (0)
  if (b == 32) SQ_WENC(32);
  else if (b == 64) SQ_WENC(64);
  else SQ_WENC(128);
#undef SQ_WENC
  return cudaGetLastError();
}

cudaError_t launch_wsq_act(const uint16_t* X, int64_t M, int64_t K, int8_t* xq, float* s_x, cudaStream_t st) {
  sqw_act_kernel<<<(unsigned)M, 256, 0, st>>>(X, K, xq, s_x);
  return cudaGetLastError();
}

cudaError_t launch_wsq_gemm(int b, int k, const int8_t* xq, const float* s_x, const uint8_t* wq4, const int8_t* w_hi,
                            const float* s_high, const float* s_low, int64_t M, int64_t N, int64_t K, uint16_t* out,
                            int32_t* acc_out, cudaStream_t st) {
  if (M < 1 || M > 4) return cudaErrorNotSupported;
  const int MT = M <= 1 ? 1 : (M <= 2 ? 2 : 4);
  const size_t smem = (size_t)MT * K + (size_t)(K / b) * (MT == 1 ? 8 : 16);
  if (smem > 200 * 1024) return cudaErrorNotSupported;
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  const int64_t pairs = (N + kWsqCh - 1) / kWsqCh;
  int64_t blocks = (pairs + kWsqWarps - 1) / kWsqWarps;
  if (blocks > 3 * (int64_t)sms) blocks = 3 * (int64_t)sms;
#define SQ_WGEMM(BB, MM)                                                                                           \
  do {                                                                                                             \
    static std::atomic<size_t> limit[64];                                                                          \
    err = ensure_smem(sqw_gemm_kernel<BB, MM>, limit, smem);                                                       \
    if (err != cudaSuccess) return err;                                                                            \
    sqw_gemm_kernel<BB, MM><<<(unsigned)blocks, kWsqWarps * 32, smem, st>>>(k, xq, s_x, wq4, w_hi, s_high, s_low,  \
                                                                          (int)M, (int)N, (int)K, out, acc_out);  \
  } while (0)
#define SQ_WGEMM_B(BB)             \
  do {                             \
    if (MT == 1) SQ_WGEMM(BB, 1);  \
    else if (MT == 2) SQ_WGEMM(BB, 2); \
    else SQ_WGEMM(BB, 4);          \
  } while (0)
  if (b == 32) SQ_WGEMM_B(32);
  else if (b == 64) SQ_WGEMM_B(64);
  else SQ_WGEMM_B(128);
#undef SQ_WGEMM_B
#undef SQ_WGEMM
  return cudaGetLastError();
}

}  // namespace sq
