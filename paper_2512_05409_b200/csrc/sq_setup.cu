// Setup kernels: static position selection (Algorithm 2) and INT4 weight packing.
// Neither is on the timed path; both are written to reproduce the definition's
// arithmetic bit for bit (sequential fp64 sums, single-rounding quantisation).
#include "sq_device.cuh"
#include "sq_host.h"

namespace sq {

// One thread per input channel j; a block covers 128 channels = 128/b whole banks.
//   Abar_j = (sum_t |calib[t,j]|)/T, r_j = sum_n W[n,j] (1 without W), I_j = |Abar_j * r_j|,
// both sums sequential in fp64 so the result does not depend on the launch shape.
// Then every channel ranks itself inside its bank (larger I first, ties to the smaller
// index) and the k winners write their bank-local index in ascending order.
__global__ void __launch_bounds__(128) calib_positions_kernel(int b, int k, const uint16_t* __restrict__ calib,
                                                              int64_t T, int64_t K,
                                                              const uint16_t* __restrict__ W, int64_t N,
                                                              uint8_t* __restrict__ positions) {
  __shared__ double sI[128];
  __shared__ unsigned char sSel[128];
  const int tid = threadIdx.x;
  const int64_t j = (int64_t)blockIdx.x * 128 + tid;

  double sum = 0.0;
  for (int64_t t = 0; t < T; ++t) sum += fabs((double)bf16_bits_to_f32(calib[t * K + j]));
  const double abar = sum / (double)T;
  double r = 1.0;
  if (W != nullptr) {
    r = 0.0;
    for (int64_t n = 0; n < N; ++n) r += (double)bf16_bits_to_f32(W[n * K + j]);
  }
  const double I = fabs(abar * r);
  sI[tid] = I;
  __syncthreads();

  const int local = tid % b;
  const int base = tid - local;
  int rank = 0;
  for (int i = 0; i < b; ++i) {
    const double o = sI[base + i];
    rank += (o > I || (o == I && i < local)) ? 1 : 0;
  }
  const bool sel = rank < k;
  sSel[tid] = sel ? 1 : 0;
  __syncthreads();
  if (sel) {
    int slot = 0;
    for (int i = 0; i < local; ++i) slot += sSel[base + i];
    positions[(j / b) * k + slot] = (uint8_t)local;
  }
}

// One block per output channel n.  Pass 1: channel maximum (bf16 magnitudes order like
// their bit patterns).  Pass 2: codes = clamp(RNE(w * 7/wmax), -7, 7), eight per thread
// packed into one 32-bit word (element 2i low nibble, 2i+1 high nibble), channel sum,
// and for static formats the gathered codes of the selected input channels.
__global__ void __launch_bounds__(256) pack_weights_kernel(int b, int k, const uint16_t* __restrict__ W, int64_t K,
                                                           const uint8_t* __restrict__ positions,
                                                           uint8_t* __restrict__ wq4, float* __restrict__ s_w,
                                                           int32_t* __restrict__ colsum,
                                                           int8_t* __restrict__ w_sparse) {
  __shared__ uint32_t sMax[8];
  __shared__ int sSum[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t n = blockIdx.x;
  const uint16_t* row = W + n * K;

  uint32_t mx = 0;
  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(row + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      mx = max(mx, w[q] & 0x7FFFu);
      mx = max(mx, (w[q] >> 16) & 0x7FFFu);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) sMax[warp] = mx;
  __syncthreads();
  mx = 0;
#pragma unroll
  for (int q = 0; q < 8; ++q) mx = max(mx, sMax[q]);
  const float wmax = bf16_bits_to_f32(mx);
  const float c = wmax > 0.f ? __fdiv_rn(7.0f, wmax) : 0.f;

  int sum = 0;
  for (int64_t i = (int64_t)tid * 8; i < K; i += 256 * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(row + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t word = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      int q0 = rne_prod(bf16_bits_to_f32(w[q] & 0xFFFFu), c);
      int q1 = rne_prod(bf16_bits_to_f32(w[q] >> 16), c);
      q0 = min(7, max(-7, q0));
      q1 = min(7, max(-7, q1));
      sum += q0 + q1;
      word |= (uint32_t)(q0 & 0xF) << (8 * q);
      word |= (uint32_t)(q1 & 0xF) << (8 * q + 4);
    }
    *reinterpret_cast<uint32_t*>(wq4 + n * (K / 2) + i / 2) = word;
  }
  sum = warp_sum(sum);
  if (lane == 0) sSum[warp] = sum;
  __syncthreads();
  if (tid == 0) {
    int s = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) s += sSum[q];
    colsum[n] = s;
    s_w[n] = wmax > 0.f ? __fdiv_rn(wmax, 7.0f) : 0.f;
  }
  if (positions != nullptr) {
    const int64_t GK = (K / b) * k;
    for (int64_t t = tid; t < GK; t += 256) {
      const int64_t g = t / k;
      const int64_t j = g * b + positions[t];
      const int q = min(7, max(-7, rne_prod(bf16_bits_to_f32(row[j]), c)));
      w_sparse[n * GK + t] = (int8_t)(16 * q);  // sixteenths: the GEMM's weight operand unit
    }
  }
}

cudaError_t launch_calib_positions(int b, int k, const uint16_t* calib, int64_t T, int64_t K,
                                   const uint16_t* W, int64_t N, uint8_t* positions,
                                   cudaStream_t st) {
  calib_positions_kernel<<<(unsigned)(K / 128), 128, 0, st>>>(b, k, calib, T, K, W, N, positions);
  return cudaGetLastError();
}

cudaError_t launch_pack_weights(int b, int k, const uint16_t* W, int64_t N, int64_t K,
                                const uint8_t* positions, const sq_weights& out, cudaStream_t st) {
  pack_weights_kernel<<<(unsigned)N, 256, 0, st>>>(b, k, W, K, positions, out.wq4, out.s_w, out.colsum,
                                                   out.w_sparse);
  return cudaGetLastError();
}

}  // namespace sq
