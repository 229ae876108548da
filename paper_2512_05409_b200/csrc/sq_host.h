// Host-side launcher prototypes shared by the translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "../../include/sq.h"

namespace sq {

// Host-side state: per-device caches (device attributes, symbol addresses, kernel attributes
// already raised, occupancy answers) filled on first use.  Readers look at atomics; whoever finds
// an entry empty fills it under this one lock, so any number of host threads may call into the
// library at the same time.
inline std::mutex& setup_mutex() {
  static std::mutex m;
  return m;
}

// Device address of the per-device status word (0 = fine, else an sq_status).
int* status_word();

cudaError_t launch_calib_positions(int b, int k, const uint16_t* calib, int64_t T, int64_t K,
                                   const uint16_t* W, int64_t N, uint8_t* positions,
                                   cudaStream_t st);

cudaError_t launch_pack_weights(int b, int k, const uint16_t* W, int64_t N, int64_t K,
                                const uint8_t* positions, const sq_weights& out, cudaStream_t st);

cudaError_t launch_encode(int b, int k, bool is_static, bool indep, const uint16_t* X, int64_t M, int64_t K,
                          const uint8_t* positions, const sq_encoded& out, int* status, cudaStream_t st,
                          uint8_t* a8 = nullptr, bool* a8_written = nullptr);
// a8 != nullptr asks for the product's merged 8-bit operand [M, K] as well; *a8_written tells whether
// the encode kernel wrote it (static positions, tied scales, row lengths the register kernel takes).

cudaError_t launch_decode(int b, int k, const sq_encoded& A, const uint8_t* positions, int64_t M,
                          int64_t K, uint16_t* out, cudaStream_t st);

// allow_stream: few-token calls the weight-streaming kernel serves go to it (it needs no workspace).
cudaError_t launch_gemm(int b, int k, bool indep, const sq_encoded& A, const sq_weights& W,
                        const uint8_t* positions, int64_t M, int64_t N, int64_t K, uint16_t* out,
                        int32_t* acc_out, int* status, void* workspace, size_t workspace_bytes, bool allow_stream,
                        cudaStream_t st, bool a8_ready = false);
// a8_ready: `workspace` already holds the merged 8-bit operand of A (M*K bytes): it is read, never written.
// The merged operand alone: what launch_gemm writes into an M*K-byte workspace before its product.
cudaError_t launch_expand_a8(int b, int k, const sq_encoded& A, const uint8_t* positions, int64_t M, int64_t K,
                             uint8_t* a8, cudaStream_t st);
// Bytes of workspace launch_gemm can make use of for this shape and format (0: none).
size_t gemm_workspace_bytes(int b, int k, bool is_static, bool indep, int64_t M, int64_t N, int64_t K);
// The weight-streaming kernel for at most 32 token rows (sq_gemm_stream.cu).
bool gemm_stream_serves(int b, int k, bool is_static, int64_t M, int64_t N, int64_t K);
cudaError_t launch_gemm_stream(int b, int k, const sq_encoded& A, const sq_weights& W, const uint8_t* positions,
                               int64_t M, int64_t N, int64_t K, uint16_t* out, int32_t* acc_out, int* status,
                               cudaStream_t st);
// The same launch with the library's own fixed scratch array as the workspace (no allocation).
cudaError_t launch_gemm_static_scratch(int b, int k, const sq_encoded& A, const sq_weights& W,
                                       const uint8_t* positions, int64_t M, int64_t N, int64_t K, uint16_t* out,
                                       int32_t* acc_out, int* status, cudaStream_t st);
size_t gemm_static_scratch_bytes();
// Measurement aid: tcgen05.mma.kind::i8 on shared-memory-resident operands, nothing else (see sq.h).
cudaError_t launch_int8_peak_probe(int iters, double* ops, int* status, cudaStream_t st);
cudaError_t launch_fp8_peak_probe(int iters, double* ops, int* status, cudaStream_t st);

// Floating-point variant (sq_fp.cu).
cudaError_t launch_fp_pack_weights(const uint16_t* W, int64_t N, int64_t K, uint8_t* wq4, float* s_w, uint8_t* w8,
                                   cudaStream_t st);
cudaError_t launch_fp_encode(int b, int k, const uint16_t* X, int64_t M, int64_t K, const uint8_t* positions,
                             const sq_encoded& out, uint8_t* a8, cudaStream_t st);
cudaError_t launch_rmsnorm_encode(int b, int k, bool fp, const uint16_t* X, const uint16_t* gamma, float eps, int64_t M,
                                  int64_t K, const uint8_t* positions, const sq_encoded& out, uint8_t* a8, int* status,
                                  cudaStream_t st);
cudaError_t launch_fp_encode_static_ring(int b, int k, const uint16_t* X, int64_t M, int64_t K, const uint8_t* positions,
                                         const sq_encoded& out, uint8_t* a8, int* status, cudaStream_t st);
cudaError_t launch_fp_encode_dynamic_rows(int b, int k, const uint16_t* X, int64_t M, int64_t K, const sq_encoded& out,
                                          uint8_t* a8, int* status, cudaStream_t st);
cudaError_t launch_fp_decode(int b, int k, const sq_encoded& A, const uint8_t* positions, int64_t M, int64_t K,
                             uint16_t* out, cudaStream_t st);
cudaError_t launch_fp_gemm(const float* s_hi, const uint8_t* a8, const float* s_w, const uint8_t* w8, int64_t M, int64_t N,
                           int64_t K, uint16_t* out, float* acc_out, int* status, cudaStream_t st);

// SQ-format on weights (sq_wsq.cu).
cudaError_t launch_wsq_encode(int b, int k, const uint16_t* W, const float* I, int64_t N, int64_t K, uint8_t* wq4,
                              int8_t* w_hi, float* s_high, float* s_low, cudaStream_t st);
cudaError_t launch_wsq_act(const uint16_t* X, int64_t M, int64_t K, int8_t* xq, float* s_x, cudaStream_t st);
cudaError_t launch_wsq_gemm(int b, int k, const int8_t* xq, const float* s_x, const uint8_t* wq4, const int8_t* w_hi,
                            const float* s_high, const float* s_low, int64_t M, int64_t N, int64_t K, uint16_t* out,
                            int32_t* acc_out, cudaStream_t st);

}  // namespace sq
