// C ABI entry points: argument validation, then one launcher per call.
#include "sq_host.h"

namespace sq {

// Per-device status word.  A kernel that gives up on a bounded wait stores an
// sq_status here; sq_device_status() reads and clears it.
__device__ int g_status_word;

int* status_word() {
  // looked up once per device (the call is not free, and decode-sized launches are host-bound)
  static std::atomic<int*> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  const bool slot = dev >= 0 && dev < 64;
  if (slot) {
    int* hit = cached[dev].load(std::memory_order_acquire);
    if (hit != nullptr) return hit;
  }
  std::lock_guard<std::mutex> lock(setup_mutex());
  int* ptr = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_status_word) != cudaSuccess) return nullptr;
  if (slot) cached[dev].store(ptr, std::memory_order_release);
  return ptr;
}

namespace {

bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }
// Static positions (tied or independent scales) / the independent-scale variant of them.
bool is_static(const sq_format* fmt) { return fmt->pos_mode != SQ_POS_DYNAMIC; }
bool is_indep(const sq_format* fmt) { return fmt->pos_mode == SQ_POS_STATIC_INDEP; }

sq_status check_format(const sq_format* fmt) {
  if (fmt == nullptr) return SQ_ERR_NULL_POINTER;
  if (fmt->version != SQ_LAYOUT_VERSION) return SQ_ERR_INVALID_ARG;
  if (fmt->bank != 32 && fmt->bank != 64 && fmt->bank != 128) return SQ_ERR_INVALID_ARG;
  if (fmt->k < 1 || fmt->k > fmt->bank / 2) return SQ_ERR_INVALID_ARG;
  if (fmt->pos_mode != SQ_POS_DYNAMIC && fmt->pos_mode != SQ_POS_STATIC && fmt->pos_mode != SQ_POS_STATIC_INDEP)
    return SQ_ERR_INVALID_ARG;
  return SQ_OK;
}

sq_status check_k(int64_t K) {
  if (K <= 0 || K % 128 != 0) return SQ_ERR_INVALID_ARG;
  if (K > SQ_MAX_K) return SQ_ERR_UNSUPPORTED;
  return SQ_OK;
}

// The kernels are built for sm_100a only; refuse anything else before launching.
sq_status check_device() {
  static std::atomic<int> major_of[64];  // per device, asked once
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SQ_ERR_CUDA;
  const bool slot = dev >= 0 && dev < 64;
  if (slot) major = major_of[dev].load(std::memory_order_acquire);
  if (major == 0) {
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SQ_ERR_CUDA;
    if (slot) major_of[dev].store(major, std::memory_order_release);
  }
  return major == 10 ? SQ_OK : SQ_ERR_ARCH;
}

#define SQ_TRY(expr)                 \
  do {                               \
    const sq_status st_ = (expr);    \
    if (st_ != SQ_OK) return st_;    \
  } while (0)

sq_status check_encoded(const sq_format* fmt, const sq_encoded* A) {
  if (A == nullptr) return SQ_ERR_NULL_POINTER;
  if (!A->dq4 || !A->vals || !A->s_hi || !A->s_lo || !A->shift) return SQ_ERR_NULL_POINTER;
  if (fmt->pos_mode == SQ_POS_DYNAMIC && !A->idx) return SQ_ERR_NULL_POINTER;
  if (!aligned16(A->dq4) || !aligned16(A->vals) || !aligned16(A->s_hi) || !aligned16(A->s_lo) ||
      !aligned16(A->shift))
    return SQ_ERR_ALIGNMENT;
  if (fmt->pos_mode == SQ_POS_DYNAMIC && !aligned16(A->idx)) return SQ_ERR_ALIGNMENT;
  return SQ_OK;
}

sq_status check_weights(const sq_format* fmt, const sq_weights* W) {
  if (W == nullptr) return SQ_ERR_NULL_POINTER;
  if (!W->wq4 || !W->s_w || !W->colsum) return SQ_ERR_NULL_POINTER;
  if (is_static(fmt) && !W->w_sparse) return SQ_ERR_NULL_POINTER;
  if (!aligned16(W->wq4) || !aligned16(W->s_w) || !aligned16(W->colsum)) return SQ_ERR_ALIGNMENT;
  if (is_static(fmt) && !aligned16(W->w_sparse)) return SQ_ERR_ALIGNMENT;
  return SQ_OK;
}

sq_status check_positions(const sq_format* fmt, const uint8_t* positions) {
  if (is_static(fmt)) {
    if (positions == nullptr) return SQ_ERR_NULL_POINTER;
    if (!aligned16(positions)) return SQ_ERR_ALIGNMENT;
  } else if (positions != nullptr) {
    return SQ_ERR_INVALID_ARG;
  }
  return SQ_OK;
}

sq_status from_cuda(cudaError_t err) { return err == cudaSuccess ? SQ_OK : SQ_ERR_CUDA; }

// The GEMM kernels address the packed tensors with 32-bit byte offsets.
sq_status check_gemm_extent(const sq_format* fmt, int64_t M, int64_t N, int64_t K) {
  const int64_t lim = 1ll << 32;
  if (M * (K / 2) >= lim || N * (K / 2) >= lim || M * ((K / fmt->bank) * fmt->k) >= lim) return SQ_ERR_UNSUPPORTED;
  return SQ_OK;
}

}  // namespace
}  // namespace sq

using namespace sq;

extern "C" {

const char* sq_status_string(sq_status status) {
  switch (status) {
    case SQ_OK: return "ok";
    case SQ_ERR_INVALID_ARG: return "invalid argument";
    case SQ_ERR_UNSUPPORTED: return "unsupported size";
    case SQ_ERR_NULL_POINTER: return "null pointer";
    case SQ_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case SQ_ERR_ARCH: return "device is not sm_100";
    case SQ_ERR_CUDA: return "CUDA runtime error";
    case SQ_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

sq_status sq_encoded_sizes(const sq_format* fmt, int64_t M, int64_t K, size_t bytes_out[6]) {
  SQ_TRY(check_format(fmt));
  if (bytes_out == nullptr) return SQ_ERR_NULL_POINTER;
  if (M < 0) return SQ_ERR_INVALID_ARG;
  SQ_TRY(check_k(K));
  const size_t m = (size_t)M, gk = (size_t)(K / fmt->bank) * (size_t)fmt->k;
  bytes_out[0] = m * (size_t)(K / 2);
  bytes_out[1] = m * gk;
  bytes_out[2] = fmt->pos_mode == SQ_POS_DYNAMIC ? m * gk : 0;
  bytes_out[3] = m * sizeof(float);
  bytes_out[4] = m * sizeof(float);
  bytes_out[5] = m;
  return SQ_OK;
}

sq_status sq_weights_sizes(const sq_format* fmt, int64_t N, int64_t K, size_t bytes_out[4]) {
  SQ_TRY(check_format(fmt));
  if (bytes_out == nullptr) return SQ_ERR_NULL_POINTER;
  if (N < 0 || N % 8 != 0) return SQ_ERR_INVALID_ARG;
  SQ_TRY(check_k(K));
  const size_t n = (size_t)N, gk = (size_t)(K / fmt->bank) * (size_t)fmt->k;
  bytes_out[0] = n * (size_t)(K / 2);
  bytes_out[1] = n * sizeof(float);
  bytes_out[2] = n * sizeof(int32_t);
  bytes_out[3] = is_static(fmt) ? n * gk : 0;
  return SQ_OK;
}

sq_status sq_calib_positions(const sq_format* fmt, const void* calib_bf16, int64_t T, int64_t K,
                             const void* W_bf16, int64_t N, uint8_t* positions, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  if (!is_static(fmt)) return SQ_ERR_INVALID_ARG;
  SQ_TRY(check_k(K));
  if (T < 1 || (W_bf16 != nullptr && N < 1)) return SQ_ERR_INVALID_ARG;
  if (calib_bf16 == nullptr || positions == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(calib_bf16) || !aligned16(positions) || !aligned16(W_bf16)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_device());
  return from_cuda(launch_calib_positions(fmt->bank, fmt->k, static_cast<const uint16_t*>(calib_bf16), T, K,
                                          static_cast<const uint16_t*>(W_bf16), N, positions,
                                          static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_pack_weights(const sq_format* fmt, const void* W_bf16, int64_t N, int64_t K,
                          const uint8_t* positions, sq_weights* out, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (N < 0 || N % 8 != 0) return SQ_ERR_INVALID_ARG;
  if (N == 0) return SQ_OK;
  if (W_bf16 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(W_bf16)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_weights(fmt, out));
  SQ_TRY(check_device());
  sq_weights o = *out;
  if (!is_static(fmt)) o.w_sparse = nullptr;
  return from_cuda(launch_pack_weights(fmt->bank, fmt->k, static_cast<const uint16_t*>(W_bf16), N, K, positions, o,
                                       static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_encode(const sq_format* fmt, const void* X_bf16, int64_t M, int64_t K,
                    const uint8_t* positions, sq_encoded* out, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (M < 0) return SQ_ERR_INVALID_ARG;
  if (M == 0) return SQ_OK;  // nothing to do: pointers of an empty tensor may be NULL
  if (X_bf16 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(X_bf16)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, out));
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  return from_cuda(launch_encode(fmt->bank, fmt->k, is_static(fmt), is_indep(fmt),
                                 static_cast<const uint16_t*>(X_bf16), M, K, positions, *out, status,
                                 static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_encode_a8(const sq_format* fmt, const void* X_bf16, int64_t M, int64_t K,
                       const uint8_t* positions, sq_encoded* out, void* a8, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (is_indep(fmt)) return SQ_ERR_UNSUPPORTED;  // two accumulators: there is no merged operand
  if (M < 0) return SQ_ERR_INVALID_ARG;
  if (M == 0) return SQ_OK;
  if (X_bf16 == nullptr || a8 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(X_bf16) || !aligned16(a8)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, out));
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  bool written = false;
  cudaError_t err = launch_encode(fmt->bank, fmt->k, is_static(fmt), false, static_cast<const uint16_t*>(X_bf16), M, K,
                                  positions, *out, status, st, static_cast<uint8_t*>(a8), &written);
  if (err == cudaSuccess && !written)
    err = launch_expand_a8(fmt->bank, fmt->k, *out, is_static(fmt) ? positions : nullptr, M, K,
                           static_cast<uint8_t*>(a8), st);
  return from_cuda(err);
}

sq_status sq_rmsnorm_encode(const sq_format* fmt, const void* X_bf16, const void* gamma_bf16, float eps, int64_t M,
                            int64_t K, const uint8_t* positions, sq_encoded* out, void* a8, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (is_indep(fmt)) return SQ_ERR_UNSUPPORTED;
  if (M < 0 || !(eps >= 0.f)) return SQ_ERR_INVALID_ARG;
  if (M == 0) return SQ_OK;
  if (X_bf16 == nullptr || gamma_bf16 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(X_bf16) || !aligned16(gamma_bf16) || !aligned16(a8)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, out));
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t err = launch_rmsnorm_encode(fmt->bank, fmt->k, false, static_cast<const uint16_t*>(X_bf16),
                                          static_cast<const uint16_t*>(gamma_bf16), eps, M, K,
                                          is_static(fmt) ? positions : nullptr, *out, static_cast<uint8_t*>(a8), status, st);
  if (err == cudaErrorNotSupported) return SQ_ERR_UNSUPPORTED;
  // dynamic positions: the merged operand, if asked for, is expanded from the codes just written
  if (err == cudaSuccess && !is_static(fmt) && a8 != nullptr)
    err = launch_expand_a8(fmt->bank, fmt->k, *out, nullptr, M, K, static_cast<uint8_t*>(a8), st);
  return from_cuda(err);
}

sq_status sq_gemm_workspace_bytes(const sq_format* fmt, int64_t M, int64_t N, int64_t K, size_t* bytes) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (bytes == nullptr) return SQ_ERR_NULL_POINTER;
  if (M < 0 || N < 0 || N % 8 != 0 || M > INT32_MAX || N > INT32_MAX) return SQ_ERR_INVALID_ARG;
  *bytes = 0;
  if (M == 0 || N == 0) return SQ_OK;
  SQ_TRY(check_device());
  *bytes = gemm_workspace_bytes(fmt->bank, fmt->k, is_static(fmt), is_indep(fmt), M, N, K);
  return SQ_OK;
}

sq_status sq_gemm_ws(const sq_format* fmt, const sq_encoded* A, const sq_weights* W,
                     const uint8_t* positions, int64_t M, int64_t N, int64_t K, void* out_bf16,
                     int32_t* acc_out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (M < 0 || N < 0 || N % 8 != 0 || M > INT32_MAX || N > INT32_MAX) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, A));
  SQ_TRY(check_weights(fmt, W));
  if (out_bf16 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(out_bf16) || !aligned16(acc_out) || !aligned16(workspace)) return SQ_ERR_ALIGNMENT;
  if ((M + 127) / 128 > 65535) return SQ_ERR_UNSUPPORTED;
  SQ_TRY(check_gemm_extent(fmt, M, N, K));
  // independent scales: the sparse product runs as TMA-fed K steps of its own, whose row pitch
  // (G*k bytes) must be a multiple of 16
  if (is_indep(fmt) && ((K / fmt->bank) * fmt->k) % 16 != 0) return SQ_ERR_UNSUPPORTED;
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  return from_cuda(launch_gemm(fmt->bank, fmt->k, is_indep(fmt), *A, *W, positions, M, N, K,
                               static_cast<uint16_t*>(out_bf16), acc_out, status, workspace,
                               workspace == nullptr ? 0 : workspace_bytes, true, static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_gemm_a8(const sq_format* fmt, const sq_encoded* A, const sq_weights* W,
                     const uint8_t* positions, int64_t M, int64_t N, int64_t K, void* out_bf16,
                     int32_t* acc_out, const void* a8, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (is_indep(fmt)) return SQ_ERR_UNSUPPORTED;
  if (M < 0 || N < 0 || N % 8 != 0 || M > INT32_MAX || N > INT32_MAX) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, A));
  SQ_TRY(check_weights(fmt, W));
  if (out_bf16 == nullptr || a8 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(out_bf16) || !aligned16(acc_out) || !aligned16(a8)) return SQ_ERR_ALIGNMENT;
  if ((M + 127) / 128 > 65535) return SQ_ERR_UNSUPPORTED;
  SQ_TRY(check_gemm_extent(fmt, M, N, K));
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  return from_cuda(launch_gemm(fmt->bank, fmt->k, false, *A, *W, positions, M, N, K, static_cast<uint16_t*>(out_bf16),
                               acc_out, status, const_cast<void*>(a8), (size_t)M * (size_t)K, true,
                               static_cast<cudaStream_t>(cuda_stream), true));
}

sq_status sq_gemm_static_scratch(const sq_format* fmt, const sq_encoded* A, const sq_weights* W,
                                 const uint8_t* positions, int64_t M, int64_t N, int64_t K, void* out_bf16,
                                 int32_t* acc_out, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (M < 0 || N < 0 || N % 8 != 0 || M > INT32_MAX || N > INT32_MAX) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  // Only the few-row case has a use for scratch, and at least two parts of K must fit.
  if (M > 128 || is_indep(fmt)) return SQ_ERR_UNSUPPORTED;
  if ((uint64_t)2 * (uint64_t)M * (uint64_t)N * 4u > (uint64_t)gemm_static_scratch_bytes()) return SQ_ERR_UNSUPPORTED;
  SQ_TRY(check_gemm_extent(fmt, M, N, K));
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, A));
  SQ_TRY(check_weights(fmt, W));
  if (out_bf16 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(out_bf16) || !aligned16(acc_out)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  return from_cuda(launch_gemm_static_scratch(fmt->bank, fmt->k, *A, *W, positions, M, N, K,
                                              static_cast<uint16_t*>(out_bf16), acc_out, status,
                                              static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_gemm(const sq_format* fmt, const sq_encoded* A, const sq_weights* W,
                  const uint8_t* positions, int64_t M, int64_t N, int64_t K, void* out_bf16,
                  int32_t* acc_out, void* cuda_stream) {
  return sq_gemm_ws(fmt, A, W, positions, M, N, K, out_bf16, acc_out, nullptr, 0, cuda_stream);
}

sq_status sq_decode(const sq_format* fmt, const sq_encoded* A, const uint8_t* positions,
                    int64_t M, int64_t K, void* out_bf16, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (M < 0) return SQ_ERR_INVALID_ARG;
  if (M == 0) return SQ_OK;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, A));
  if (out_bf16 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(out_bf16)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_device());
  sq_encoded a = *A;
  if (is_static(fmt)) a.idx = nullptr;
  return from_cuda(launch_decode(fmt->bank, fmt->k, a, positions, M, K, static_cast<uint16_t*>(out_bf16),
                                 static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_fp_pack_weights(const void* W_bf16, int64_t N, int64_t K, uint8_t* wq4, float* s_w, uint8_t* w8,
                             void* cuda_stream) {
  SQ_TRY(check_k(K));
  if (N < 0 || N % 8 != 0) return SQ_ERR_INVALID_ARG;
  if (N == 0) return SQ_OK;
  if (!W_bf16 || !wq4 || !s_w || !w8) return SQ_ERR_NULL_POINTER;
  if (!aligned16(W_bf16) || !aligned16(wq4) || !aligned16(s_w) || !aligned16(w8)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_device());
  return from_cuda(launch_fp_pack_weights(static_cast<const uint16_t*>(W_bf16), N, K, wq4, s_w, w8,
                                          static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_fp_encode(const sq_format* fmt, const void* X_bf16, int64_t M, int64_t K, const uint8_t* positions,
                       sq_encoded* out, uint8_t* a8, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  if (is_indep(fmt)) return SQ_ERR_INVALID_ARG;
  SQ_TRY(check_k(K));
  if (M < 0) return SQ_ERR_INVALID_ARG;
  if (M == 0) return SQ_OK;
  if (X_bf16 == nullptr || a8 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(X_bf16) || !aligned16(a8)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, out));
  SQ_TRY(check_device());
  sq_encoded o = *out;
  if (is_static(fmt)) o.idx = nullptr;
  if (is_static(fmt)) {
    // static positions: rows streamed through shared-memory slots (bounded waits, hence the status word)
    int* status = status_word();
    if (status == nullptr) return SQ_ERR_CUDA;
    const cudaError_t err = launch_fp_encode_static_ring(fmt->bank, fmt->k, static_cast<const uint16_t*>(X_bf16), M, K,
                                                         positions, o, a8, status, static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaErrorNotSupported) return from_cuda(err);
  }
  if (!is_static(fmt)) {
    // dynamic positions at the integer path's fast ratios: its row-group kernel (selection by
    // sorting network) with this format's scales and roundings
    int* status = status_word();
    if (status == nullptr) return SQ_ERR_CUDA;
    const cudaError_t err = launch_fp_encode_dynamic_rows(fmt->bank, fmt->k, static_cast<const uint16_t*>(X_bf16), M, K, o, a8,
                                                          status, static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaErrorNotSupported) return from_cuda(err);
  }
  return from_cuda(launch_fp_encode(fmt->bank, fmt->k, static_cast<const uint16_t*>(X_bf16), M, K, positions, o, a8,
                                    static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_fp_rmsnorm_encode(const sq_format* fmt, const void* X_bf16, const void* gamma_bf16, float eps, int64_t M,
                               int64_t K, const uint8_t* positions, sq_encoded* out, uint8_t* a8, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (!is_static(fmt) || is_indep(fmt)) return SQ_ERR_UNSUPPORTED;
  if (M < 0 || !(eps >= 0.f)) return SQ_ERR_INVALID_ARG;
  if (M == 0) return SQ_OK;
  if (X_bf16 == nullptr || gamma_bf16 == nullptr || a8 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(X_bf16) || !aligned16(gamma_bf16) || !aligned16(a8)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, out));
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  sq_encoded o = *out;
  o.idx = nullptr;
  const cudaError_t err = launch_rmsnorm_encode(fmt->bank, fmt->k, true, static_cast<const uint16_t*>(X_bf16),
                                                static_cast<const uint16_t*>(gamma_bf16), eps, M, K, positions, o, a8,
                                                status, static_cast<cudaStream_t>(cuda_stream));
  return err == cudaErrorNotSupported ? SQ_ERR_UNSUPPORTED : from_cuda(err);
}

sq_status sq_fp_gemm(const float* s_hi, const uint8_t* a8, const float* s_w, const uint8_t* w8, int64_t M, int64_t N,
                     int64_t K, void* out_bf16, float* acc_out, void* cuda_stream) {
  SQ_TRY(check_k(K));
  if (M < 0 || N < 0 || N % 8 != 0 || M > INT32_MAX || N > INT32_MAX) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  if (!s_hi || !a8 || !s_w || !w8 || !out_bf16) return SQ_ERR_NULL_POINTER;
  if (!aligned16(a8) || !aligned16(w8) || !aligned16(out_bf16) || !aligned16(acc_out)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  return from_cuda(launch_fp_gemm(s_hi, a8, s_w, w8, M, N, K, static_cast<uint16_t*>(out_bf16), acc_out, status,
                                  static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_fp_decode(const sq_format* fmt, const sq_encoded* A, const uint8_t* positions, int64_t M, int64_t K,
                       void* out_bf16, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  if (is_indep(fmt)) return SQ_ERR_INVALID_ARG;
  SQ_TRY(check_k(K));
  if (M < 0) return SQ_ERR_INVALID_ARG;
  if (M == 0) return SQ_OK;
  SQ_TRY(check_positions(fmt, positions));
  SQ_TRY(check_encoded(fmt, A));
  if (out_bf16 == nullptr) return SQ_ERR_NULL_POINTER;
  if (!aligned16(out_bf16)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_device());
  sq_encoded a = *A;
  if (is_static(fmt)) a.idx = nullptr;
  return from_cuda(launch_fp_decode(fmt->bank, fmt->k, a, positions, M, K, static_cast<uint16_t*>(out_bf16),
                                    static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_w_encode(const sq_format* fmt, const void* W_bf16, const float* importance, int64_t N, int64_t K,
                      uint8_t* wq4, int8_t* w_hi, float* s_high, float* s_low, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (N < 0) return SQ_ERR_INVALID_ARG;
  if (N == 0) return SQ_OK;
  if (!W_bf16 || !importance || !wq4 || !w_hi || !s_high || !s_low) return SQ_ERR_NULL_POINTER;
  if (!aligned16(W_bf16) || !aligned16(importance) || !aligned16(wq4) || !aligned16(w_hi)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_device());
  return from_cuda(launch_wsq_encode(fmt->bank, fmt->k, static_cast<const uint16_t*>(W_bf16), importance, N, K, wq4,
                                     w_hi, s_high, s_low, static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_w_act_quant(const void* X_bf16, int64_t M, int64_t K, int8_t* xq, float* s_x, void* cuda_stream) {
  SQ_TRY(check_k(K));
  if (M < 0) return SQ_ERR_INVALID_ARG;
  if (M == 0) return SQ_OK;
  if (!X_bf16 || !xq || !s_x) return SQ_ERR_NULL_POINTER;
  if (!aligned16(X_bf16) || !aligned16(xq)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_device());
  return from_cuda(launch_wsq_act(static_cast<const uint16_t*>(X_bf16), M, K, xq, s_x,
                                  static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_w_gemm(const sq_format* fmt, const int8_t* xq, const float* s_x, const uint8_t* wq4, const int8_t* w_hi,
                    const float* s_high, const float* s_low, int64_t M, int64_t N, int64_t K, void* out_bf16,
                    int32_t* acc_out, void* cuda_stream) {
  SQ_TRY(check_format(fmt));
  SQ_TRY(check_k(K));
  if (M < 0 || N < 0 || N % 8 != 0 || N > INT32_MAX) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  if (M > 4) return SQ_ERR_UNSUPPORTED;
  if (!xq || !s_x || !wq4 || !w_hi || !s_high || !s_low || !out_bf16) return SQ_ERR_NULL_POINTER;
  if (!aligned16(xq) || !aligned16(wq4) || !aligned16(w_hi) || !aligned16(out_bf16)) return SQ_ERR_ALIGNMENT;
  SQ_TRY(check_device());
  const cudaError_t err = launch_wsq_gemm(fmt->bank, fmt->k, xq, s_x, wq4, w_hi, s_high, s_low, M, N, K,
                                          static_cast<uint16_t*>(out_bf16), acc_out, static_cast<cudaStream_t>(cuda_stream));
  return err == cudaErrorNotSupported ? SQ_ERR_UNSUPPORTED : from_cuda(err);
}

sq_status sq_device_status(void* cuda_stream) {
  SQ_TRY(check_device());
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return SQ_ERR_CUDA;
  int word = 0;
  if (cudaMemcpyFromSymbol(&word, g_status_word, sizeof(int)) != cudaSuccess) return SQ_ERR_CUDA;
  if (word != 0) {
    const int zero = 0;
    if (cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int)) != cudaSuccess) return SQ_ERR_CUDA;
    return static_cast<sq_status>(word);
  }
  return SQ_OK;
}


sq_status sq_probe_int8_tensor_rate(int iterations, double* int8_ops, void* cuda_stream) {
  if (iterations < 1 || iterations > (1 << 24)) return SQ_ERR_INVALID_ARG;
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  return from_cuda(launch_int8_peak_probe(iterations, int8_ops, status, static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_probe_fp8_tensor_rate(int iterations, double* fp8_ops, void* cuda_stream) {
  if (iterations < 1 || iterations > (1 << 24)) return SQ_ERR_INVALID_ARG;
  SQ_TRY(check_device());
  int* status = status_word();
  if (status == nullptr) return SQ_ERR_CUDA;
  return from_cuda(launch_fp8_peak_probe(iterations, fp8_ops, status, static_cast<cudaStream_t>(cuda_stream)));
}

sq_status sq_device_status_word(int** device_word) {
  if (device_word == nullptr) return SQ_ERR_NULL_POINTER;
  SQ_TRY(check_device());
  *device_word = status_word();
  return *device_word != nullptr ? SQ_OK : SQ_ERR_CUDA;
}

}  // extern "C"
