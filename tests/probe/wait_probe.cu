// TEST-ONLY kernel (never part of libsq_b200.so): makes the library's bounded device-side waits
// run out, the allowed way.  One block initialises an mbarrier that nobody ever completes and
// calls each wait helper of sq_device.cuh with a poll limit of a few hundred to a thousand; every
// helper must give up, raise the abort flag and return false, and the kernel then records
// SQ_ERR_TIMEOUT in the status word exactly as the product kernels do at their end.  Nothing here
// waits without a bound, traps or touches tensor memory.
#include "../../paper_2512_05409_b200/csrc/sq_device.cuh"

namespace {

// report[0..3]: 1 if mbar_wait / mbar_wait_park / mbar_wait_idle / mbar_wait_cluster returned false
// report[4..7]: the abort flag after each of them (cleared in between)
// report[8]:    1 if a wait on a barrier whose phase HAS completed returned true
// report[9]:    1 if a second waiter was released by the abort flag (before its own limit)
__global__ void expire_waits_kernel(int* status, int* report) {
  __shared__ __align__(8) uint64_t bar_never, bar_done;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;
  const uint32_t never = sq::smem_u32(&bar_never), done = sq::smem_u32(&bar_done);
  if (threadIdx.x == 0) {
    sq::mbar_init(never, 1);
    sq::mbar_init(done, 1);
    sq::fence_mbar_init();
    abort_s = 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    sq::mbar_arrive(done);  // phase 0 of `done` completes; `never` stays in phase 0 for good
    report[8] = sq::mbar_wait<1024>(done, 0, abort_flag) ? 1 : 0;
    report[0] = sq::mbar_wait<1024>(never, 0, abort_flag) ? 0 : 1;
    report[4] = abort_s;
    abort_s = 0;
    report[1] = sq::mbar_wait_park<8>(never, 0, abort_flag) ? 0 : 1;
    report[5] = abort_s;
    abort_s = 0;
    report[2] = sq::mbar_wait_idle<256>(never, 0, abort_flag) ? 0 : 1;
    report[6] = abort_s;
    abort_s = 0;
    report[3] = sq::mbar_wait_cluster<1024>(never, 0, abort_flag) ? 0 : 1;
    report[7] = abort_s;  // left raised: releases the second waiter below
  }
  if (threadIdx.x == 32) {
    // a role that waits with the product's (long) limit is released by another role's failure
    const long long t0 = clock64();
    const bool ok = sq::mbar_wait_idle(never, 0, abort_flag);
    report[9] = (!ok && clock64() - t0 < (1ll << 31)) ? 1 : 0;
  }
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, (int)SQ_ERR_TIMEOUT);
}

}  // namespace

// status_word: device pointer (sq_device_status_word); report: device int[10]; stream: cudaStream_t.
extern "C" int sqt_expire_waits(int* status_word, int* report, void* stream) {
  expire_waits_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(status_word, report);
  return (int)cudaGetLastError();
}
