// Self-test of the bounded waits: a one-warp kernel that waits on something nothing will ever signal,
// with a short limit, so that the expiry path (status word, abort flag, orderly return) can be exercised
// without any copy, MMA or tensor-memory allocation in flight and without disturbing the device.
#include "gemm_epilogue.cuh"

namespace lazy {

namespace {

__device__ unsigned g_never_signalled;  // stays zero for the life of the process

__global__ void wait_selftest_kernel(int which, unsigned long long limit_ns, DevStatus *status) {
  __shared__ unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (which == 0) {
    // phase 0 of a barrier that expects one arrival and gets none
    if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0u, &abort_flag, status, W_WAIT_SELFTEST, limit_ns);
  } else {
    // the arrival-counter wait of the split last wave, on a counter that stays at zero
    gemm_tail_wait(&g_never_signalled, 1u, &abort_flag, status, limit_ns);
  }
}

}  // namespace

}  // namespace lazy

extern "C" int lazy_k_wait_selftest(void *stream, int32_t which, uint32_t limit_us) {
  using namespace lazy;
  if ((which != 0 && which != 1) || limit_us < 1 || limit_us > 100000) return LAZY_E_BADARG;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(which, (unsigned long long)limit_us * 1000ull, status);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

extern "C" int lazy_status_detail(int32_t *where, int32_t *a, int32_t *b) {
  int w = 0, x = 0, y = 0;
  lazy::last_status_detail(&w, &x, &y);
  if (where) *where = w;
  if (a) *a = x;
  if (b) *b = y;
  return LAZY_OK;
}
