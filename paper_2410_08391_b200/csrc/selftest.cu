// Self-test of the bounded device-side wait that every kernel of the library uses: a one-block kernel waits on a
// barrier that nothing will ever complete, with a limit of a few thousand polls.  The wait must run out, the kernel
// must return, and the status word must read DEV_TIMEOUT, which kvp_poll_status reports as KVP_ERR_TIMEOUT.
#include "kvp_internal.h"
#include "tc_ptx.cuh"

namespace {
using namespace tcp;

__global__ void __launch_bounds__(64) wait_timeout_kernel(int* status, uint32_t limit) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_mem;
  volatile int* abort_flag = &abort_mem;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // thread 0 plays a consumer whose producer never arrives; thread 32 a second role that watches the abort flag
  if (threadIdx.x == 0 || threadIdx.x == 32) mbar_wait(smem_u32(&bar), 0, abort_flag, status, limit);
  __syncthreads();
}
}  // namespace

extern "C" kvp_status kvp_selftest_wait_timeout(kvp_handle* h, void* workspace, void* stream) {
  if (!h || !workspace) return KVP_ERR_INVALID_ARG;
  h->err.clear();
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != h->device) {
    cudaGetLastError();
    h->err = "current device is not the handle's device";
    return KVP_ERR_INVALID_ARG;
  }
  ++h->n_launch;
  wait_timeout_kernel<<<1, 64, 0, (cudaStream_t)stream>>>((int*)workspace, 4096u);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    h->err = std::string("kvp_selftest_wait_timeout: ") + cudaGetErrorString(e);
    return KVP_ERR_CUDA;
  }
  return KVP_OK;
}
