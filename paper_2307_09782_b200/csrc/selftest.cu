// zq_selftest_bounded_wait: makes one of the library's bounded waits run out on purpose, safely.
//
// Every wait inside the kernels of this library (on an mbarrier, on a hand-over flag) has a limit; when it
// runs out the kernel records ZQ_ERR_DEVICE_TIMEOUT in the workspace status words and returns by itself, so
// that the context stays usable.  That path cannot be reached with valid inputs.  This entry point launches
// one CTA that initializes an mbarrier nobody will ever arrive at and waits on it with the same wait routine
// and a short limit: the wait gives up, the kernel reports exactly as the GEMM kernels do, and exits.
// Nothing faults, traps or keeps spinning.
#include "zq_common.cuh"

namespace zq {
namespace {

__global__ void bounded_wait_selftest_kernel(int* status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) {
    ok = mbar_wait(&bar, 0, &abort_flag, limit_ns);  // phase 0 never completes: there is no arrival
    if (!ok && atomicCAS(status, 0, ZQ_ERR_DEVICE_TIMEOUT) == 0) status[1] = kErrDetailSelfTest;
  }
  __syncthreads();
}

}  // namespace
}  // namespace zq

extern "C" int zq_selftest_bounded_wait(void* workspace, size_t workspace_bytes, uint32_t limit_us, void* stream) {
  using namespace zq;
  if (!workspace) return ZQ_ERR_NULL;
  if (workspace_bytes < kWsHeadBytes) return ZQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return ZQ_ERR_ALIGN;
  if (limit_us == 0 || limit_us > 1000000u) return ZQ_ERR_SHAPE;
  if (int e = check_device_sm100()) return e;
  bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<int*>(workspace), static_cast<uint64_t>(limit_us) * 1000ull);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? ZQ_OK : ZQ_ERR_CUDA;
}
