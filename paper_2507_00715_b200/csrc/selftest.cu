// Self-test of the failure path of the tensor-core kernels: a wait on an mbarrier that nothing ever completes.
// The wait is the same bounded wait the prefill kernel uses; here its limit is short and chosen by the caller.
// When it runs out the kernel records EARN_ERR_TIMEOUT in the workspace status word and returns normally, so the
// context stays usable -- which is what the test of this entry point checks.
#include "earn_common.cuh"
#include "sm100_ptx.cuh"

namespace earn {
namespace {

__global__ void __launch_bounds__(64) wait_timeout_kernel(int32_t* status, long long limit_cycles) {
  __shared__ __align__(8) unsigned long long barrier;
  __shared__ int abort_flag;
  const uint32_t bar = ptx::smem_u32(&barrier);
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar, 1);   // one arrival expected; none will come
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const bool done = ptx::mbar_wait_bounded(bar, 0, &abort_flag, limit_cycles);
  __syncthreads();
  if (threadIdx.x == 0 && (!done || abort_flag)) atomicExch(status, (int32_t)EARN_ERR_TIMEOUT);
}

}  // namespace
}  // namespace earn

extern "C" earn_status_t earn_selftest_wait_timeout(void* workspace, size_t workspace_bytes, int64_t limit_cycles,
                                                    earn_stream_t stream) {
  using namespace earn;
  if (workspace == nullptr || workspace_bytes < (size_t)kStatusBytes || (reinterpret_cast<uintptr_t>(workspace) & 15u))
    return EARN_ERR_WORKSPACE;
  if (limit_cycles < 1 || limit_cycles > 2000000000LL) return EARN_ERR_INVALID_ARG;   // at most about a second
  wait_timeout_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(reinterpret_cast<int32_t*>(workspace), (long long)limit_cycles);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}
