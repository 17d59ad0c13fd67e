// Test hook for the time-out path of the kernels' bounded waits (see mate_debug_expire_wait in mate.h).
#include "mate_internal.h"
#include "sm100_ptx.cuh"

namespace mate {
namespace {

// One thread waits, with the same bounded helper the attention kernels use and a limit of a few
// tries, for a phase of a barrier on which nothing ever arrives; when the wait gives up it raises
// the plan's time-out word, exactly as the kernels do, and the kernel returns.
__global__ void expire_wait_kernel(int32_t *status) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = ptx::smem_u32(&bar);
    ptx::mbar_init(b, 1);
    ptx::fence_mbar_init();
    if (!ptx::mbar_wait_bounded(b, 0, 4)) atomicOr(status + 1, 1);
}

}  // namespace
}  // namespace mate

extern "C" int mate_debug_expire_wait(const mate_plan_t *plan, void *stream) {
    if (!plan) return MATE_ERR_INVALID_ARG;
    mate::expire_wait_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(plan->status_dev);
    return cudaGetLastError() == cudaSuccess ? MATE_OK : MATE_ERR_CUDA;
}
