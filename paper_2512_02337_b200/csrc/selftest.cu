// Self-test kernels (see include/specpv_selftest.h): the give-up path of the bounded barrier wait.
#include "../../include/specpv_selftest.h"
#include "tc_common.cuh"

namespace specpv {
namespace {

using namespace tc;

// One CTA: allocate tensor memory as the product kernels do, wait on a barrier nobody arrives on, give up after the
// limit, then go through the product kernels' teardown (abort flag seen, tensor memory freed).
__global__ void __launch_bounds__(64) wait_timeout_kernel(void* workspace, unsigned long long limit_ns, unsigned long long* observed_ns) {
    __shared__ uint64_t never;
    __shared__ uint32_t tmem_base;
    __shared__ int abort_flag_storage;
    volatile int* abort_flag = &abort_flag_storage;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&never), 1);
        abort_flag_storage = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 32;" ::"r"(smem_u32(&tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) {
        const uint64_t t0 = global_ns();
        const bool ok = mbar_wait(smem_u32(&never), 0, abort_flag, workspace, SPECPV_SELFTEST_WHERE, limit_ns);
        if (lane == 0 && observed_ns) *observed_ns = ok ? 0ull : (unsigned long long)(global_ns() - t0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 32;" ::"r"(tmem_base) : "memory");
    }
}

}  // namespace
}  // namespace specpv

extern "C" __attribute__((visibility("default"))) specpv_status specpv_selftest_wait_timeout(
    void* workspace, size_t workspace_bytes, int limit_us, unsigned long long* observed_ns, void* stream) {
    using namespace specpv;
    if (!workspace || workspace_bytes < kHeaderBytes || limit_us < 1 || limit_us > 1000000) return SPECPV_ERR_INVALID_ARG;
    wait_timeout_kernel<<<1, 64, 0, reinterpret_cast<cudaStream_t>(stream)>>>(workspace, (unsigned long long)limit_us * 1000ull,
                                                                             observed_ns);
    if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
    count_launch();
    return SPECPV_OK;
}
