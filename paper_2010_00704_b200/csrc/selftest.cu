// Self-test of the bounded device-side waits (bcnn_selftest_wait_timeout): the same helpers the tcgen05 engines
// use - tensor-memory allocation, mbarrier waits with a poll limit and back-off, the CTA's abort flag, the device
// error word - in a kernel where one wait runs out by construction.  Nothing arrives on either barrier:
//   warp 1    waits on barrier 0 with the caller's small limit, gives up, raises the abort flag and records the code;
//   warps 2-3 wait on barrier 1 with the engines' full limit and leave as soon as they see the abort flag
//             (the path every other role of an engine takes after one of its waits has run out);
//   warp 0    allocates tensor memory before, and frees it after, the CTA-wide barrier all warps reach.
// The kernel ends normally; the host reads the code from the error word.
#include "tc_common.cuh"

namespace bcnn {

namespace {

using namespace tc;

__global__ void __launch_bounds__(128, 1) selftest_wait_timeout_kernel(int *err, uint32_t polls)
{
    __shared__ __align__(8) unsigned long long bars[2];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;
    const int warp = threadIdx.x >> 5;
    volatile int *abort_flag = &abort_flag_smem;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        abort_flag_smem = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(32u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;
    if (warp == 1) {
        mbar_wait_warp(smem_u32(&bars[0]), 0, abort_flag, err, BCNN_SELFTEST_TIMEOUT_CODE, polls);
    } else if (warp >= 2) {
        mbar_wait_warp(smem_u32(&bars[1]), 0, abort_flag, err, BCNN_SELFTEST_TIMEOUT_CODE + 1);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(32u) : "memory");
}

}  // namespace

int launch_selftest_wait_timeout(int polls, cudaStream_t stream)
{
    int *err = device_error_word();
    if (!err) return BCNN_ERR_CUDA;
    selftest_wait_timeout_kernel<<<1, 128, 0, stream>>>(err, (uint32_t)polls);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace bcnn
