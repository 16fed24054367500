// Instruction-throughput probes of the inner-product choices on sm_100a, used by bench.py for the roofline
// denominators.  No global-memory traffic inside the timed kernels:
//   * mma.sync .b1 (and.popc / xor.popc), mma.sync .s8 m16n8k32 and CUDA-core xor + popc: register-resident;
//   * tcgen05.mma kind::i8: A operand resident in tensor memory, B in shared memory, int32 accumulators in tensor
//     memory; one thread per SM issues M = 128, K = 32 instructions of width N back to back (N = 256 runs at the
//     pipe's rate, narrower instructions show the issue-bound regime).
// Built on demand into bench_probes.so (nvcc -shared, sm_100a) and called through ctypes; every function runs its
// kernel three times and writes the best time in milliseconds.
#include <cstdint>
#include <cuda_runtime.h>
#include "tc_common.cuh"

using namespace bcnn::tc;

namespace {

template <int MODE>
__global__ void __launch_bounds__(256) k_mma_sync(int iters, int *out, uint32_t seed)
{
    uint32_t a[4] = {seed + threadIdx.x, seed * 3 + threadIdx.x, seed * 5, seed * 7}, b0 = seed * 11 + threadIdx.x, b1 = seed * 13;
    int d[8][4];
#pragma unroll
    for (int i = 0; i < 8; i++)
        for (int j = 0; j < 4; j++) d[i][j] = 0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 8; i++) {
            if (MODE == 0)
                asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                             : "+r"(d[i][0]), "+r"(d[i][1]), "+r"(d[i][2]), "+r"(d[i][3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
            else if (MODE == 1)
                asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                             : "+r"(d[i][0]), "+r"(d[i][1]), "+r"(d[i][2]), "+r"(d[i][3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
            else
                asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                             : "+r"(d[i][0]), "+r"(d[i][1]), "+r"(d[i][2]), "+r"(d[i][3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
        }
    }
    int s = 0;
#pragma unroll
    for (int i = 0; i < 8; i++)
        for (int j = 0; j < 4; j++) s += d[i][j];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

__global__ void __launch_bounds__(256) k_popc(int iters, int *out, uint32_t seed)
{
    uint32_t a[4] = {seed + threadIdx.x, seed * 3 + threadIdx.x, seed * 5 + blockIdx.x, seed * 7};
    uint32_t w[4] = {seed * 11 + threadIdx.x, seed * 13, seed * 17, seed * 19 + threadIdx.x};
    int acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; i++)
        for (int j = 0; j < 4; j++) acc[i][j] = 0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 4; i++)
#pragma unroll
            for (int j = 0; j < 4; j++) acc[i][j] += __popc(a[i] ^ w[j]);
#pragma unroll
        for (int i = 0; i < 4; i++) a[i] = a[i] * 1664525u + 1013904223u;
    }
    int s = 0;
#pragma unroll
    for (int i = 0; i < 4; i++)
        for (int j = 0; j < 4; j++) s += acc[i][j];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

// One CTA per SM (the shared-memory request keeps a second one out).  Thread 0 of warp 0 issues `iters` groups of
// four MMAs (128 bits of K) into one accumulator, A from tensor memory, then one commit; warp 1 waits for it with
// the library's bounded wait.  The operands' contents do not matter (the weight tile is zeroed, the activation
// columns are whatever tensor memory holds): integer MMAs take the same time on any data.
template <int N>
__global__ void __launch_bounds__(128, 1) k_tcgen05_i8(int iters, int *err)
{
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;
    const int warp = threadIdx.x >> 5;
    const uint32_t wtile = (smem_u32(smem_raw) + 1023u) & ~1023u;          // [N rows][128 B], K-major, 128-byte swizzle
    for (int i = threadIdx.x; i < N * ROWB / 16; i += 128) st_shared_v4(wtile + 16u * i, 0u, 0u, 0u, 0u);
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag_smem = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_async_proxy();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;
    if (warp == 0) {
        constexpr uint32_t idesc = make_idesc(N);
        const uint64_t desc0 = make_desc(wtile);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32), b_lo = (uint32_t)desc0;
        const uint32_t a_t = tmem_base + 256u;                              // 32 columns of A behind the accumulator
        if (elect_one()) {
            for (int it = 0; it < iters; ++it) {
                tc_mma_i8_ts(tmem_base, a_t, b_lo, desc_hi, idesc, 1u);
                tc_mma_i8_ts(tmem_base, a_t + 8u, b_lo + 2u, desc_hi, idesc, 1u);
                tc_mma_i8_ts(tmem_base, a_t + 16u, b_lo + 4u, desc_hi, idesc, 1u);
                tc_mma_i8_ts(tmem_base, a_t + 24u, b_lo + 6u, desc_hi, idesc, 1u);
            }
            tc_commit(smem_u32(&bar));
        }
        __syncwarp();
    } else if (warp == 1) {
        mbar_wait_warp(smem_u32(&bar), 0, &abort_flag_smem, err, 130);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

template <typename F>
int best_of_three(F launch, double *ms_out)
{
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return -4;
    float best = 1e30f;
    for (int rep = 0; rep < 3; ++rep) {
        cudaEventRecord(e0);
        launch();
        cudaEventRecord(e1);
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaGetLastError() != cudaSuccess) return -4;
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (ms < best) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *ms_out = best;
    return 0;
}

int sm_count()
{
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

}  // namespace

extern "C" {

// mode 0: mma.sync b1 and.popc (K = 256), 1: b1 xor.popc, 2: s8 (K = 32).  *macs = multiply-accumulates per run.
int probe_mma_sync(int mode, int iters, double *ms, double *macs)
{
    if (mode < 0 || mode > 2 || iters <= 0 || !ms || !macs) return -1;
    const int sms = sm_count(), blocks = sms * 4;
    int *out = nullptr;
    if (cudaMalloc(&out, (size_t)blocks * 256 * 4) != cudaSuccess) return -4;
    const int st = best_of_three([&] {
        if (mode == 0) k_mma_sync<0><<<blocks, 256>>>(iters, out, 12345u);
        else if (mode == 1) k_mma_sync<1><<<blocks, 256>>>(iters, out, 12345u);
        else k_mma_sync<2><<<blocks, 256>>>(iters, out, 12345u);
    }, ms);
    cudaFree(out);
    *macs = (double)blocks * 8 * iters * 8 * 16 * 8 * (mode < 2 ? 256.0 : 32.0);
    return st;
}

int probe_popc(int iters, double *ms, double *macs)
{
    if (iters <= 0 || !ms || !macs) return -1;
    const int sms = sm_count(), blocks = sms * 8;
    int *out = nullptr;
    if (cudaMalloc(&out, (size_t)blocks * 256 * 4) != cudaSuccess) return -4;
    const int st = best_of_three([&] { k_popc<<<blocks, 256>>>(iters, out, 999u); }, ms);
    cudaFree(out);
    *macs = (double)blocks * 256 * iters * 16 * 32;
    return st;
}

// n in {32, 64, 128, 256}: width of the instruction.  *dev_err receives the error word of the bounded wait (0 = fine).
int probe_tcgen05_i8(int n, int iters, double *ms, double *macs, int *dev_err)
{
    if (iters <= 0 || !ms || !macs || !dev_err) return -1;
    if (n != 32 && n != 64 && n != 128 && n != 256) return -1;
    const int sms = sm_count();
    int *err = nullptr;
    if (cudaMalloc(&err, 4) != cudaSuccess) return -4;
    cudaMemset(err, 0, 4);
    const int smem = 160 * 1024;                  // more than half an SM: one CTA per SM
    void (*k)(int, int *) = n == 32 ? k_tcgen05_i8<32> : (n == 64 ? k_tcgen05_i8<64> : (n == 128 ? k_tcgen05_i8<128> : k_tcgen05_i8<256>));
    int st = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) == cudaSuccess ? 0 : -4;
    if (st == 0) st = best_of_three([&] { k<<<sms, 128, smem>>>(iters, err); }, ms);
    *dev_err = 0;
    if (st == 0 && cudaMemcpy(dev_err, err, 4, cudaMemcpyDeviceToHost) != cudaSuccess) st = -4;
    cudaFree(err);
    *macs = (double)sms * iters * 4.0 * 128.0 * n * 32.0;
    return st;
}

}  // extern "C"
