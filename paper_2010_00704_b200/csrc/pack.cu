// Binarize + pack kernel: real NHWC fp32 -> sign bits (bit 1 = +1), with optional
// per-channel bias and channel replication (paper Section 4.2.1 bias + sign, Section
// 4.2.2 replication by bookkeeping).  A pure HBM stream: 4 bytes read per input value,
// 1 bit written per output channel.
#include "bcnn_common.cuh"

namespace bcnn {

// Streaming path, no replication, C_in % 32 == 0: the tensor is a flat array of
// fp32 values and every aligned group of 32 values becomes one output word.  Lane l of
// a warp reads value l of a group (one coalesced 128-byte request per group) and the
// warp vote assembles the word, bit l = lane l = channel l of the group (LSB first).
// UNROLL groups are in flight per warp to cover HBM latency.
template <int UNROLL, bool HAS_BIAS>
__global__ void __launch_bounds__(256)
pack_stream_kernel(const float *__restrict__ x, const float *__restrict__ bias,
                   uint32_t *__restrict__ out, long nwords, int cwords)
{
    const int lane = threadIdx.x & 31;
    const long warp = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long nwarps = (long)gridDim.x * (blockDim.x >> 5);
    for (long w0 = warp * UNROLL; w0 < nwords; w0 += nwarps * UNROLL) {
        float v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long wi = w0 + u;
            v[u] = (wi < nwords) ? __ldcs(x + wi * 32 + lane) : -1.0f;
        }
        uint32_t word[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            float s = v[u];
            if (HAS_BIAS) {
                const long wi = w0 + u;
                const int cword = (int)(wi % cwords);
                s = __fadd_rn(s, __ldg(bias + cword * 32 + lane));
            }
            word[u] = __ballot_sync(0xffffffffu, s >= 0.0f);
        }
        // lane u stores word u: one contiguous UNROLL*4-byte segment per warp
        uint32_t mine = 0;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (lane == u) mine = word[u];
        if (lane < UNROLL && w0 + lane < nwords) out[w0 + lane] = mine;
    }
}

// General path: any C_in and replication factor R with R*C_in % 32 == 0.  One warp
// per output word; lane l evaluates channel c = 32*word + l, which reads input channel
// c mod C_in of the same pixel.
__global__ void __launch_bounds__(256)
pack_general_kernel(const float *__restrict__ x, const float *__restrict__ bias,
                    uint32_t *__restrict__ out, long nwords, int C_in, int cwords)
{
    const int lane = threadIdx.x & 31;
    const long warp = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long nwarps = (long)gridDim.x * (blockDim.x >> 5);
    for (long wi = warp; wi < nwords; wi += nwarps) {
        const long pix = wi / cwords;
        const int c = (int)(wi - pix * cwords) * 32 + lane;
        float s = __ldg(x + pix * C_in + (c % C_in));
        if (bias) s = __fadd_rn(s, __ldg(bias + c));
        const uint32_t word = __ballot_sync(0xffffffffu, s >= 0.0f);
        if (lane == 0) out[wi] = word;
    }
}

// Stem path (Table 1 "stem replicate": 4 real channels replicated 8x to 32 sign
// channels): one thread per pixel reads its 4 values as one 16-byte load and emits the
// pixel's single 32-bit word; the 32 biases sit in shared memory.
__global__ void __launch_bounds__(256)
pack_c4r8_kernel(const float4 *__restrict__ x, const float *__restrict__ bias,
                 uint32_t *__restrict__ out, long npix)
{
    constexpr int U = 4;                       // pixels in flight per thread
    __shared__ float sb[32];
    if (threadIdx.x < 32) sb[threadIdx.x] = bias ? bias[threadIdx.x] : 0.0f;
    __syncthreads();
    float b[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) b[c] = sb[c];
    const long stride = (long)gridDim.x * blockDim.x;
    for (long p0 = (long)blockIdx.x * blockDim.x + threadIdx.x; p0 < npix; p0 += stride * U) {
        float4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long p = p0 + u * stride;
            v[u] = (p < npix) ? __ldcs(x + p) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long p = p0 + u * stride;
            const float f[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            uint32_t word = 0;
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                const float s = bias ? __fadd_rn(f[c & 3], b[c]) : f[c & 3];
                word |= (s >= 0.0f ? 1u : 0u) << c;
            }
            if (p < npix) __stcs(out + p, word);
        }
    }
}

int launch_pack(const float *x, const float *bias, uint32_t *out, long npix, int C_in, int R,
                cudaStream_t stream)
{
    const int C = C_in * R;
    const int cwords = C / 32;
    const long nwords = npix * cwords;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int threads = 256;
    if (R == 1 && C_in % 32 == 0) {
        constexpr int UNROLL = 8;
        const long warps_needed = (nwords + UNROLL - 1) / UNROLL;
        long blocks = (warps_needed + 7) / 8;
        const long cap = (long)sms * 8;
        if (blocks > cap) blocks = cap;
        if (blocks < 1) blocks = 1;
        if (bias)
            pack_stream_kernel<UNROLL, true><<<(int)blocks, threads, 0, stream>>>(x, bias, out, nwords, cwords);
        else
            pack_stream_kernel<UNROLL, false><<<(int)blocks, threads, 0, stream>>>(x, bias, out, nwords, cwords);
    } else if (C_in == 4 && R == 8) {
        long blocks = (npix + threads * 4 - 1) / (threads * 4);
        const long cap = (long)sms * 6;
        if (blocks > cap) blocks = cap;
        if (blocks < 1) blocks = 1;
        pack_c4r8_kernel<<<(int)blocks, threads, 0, stream>>>(reinterpret_cast<const float4 *>(x), bias, out, npix);
    } else {
        long blocks = (nwords + 7) / 8;
        const long cap = (long)sms * 8;
        if (blocks > cap) blocks = cap;
        pack_general_kernel<<<(int)blocks, threads, 0, stream>>>(x, bias, out, nwords, C_in, cwords);
    }
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace bcnn
