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

// Stem path (Table 1 "stem replicate": 4 real channels replicated 8x to 32 sign channels): one
// thread per pixel reads its 4 values as one 16-byte load and emits the pixel's single 32-bit word.
//
// Fast path (all biases finite).  For finite b, fl(x + b) >= 0 exactly when x >= -b (a sum of two
// floats never rounds to zero unless it is zero, and NaN / infinite x behave the same on both sides),
// so input value i only has to be ranked among its 8 thresholds -b[4r+i]: they are sorted once per
// CTA, a 4-compare search counts how many are <= x, and a 9-entry table per input gives the bits.
// That is ~13 instructions per input value instead of 3 per output channel; the kernel becomes
// HBM-bound.  With a NaN or infinite bias (inf - inf = NaN -> -1) the plain per-channel path runs.
__global__ void __launch_bounds__(256)
pack_c4r8_kernel(const float4 *__restrict__ x, const float *__restrict__ bias,
                 uint32_t *__restrict__ out, long npix)
{
    constexpr int U = 4;                       // pixels in flight per thread
    __shared__ float sb[32];
    __shared__ float sts[4][8];                // sorted thresholds of input i
    __shared__ uint32_t lut[4][9];             // bits set when c thresholds are <= x
    __shared__ int all_finite;
    if (threadIdx.x == 0) all_finite = 1;
    __syncthreads();
    if (threadIdx.x < 32) {
        const float b = bias ? bias[threadIdx.x] : 0.0f;
        sb[threadIdx.x] = b;
        if (!(fabsf(b) <= 3.402823466e38f)) all_finite = 0;      // NaN or infinity
    }
    __syncthreads();
    if (threadIdx.x < 4 && all_finite) {
        const int i = threadIdx.x;
        float t[8];
        int r[8];
        for (int k = 0; k < 8; ++k) { t[k] = -sb[4 * k + i]; r[k] = k; }
        for (int a = 1; a < 8; ++a)            // insertion sort, ascending
            for (int k = a; k > 0 && t[k] < t[k - 1]; --k) {
                const float tf = t[k]; t[k] = t[k - 1]; t[k - 1] = tf;
                const int ti = r[k]; r[k] = r[k - 1]; r[k - 1] = ti;
            }
        uint32_t m = 0;
        lut[i][0] = 0;
        for (int k = 0; k < 8; ++k) {
            sts[i][k] = t[k];
            m |= 1u << (4 * r[k] + i);
            lut[i][k + 1] = m;
        }
    }
    __syncthreads();
    const long stride = (long)gridDim.x * blockDim.x;
    if (all_finite) {
        float ts[4][8];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int k = 0; k < 8; ++k) ts[i][k] = sts[i][k];
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
                for (int i = 0; i < 4; ++i) {
                    const float xv = f[i];
                    const bool pp = xv >= ts[i][3];
                    const bool qq = xv >= (pp ? ts[i][5] : ts[i][1]);
                    const float tl = pp ? (qq ? ts[i][6] : ts[i][4]) : (qq ? ts[i][2] : ts[i][0]);
                    const bool rr = xv >= tl;
                    const int c = (pp ? 4 : 0) + (qq ? 2 : 0) + (rr ? 1 : 0) + (xv >= ts[i][7] ? 1 : 0);
                    word |= lut[i][c];
                }
                if (p < npix) __stcs(out + p, word);
            }
        }
        return;
    }
    float b[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) b[c] = sb[c];
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
                const float s = __fadd_rn(f[c & 3], b[c]);
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
        int per_sm = 4;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pack_c4r8_kernel, threads, 0) != cudaSuccess || per_sm < 1)
            per_sm = 4;
        const long cap = (long)sms * per_sm;       // one wave of resident CTAs, grid-stride inside
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
