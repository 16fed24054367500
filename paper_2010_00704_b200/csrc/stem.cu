// Fused stem: binarize + pack (Section 4.2.1 bias + sign, Table 1 "stem replicate": 4 real channels
// replicated 8x to 32 sign channels) followed by the first binary 1x1 convolution (32 -> 32 channels)
// with its threshold epilogue, in one pass over the real input.  The 32-channel sign tensor is never
// written: per pixel the kernel reads 16 bytes and writes the 4 bytes of the convolution's packed output.
//
// Why a table.  Sign channel c = 4r + i is (x_i + bias_c >= 0): the 8 replicas of real channel i are a
// thermometer code of x_i against its 8 thresholds -bias, so a pixel's 32 sign bits are fixed by four
// levels c_i in 0..8 (how many thresholds of channel i are <= x_i): 9^4 = 6561 distinct sign words.  The
// whole 1x1 layer - K - 2 popc(word XOR w_n) >= thr_n for the 32 outputs n - is therefore a function of
// e = c_0 + 9 c_1 + 81 c_2 + 729 c_3, tabulated once per CTA in shared memory (26 KB); the pixel loop is
// the level search of the pack kernel plus one table read.  The result is bit-identical to bcnn_pack
// followed by bcnn_conv2d_b1_fused.
//
// Table build (per CTA, ~2 us): mismatches split as popc over channels {0,1} + popc over channels {2,3};
// two 81-entry tables of 32 byte fields (one per output n, four per word) are added word-wise; the first
// carries 127 - theta_n, theta_n = floor((32 - thr_n) / 2) clamped to [-1, 32], so that bit 7 of field n
// is set exactly when mismatches > theta_n, i.e. when the output bit is 0.
//
// With a NaN or infinite bias the thermometer argument fails (inf - inf = NaN -> -1): the plain
// per-channel path runs instead (32 fp32 adds + compares, 32 popcounts per pixel).
#include "bcnn_common.cuh"

namespace bcnn {

namespace {

constexpr int STEM_THREADS = 1024;
constexpr int STEM_LEVELS = 9 * 9 * 9 * 9;

__global__ void __launch_bounds__(STEM_THREADS, 1)
stem_c4r8_k32_kernel(const float4 *__restrict__ x, const float *__restrict__ bias, const uint32_t *__restrict__ w,
                     const int32_t *__restrict__ thr, uint32_t *__restrict__ out, long npix)
{
    constexpr int U = 4;                        // pixels in flight per thread
    __shared__ float sb[32];
    __shared__ float sts[4][8];                 // sorted thresholds of input i
    __shared__ uint32_t lut[4][9];              // sign bits of input i set at level c
    __shared__ uint32_t sw[32];                 // weight word of output n
    __shared__ int stheta[32];
    __shared__ __align__(16) uint32_t ta[81][8];  // byte field n: 127 - theta_n + mismatches over channels {0, 1}
    __shared__ __align__(16) uint32_t tb[81][8];  // byte field n: mismatches over channels {2, 3}
    __shared__ uint32_t table[STEM_LEVELS];     // output word of the level tuple e
    __shared__ int all_finite;

    const int tid = threadIdx.x;
    if (tid == 0) all_finite = 1;
    __syncthreads();
    if (tid < 32) {
        const float b = bias ? bias[tid] : 0.0f;
        sb[tid] = b;
        if (!(fabsf(b) <= 3.402823466e38f)) all_finite = 0;      // NaN or infinity
        sw[tid] = w[tid];
        // out bit n = (32 - 2*mism >= thr)  <=>  mism <= floor((32 - thr) / 2)
        long long th = (32LL - (long long)thr[tid]) >> 1;
        th = th < -1 ? -1 : (th > 32 ? 32 : th);
        stheta[tid] = (int)th;
    }
    __syncthreads();
    const long stride = (long)gridDim.x * blockDim.x;

    if (!all_finite) {
        // plain path: every sign channel evaluated as written, then 32 XOR + popcount
        for (long p = (long)blockIdx.x * blockDim.x + tid; p < npix; p += stride) {
            const float4 v = __ldcs(x + p);
            const float f[4] = {v.x, v.y, v.z, v.w};
            uint32_t word = 0;
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                const float s = __fadd_rn(f[c & 3], sb[c]);
                word |= (s >= 0.0f ? 1u : 0u) << c;
            }
            uint32_t o = 0;
#pragma unroll 8
            for (int n = 0; n < 32; ++n) o |= (__popc(word ^ sw[n]) <= stheta[n] ? 1u : 0u) << n;
            __stcs(out + p, o);
        }
        return;
    }

    if (tid < 4) {
        const int i = tid;
        float t[8];
        int r[8];
        for (int k = 0; k < 8; ++k) { t[k] = -sb[4 * k + i]; r[k] = k; }
        for (int a = 1; a < 8; ++a)             // insertion sort, ascending
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
    // the two half tables: entry (c_lo + 9 c_hi), output n -> one byte
    for (int idx = tid; idx < 2 * 81 * 32; idx += STEM_THREADS) {
        const int half = idx / (81 * 32), rem = idx - half * (81 * 32);
        const int e = rem >> 5, n = rem & 31;
        const int clo = e % 9, chi = e / 9;
        const uint32_t word = lut[2 * half][clo] | lut[2 * half + 1][chi];
        const uint32_t mask = half ? 0xCCCCCCCCu : 0x33333333u;    // sign channels c with c % 4 in {2,3} / {0,1}
        int v = __popc((word ^ sw[n]) & mask);
        if (half == 0) v += 127 - stheta[n];
        unsigned char *dst = reinterpret_cast<unsigned char *>(half ? &tb[e][0] : &ta[e][0]);
        dst[n] = (unsigned char)v;
    }
    __syncthreads();
    for (int e = tid; e < STEM_LEVELS; e += STEM_THREADS) {
        const int e01 = e % 81, e23 = e / 81;
        uint32_t o = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t v = ta[e01][k] + tb[e23][k];            // fields stay below 256: no carries between them
            // bit 7 of field j clear -> output bit 4k + j set; the multiply gathers bits 7, 15, 23, 31 into 28..31
            o |= (((~v & 0x80808080u) * 0x00204081u) >> 28) << (4 * k);
        }
        table[e] = o;
    }
    __syncthreads();

    float ts[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int k = 0; k < 8; ++k) ts[i][k] = sts[i][k];
    for (long p0 = (long)blockIdx.x * blockDim.x + tid; p0 < npix; p0 += stride * U) {
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
            // level of value i = how many of its sorted thresholds are <= x: eight compares that yield 1.0f / 0.0f
            // and a sum on the fp32 pipe (cheaper than a search made of selects on the integer pipe); the tuple index
            // c_0 + 9 c_1 + 81 c_2 + 729 c_3 <= 6560 is exact in fp32
            float ef = 0.0f;
#pragma unroll
            for (int i = 3; i >= 0; --i) {
                const float xv = f[i];
                float c = 0.0f;
#pragma unroll
                for (int k = 0; k < 8; ++k) c += (xv >= ts[i][k]) ? 1.0f : 0.0f;
                ef = fmaf(ef, 9.0f, c);
            }
            const int e = __float2int_rn(ef);
            if (p < npix) __stcs(out + p, table[e]);
        }
    }
}

}  // namespace

int launch_stem_c4r8_k32(const float *x, const float *bias, const uint32_t *w, const int32_t *thr, uint32_t *out,
                         long npix, cudaStream_t stream)
{
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    long blocks = (npix + STEM_THREADS * 4 - 1) / (STEM_THREADS * 4);
    if (blocks > sms) blocks = sms;             // one resident CTA per SM builds the table once, grid-stride inside
    if (blocks < 1) blocks = 1;
    stem_c4r8_k32_kernel<<<(int)blocks, STEM_THREADS, 0, stream>>>(reinterpret_cast<const float4 *>(x), bias, w, thr, out, npix);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace bcnn
