// CUDA-core engine of the binary implicit GEMM: XOR + popcount on 32-bit words.
// It accepts every shape the API accepts (any kh, kw, stride, pad, any C_out) and is
// the fallback of the faster engines.
//
// CTA tile: 64 output pixels x 64 output channels, 256 threads, each thread a 4x4
// register tile (rows ty+16*i, columns tx+16*j).  K advances 8 words (256 bits) per
// step through shared memory; rows of the implicit patch matrix are gathered straight
// from the packed NHWC tensor, out-of-image taps read as zero words (= all -1).
#include "bcnn_common.cuh"

namespace bcnn {

namespace {

constexpr int BM = 64, BN = 64, KC = 8, LDS_STRIDE = 12;  // 12-word rows: 16-byte aligned, bank-spread

template <bool FUSED>
__global__ void __launch_bounds__(256)
conv_lop3_kernel(const ConvProblem p)
{
    __shared__ __align__(16) uint32_t As[BM * LDS_STRIDE];
    __shared__ __align__(16) uint32_t Ws[BN * LDS_STRIDE];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;

    // staging role: thread loads word kk of rows r0 and r0+32
    const int kk = tid & 7, r0 = tid >> 3;
    RowCoord rc[2];
    bool row_ok[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int m = m0 + r0 + 32 * h;
        row_ok[h] = m < p.M;
        rc[h] = row_coord(p, row_ok[h] ? m : 0);
    }

    int acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;

    for (int k0 = 0; k0 < p.kwords; k0 += KC) {
        const int kword = k0 + kk;
        const bool k_ok = kword < p.kwords;
        int r = 0, t = 0, cj = 0;
        if (k_ok) {
            const int tap = kword / p.cw;
            cj = kword - tap * p.cw;
            r = tap / p.kw;
            t = tap - r * p.kw;
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t av = 0;
            if (k_ok && row_ok[h]) {
                const int ih = rc[h].ih0 + r, iw = rc[h].iw0 + t;
                if (ih >= 0 && ih < p.H && iw >= 0 && iw < p.W)
                    av = __ldg(p.x + (((long)rc[h].b * p.H + ih) * p.W + iw) * p.cw + cj);
            }
            As[(r0 + 32 * h) * LDS_STRIDE + kk] = av;
            uint32_t wv = 0;
            const int n = n0 + r0 + 32 * h;
            if (k_ok && n < p.C_out) wv = __ldg(p.w + (long)n * p.kwords + kword);
            Ws[(r0 + 32 * h) * LDS_STRIDE + kk] = wv;
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < KC / 4; ++q) {
            uint4 a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                a[i] = *reinterpret_cast<const uint4 *>(&As[(ty + 16 * i) * LDS_STRIDE + 4 * q]);
#pragma unroll
            for (int j = 0; j < 4; ++j)
                w[j] = *reinterpret_cast<const uint4 *>(&Ws[(tx + 16 * j) * LDS_STRIDE + 4 * q]);
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    acc[i][j] += __popc(a[i].x ^ w[j].x) + __popc(a[i].y ^ w[j].y) +
                                 __popc(a[i].z ^ w[j].z) + __popc(a[i].w ^ w[j].w);
        }
        __syncthreads();
    }

    // epilogue: value = K - 2 * (number of differing bits)
    if (!FUSED) {
        int32_t *out = static_cast<int32_t *>(p.out);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = m0 + ty + 16 * i;
            if (m >= p.M) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int n = n0 + tx + 16 * j;
                if (n < p.C_out) out[(long)m * p.C_out + n] = p.K - 2 * acc[i][j];
            }
        }
    } else {
        // C_out % 32 == 0.  A warp holds rows ty = 2*warp (lanes 0-15) and 2*warp+1
        // (lanes 16-31); for fixed (i, j) the vote collects columns n0+16*j+tx.
        uint32_t *out = static_cast<uint32_t *>(p.out);
        const int owords = p.C_out >> 5;
        const int lane = tid & 31;
        int thr[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx + 16 * j;
            thr[j] = (n < p.C_out) ? __ldg(p.thr + n) : 0;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                v[j] = __ballot_sync(0xffffffffu, (p.K - 2 * acc[i][j]) >= thr[j]);
            const int m = m0 + ty + 16 * i;
            // lane 0 writes the row of lanes 0-15, lane 16 the row of lanes 16-31
            if ((lane & 15) == 0 && m < p.M) {
                const int sh = lane;  // 0 or 16
#pragma unroll
                for (int wd = 0; wd < 2; ++wd) {
                    const int nword = (n0 >> 5) + wd;
                    if (nword < owords) {
                        const uint32_t lo = (v[2 * wd] >> sh) & 0xffffu;
                        const uint32_t hi = (v[2 * wd + 1] >> sh) & 0xffffu;
                        out[(long)m * owords + nword] = lo | (hi << 16);
                    }
                }
            }
        }
    }
}

// Pointwise layer with one word of K (1x1, stride 1, no padding, C_in = 32, C_out <= 32): a pixel is one
// 32-bit word and an output is one XOR + popcount, so a tile engine only adds overhead.  Each thread
// turns four pixels per step into four output words: per output bit XOR, POPC, subtract and a funnel
// shift that collects the sign; the popcount pipe is the bound (measured 13 outputs per clock per SM).  K - 2*pc >= thr  <=>  pc <= floor((K - thr) / 2) =: lim, and the sign bit of lim - pc is the
// complement of the output bit.
template <bool FUSED>
__global__ void __launch_bounds__(256)
conv_k32_kernel(const ConvProblem p)
{
    uint32_t w[32];       // uniform across the grid: weight words and popcount limits
    int lim[32];
#pragma unroll
    for (int n = 0; n < 32; ++n) {
        w[n] = n < p.C_out ? __ldg(p.w + n) : 0u;
        lim[n] = 0;
        if (FUSED) {
            int t = __ldg(p.thr + n);
            t = t < -64 ? -64 : (t > 64 ? 64 : t);        // beyond +-K the comparison is constant
            lim[n] = (32 - t) >> 1;                        // floor: arithmetic shift
        }
    }
    const long groups = p.M >> 2;                          // four consecutive pixels per step
    const long stride = (long)gridDim.x * blockDim.x;
    const long first = (long)blockIdx.x * blockDim.x + threadIdx.x;
    const uint4 *x4 = reinterpret_cast<const uint4 *>(p.x);

    auto pixel = [&](uint32_t xv, long m) -> uint32_t {
        if (FUSED) {
            uint32_t acc = 0;
#pragma unroll
            for (int n = 31; n >= 0; --n) acc = __funnelshift_l((uint32_t)(lim[n] - __popc(xv ^ w[n])), acc, 1);
            return ~acc;
        } else {
            int32_t *dst = static_cast<int32_t *>(p.out) + m * p.C_out;
            if (p.C_out == 32) {
#pragma unroll
                for (int n4 = 0; n4 < 8; ++n4)
                    *reinterpret_cast<int4 *>(dst + 4 * n4) =
                        make_int4(32 - 2 * __popc(xv ^ w[4 * n4]), 32 - 2 * __popc(xv ^ w[4 * n4 + 1]),
                                  32 - 2 * __popc(xv ^ w[4 * n4 + 2]), 32 - 2 * __popc(xv ^ w[4 * n4 + 3]));
            } else {
#pragma unroll
                for (int n = 0; n < 32; ++n)
                    if (n < p.C_out) dst[n] = 32 - 2 * __popc(xv ^ w[n]);
            }
            return 0;
        }
    };

    for (long g = first; g < groups; g += stride) {
        const uint4 xv = __ldg(x4 + g);
        uint4 o;
        o.x = pixel(xv.x, 4 * g);
        o.y = pixel(xv.y, 4 * g + 1);
        o.z = pixel(xv.z, 4 * g + 2);
        o.w = pixel(xv.w, 4 * g + 3);
        if (FUSED) reinterpret_cast<uint4 *>(p.out)[g] = o;
    }
    const long m = 4 * groups + first;                     // up to three tail pixels
    if (m < p.M) {
        const uint32_t o = pixel(__ldg(p.x + m), m);
        if (FUSED) static_cast<uint32_t *>(p.out)[m] = o;
    }
}

template <bool FUSED>
int launch_k32(const ConvProblem &p, cudaStream_t stream)
{
    int dev = 0, sms = 148, per_sm = 1;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, conv_k32_kernel<FUSED>, 256, 0) != cudaSuccess || per_sm < 1)
        per_sm = 1;
    const long groups = ((long)p.M + 3) / 4;
    long blocks = (groups + 255) / 256;
    const long wave = (long)sms * per_sm;                 // one resident wave, grid-stride beyond it
    if (blocks > wave) blocks = wave;
    conv_k32_kernel<FUSED><<<(unsigned)blocks, 256, 0, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace

bool conv_lop3_pointwise_k32(const ConvProblem &p)
{
    return p.kh * p.kw == 1 && p.stride == 1 && p.pad == 0 && p.C_in == 32 &&
           (p.thr ? p.C_out == 32 : p.C_out <= 32);
}

int launch_conv_lop3(const ConvProblem &p, cudaStream_t stream)
{
    if (conv_lop3_pointwise_k32(p)) return p.thr ? launch_k32<true>(p, stream) : launch_k32<false>(p, stream);
    dim3 grid((unsigned)(((long)p.M + BM - 1) / BM), (p.C_out + BN - 1) / BN);
    if (grid.y > 65535) return BCNN_ERR_UNSUPPORTED;
    if (p.thr)
        conv_lop3_kernel<true><<<grid, 256, 0, stream>>>(p);
    else
        conv_lop3_kernel<false><<<grid, 256, 0, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace bcnn
