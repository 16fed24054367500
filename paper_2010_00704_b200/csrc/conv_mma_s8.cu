// Narrow-layer engine of the binary implicit GEMM: warp-level int8 tensor-core MMA
// (mma.sync.m16n8k32, u8 x u8 -> s32) fed straight from registers.
//
// For layers with few output channels and a short K (the stem-like layers: K = 32..576,
// C_out <= 64) a 128-row tensor-memory tile is mostly set-up cost.  Here every warp
// streams 32 output pixels at a time and never touches shared memory for activations:
// the A fragment of thread (g, q) of m16n8k32 holds row g (and g+8), K bytes 4q..4q+3
// (and 16+4q..), and since the sum over K is order-free we let those bytes carry bits
// q+8i (and q+4+8i) of the row's 32-bit word, so a fragment register is one AND:
//     a = word & (0x01010101 << q)          -> bytes 0 or 2^q
// The weight fragments carry the matching bits with bytes 0 or 2^(7-q), are built once
// per CTA into shared memory in fragment order, and every product of two set bits is
// 128.  With the row / column popcounts,
//     sum a*g = K - 2*popc(A) - 2*popc(G) + 4*popc(A and G) = K - 2pa - 2pg + (acc >> 5).
// Out-of-image taps are zero words (value -1).
#include "bcnn_common.cuh"

namespace bcnn {

namespace {

constexpr int THREADS = 256;
constexpr int MA = 2;                 // m16 atoms per warp iteration (32 output pixels)
constexpr int MAX_SMEM = 200 * 1024;

__device__ __forceinline__ void mma_u8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint2 b)
{
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b.x), "r"(b.y));
}

template <int NA, bool FUSED>
__global__ void __launch_bounds__(THREADS, 2)
conv_mma_s8_kernel(const ConvProblem p)
{
    constexpr int BN = 8 * NA;
    extern __shared__ __align__(16) unsigned char smem[];
    uint2 *wfrag = reinterpret_cast<uint2 *>(smem);                 // [kwords][NA][32 lanes]
    int *colc = reinterpret_cast<int *>(wfrag + (size_t)p.kwords * NA * 32);   // [BN] per-column constant

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, q = lane & 3;
    const int n0 = blockIdx.y * BN;

    // ---- weight fragments in fragment order + per-column constants
    for (int idx = tid; idx < p.kwords * NA * 32; idx += THREADS) {
        const int l = idx & 31, j = (idx >> 5) % NA, kw = idx / (32 * NA);
        const int n = n0 + 8 * j + (l >> 2), ql = l & 3;
        const uint32_t w = (n < p.C_out) ? __ldg(p.w + (long)n * p.kwords + kw) : 0u;
        uint2 f;
        f.x = ((w >> ql) & 0x01010101u) << (7 - ql);
        f.y = ((w >> (ql + 4)) & 0x01010101u) << (3 - ql);
        wfrag[idx] = f;
    }
    for (int c = tid; c < BN; c += THREADS) {
        const int n = n0 + c;
        int pop = 0;
        if (n < p.C_out)
            for (int kw = 0; kw < p.kwords; ++kw) pop += __popc(__ldg(p.w + (long)n * p.kwords + kw));
        // int32 output: value = colc - 2*pa + (acc >> 5);  fused: bit = (acc >> 5) - 2*pa >= thr - colc
        const int base = p.K - 2 * pop;
        colc[c] = FUSED ? ((n < p.C_out ? __ldg(p.thr + n) : 0) - base) : base;
    }
    __syncthreads();

    // per-thread column constants: columns 8j + 2q + e
    int cc[NA][2];
#pragma unroll
    for (int j = 0; j < NA; ++j) {
        cc[j][0] = colc[8 * j + 2 * q];
        cc[j][1] = colc[8 * j + 2 * q + 1];
    }

    const uint32_t mlo = 0x01010101u << q, mhi = 0x10101010u << q;
    const int rows_per_iter = 16 * MA;
    const long nblocks = ((long)p.M + rows_per_iter - 1) / rows_per_iter;
    const long wstride = (long)gridDim.x * (THREADS / 32);
    const int owords = p.C_out >> 5;

    for (long blk = (long)blockIdx.x * (THREADS / 32) + warp; blk < nblocks; blk += wstride) {
        const int mbase = (int)(blk * rows_per_iter);
        // rows handled by this thread: mbase + 16*a + g + 8*h
        const uint32_t *xb[MA][2];
        int ih0[MA][2], iw0[MA][2];
        bool ok[MA][2];
#pragma unroll
        for (int a = 0; a < MA; ++a)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int m = mbase + 16 * a + g + 8 * h;
                ok[a][h] = m < p.M;
                const RowCoord rc = row_coord(p, ok[a][h] ? m : 0);
                xb[a][h] = p.x + (long)rc.b * p.H * p.W * p.cw;
                ih0[a][h] = rc.ih0;
                iw0[a][h] = rc.iw0;
            }
        int acc[MA][NA][4];
        int pa[MA][2];
#pragma unroll
        for (int a = 0; a < MA; ++a) {
            pa[a][0] = pa[a][1] = 0;
#pragma unroll
            for (int j = 0; j < NA; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[a][j][e] = 0;
        }

        // K loop, software-pipelined: the words of step kw+1 are in flight while step kw is multiplied
        int r = 0, t = 0, cj = 0;      // tap and channel word of the K word being loaded (warp-uniform)
        auto load_words = [&](uint32_t (&w)[MA][2]) {
#pragma unroll
            for (int a = 0; a < MA; ++a)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int ih = ih0[a][h] + r, iw = iw0[a][h] + t;
                    uint32_t v = 0;
                    if (ok[a][h] && ih >= 0 && ih < p.H && iw >= 0 && iw < p.W)
                        v = __ldg(xb[a][h] + ((long)ih * p.W + iw) * p.cw + cj);
                    w[a][h] = v;
                }
            if (++cj == p.cw) {
                cj = 0;
                if (++t == p.kw) { t = 0; ++r; }
            }
        };
        uint32_t w[MA][2], wn[MA][2];
        load_words(w);
        for (int kw = 0; kw < p.kwords; ++kw) {
            if (kw + 1 < p.kwords) load_words(wn);
            const uint2 *wf = wfrag + (size_t)kw * NA * 32 + lane;
#pragma unroll
            for (int a = 0; a < MA; ++a) {
                pa[a][0] += __popc(w[a][0]);
                pa[a][1] += __popc(w[a][1]);
            }
#pragma unroll
            for (int j = 0; j < NA; ++j) {
                const uint2 b = wf[j * 32];
#pragma unroll
                for (int a = 0; a < MA; ++a)
                    mma_u8(acc[a][j], w[a][0] & mlo, w[a][1] & mlo, w[a][0] & mhi, w[a][1] & mhi, b);
            }
#pragma unroll
            for (int a = 0; a < MA; ++a) {
                w[a][0] = wn[a][0];
                w[a][1] = wn[a][1];
            }
        }

        // ---- epilogue.  acc[a][j][0,1] -> row g, columns 8j+2q, 8j+2q+1;  [2,3] -> row g+8.
#pragma unroll
        for (int a = 0; a < MA; ++a)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int m = mbase + 16 * a + g + 8 * h;
                const int pa2 = 2 * pa[a][h];
                if (!FUSED) {
                    if (m < p.M) {
                        int32_t *dst = static_cast<int32_t *>(p.out) + (long)m * p.C_out + n0 + 2 * q;
#pragma unroll
                        for (int j = 0; j < NA; ++j) {
                            const int n = n0 + 8 * j + 2 * q;
                            const int v0 = cc[j][0] - pa2 + (acc[a][j][2 * h] >> 5);
                            const int v1 = cc[j][1] - pa2 + (acc[a][j][2 * h + 1] >> 5);
                            if (n + 1 < p.C_out && (p.C_out & 1) == 0) {
                                *reinterpret_cast<int2 *>(dst + 8 * j) = make_int2(v0, v1);
                            } else {
                                if (n < p.C_out) dst[8 * j] = v0;
                                if (n + 1 < p.C_out) dst[8 * j + 1] = v1;
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int wd = 0; wd < NA / 4; ++wd) {
                        uint32_t bits = 0;
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) {
                            const int j = 4 * wd + jj;
                            const int v0 = (acc[a][j][2 * h] >> 5) - pa2;
                            const int v1 = (acc[a][j][2 * h + 1] >> 5) - pa2;
                            bits |= (v0 >= cc[j][0] ? 1u : 0u) << (8 * jj + 2 * q);
                            bits |= (v1 >= cc[j][1] ? 1u : 0u) << (8 * jj + 2 * q + 1);
                        }
                        bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
                        bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
                        const int nword = (n0 >> 5) + wd;
                        if (q == 0 && m < p.M && nword < owords)
                            static_cast<uint32_t *>(p.out)[(long)m * owords + nword] = bits;
                    }
                }
            }
    }
}

size_t smem_bytes(const ConvProblem &p, int NA) { return (size_t)p.kwords * NA * 32 * sizeof(uint2) + 8 * NA * sizeof(int); }

template <int NA>
int launch_na(const ConvProblem &p, cudaStream_t stream)
{
    const size_t smem = smem_bytes(p, NA);
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long nblocks = ((long)p.M + 16 * MA - 1) / (16 * MA);
    void (*k)(const ConvProblem) = p.thr ? conv_mma_s8_kernel<NA, true> : conv_mma_s8_kernel<NA, false>;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return BCNN_ERR_CUDA;
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, THREADS, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    // persistent grid: every resident CTA slot of the chip, split over the N tiles
    const long ny = (p.C_out + 8 * NA - 1) / (8 * NA);
    if (ny > 65535) return BCNN_ERR_UNSUPPORTED;
    long gx = (nblocks + THREADS / 32 - 1) / (THREADS / 32);
    long cap = ((long)sms * per_sm) / ny;
    if (cap < 1) cap = 1;
    if (gx > cap) gx = cap;
    if (gx < 1) gx = 1;
    dim3 grid((unsigned)gx, (unsigned)ny);
    k<<<grid, THREADS, smem, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace

bool conv_mma_s8_supports(const ConvProblem &p)
{
    if (p.thr != nullptr && (p.C_out % 32 != 0)) return false;
    const int NA = p.C_out <= 32 ? 4 : 8;
    return smem_bytes(p, NA) <= (size_t)MAX_SMEM && p.K <= (1 << 20);
}

int launch_conv_mma_s8(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_mma_s8_supports(p)) return BCNN_ERR_UNSUPPORTED;
    if (p.C_out <= 32) return launch_na<4>(p, stream);
    return launch_na<8>(p, stream);
}

}  // namespace bcnn
