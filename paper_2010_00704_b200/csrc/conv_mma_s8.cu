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

// Output-channel permutation.  Inside each group of 32 output channels, column c (0..7) of
// MMA atom j (0..3) carries channel 8*(c >> 1) + 2*j + (c & 1).  Thread q of a quad holds
// columns 2q, 2q+1 of every atom, i.e. the eight consecutive channels 8q .. 8q+7: one byte
// of the packed output word, or two 16-byte int32 stores.
__device__ __forceinline__ int atom_col_to_channel(int atom, int c)
{
    return 32 * (atom >> 2) + 8 * (c >> 1) + 2 * (atom & 3) + (c & 1);
}

template <int NA, bool FUSED>
__global__ void __launch_bounds__(THREADS, 2)
conv_mma_s8_kernel(const ConvProblem p)
{
    constexpr int BN = 8 * NA;
    extern __shared__ __align__(16) unsigned char smem[];
    uint2 *wfrag = reinterpret_cast<uint2 *>(smem);                 // [kwords][NA][32 lanes]
    int *colc = reinterpret_cast<int *>(wfrag + (size_t)p.kwords * NA * 32);   // [BN] per-channel constant
    int *tapoff = colc + BN;                                         // [kh*kw] word offset of each tap

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, q = lane & 3;
    const int n0 = blockIdx.y * BN;
    const int ntaps = p.kh * p.kw;

    // ---- weight fragments in fragment order, per-channel constants, tap offsets
    for (int idx = tid; idx < p.kwords * NA * 32; idx += THREADS) {
        const int l = idx & 31, j = (idx >> 5) % NA, kw = idx / (32 * NA);
        const int n = n0 + atom_col_to_channel(j, l >> 2), ql = l & 3;
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
        // with acc = 128 * popc(A and G) and pa = popc(A):
        //   int32:  value = (acc >> 5) - 2*pa + (K - 2*pop)
        //   fused:  bit   = acc - 64*pa - 32*(thr - K + 2*pop) >= 0
        // (a threshold beyond +-(K + 1) decides like that bound; clamping keeps the constant inside int32)
        const int thr_n = max(min(FUSED && n < p.C_out ? __ldg(p.thr + n) : 0, p.K + 1), -p.K - 1);
        colc[c] = FUSED ? -32 * (thr_n - p.K + 2 * pop) : p.K - 2 * pop;
    }
    for (int tp = tid; tp < ntaps; tp += THREADS) tapoff[tp] = ((tp / p.kw) * p.W + (tp % p.kw)) * p.cw;
    __syncthreads();

    // per-thread channel constants: atom j, column 2q+e -> channel 32*(j/4) + 8q + 2*(j%4) + e
    int cc[NA][2];
#pragma unroll
    for (int j = 0; j < NA; ++j) {
        cc[j][0] = colc[atom_col_to_channel(j, 2 * q)];
        cc[j][1] = colc[atom_col_to_channel(j, 2 * q + 1)];
    }

    const uint32_t mlo = 0x01010101u << q, mhi = 0x10101010u << q;
    const int rows_per_iter = 16 * MA;
    const long nblocks = ((long)p.M + rows_per_iter - 1) / rows_per_iter;
    const long wstride = (long)gridDim.x * (THREADS / 32);
    const int owords = p.C_out >> 5;
    const bool plain = (ntaps == 1 && p.stride == 1 && p.pad == 0);   // 1x1: row m is pixel m

    // Row set-up of one 32-row block: pointer to each window's top-left pixel (may lie outside the
    // image) and one validity bit per tap.  Rows of this thread: mbase + 16*a + g + 8*h.
    auto setup_rows = [&](long blk, const uint32_t *(&xb)[MA][2], uint32_t (&vmask)[MA][2]) {
        const int mbase = (int)(blk * rows_per_iter);
#pragma unroll
        for (int a = 0; a < MA; ++a)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int m = mbase + 16 * a + g + 8 * h;
                const bool ok = m < p.M;
                if (plain) {
                    xb[a][h] = p.x + (long)(ok ? m : 0) * p.cw;
                    vmask[a][h] = ok ? 1u : 0u;
                } else {
                    const RowCoord rc = row_coord(p, ok ? m : 0);
                    xb[a][h] = p.x + (((long)rc.b * p.H + rc.ih0) * p.W + rc.iw0) * p.cw;
                    uint32_t colbits = 0, mask = 0;
                    for (int t = 0; t < p.kw; ++t)
                        if (rc.iw0 + t >= 0 && rc.iw0 + t < p.W) colbits |= 1u << t;
                    for (int r = 0; r < p.kh; ++r)
                        if (rc.ih0 + r >= 0 && rc.ih0 + r < p.H) mask |= colbits << (r * p.kw);
                    vmask[a][h] = ok ? mask : 0u;
                }
            }
    };
    auto load_words = [&](uint32_t (&w)[MA][2], const uint32_t *const (&xb)[MA][2], const uint32_t (&vmask)[MA][2],
                          int tap, int cj) {
        const int off = tapoff[tap] + cj;
#pragma unroll
        for (int a = 0; a < MA; ++a)
#pragma unroll
            for (int h = 0; h < 2; ++h)
                w[a][h] = ((vmask[a][h] >> tap) & 1u) ? __ldg(xb[a][h] + off) : 0u;
    };

    long blk = (long)blockIdx.x * (THREADS / 32) + warp;
    const uint32_t *xb[MA][2];
    uint32_t vmask[MA][2];
    uint32_t w[MA][2];
    if (blk < nblocks) {
        setup_rows(blk, xb, vmask);
        load_words(w, xb, vmask, 0, 0);
    }
    for (; blk < nblocks; blk += wstride) {
        const int mbase = (int)(blk * rows_per_iter);
        // the next block's rows are set up now so that its first words can be requested
        // before this block's epilogue (the whole flattened K sequence is software-pipelined)
        const long nblk = blk + wstride;
        const uint32_t *xbn[MA][2];
        uint32_t vmaskn[MA][2];
        if (nblk < nblocks) setup_rows(nblk, xbn, vmaskn);

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

        int tap = 0, cj = 0;           // tap and channel word of the K word being loaded (warp-uniform)
        for (int kw = 0; kw < p.kwords; ++kw) {
            uint32_t wn[MA][2];
            if (++cj == p.cw) { cj = 0; ++tap; }
            if (kw + 1 < p.kwords) load_words(wn, xb, vmask, tap, cj);
            else if (nblk < nblocks) load_words(wn, xbn, vmaskn, 0, 0);
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
#pragma unroll
        for (int a = 0; a < MA; ++a)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                xb[a][h] = xbn[a][h];
                vmask[a][h] = vmaskn[a][h];
            }

        // ---- epilogue.  acc[a][j][0,1] -> row g, columns 2q, 2q+1 of atom j;  [2,3] -> row g+8.
#pragma unroll
        for (int a = 0; a < MA; ++a)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int m = mbase + 16 * a + g + 8 * h;
                if (!FUSED) {
                    const int rowc = -2 * pa[a][h];
                    if (m < p.M) {
#pragma unroll
                        for (int gi = 0; gi < NA / 4; ++gi) {
                            const int n = n0 + 32 * gi + 8 * q;      // this thread's 8 consecutive channels
                            int v[8];
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj)
#pragma unroll
                                for (int e = 0; e < 2; ++e)
                                    v[2 * jj + e] = (acc[a][4 * gi + jj][2 * h + e] >> 5) + rowc + cc[4 * gi + jj][e];
                            int32_t *dst = static_cast<int32_t *>(p.out) + (long)m * p.C_out + n;
                            if ((p.C_out & 3) == 0 && n + 8 <= p.C_out) {
                                *reinterpret_cast<int4 *>(dst) = make_int4(v[0], v[1], v[2], v[3]);
                                *reinterpret_cast<int4 *>(dst + 4) = make_int4(v[4], v[5], v[6], v[7]);
                            } else {
#pragma unroll
                                for (int i = 0; i < 8; ++i)
                                    if (n + i < p.C_out) dst[i] = v[i];
                            }
                        }
                    }
                } else {
                    const int rowc = -64 * pa[a][h];
#pragma unroll
                    for (int gi = 0; gi < NA / 4; ++gi) {
                        // shift the sign bits of (acc + rowc + colc) in, highest channel first
                        uint32_t sb = 0;
#pragma unroll
                        for (int jj = 3; jj >= 0; --jj)
#pragma unroll
                            for (int e = 1; e >= 0; --e)
                                sb = __funnelshift_l((uint32_t)(acc[a][4 * gi + jj][2 * h + e] + rowc + cc[4 * gi + jj][e]), sb, 1);
                        uint32_t bits = (~sb & 0xffu) << (8 * q);
                        bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
                        bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
                        const int nword = (n0 >> 5) + gi;
                        if (q == 0 && m < p.M && nword < owords)
                            static_cast<uint32_t *>(p.out)[(long)m * owords + nword] = bits;
                    }
                }
            }
    }
}

size_t smem_bytes(const ConvProblem &p, int NA)
{
    return (size_t)p.kwords * NA * 32 * sizeof(uint2) + 8 * NA * sizeof(int) + (size_t)p.kh * p.kw * sizeof(int);
}

template <int NA>
int launch_na(const ConvProblem &p, cudaStream_t stream)
{
    const size_t smem = smem_bytes(p, NA);
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long nblocks = ((long)p.M + 16 * MA - 1) / (16 * MA);
    void (*k)(const ConvProblem) = p.thr ? conv_mma_s8_kernel<NA, true> : conv_mma_s8_kernel<NA, false>;
    // a property of the kernel, not of the launch: always the limit, so that captured launches stay valid
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM) != cudaSuccess) return BCNN_ERR_CUDA;
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
    if (p.kh * p.kw > 32) return false;     // one validity bit per tap in a 32-bit mask
    return smem_bytes(p, NA) <= (size_t)MAX_SMEM && p.K <= (1 << 20);
}

int launch_conv_mma_s8(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_mma_s8_supports(p)) return BCNN_ERR_UNSUPPORTED;
    if (p.C_out <= 32) return launch_na<4>(p, stream);
    return launch_na<8>(p, stream);
}

}  // namespace bcnn
