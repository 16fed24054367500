// Warp-level tensor-core engine of the binary implicit GEMM:
// mma.sync.m16n8k256 on single-bit operands with AND + popcount accumulation.
//
// With sign bits A (activations) and G (weights) of a K-bit row / column,
//   popcount(A xor G) = popcount(A) + popcount(G) - 2*popcount(A and G),
// so  sum a*g = K - 2*popcount(A) - 2*popcount(G) + 4*popcount(A and G).
// The tensor cores produce popcount(A and G); the row and column popcounts are taken
// from the same shared-memory tiles while they stream by.  Out-of-image taps and the
// K tail are zero words, which is both "value -1" and "adds nothing to any popcount".
//
// CTA tile 128 x BN (BN = 128, 64 or 32), 8 warps, K advances 512 bits per stage
// through a 4-stage cp.async pipeline.  Shared-memory rows are 64 bytes with the
// 16-byte chunks XOR-swizzled by (row >> 1) & 3 so that ldmatrix reads and the
// gathering cp.async writes are bank-conflict free.
#include "bcnn_common.cuh"

namespace bcnn {

namespace {

constexpr int BM = 128;
constexpr int STAGES = 4;
constexpr int ROW_BYTES = 64;                 // 512 bits of K per stage
constexpr int STAGE_WORDS = ROW_BYTES / 4;    // 16 words
constexpr int THREADS = 256;

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

template <int BYTES>
__device__ __forceinline__ void cp_async_zfill(uint32_t dst, const void *src, bool valid)
{
    const int n = valid ? BYTES : 0;
    if (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(n));
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;\n" ::"r"(dst), "l"(src), "n"(BYTES), "r"(n));
}

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

__device__ __forceinline__ void mma_b1_and(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc "
        "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// byte offset of 16-byte chunk `chunk` of row `row` inside a tile of 64-byte rows
__device__ __forceinline__ int swz(int row, int chunk)
{
    return row * ROW_BYTES + ((chunk ^ ((row >> 1) & 3)) << 4);
}

// GW = words per gather granule (1, 2 or 4): the largest power of two dividing C_in/32
// (capped at 4), so that a granule never straddles two taps.
template <int WN, int GW, bool FUSED>
__global__ void __launch_bounds__(THREADS)
conv_mma_b1_kernel(const ConvProblem p)
{
    constexpr int BN = 32 * WN;
    constexpr int WM = 8 / WN;
    constexpr int MI = BM / WM / 16;           // m16 atoms per warp
    constexpr int A_BYTES = BM * ROW_BYTES;
    constexpr int W_BYTES = BN * ROW_BYTES;
    constexpr int W_CHUNKS = BN * 4;

    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *As = smem;                          // STAGES x A_BYTES
    unsigned char *Ws = smem + STAGES * A_BYTES;       // STAGES x W_BYTES
    __shared__ int row_pop[BM];
    __shared__ int col_pop[BN];

    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int warp_m = warp / WN, warp_n = warp % WN;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;

    // ---- loader role: chunk (tid & 3) of rows (tid >> 2) and (tid >> 2) + 64
    const int lchunk = tid & 3, lrow = tid >> 2;
    RowCoord rc[2];
    bool row_ok[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int m = m0 + lrow + 64 * h;
        row_ok[h] = m < p.M;
        rc[h] = row_coord(p, row_ok[h] ? m : 0);
    }

    auto load_stage = [&](int kt, int slot) {
        const int kbase = kt * STAGE_WORDS + lchunk * 4;
        const uint32_t a_dst = smem_u32(As + slot * A_BYTES);
        const uint32_t w_dst = smem_u32(Ws + slot * W_BYTES);
#pragma unroll
        for (int g = 0; g < 4 / GW; ++g) {
            const int kword = kbase + g * GW;
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
                const int ih = rc[h].ih0 + r, iw = rc[h].iw0 + t;
                const bool ok = k_ok && row_ok[h] && ih >= 0 && ih < p.H && iw >= 0 && iw < p.W;
                const uint32_t *src = ok ? p.x + (((long)rc[h].b * p.H + ih) * p.W + iw) * p.cw + cj : p.x;
                cp_async_zfill<GW * 4>(a_dst + swz(lrow + 64 * h, lchunk) + g * GW * 4, src, ok);
            }
#pragma unroll
            for (int c = tid; c < W_CHUNKS; c += THREADS) {
                const int wrow = c >> 2;            // chunk index c & 3 == lchunk
                const int n = n0 + wrow;
                const bool ok = k_ok && n < p.C_out;
                const uint32_t *src = ok ? p.w + (long)n * p.kwords + kword : p.w;
                cp_async_zfill<GW * 4>(w_dst + swz(wrow, lchunk) + g * GW * 4, src, ok);
            }
        }
    };

    int acc[MI][4][4];
#pragma unroll
    for (int i = 0; i < MI; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[i][j][q] = 0;
    int my_pop = 0;   // popcount of row `tid` of A (tid < 128) or row `tid - 128` of W

    const int ktiles = (p.kwords + STAGE_WORDS - 1) / STAGE_WORDS;
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < ktiles) load_stage(s, s);
        cp_async_commit();
    }

    // ldmatrix lane roles
    const int lmat = lane >> 3, lr = lane & 7;
    const int a_row_in = lr + ((lmat & 1) << 3), a_chunk_in = lmat >> 1;   // A: rows 0-15, chunk pair
    const int b_row_in = lr + ((lmat >> 1) << 3), b_chunk_in = lmat & 1;   // W: two n8 atoms, chunk pair

    for (int kt = 0; kt < ktiles; ++kt) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        {
            const int nk = kt + STAGES - 1;
            if (nk < ktiles) load_stage(nk, nk % STAGES);
            cp_async_commit();
        }
        const int slot = kt % STAGES;
        const unsigned char *At = As + slot * A_BYTES;
        const unsigned char *Wt = Ws + slot * W_BYTES;

        // row / column popcounts from the tiles in flight
        {
            const unsigned char *tile = (tid < BM) ? At : Wt;
            const int row = (tid < BM) ? tid : tid - BM;
            if (tid < BM || row < BN) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 v = *reinterpret_cast<const uint4 *>(tile + swz(row, c));
                    my_pop += __popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w);
                }
            }
        }

        const uint32_t a_base = smem_u32(At), w_base = smem_u32(Wt);
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {       // two k256 steps per stage
            uint32_t bfrag[4][2];
#pragma unroll
            for (int jp = 0; jp < 2; ++jp) {
                const int row = warp_n * 32 + jp * 16 + b_row_in;
                ldmatrix_x4(w_base + swz(row, 2 * ks + b_chunk_in),
                            bfrag[2 * jp][0], bfrag[2 * jp][1], bfrag[2 * jp + 1][0], bfrag[2 * jp + 1][1]);
            }
#pragma unroll
            for (int i = 0; i < MI; ++i) {
                uint32_t afrag[4];
                const int row = warp_m * (MI * 16) + i * 16 + a_row_in;
                ldmatrix_x4(a_base + swz(row, 2 * ks + a_chunk_in), afrag[0], afrag[1], afrag[2], afrag[3]);
#pragma unroll
                for (int j = 0; j < 4; ++j) mma_b1_and(acc[i][j], afrag, bfrag[j][0], bfrag[j][1]);
            }
        }
    }
    cp_async_wait<0>();

    if (tid < BM) row_pop[tid] = my_pop;
    else if (tid - BM < BN) col_pop[tid - BM] = my_pop;
    __syncthreads();

    // ---- epilogue.  Fragment: c0,c1 -> row g, columns 2q,2q+1; c2,c3 -> row g+8.
    const int g = lane >> 2, q = lane & 3;
    if (!FUSED) {
        int32_t *out = static_cast<int32_t *>(p.out);
#pragma unroll
        for (int i = 0; i < MI; ++i)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int rloc = warp_m * (MI * 16) + i * 16 + g + 8 * hh;
                const int m = m0 + rloc;
                if (m >= p.M) continue;
                const int base = p.K - 2 * row_pop[rloc];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int cloc = warp_n * 32 + j * 8 + 2 * q;
                    const int n = n0 + cloc;
                    const int v0 = base - 2 * col_pop[cloc] + 4 * acc[i][j][2 * hh];
                    const int v1 = base - 2 * col_pop[cloc + 1] + 4 * acc[i][j][2 * hh + 1];
                    int32_t *dst = out + (long)m * p.C_out + n;
                    if (n + 1 < p.C_out && (p.C_out & 1) == 0) {
                        *reinterpret_cast<int2 *>(dst) = make_int2(v0, v1);
                    } else {
                        if (n < p.C_out) dst[0] = v0;
                        if (n + 1 < p.C_out) dst[1] = v1;
                    }
                }
            }
    } else {
        uint32_t *out = static_cast<uint32_t *>(p.out);
        const int owords = p.C_out >> 5;
        const int nword = (n0 >> 5) + warp_n;
        int thr[4][2], cp2[4][2];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int cloc = warp_n * 32 + j * 8 + 2 * q + e;
                const int n = n0 + cloc;
                thr[j][e] = (n < p.C_out) ? __ldg(p.thr + n) : 0;
                cp2[j][e] = 2 * col_pop[cloc];
            }
#pragma unroll
        for (int i = 0; i < MI; ++i)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int rloc = warp_m * (MI * 16) + i * 16 + g + 8 * hh;
                const int m = m0 + rloc;
                const int base = p.K - 2 * row_pop[rloc];
                uint32_t bits = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int v = base - cp2[j][e] + 4 * acc[i][j][2 * hh + e];
                        bits |= (v >= thr[j][e] ? 1u : 0u) << (j * 8 + 2 * q + e);
                    }
                bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
                bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
                if (q == 0 && m < p.M && nword < owords) out[(long)m * owords + nword] = bits;
            }
    }
}

template <int WN, int GW>
int launch_variant(const ConvProblem &p, cudaStream_t stream)
{
    constexpr int BN = 32 * WN;
    const int smem = STAGES * (BM + BN) * ROW_BYTES;
    dim3 grid((unsigned)(((long)p.M + BM - 1) / BM), (p.C_out + BN - 1) / BN);
    if (grid.y > 65535) return BCNN_ERR_UNSUPPORTED;
    cudaError_t e;
    if (p.thr) {
        auto k = conv_mma_b1_kernel<WN, GW, true>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return BCNN_ERR_CUDA;
        k<<<grid, THREADS, smem, stream>>>(p);
    } else {
        auto k = conv_mma_b1_kernel<WN, GW, false>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return BCNN_ERR_CUDA;
        k<<<grid, THREADS, smem, stream>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

template <int WN>
int launch_gw(const ConvProblem &p, cudaStream_t stream)
{
    if (p.cw % 4 == 0) return launch_variant<WN, 4>(p, stream);
    if (p.cw % 2 == 0) return launch_variant<WN, 2>(p, stream);
    return launch_variant<WN, 1>(p, stream);
}

}  // namespace

bool conv_mma_b1_supports(const ConvProblem &p)
{
    // the fused epilogue writes whole 32-channel words; the int32 one handles any C_out
    return p.thr == nullptr || (p.C_out % 32 == 0);
}

int launch_conv_mma_b1(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_mma_b1_supports(p)) return BCNN_ERR_UNSUPPORTED;
    if (p.C_out > 64) return launch_gw<4>(p, stream);
    if (p.C_out > 32) return launch_gw<2>(p, stream);
    return launch_gw<1>(p, stream);
}

}  // namespace bcnn
