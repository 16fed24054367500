// Fifth-generation tensor-core engine of the binary implicit GEMM (tcgen05, kind::i8).
//
// The tensor cores of sm_100a have no fast single-bit path, so sign bits are expanded
// to bytes on the fly, in shared memory, and fed to the dense 8-bit integer MMA with
// int32 accumulators in tensor memory.  Nothing expanded ever touches global memory.
//
// Expansion.  Inside every 32-bit group of K the byte at position 4*j + i carries input
// bit j + 8*i (the sum over K does not care about the order as long as both operands
// agree).  With that order one 32-bit word of bits w turns into its eight output words
// with one logic op each:   activations:  w & (0x01010101 << j)         -> byte 0 or 2^j
//                           weights:      shift(w) & (0x01010101 << 7-j) -> byte 0 or 2^(7-j)
// so every product of two set bits is exactly 128 and the accumulator holds
// 128 * popcount(A and G).  As in the warp-level engine,
//   sum a*g = K - 2*popcount(A) - 2*popcount(G) + 4*popcount(A and G),
// with the row / column popcounts taken from the words as they are expanded.  Zero
// words stand for out-of-image taps (value -1), for rows past M, columns past C_out
// and for the K tail.
//
// CTA = one 128 x BN output tile.  Warps 0-7 gather + expand (two threads per tile
// row and stage, 128 bits of K per stage) into a ring of 128-byte-swizzled K-major
// tiles; warp 8 issues the MMAs (one thread) and releases ring slots with
// tcgen05.commit; warps 0-7 then read the accumulators (tcgen05.ld), apply the
// epilogue and store int32 values or thresholded packed bits.
// Every mbarrier wait is bounded: on expiry the kernel records an error code in the
// device error word and all roles fall through to the common exit.
#include "bcnn_common.cuh"

namespace bcnn {

namespace {

constexpr int BM = 128;
constexpr int ROWB = 128;                 // bytes of one expanded tile row per stage (= 128 bits of K)
constexpr int PRODUCER_THREADS = 256;
constexpr int THREADS = PRODUCER_THREADS + 32;
constexpr uint32_t WAIT_LIMIT = 1u << 22; // polls before a wait gives up

constexpr int ERR_PRODUCER_TIMEOUT = 101;
constexpr int ERR_MMA_TIMEOUT = 102;
constexpr int ERR_EPILOGUE_TIMEOUT = 103;

template <int BN> struct Cfg {
    static constexpr int STAGES = (BN == 256) ? 4 : (BN == 128 ? 6 : 6);
    static constexpr int A_BYTES = BM * ROWB;
    static constexpr int W_BYTES = BN * ROWB;
    static constexpr int STAGE_BYTES = A_BYTES + W_BYTES;
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024;   // + slack to align the ring to 1024 bytes
};

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err, int code)
{
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    if (err) atomicCAS(err, 0, code);
    return false;
}

__device__ __forceinline__ void fence_async_proxy()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, 8-bit integer operands, int32 accumulators.
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile with 128-byte rows and the 128-byte
// swizzle: 8-row groups are 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr)
{
    const uint32_t lo = ((saddr & 0x3FFFFu) >> 4) | (1u << 16);
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    return (static_cast<uint64_t>(hi) << 32) | lo;
}

// Instruction descriptor: unsigned 8-bit A and B (K-major), int32 accumulate, M = 128, N = BN.
template <int BN>
__device__ __forceinline__ constexpr uint32_t make_idesc()
{
    return (2u << 4) | (0u << 7) | (0u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

// physical byte offset of 16-byte chunk `c` of tile row `row`
__device__ __forceinline__ uint32_t swz(int row, int c) { return (uint32_t)row * ROWB + (uint32_t)((c ^ (row & 7)) << 4); }

// One word of activation bits -> two 16-byte chunks (bytes 0 or 2^j).
__device__ __forceinline__ void expand_a(uint32_t w, uint4 &c0, uint4 &c1)
{
    c0.x = w & 0x01010101u; c0.y = w & 0x02020202u; c0.z = w & 0x04040404u; c0.w = w & 0x08080808u;
    c1.x = w & 0x10101010u; c1.y = w & 0x20202020u; c1.z = w & 0x40404040u; c1.w = w & 0x80808080u;
}

// One word of weight bits -> two 16-byte chunks (bytes 0 or 2^(7-j)).
__device__ __forceinline__ void expand_w(uint32_t w, uint4 &c0, uint4 &c1)
{
    c0.x = (w << 7) & 0x80808080u; c0.y = (w << 5) & 0x40404040u; c0.z = (w << 3) & 0x20202020u; c0.w = (w << 1) & 0x10101010u;
    c1.x = (w >> 1) & 0x08080808u; c1.y = (w >> 3) & 0x04040404u; c1.z = (w >> 5) & 0x02020202u; c1.w = (w >> 7) & 0x01010101u;
}

template <int BN, bool FUSED>
__global__ void __launch_bounds__(THREADS, 1)
conv_tc_i8_kernel(const ConvProblem p)
{
    using C = Cfg<BN>;
    constexpr int STAGES = C::STAGES;
    constexpr int WP = BN / 128 > 0 ? BN / 128 : 1;   // weight passes of 128 rows (BN = 64: half the threads idle)

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * STAGES + 1];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;
    __shared__ int row_pop[BM];
    __shared__ int col_pop[BN];
    __shared__ int thr_s[BN];

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int ktiles = (p.kwords + 3) >> 2;

    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    const uint32_t accum_bar = bar0 + 8u * (2 * STAGES);
    volatile int *abort_flag = &abort_flag_smem;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), PRODUCER_THREADS);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(accum_bar, 1);
        abort_flag_smem = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"((uint32_t)BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (FUSED) {
        for (int i = tid; i < BN; i += THREADS) thr_s[i] = (n0 + i < p.C_out) ? __ldg(p.thr + n0 + i) : 0;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;

    if (warp < 8) {
        // ------------------------------------------------------------------ producers
        const int row = tid >> 1, half = tid & 1;
        const int m = m0 + row;
        const bool row_ok = m < p.M;
        const RowCoord rc = row_coord(p, row_ok ? m : 0);
        const uint32_t *xrow = p.x + (long)rc.b * p.H * p.W * p.cw;

        auto load_a = [&](int kt, uint32_t (&a)[2]) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int kword = kt * 4 + half * 2 + e;
                uint32_t v = 0;
                if (row_ok && kword < p.kwords) {
                    const int tap = fast_div(kword, p.cw_magic);
                    const int cj = kword - tap * p.cw;
                    const int r = fast_div(tap, p.kw_magic);
                    const int t = tap - r * p.kw;
                    const int ih = rc.ih0 + r, iw = rc.iw0 + t;
                    if (ih >= 0 && ih < p.H && iw >= 0 && iw < p.W)
                        v = __ldg(xrow + ((long)ih * p.W + iw) * p.cw + cj);
                }
                a[e] = v;
            }
        };
        auto load_w = [&](int kt, uint32_t (&w)[WP][2]) {
#pragma unroll
            for (int q = 0; q < WP; ++q) {
                const int wrow = q * 128 + row;
                const int n = n0 + wrow;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int kword = kt * 4 + half * 2 + e;
                    uint32_t v = 0;
                    if (wrow < BN && n < p.C_out && kword < p.kwords) v = __ldg(p.w + (long)n * p.kwords + kword);
                    w[q][e] = v;
                }
            }
        };

        uint32_t a_cur[2], w_cur[WP][2];
        int a_pop = 0, w_pop[WP];
#pragma unroll
        for (int q = 0; q < WP; ++q) w_pop[q] = 0;
        load_a(0, a_cur);
        load_w(0, w_cur);
        bool alive = true;
        for (int kt = 0; kt < ktiles && alive; ++kt) {
            const int s = kt % STAGES;
            uint32_t a_nxt[2], w_nxt[WP][2];
            if (kt + 1 < ktiles) {
                load_a(kt + 1, a_nxt);
                load_w(kt + 1, w_nxt);
            }
            alive = mbar_wait(empty_bar(s), ((kt / STAGES) & 1) ^ 1, abort_flag, p.err, ERR_PRODUCER_TIMEOUT);
            if (!alive) break;
            const uint32_t a_tile = ring + (uint32_t)s * C::STAGE_BYTES;
            const uint32_t w_tile = a_tile + C::A_BYTES;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                uint4 c0, c1;
                expand_a(a_cur[e], c0, c1);
                a_pop += __popc(a_cur[e]);
                const int c = half * 4 + e * 2;
                asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a_tile + swz(row, c)), "r"(c0.x), "r"(c0.y), "r"(c0.z), "r"(c0.w) : "memory");
                asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a_tile + swz(row, c + 1)), "r"(c1.x), "r"(c1.y), "r"(c1.z), "r"(c1.w) : "memory");
            }
#pragma unroll
            for (int q = 0; q < WP; ++q) {
                const int wrow = q * 128 + row;
                if (wrow < BN) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        uint4 c0, c1;
                        expand_w(w_cur[q][e], c0, c1);
                        w_pop[q] += __popc(w_cur[q][e]);
                        const int c = half * 4 + e * 2;
                        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(w_tile + swz(wrow, c)), "r"(c0.x), "r"(c0.y), "r"(c0.z), "r"(c0.w) : "memory");
                        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(w_tile + swz(wrow, c + 1)), "r"(c1.x), "r"(c1.y), "r"(c1.z), "r"(c1.w) : "memory");
                    }
                }
            }
            fence_async_proxy();
            mbar_arrive(full_bar(s));
            if (kt + 1 < ktiles) {
#pragma unroll
                for (int e = 0; e < 2; ++e) a_cur[e] = a_nxt[e];
#pragma unroll
                for (int q = 0; q < WP; ++q)
#pragma unroll
                    for (int e = 0; e < 2; ++e) w_cur[q][e] = w_nxt[q][e];
            }
        }

        // row / column popcounts: the two halves of a row sit in neighbouring lanes
        a_pop += __shfl_xor_sync(0xffffffffu, a_pop, 1);
        if (half == 0) row_pop[row] = a_pop;
#pragma unroll
        for (int q = 0; q < WP; ++q) {
            int v = w_pop[q];
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            const int wrow = q * 128 + row;
            if (half == 0 && wrow < BN) col_pop[wrow] = v;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");

        // ------------------------------------------------------------------ epilogue
        // (tcgen05.ld is warp-collective: keep the go / no-go decision warp-uniform)
        if (alive) alive = mbar_wait(accum_bar, 0, abort_flag, p.err, ERR_EPILOGUE_TIMEOUT);
        alive = __all_sync(0xffffffffu, alive && !*abort_flag);
        if (alive) {
            tc_fence_after();
            const int quad = warp & 3, colhalf = warp >> 2;
            const int erow = quad * 32 + lane;
            const int em = m0 + erow;
            const int base = p.K - 2 * row_pop[erow];
            constexpr int CH = BN / 2 / 32;      // 32-column chunks per warp
#pragma unroll 1
            for (int ch = 0; ch < CH; ++ch) {
                const int col0 = colhalf * (BN / 2) + ch * 32;
                if (n0 + col0 >= p.C_out) break;           // warp-uniform
                uint32_t v[32];
                tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)col0, v);
                if (!FUSED) {
                    int32_t *dst = static_cast<int32_t *>(p.out) + (long)em * p.C_out + n0 + col0;
                    const bool vec = (p.C_out & 3) == 0 && (n0 + col0 + 32 <= p.C_out);
                    if (em < p.M) {
                        if (vec) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4) {
                                int4 o;
                                o.x = base - 2 * col_pop[col0 + i] + (int)(v[i] >> 5);
                                o.y = base - 2 * col_pop[col0 + i + 1] + (int)(v[i + 1] >> 5);
                                o.z = base - 2 * col_pop[col0 + i + 2] + (int)(v[i + 2] >> 5);
                                o.w = base - 2 * col_pop[col0 + i + 3] + (int)(v[i + 3] >> 5);
                                *reinterpret_cast<int4 *>(dst + i) = o;
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (n0 + col0 + i < p.C_out) dst[i] = base - 2 * col_pop[col0 + i] + (int)(v[i] >> 5);
                        }
                    }
                } else {
                    uint32_t word = 0;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int val = base - 2 * col_pop[col0 + i] + (int)(v[i] >> 5);
                        word |= (val >= thr_s[col0 + i] ? 1u : 0u) << i;
                    }
                    if (em < p.M)
                        static_cast<uint32_t *>(p.out)[(long)em * (p.C_out >> 5) + ((n0 + col0) >> 5)] = word;
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc<BN>();
            bool alive = true;
            for (int kt = 0; kt < ktiles; ++kt) {
                const int s = kt % STAGES;
                alive = mbar_wait(full_bar(s), (kt / STAGES) & 1, abort_flag, p.err, ERR_MMA_TIMEOUT);
                if (!alive) break;
                tc_fence_after();
                const uint32_t a_tile = ring + (uint32_t)s * C::STAGE_BYTES;
                const uint64_t a_desc = make_desc(a_tile);
                const uint64_t b_desc = make_desc(a_tile + C::A_BYTES);
#pragma unroll
                for (int k = 0; k < 4; ++k)   // 32 bytes of K per instruction: +2 in 16-byte address units
                    tc_mma_i8(tmem_base, a_desc + 2u * k, b_desc + 2u * k, idesc, (kt > 0 || k > 0) ? 1u : 0u);
                tc_commit(empty_bar(s));
            }
            if (alive) tc_commit(accum_bar);
        }
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)BN) : "memory");
    }
}

template <int BN>
int launch_bn(const ConvProblem &p0, cudaStream_t stream)
{
    ConvProblem p = p0;
    p.err = device_error_word();
    dim3 grid((p.M + BM - 1) / BM, (p.C_out + BN - 1) / BN);
    if (grid.y > 65535) return BCNN_ERR_UNSUPPORTED;
    const int smem = Cfg<BN>::SMEM;
    cudaError_t e;
    if (p.thr) {
        auto k = conv_tc_i8_kernel<BN, true>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return BCNN_ERR_CUDA;
        k<<<grid, THREADS, smem, stream>>>(p);
    } else {
        auto k = conv_tc_i8_kernel<BN, false>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return BCNN_ERR_CUDA;
        k<<<grid, THREADS, smem, stream>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace

bool conv_tc_i8_supports(const ConvProblem &p)
{
    if (p.thr != nullptr && (p.C_out % 32 != 0)) return false;
    // the multiplier-based divisions need kword * cw < 2^32 and the accumulator 128 * K < 2^31
    return p.K <= (1 << 20);
}

int launch_conv_tc_i8(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_tc_i8_supports(p)) return BCNN_ERR_UNSUPPORTED;
    if (p.C_out > 128) return launch_bn<256>(p, stream);
    if (p.C_out > 64) return launch_bn<128>(p, stream);
    return launch_bn<64>(p, stream);
}

}  // namespace bcnn
