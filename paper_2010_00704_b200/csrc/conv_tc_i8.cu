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
// 128 * popcount(A and G).  With the row / column popcounts,
//   sum a*g = K - 2*popcount(A) - 2*popcount(G) + 4*popcount(A and G),
// the popcounts being taken from the words as they are expanded.  Zero words stand for
// out-of-image taps (value -1), for rows past M, columns past C_out and for the K tail.
//
// Persistent, warp-specialised kernel; each CTA walks a static list of 128 x BN tiles.
//   warp 0        : issues the MMAs (one thread), releases ring slots with tcgen05.commit
//   warps 1-4     : epilogue - read an accumulator buffer (tcgen05.ld), threshold / pack or
//                   write int32, hand the buffer back; overlaps the next tile's main loop
//                   because the accumulators are double-buffered in tensor memory
//   warps 5...    : producers, one thread per tile row (128 activation rows + BN weight
//                   rows).  Packed words are staged ahead with cp.async (16 bytes per row
//                   and stage, zero-filled when out of range), then expanded into a ring of
//                   128-byte-swizzled K-major tiles, 128 bits of K per stage.
// Every mbarrier wait is bounded: on expiry the kernel records an error code in the
// device error word and all roles fall through to the common exit.
#include "bcnn_common.cuh"

namespace bcnn {

namespace {

constexpr int BM = 128;
constexpr int ROWB = 128;                 // bytes of one expanded tile row per stage (= 128 bits of K)
constexpr int EPI_WARPS = 4;
constexpr int FIRST_PRODUCER_THREAD = 32 * (1 + EPI_WARPS);
constexpr uint32_t WAIT_LIMIT = 1u << 17;
// upper bound (ns) for which one try_wait may suspend the thread: waiting warps then leave
// the issue slots to the warps that have work; the wake-up on phase completion is immediate
constexpr uint32_t SUSPEND_HINT_NS = 20000;

constexpr int ERR_PRODUCER_TIMEOUT = 101;
constexpr int ERR_MMA_TIMEOUT = 102;
constexpr int ERR_EPILOGUE_TIMEOUT = 103;

template <int BN> struct Cfg {
    static constexpr int PROD_THREADS = BM + BN;
    static constexpr int THREADS = FIRST_PRODUCER_THREAD + PROD_THREADS;
    static constexpr int STAGES = BN == 256 ? 4 : (BN == 128 ? 6 : 8);
    static constexpr int A_BYTES = BM * ROWB;
    static constexpr int STAGE_BYTES = (BM + BN) * ROWB;
    static constexpr int SLOTS = STAGES + 3;             // per-tile constant slots: producers run at most STAGES
                                                         // tiles ahead of the MMAs, the MMAs two tiles ahead of the epilogue
    static constexpr int PF = BN == 256 ? 3 : 4;         // stages of packed words in flight per producer thread
    static constexpr int BITS_BYTES = PF * PROD_THREADS * 16;
    static constexpr int CONST_BYTES = SLOTS * (BM + BN) * 4;
    static constexpr int SMEM = 1024 + STAGES * STAGE_BYTES + BITS_BYTES + CONST_BYTES;
    static constexpr int TMEM_COLS = 2 * BN;             // two accumulator buffers
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
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(SUSPEND_HINT_NS) : "memory");
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

__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
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

// 32 accumulator columns of this warp's 32 rows.  The load and its completion wait are one asm
// statement so that no use of the destination registers can be scheduled between them.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
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

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    const int n = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}

__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src, bool valid)
{
    const int n = valid ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// One word of activation bits -> two 16-byte chunks (bytes 0 or 2^j), stored to chunks c, c+1 of a row.
__device__ __forceinline__ void expand_store_a(uint32_t w, uint32_t row_addr, int xr, int c)
{
    st_shared_v4(row_addr + (uint32_t)(((c) ^ xr) << 4),
                 w & 0x01010101u, w & 0x02020202u, w & 0x04040404u, w & 0x08080808u);
    st_shared_v4(row_addr + (uint32_t)(((c + 1) ^ xr) << 4),
                 w & 0x10101010u, w & 0x20202020u, w & 0x40404040u, w & 0x80808080u);
}

// One word of weight bits -> two 16-byte chunks (bytes 0 or 2^(7-j)).
__device__ __forceinline__ void expand_store_w(uint32_t w, uint32_t row_addr, int xr, int c)
{
    st_shared_v4(row_addr + (uint32_t)(((c) ^ xr) << 4),
                 (w << 7) & 0x80808080u, (w << 5) & 0x40404040u, (w << 3) & 0x20202020u, (w << 1) & 0x10101010u);
    st_shared_v4(row_addr + (uint32_t)(((c + 1) ^ xr) << 4),
                 (w >> 1) & 0x08080808u, (w >> 3) & 0x04040404u, (w >> 5) & 0x02020202u, (w >> 7) & 0x01010101u);
}

template <int BN, bool FUSED>
__global__ void __launch_bounds__(Cfg<BN>::THREADS, 1)
conv_tc_i8_kernel(const ConvProblem p)
{
    using C = Cfg<BN>;
    constexpr int STAGES = C::STAGES;
    constexpr int SLOTS = C::SLOTS;
    constexpr int PT = C::PROD_THREADS;
    constexpr int PF = C::PF;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * STAGES + 4];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int ktiles = (p.kwords + 3) >> 2;
    const int m_tiles = (p.M + BM - 1) / BM;
    const int n_tiles = (p.C_out + BN - 1) / BN;
    const int total_tiles = m_tiles * n_tiles;
    const int my_tiles = ((int)blockIdx.x < total_tiles) ? (total_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bits_ring = ring + STAGES * C::STAGE_BYTES;
    const uint32_t consts = bits_ring + C::BITS_BYTES;        // [SLOTS][BM + BN] int32
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
    volatile int *abort_flag = &abort_flag_smem;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), PT / 32);      // one arrival per producer warp
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), EPI_WARPS);
        }
        abort_flag_smem = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"((uint32_t)C::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;

    if (warp == 0) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc<BN>();
            int s = 0;
            uint32_t ring_phase = 0;
            bool alive = true;
            for (int ti = 0; ti < my_tiles && alive; ++ti) {
                const int buf = ti & 1;
                alive = mbar_wait(tempty_bar(buf), ((ti >> 1) & 1) ^ 1, abort_flag, p.err, ERR_MMA_TIMEOUT);
                if (!alive) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kt = 0; kt < ktiles; ++kt) {
                    alive = mbar_wait(full_bar(s), ring_phase, abort_flag, p.err, ERR_MMA_TIMEOUT);
                    if (!alive) break;
                    tc_fence_after();
                    const uint32_t a_tile = ring + (uint32_t)s * C::STAGE_BYTES;
                    const uint64_t a_desc = make_desc(a_tile);
                    const uint64_t b_desc = make_desc(a_tile + C::A_BYTES);
#pragma unroll
                    for (int k = 0; k < 4; ++k)   // 32 bytes of K per instruction: +2 in 16-byte address units
                        tc_mma_i8(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kt > 0 || k > 0) ? 1u : 0u);
                    tc_commit(empty_bar(s));
                    if (++s == STAGES) { s = 0; ring_phase ^= 1u; }
                }
                if (alive) tc_commit(tfull_bar(buf));
            }
        }
        __syncwarp();
    } else if (warp <= EPI_WARPS) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;                 // tensor-memory lane quadrant this warp may read
        const int erow = quad * 32 + lane;
        bool alive = true;
        for (int ti = 0; ti < my_tiles; ++ti) {
            const int tile = (int)blockIdx.x + ti * (int)gridDim.x;
            const int n_tile = tile / m_tiles, m_tile = tile - n_tile * m_tiles;
            const int m0 = m_tile * BM, n0 = n_tile * BN;
            const int buf = ti & 1;
            const uint32_t slot = consts + (uint32_t)((ti % SLOTS) * (BM + BN) * 4);
            if (alive) alive = mbar_wait(tfull_bar(buf), (ti >> 1) & 1, abort_flag, p.err, ERR_EPILOGUE_TIMEOUT);
            alive = __all_sync(0xffffffffu, alive && !*abort_flag);
            if (!alive) break;
            tc_fence_after();
            const int em = m0 + erow;
            int rowc;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(rowc) : "r"(slot + 4u * erow) : "memory");
            const uint32_t colc_addr = slot + 4u * BM;
            const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BN);
            uint32_t words[BN / 32];
#pragma unroll
            for (int ch = 0; ch < BN / 32; ++ch) {
                const int col0 = ch * 32;
                words[ch] = 0;
                if (n0 + col0 < p.C_out) {             // warp-uniform
                    uint32_t v[32];
                    tc_ld32(t_addr + (uint32_t)col0, v);
                    if (FUSED) {
                        // bit = (v + rowc + colc >= 0); sign bits are shifted in last column first
                        uint32_t acc = 0;
#pragma unroll
                        for (int i4 = 7; i4 >= 0; --i4) {
                            const uint4 cc = ld_shared_v4(colc_addr + 4u * (col0 + 4 * i4));
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 3] + rowc + (int)cc.w), acc, 1);
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 2] + rowc + (int)cc.z), acc, 1);
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 1] + rowc + (int)cc.y), acc, 1);
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 0] + rowc + (int)cc.x), acc, 1);
                        }
                        words[ch] = ~acc;
                    } else if (em < p.M) {
                        int32_t *dst = static_cast<int32_t *>(p.out) + (long)em * p.C_out + n0 + col0;
                        const bool vec = (p.C_out & 3) == 0 && (n0 + col0 + 32 <= p.C_out);
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            const uint4 cc = ld_shared_v4(colc_addr + 4u * (col0 + 4 * i4));
                            int4 o;
                            o.x = (int)(v[4 * i4 + 0] >> 5) + rowc + (int)cc.x;
                            o.y = (int)(v[4 * i4 + 1] >> 5) + rowc + (int)cc.y;
                            o.z = (int)(v[4 * i4 + 2] >> 5) + rowc + (int)cc.z;
                            o.w = (int)(v[4 * i4 + 3] >> 5) + rowc + (int)cc.w;
                            if (vec) {
                                *reinterpret_cast<int4 *>(dst + 4 * i4) = o;
                            } else {
                                const int n = n0 + col0 + 4 * i4;
                                if (n < p.C_out) dst[4 * i4] = o.x;
                                if (n + 1 < p.C_out) dst[4 * i4 + 1] = o.y;
                                if (n + 2 < p.C_out) dst[4 * i4 + 2] = o.z;
                                if (n + 3 < p.C_out) dst[4 * i4 + 3] = o.w;
                            }
                        }
                    }
                }
            }
            // all reads of this accumulator buffer are complete: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
            if (FUSED && em < p.M) {
                const int owords = p.C_out >> 5;
                uint32_t *dst = static_cast<uint32_t *>(p.out) + (long)em * owords + (n0 >> 5);
                if (BN >= 128 && (owords & 3) == 0 && n0 + BN <= p.C_out) {
#pragma unroll
                    for (int c4 = 0; c4 < BN / 128; ++c4)
                        *reinterpret_cast<uint4 *>(dst + 4 * c4) =
                            make_uint4(words[4 * c4], words[4 * c4 + 1], words[4 * c4 + 2], words[4 * c4 + 3]);
                } else {
#pragma unroll
                    for (int ch = 0; ch < BN / 32; ++ch)
                        if (n0 + ch * 32 < p.C_out) dst[ch] = words[ch];
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ producers
        const int ptid = tid - FIRST_PRODUCER_THREAD;
        const bool is_a = ptid < BM;
        const int row = is_a ? ptid : ptid - BM;                 // row inside the A or the W tile
        const int xr = row & 7;                                  // swizzle term of this row
        const uint32_t row_off = (is_a ? 0u : (uint32_t)C::A_BYTES) + (uint32_t)row * ROWB;
        const uint32_t my_bits = bits_ring + (uint32_t)ptid * 16u;
        const bool a16 = (p.cw & 3) == 0;                        // a stage never straddles two taps
        const bool w16 = (p.kwords & 3) == 0;
        const int total_items = my_tiles * ktiles;

        // ---- load cursor (runs PF - 1 items ahead of the expand cursor)
        int l_ti = 0, l_kt = 0, l_r = 0, l_t = 0, l_cj = 0, l_slot = 0;
        bool l_ok = false;
        const uint32_t *l_base = p.x;
        int l_ih0 = 0, l_iw0 = 0;
        auto l_new_tile = [&]() {
            const int tile = (int)blockIdx.x + l_ti * (int)gridDim.x;
            const int n_tile = tile / m_tiles, m_tile = tile - n_tile * m_tiles;
            if (is_a) {
                const int m = m_tile * BM + row;
                l_ok = m < p.M;
                const RowCoord rc = row_coord(p, l_ok ? m : 0);
                l_base = p.x + (long)rc.b * p.H * p.W * p.cw;
                l_ih0 = rc.ih0;
                l_iw0 = rc.iw0;
            } else {
                const int n = n_tile * BN + row;
                l_ok = n < p.C_out;
                l_base = p.w + (long)(l_ok ? n : 0) * p.kwords;
            }
            l_kt = 0; l_r = 0; l_t = 0; l_cj = 0;
        };
        auto issue_load = [&]() {
            const uint32_t dst = my_bits + (uint32_t)l_slot * (PT * 16u);
            if (is_a) {
                if (a16) {
                    const int ih = l_ih0 + l_r, iw = l_iw0 + l_t;
                    const bool ok = l_ok && ih >= 0 && ih < p.H && iw >= 0 && iw < p.W;
                    cp_async16(dst, ok ? l_base + ((long)ih * p.W + iw) * p.cw + l_cj : p.x, ok);
                    l_cj += 4;
                    if (l_cj == p.cw) {
                        l_cj = 0;
                        if (++l_t == p.kw) { l_t = 0; ++l_r; }
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int kword = l_kt * 4 + e;
                        bool ok = l_ok && kword < p.kwords;
                        const uint32_t *src = p.x;
                        if (ok) {
                            const int tap = fast_div(kword, p.cw_magic);
                            const int cj = kword - tap * p.cw;
                            const int r = fast_div(tap, p.kw_magic);
                            const int t = tap - r * p.kw;
                            const int ih = l_ih0 + r, iw = l_iw0 + t;
                            ok = ih >= 0 && ih < p.H && iw >= 0 && iw < p.W;
                            if (ok) src = l_base + ((long)ih * p.W + iw) * p.cw + cj;
                        }
                        cp_async4(dst + 4u * e, src, ok);
                    }
                }
            } else {
                if (w16) {
                    cp_async16(dst, l_ok ? l_base + l_kt * 4 : p.w, l_ok);
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int kword = l_kt * 4 + e;
                        const bool ok = l_ok && kword < p.kwords;
                        cp_async4(dst + 4u * e, ok ? l_base + kword : p.w, ok);
                    }
                }
            }
            if (++l_kt == ktiles) {
                ++l_ti;
                if (l_ti < my_tiles) l_new_tile();
            }
            if (++l_slot == PF) l_slot = 0;
        };

        if (my_tiles > 0) l_new_tile();
        int issued = 0;
#pragma unroll 1
        for (; issued < PF - 1; ++issued) {
            if (issued < total_items) issue_load();
            cp_async_commit();
        }

        // ---- expand cursor
        int s = 0, c_slot = 0, c_kt = 0, c_ti = 0, pop = 0;
        uint32_t ring_phase = 1;             // first pass through the ring: slots are free
        int thr_n = 0;
        bool n_ok = false;
        auto c_new_tile = [&]() {
            if (!is_a) {
                const int tile = (int)blockIdx.x + c_ti * (int)gridDim.x;
                const int n = (tile / m_tiles) * BN + row;
                n_ok = n < p.C_out;
                thr_n = (FUSED && n_ok) ? __ldg(p.thr + n) : 0;
            }
        };
        if (my_tiles > 0) c_new_tile();
        bool alive = true;
        for (int it = 0; it < total_items; ++it) {
            if (issued < total_items) issue_load();
            ++issued;
            cp_async_commit();
            cp_async_wait<PF - 1>();
            const uint4 bits = ld_shared_v4(my_bits + (uint32_t)c_slot * (PT * 16u));
            if (++c_slot == PF) c_slot = 0;
            alive = mbar_wait(empty_bar(s), ring_phase, abort_flag, p.err, ERR_PRODUCER_TIMEOUT);
            alive = __all_sync(0xffffffffu, alive);
            if (!alive) break;
            const uint32_t row_addr = ring + (uint32_t)s * C::STAGE_BYTES + row_off;
            if (is_a) {
                expand_store_a(bits.x, row_addr, xr, 0);
                expand_store_a(bits.y, row_addr, xr, 2);
                expand_store_a(bits.z, row_addr, xr, 4);
                expand_store_a(bits.w, row_addr, xr, 6);
            } else {
                expand_store_w(bits.x, row_addr, xr, 0);
                expand_store_w(bits.y, row_addr, xr, 2);
                expand_store_w(bits.z, row_addr, xr, 4);
                expand_store_w(bits.w, row_addr, xr, 6);
            }
            pop += __popc(bits.x) + __popc(bits.y) + __popc(bits.z) + __popc(bits.w);
            if (++c_kt == ktiles) {
                // per-tile constants of this row / column, read by the epilogue of this tile
                int cst;
                if (is_a) cst = FUSED ? -64 * pop : -2 * pop;
                else      cst = FUSED ? -32 * (thr_n - p.K + 2 * pop) : p.K - 2 * pop;
                const uint32_t slot = consts + (uint32_t)((c_ti % SLOTS) * (BM + BN) * 4);
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(slot + 4u * ptid), "r"(cst) : "memory");
                pop = 0;
                c_kt = 0;
                ++c_ti;
                if (c_ti < my_tiles) c_new_tile();
            }
            fence_async_proxy();          // make this thread's generic-proxy stores visible to the MMA (async proxy)
            __syncwarp();
            if (lane == 0) mbar_arrive(full_bar(s));
            if (++s == STAGES) { s = 0; ring_phase ^= 1u; }
        }
        cp_async_wait<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
    }
}

template <int BN>
int launch_bn(const ConvProblem &p0, cudaStream_t stream)
{
    ConvProblem p = p0;
    p.err = device_error_word();
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long m_tiles = ((long)p.M + BM - 1) / BM;
    const long n_tiles = ((long)p.C_out + BN - 1) / BN;
    const long total = m_tiles * n_tiles;
    if (total >= (1L << 31)) return BCNN_ERR_UNSUPPORTED;
    const unsigned grid = (unsigned)(total < sms ? total : sms);
    const int smem = Cfg<BN>::SMEM;
    cudaError_t e;
    if (p.thr) {
        auto k = conv_tc_i8_kernel<BN, true>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return BCNN_ERR_CUDA;
        k<<<grid, Cfg<BN>::THREADS, smem, stream>>>(p);
    } else {
        auto k = conv_tc_i8_kernel<BN, false>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return BCNN_ERR_CUDA;
        k<<<grid, Cfg<BN>::THREADS, smem, stream>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace

bool conv_tc_i8_supports(const ConvProblem &p)
{
    if (p.thr != nullptr && (p.C_out % 32 != 0)) return false;
    // the multiplier-based divisions need kword * cw < 2^32 and the epilogue constants (3K << 5) < 2^31
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
