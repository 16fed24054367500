// Weight-stationary variant of the tcgen05 engine for layers with few output channels and a
// short K (C_out <= 128 and the expanded weights fit in shared memory).
//
// Same arithmetic as conv_tc_i8.cu: sign bits are expanded to bytes on chip (activations to
// {0, 2^j}, weights to {0, 2^(7-j)}, byte 4j+i of a 32-bit group carrying bit j+8i), every
// product of two set bits is 128, accumulators are int32 in tensor memory and
//   sum a*g = K - 2*popc(A) - 2*popc(G) + 4*popc(A and G).
// Differences, all aimed at short tiles (a 128 x 32 x 32 tile is one MMA instruction):
//   * the CTA expands its weight tile ONCE into shared memory and keeps it for all its
//     output tiles; only activations stream through the ring;
//   * the activation ring lives in TENSOR memory, not shared memory: producers write expanded rows
//     with tcgen05.st and the MMA takes its A operand from tensor memory.  A narrow MMA is bound by
//     operand fetch from shared memory (128 x 32 bytes of A per instruction whatever N is); with A in
//     tensor memory only the small weight slice is fetched;
//   * one extra all-ones weight row is appended, so column BN of every accumulator holds
//     128 * popc(A) for its row: the epilogue reads the row popcount from tensor memory and
//     no per-tile constants travel through shared memory;
//   * G producer groups of 128 threads take the ring's stages round-robin, so that G stages
//     are being gathered / expanded at any time (one thread's stage latency is several
//     hundred cycles, an MMA stage as little as 64);
//   * up to four accumulator buffers, so the epilogue of one tile overlaps the MMAs of the next ones;
//   * the warp that issues the MMAs waits only on named barriers; a separate control warp does the
//     mbarrier waits for it (a memory instruction after tensor-core instructions stalls the issuer);
//   * the implicit-im2col gather uses a per-K-word table (tap, word offset) and a per-row
//     tap-validity mask instead of divisions; out-of-image taps are zero-filled by cp.async.
// Every mbarrier wait is bounded and reports through the device error word.
#include "bcnn_common.cuh"

namespace bcnn {

namespace {

constexpr int BM = 128;
constexpr int ROWB = 128;                 // bytes of one expanded row per stage (= 128 bits of K)
constexpr int EPI_WARPS = 4;
constexpr int FIRST_PRODUCER_THREAD = 32 * (1 + EPI_WARPS);
constexpr int PF = 3;                     // packed-word stages in flight per producer thread
constexpr int MAX_SMEM = 227 * 1024;
constexpr uint32_t WAIT_LIMIT = 1u << 17;
// upper bound (ns) for which one try_wait may suspend the thread: waiting warps then leave
// the issue slots to the warps that have work; the wake-up on phase completion is immediate
constexpr uint32_t SUSPEND_HINT_NS = 20000;
constexpr uint32_t SLEEP_NS = 100;

constexpr int ERR_PRODUCER_TIMEOUT = 111;
constexpr int ERR_MMA_TIMEOUT = 112;
constexpr int ERR_EPILOGUE_TIMEOUT = 113;

// DUAL: two CTAs share an SM (two independent MMA issuers), each with half of tensor memory.
template <int BN, int G, bool DUAL> struct Cfg {
    static constexpr int BNX = BN + 16;                       // + the all-ones row (MMA N is a multiple of 16)
    static constexpr int PROD_THREADS = G * BM;
    static constexpr int CONTROL_WARP = (FIRST_PRODUCER_THREAD + PROD_THREADS) / 32;   // last warp
    static constexpr int THREADS = FIRST_PRODUCER_THREAD + PROD_THREADS + 32;
    // Tensor memory (512 columns): NBUF accumulator buffers of BNX columns, then the activation ring,
    // one stage = 128 rows x 128 expanded bytes = 32 columns.
    static constexpr int TMEM_COLS = DUAL ? 256 : 512;
    static constexpr int NBUF = DUAL ? (BN == 128 ? 1 : 2) : (BN == 32 ? 4 : (BN == 64 ? 3 : 2));
    static constexpr int A_COL0 = NBUF * BNX;
    static constexpr int STAGES = (TMEM_COLS - A_COL0) / 32 > 8 ? 8 : (TMEM_COLS - A_COL0) / 32;
    static constexpr int CTAS_PER_SM = DUAL ? 2 : 1;
    // registers are granted in blocks of 8 per thread: bound the pair of CTAs to 64 registers per thread
    static constexpr int BOUND_THREADS = DUAL ? 512 : THREADS;
    static_assert(A_COL0 + STAGES * 32 <= TMEM_COLS, "tensor memory budget");
    static_assert(STAGES >= G, "a producer group must not lap the ring (parity waits)");
    static constexpr int W_TILE_BYTES = BNX * ROWB;           // one K stage of the expanded weights
    static constexpr int BITS_BYTES = PF * PROD_THREADS * 16;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

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
// Bounded wait with back-off.  A polling warp competes with the MMA-issuing warp for issue
// slots, so after a first failed poll the waiter sleeps between polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err, int code)
{
    if (mbar_try_wait(bar, parity)) return true;
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        __nanosleep(SLEEP_NS);
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
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}
// Predicated forms for the issuer warp: every lane executes the same straight-line code and
// only the elected lane's predicate is true, so there is no branch to reconverge from.  The
// descriptors are passed as (low word, high word); only the low word (start address) varies.
__device__ __forceinline__ void tc_mma_i8_pred(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                               uint32_t idesc, uint32_t accumulate, uint32_t pred)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "setp.ne.b32 q, %6, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, {%7, %7, %7, %7}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(pred), "r"(0u)
        : "memory");
}
// A operand from tensor memory (128 lanes x 8 columns = 128 rows x 32 bytes of K), B from shared memory.
__device__ __forceinline__ void tc_mma_i8_ts_pred(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi,
                                                  uint32_t idesc, uint32_t accumulate, uint32_t pred)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "setp.ne.b32 q, %6, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], db, %4, {%7, %7, %7, %7}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(pred), "r"(0u)
        : "memory");
}
// 32 columns of this warp's 32 lanes <- 32 registers; returns once the store has completed.
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n\t"
        "tcgen05.wait::st.sync.aligned;"
        ::"r"(taddr),
          "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tc_commit_pred(uint32_t bar, uint32_t pred)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(bar), "r"(pred) : "memory");
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
__device__ __forceinline__ uint32_t tc_ld1(uint32_t taddr)
{
    uint32_t v;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];\n\ttcgen05.wait::ld.sync.aligned;"
                 : "=r"(v) : "r"(taddr) : "memory");
    return v;
}

// K-major tile, 128-byte rows, 128-byte swizzle, 8-row groups 1024 bytes apart, descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr)
{
    const uint32_t lo = ((saddr & 0x3FFFFu) >> 4) | (1u << 16);
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    return (static_cast<uint64_t>(hi) << 32) | lo;
}
// unsigned 8-bit A and B (K-major), int32 accumulate, M = 128, N = n.
__device__ __forceinline__ constexpr uint32_t make_idesc(int n)
{
    return (2u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
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

__device__ __forceinline__ void expand_store_a(uint32_t w, uint32_t row_addr, int xr, int c)
{
    st_shared_v4(row_addr + (uint32_t)(((c) ^ xr) << 4),
                 w & 0x01010101u, w & 0x02020202u, w & 0x04040404u, w & 0x08080808u);
    st_shared_v4(row_addr + (uint32_t)(((c + 1) ^ xr) << 4),
                 w & 0x10101010u, w & 0x20202020u, w & 0x40404040u, w & 0x80808080u);
}
__device__ __forceinline__ void expand_store_w(uint32_t w, uint32_t row_addr, int xr, int c)
{
    st_shared_v4(row_addr + (uint32_t)(((c) ^ xr) << 4),
                 (w << 7) & 0x80808080u, (w << 5) & 0x40404040u, (w << 3) & 0x20202020u, (w << 1) & 0x10101010u);
    st_shared_v4(row_addr + (uint32_t)(((c + 1) ^ xr) << 4),
                 (w >> 1) & 0x08080808u, (w >> 3) & 0x04040404u, (w >> 5) & 0x02020202u, (w >> 7) & 0x01010101u);
}

struct WsLayout {
    int ktiles;       // 128-bit K stages
    int smem;         // dynamic shared memory in bytes
};

template <int BN, int G, bool DUAL>
__host__ __device__ inline WsLayout ws_layout(int kwords)
{
    using C = Cfg<BN, G, DUAL>;
    WsLayout l;
    l.ktiles = (kwords + 3) >> 2;
    l.smem = 1024 + l.ktiles * C::W_TILE_BYTES + C::BITS_BYTES + BN * 4 + l.ktiles * 4 * 4;
    // Tensor memory is shared out by the resident CTAs (all 512 columns, or 256 each for two): ask
    // for enough shared memory that no further CTA of this kernel fits on the SM (it would sit in
    // tcgen05.alloc until a neighbour exits).
    const int floor_bytes = DUAL ? 78 * 1024 : 120 * 1024;
    if (l.smem < floor_bytes) l.smem = floor_bytes;
    return l;
}

template <int BN, int G, bool DUAL, bool FUSED>
__global__ void __launch_bounds__(Cfg<BN, G, DUAL>::BOUND_THREADS, Cfg<BN, G, DUAL>::CTAS_PER_SM)
conv_tc_ws_kernel(const ConvProblem p)
{
    using C = Cfg<BN, G, DUAL>;
    constexpr int BNX = C::BNX;
    constexpr int NBUF = C::NBUF;
    constexpr int MAX_STAGES = 8;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * MAX_STAGES + 2 * 4];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const WsLayout L = ws_layout<BN, G, DUAL>(p.kwords);
    const int ktiles = L.ktiles;
    constexpr int STAGES = C::STAGES;
    const int m_tiles = (p.M + BM - 1) / BM;
    const int my_tiles = ((int)blockIdx.x < m_tiles) ? (m_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int total_items = my_tiles * ktiles;

    // shared-memory map (all 1024-byte aligned where the MMA reads)
    const uint32_t wexp = (smem_u32(smem_raw) + 1023u) & ~1023u;          // [ktiles][BNX rows][128 B]
    const uint32_t bits_ring = wexp + (uint32_t)ktiles * C::W_TILE_BYTES; // [PF][PROD_THREADS][16 B]
    const uint32_t colc_addr = bits_ring + C::BITS_BYTES;                 // [BN] int32
    const uint32_t ktab_addr = colc_addr + BN * 4;                        // [ktiles*4] int32: (word offset << 5) | tap
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (MAX_STAGES + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * MAX_STAGES + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * MAX_STAGES + 4 + b); };
    volatile int *abort_flag = &abort_flag_smem;

    if (tid == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) {
            mbar_init(full_bar(s), 4);          // the four warps of the group that owns the stage
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 4; ++b) {
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

    // ---- one-off: expand the weight tile (+ the all-ones row), column constants, K-word table
    for (int idx = tid; idx < ktiles * BNX; idx += C::THREADS) {
        const int kt = idx / BNX, row = idx - kt * BNX;
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int kword = kt * 4 + e;
            uint32_t v = 0;
            if (kword < p.kwords) {
                if (row < BN) v = (row < p.C_out) ? __ldg(p.w + (long)row * p.kwords + kword) : 0u;
                else if (row == BN) v = 0xffffffffu;
            }
            w[e] = v;
        }
        const uint32_t row_addr = wexp + (uint32_t)kt * C::W_TILE_BYTES + (uint32_t)row * ROWB;
#pragma unroll
        for (int e = 0; e < 4; ++e) expand_store_w(w[e], row_addr, row & 7, 2 * e);
    }
    for (int c = tid; c < BN; c += C::THREADS) {
        int pop = 0;
        if (c < p.C_out)
            for (int kw = 0; kw < p.kwords; ++kw) pop += __popc(__ldg(p.w + (long)c * p.kwords + kw));
        // with acc = 128*popc(A and G), pa = popc(A):  int32: (acc >> 5) - 2*pa + (K - 2*pop)
        //                                             fused: acc - 64*pa - 32*(thr - K + 2*pop) >= 0
        const int cst = FUSED ? -32 * ((c < p.C_out ? __ldg(p.thr + c) : 0) - p.K + 2 * pop) : p.K - 2 * pop;
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(colc_addr + 4u * c), "r"(cst) : "memory");
    }
    for (int kword = tid; kword < ktiles * 4; kword += C::THREADS) {
        int entry = 0;
        if (kword < p.kwords) {
            const int tap = kword / p.cw, cj = kword - tap * p.cw;
            const int r = tap / p.kw, t = tap - r * p.kw;
            entry = (((r * p.W + t) * p.cw + cj) << 5) | tap;
        } else {
            entry = 31;                      // tap 31 is never valid (at most 31 taps are supported)
        }
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(ktab_addr + 4u * kword), "r"(entry) : "memory");
    }
    fence_async_proxy();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;

    if (warp == 0) {
        // ------------------------------------------------------------------ MMA issuer
        // This warp never touches memory: a load or an mbarrier wait issued after tensor-core
        // instructions holds the issuing thread until they have drained (measured: +230 cycles per
        // stage), a named barrier does not.  The control warp does the waiting and releases one
        // stage at a time through named barrier 1 + slot.
        constexpr uint32_t idesc = make_idesc(BNX);
        const uint64_t desc0 = make_desc(0);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32);
        const uint32_t a_tmem0 = tmem_base + (uint32_t)C::A_COL0;                // + slot * 32 columns
        const uint32_t b_lo0 = (uint32_t)desc0 | ((wexp & 0x3FFFFu) >> 4);       // + kt * (W_TILE_BYTES / 16)
        const uint32_t elected = lane == 0 ? 1u : 0u;
        int s = 0, buf = 0;
        for (int ti = 0; ti < my_tiles; ++ti) {
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BNX);
            const uint32_t tfull = tfull_bar(buf);
            for (int kt = 0; kt < ktiles; ++kt) {
                const uint32_t a_t = a_tmem0 + (uint32_t)s * 32u;
                const uint32_t b_lo = b_lo0 + (uint32_t)kt * (C::W_TILE_BYTES >> 4);
                const int nk = p.kwords - 4 * kt;                 // 32 bits of K per instruction; skip the zero tail
                const uint32_t e1 = nk > 1 ? elected : 0u, e2 = nk > 2 ? elected : 0u, e3 = nk > 3 ? elected : 0u;
                const uint32_t last = (kt == ktiles - 1) ? elected : 0u;
                const uint32_t ebar = empty_bar(s);
                asm volatile("bar.sync %0, 64;" ::"r"(1 + s) : "memory");
                tc_fence_after();
                // per 32 bytes of K: 8 tensor-memory columns of A, +2 (16-byte units) in the B descriptor
                tc_mma_i8_ts_pred(d_tmem, a_t, b_lo, desc_hi, idesc, kt > 0 ? 1u : 0u, elected);
                tc_mma_i8_ts_pred(d_tmem, a_t + 8u, b_lo + 2u, desc_hi, idesc, 1u, e1);
                tc_mma_i8_ts_pred(d_tmem, a_t + 16u, b_lo + 4u, desc_hi, idesc, 1u, e2);
                tc_mma_i8_ts_pred(d_tmem, a_t + 24u, b_lo + 6u, desc_hi, idesc, 1u, e3);
                tc_commit_pred(ebar, elected);
                tc_commit_pred(tfull, last);
                if (++s == STAGES) s = 0;
            }
            if (++buf == NBUF) buf = 0;
        }
    } else if (warp == C::CONTROL_WARP) {
        // ------------------------------------------------------------------ control: waits for the issuer
        // Stage `it` is released (bar.arrive on 1 + slot) once its ring slot is full and, for a tile's
        // first stage, once the accumulator buffer is free.  The slot being full implies that the
        // issuer is past the previous use of the same named barrier (it committed that slot's release).
        // After a time-out the remaining stages are released without waiting so that the issuer,
        // whose barrier wait has no time limit, always terminates; the error word tells the host.
        int s = 0, buf = 0;
        uint32_t ring_phase = 0, buf_phase = 1;      // first use of every accumulator buffer: free
        bool alive = true;
        for (int ti = 0; ti < my_tiles; ++ti) {
            if (lane == 0 && alive) alive = mbar_wait(tempty_bar(buf), buf_phase, abort_flag, p.err, ERR_MMA_TIMEOUT);
            for (int kt = 0; kt < ktiles; ++kt) {
                if (lane == 0 && alive) alive = mbar_wait(full_bar(s), ring_phase, abort_flag, p.err, ERR_MMA_TIMEOUT);
                __syncwarp();
                asm volatile("bar.arrive %0, 64;" ::"r"(1 + s) : "memory");
                if (++s == STAGES) { s = 0; ring_phase ^= 1u; }
            }
            if (++buf == NBUF) { buf = 0; buf_phase ^= 1u; }
        }
    } else if (warp <= EPI_WARPS) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;
        const int erow = quad * 32 + lane;
        bool alive = true;
        int buf = 0;
        uint32_t buf_phase = 0;
        for (int ti = 0; ti < my_tiles; ++ti) {
            const int m_tile = (int)blockIdx.x + ti * (int)gridDim.x;
            const int em = m_tile * BM + erow;
            if (alive) alive = mbar_wait(tfull_bar(buf), buf_phase, abort_flag, p.err, ERR_EPILOGUE_TIMEOUT);
            alive = __all_sync(0xffffffffu, alive && !*abort_flag);
            if (!alive) break;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BNX);
            const uint32_t pa128 = tc_ld1(t_addr + BN);        // 128 * popc(A) of this row
            uint32_t words[BN / 32];
#pragma unroll
            for (int ch = 0; ch < BN / 32; ++ch) {
                const int col0 = ch * 32;
                words[ch] = 0;
                if (col0 < p.C_out) {                                 // warp-uniform
                    uint32_t v[32];
                    tc_ld32(t_addr + (uint32_t)col0, v);
                    if (FUSED) {
                        const int rowc = -(int)(pa128 >> 1);          // -64 * popc(A)
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
                        const int rowc = -(int)(pa128 >> 6);          // -2 * popc(A)
                        int32_t *dst = static_cast<int32_t *>(p.out) + (long)em * p.C_out + col0;
                        const bool vec = (p.C_out & 3) == 0 && (col0 + 32 <= p.C_out);
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
                                const int n = col0 + 4 * i4;
                                if (n < p.C_out) dst[4 * i4] = o.x;
                                if (n + 1 < p.C_out) dst[4 * i4 + 1] = o.y;
                                if (n + 2 < p.C_out) dst[4 * i4 + 2] = o.z;
                                if (n + 3 < p.C_out) dst[4 * i4 + 3] = o.w;
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
            if (++buf == NBUF) { buf = 0; buf_phase ^= 1u; }
            if (FUSED && em < p.M) {
                const int owords = p.C_out >> 5;
                uint32_t *dst = static_cast<uint32_t *>(p.out) + (long)em * owords;
                if (BN == 128 && owords == 4) {
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(words[0], words[1], words[2], words[3]);
                } else if (BN >= 64 && owords == 2) {
                    *reinterpret_cast<uint2 *>(dst) = make_uint2(words[0], words[1]);
                } else {
#pragma unroll
                    for (int ch = 0; ch < BN / 32; ++ch)
                        if (ch < owords) dst[ch] = words[ch];
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ producers
        const int ptid = tid - FIRST_PRODUCER_THREAD;
        const int grp = ptid >> 7;                               // group = 4 consecutive warps
        const int quad = warp & 3;                               // tensor-memory lane quadrant this warp may write
        const int row = quad * 32 + lane;                        // the four warps of a group cover rows 0..127
        const uint32_t my_bits = bits_ring + (uint32_t)ptid * 16u;
        const bool a16 = (p.cw & 3) == 0;
        const bool plain = (p.kh * p.kw == 1 && p.stride == 1 && p.pad == 0);

        // this thread's items: grp, grp + G, grp + 2G, ... of the CTA's flattened (tile, stage) list
        // ---- load cursor
        int l_it = grp, l_ti = 0, l_kt = grp, l_slot = 0;
        bool l_fresh = true;                 // the row set-up of tile l_ti is still to be done
        const uint32_t *l_base = p.x;
        uint32_t l_mask = 0;
        auto l_locate = [&]() {              // (tile, stage) of l_it; refresh the row when the tile changes
            while (l_kt >= ktiles) { l_kt -= ktiles; ++l_ti; l_fresh = true; }
            if (l_fresh) {
                l_fresh = false;
                const int m = ((int)blockIdx.x + l_ti * (int)gridDim.x) * BM + row;
                const bool ok = m < p.M;
                if (plain) {
                    l_base = p.x + (long)(ok ? m : 0) * p.cw;
                    l_mask = ok ? 1u : 0u;
                } else {
                    const RowCoord rc = row_coord(p, ok ? m : 0);
                    l_base = p.x + (((long)rc.b * p.H + rc.ih0) * p.W + rc.iw0) * p.cw;
                    uint32_t colbits = 0, mask = 0;
                    for (int t = 0; t < p.kw; ++t)
                        if (rc.iw0 + t >= 0 && rc.iw0 + t < p.W) colbits |= 1u << t;
                    for (int r = 0; r < p.kh; ++r)
                        if (rc.ih0 + r >= 0 && rc.ih0 + r < p.H) mask |= colbits << (r * p.kw);
                    l_mask = ok ? mask : 0u;
                }
            }
        };
        auto issue_load = [&]() {
            l_locate();
            const uint32_t dst = my_bits + (uint32_t)l_slot * (C::PROD_THREADS * 16u);
            if (a16) {
                int entry;
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(entry) : "r"(ktab_addr + 16u * l_kt));
                const bool ok = (l_mask >> (entry & 31)) & 1u;
                cp_async16(dst, ok ? l_base + (entry >> 5) : p.x, ok);
            } else {
                const uint4 e4 = ld_shared_v4(ktab_addr + 16u * l_kt);
                const int ent[4] = {(int)e4.x, (int)e4.y, (int)e4.z, (int)e4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool ok = (l_mask >> (ent[e] & 31)) & 1u;
                    cp_async4(dst + 4u * e, ok ? l_base + (ent[e] >> 5) : p.x, ok);
                }
            }
            l_it += G;
            l_kt += G;
            if (++l_slot == PF) l_slot = 0;
        };

        int issued = 0;                       // groups committed so far
#pragma unroll 1
        for (; issued < PF - 1; ++issued) {
            if (l_it < total_items) issue_load();
            cp_async_commit();
        }

        // ---- expand cursor
        int c_slot = 0;
        int s = grp;                          // ring slot of item `it` and its parity, kept incrementally
        uint32_t phase = 1;                   // first pass through the ring: slots are free
        while (s >= STAGES) { s -= STAGES; phase ^= 1u; }
        bool alive = true;
        for (int it = grp; it < total_items; it += G) {
            if (l_it < total_items) issue_load();
            cp_async_commit();
            cp_async_wait<PF - 1>();
            const uint4 bits = ld_shared_v4(my_bits + (uint32_t)c_slot * (C::PROD_THREADS * 16u));
            if (++c_slot == PF) c_slot = 0;
            alive = mbar_wait(empty_bar(s), phase, abort_flag, p.err, ERR_PRODUCER_TIMEOUT);
            alive = __all_sync(0xffffffffu, alive);
            if (!alive) break;
            tc_fence_after();     // the MMAs that read this slot are complete (their commit released it)
            // expanded row -> 32 columns of this lane: column 8*e + j = word j of K word e (bytes 0 or 2^j)
            uint32_t v[32];
            const uint32_t wds[4] = {bits.x, bits.y, bits.z, bits.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
#pragma unroll
                for (int j = 0; j < 8; ++j) v[8 * e + j] = wds[e] & (0x01010101u << j);
            tc_st32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(C::A_COL0 + s * 32), v);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(full_bar(s));
            s += G;
            while (s >= STAGES) { s -= STAGES; phase ^= 1u; }
        }
        cp_async_wait<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
    }
}

template <int BN, int G, bool DUAL>
int launch_ws(const ConvProblem &p0, cudaStream_t stream)
{
    ConvProblem p = p0;
    p.err = device_error_word();
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    using C = Cfg<BN, G, DUAL>;
    const WsLayout L = ws_layout<BN, G, DUAL>(p.kwords);
    const long m_tiles = ((long)p.M + BM - 1) / BM;
    const long slots = (long)sms * C::CTAS_PER_SM;
    const unsigned grid = (unsigned)(m_tiles < slots ? m_tiles : slots);
    void (*k)(const ConvProblem) = p.thr ? conv_tc_ws_kernel<BN, G, DUAL, true> : conv_tc_ws_kernel<BN, G, DUAL, false>;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, L.smem) != cudaSuccess) return BCNN_ERR_CUDA;
    k<<<grid, C::THREADS, L.smem, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

// The expanded weights, the packed-word staging ring and the tables must fit in shared memory
// (in half of it when two CTAs share an SM).
template <int BN, int G, bool DUAL>
bool fits(const ConvProblem &p)
{
    return ws_layout<BN, G, DUAL>(p.kwords).smem + 512 <= (DUAL ? 113 * 1024 : MAX_SMEM);
}

}  // namespace

bool conv_tc_ws_supports(const ConvProblem &p)
{
    if (p.thr != nullptr && (p.C_out % 32 != 0)) return false;
    if (p.C_out > 128 || p.kh * p.kw > 31 || p.K > (1 << 16)) return false;
    // word offsets of the K-word table are shifted left by 5 bits
    if ((long)(p.kh * (long)p.W + p.kw) * p.cw >= (1L << 26)) return false;
    if (p.C_out <= 32) return fits<32, 4, false>(p);
    if (p.C_out <= 64) return fits<64, 4, false>(p);
    return fits<128, 4, false>(p) || fits<128, 2, false>(p);
}

int launch_conv_tc_ws(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_tc_ws_supports(p)) return BCNN_ERR_UNSUPPORTED;
    // narrow layers: the per-stage cost of issuing MMAs exceeds their execution time, so two CTAs
    // per SM (two issuers) when the resident weights leave room for it
    if (p.C_out <= 32) return fits<32, 2, true>(p) ? launch_ws<32, 2, true>(p, stream) : launch_ws<32, 4, false>(p, stream);
    if (p.C_out <= 64) return fits<64, 2, true>(p) ? launch_ws<64, 2, true>(p, stream) : launch_ws<64, 4, false>(p, stream);
    if (fits<128, 2, true>(p)) return launch_ws<128, 2, true>(p, stream);
    if (fits<128, 4, false>(p)) return launch_ws<128, 4, false>(p, stream);
    return launch_ws<128, 2, false>(p, stream);     // long K: fewer producer groups, smaller staging ring
}

}  // namespace bcnn
