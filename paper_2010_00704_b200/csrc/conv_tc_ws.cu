// Weight-stationary variant of the tcgen05 engine for layers with a short K: the expanded weights of up to
// 128 output channels fit in shared memory.  Wider layers run as slices of 128 (or 64) output channels: a CTA
// keeps one slice's weights, so the activations are expanded once per slice.
//
// Arithmetic.  Sign bits are expanded to bytes on chip; byte 4j+i of a 32-bit group carries bit j+8i.
//   activations (unsigned bytes): 0 where the bit is clear, else 2^j (j <= 6) or 64 (j = 7)
//   weights     (signed bytes):   +-2^(6-j) (j <= 6) or +-1 (j = 7), sign = the weight's sign
// Every product with a set activation bit is +-64, accumulators are int32 in tensor memory, and with
// S = sum over set activation bits of the weight signs (acc = 64 S):
//   sum a*g = 2 S + K - 2 popc(G)          (a, g in {-1,+1})
// so the epilogue needs one constant per output channel and nothing per row - and not even an addition: the
// accumulator buffers START from that constant (scaled by 32; the threshold folded in for the packed output).  The
// epilogue team writes the constants into its buffers once, and again right after reading a tile out of one; every
// MMA accumulates.  The packed output is then the complement of the accumulators' sign bits.
// Differences to conv_tc_i8.cu, all aimed at short tiles (a 128 x 32 x 32 tile is one MMA instruction):
//   * the CTA expands its weight tile ONCE into shared memory and keeps it for all its
//     output tiles; only activations stream through the ring;
//   * the activation ring lives in TENSOR memory, not shared memory: producers write expanded rows
//     with tcgen05.st and the MMA takes its A operand from tensor memory.  A narrow MMA is bound by
//     operand fetch from shared memory (128 x 32 bytes of A per instruction whatever N is); with A in
//     tensor memory only the small weight slice is fetched;
//   * G producer groups of 128 threads take the ring's stages round-robin, so that G stages
//     are being gathered / expanded at any time (one thread's stage latency is several
//     hundred cycles, an MMA stage as little as 64);
//   * up to four accumulator buffers, so the epilogue of one tile overlaps the MMAs of the next ones;
//   * the warp that issues the MMAs waits only on named barriers; a separate control warp does the
//     mbarrier waits for it (a memory instruction after tensor-core instructions stalls the issuer);
//   * the implicit-im2col gather uses a per-K-word table (tap, word offset) and a per-row
//     tap-validity mask instead of divisions; out-of-image taps are zero-filled by cp.async.
// Every mbarrier wait is bounded and reports through the device error word.
#include "tc_common.cuh"

namespace bcnn {

namespace {

using namespace tc;

constexpr int EPI_WARPS = 4;              // warps of one epilogue team (one per tensor-memory lane quadrant)
constexpr int PF = 3;                     // packed-word stages in flight per producer thread
constexpr int MAX_SMEM = 227 * 1024;

constexpr int ERR_PRODUCER_TIMEOUT = 111;
constexpr int ERR_MMA_TIMEOUT = 112;
constexpr int ERR_EPILOGUE_TIMEOUT = 113;

// DUAL: two CTAs share an SM (two independent MMA issuers), each with half of tensor memory.
// TEAMS: epilogue teams of four warps; team t takes the tiles t, t + TEAMS, ... of the CTA (their accumulator
// buffers are then a fixed subset, so NBUF is a multiple of TEAMS).  Two teams serve the module epilogue, which is
// bound by the epilogue warps.
template <int BN, int G, bool DUAL, int TEAMS = 1> struct Cfg {
    static constexpr int FIRST_PRODUCER_THREAD = 32 * (1 + EPI_WARPS * TEAMS);
    static constexpr int PROD_THREADS = G * BM;
    // Tensor memory (512 columns): NBUF accumulator buffers of BN columns, then the activation ring,
    // one stage = 128 rows x 128 expanded bytes = 32 columns.
    static constexpr int TMEM_COLS = DUAL ? 256 : 512;
    static constexpr int NBUF = DUAL ? (BN == 128 ? 1 : 2) : (BN == 32 ? 4 : (BN == 64 ? 3 : 2));
    static constexpr int CONTROL_WARP = (FIRST_PRODUCER_THREAD + PROD_THREADS) / 32;
    static constexpr int THREADS = FIRST_PRODUCER_THREAD + PROD_THREADS + 32;
    static constexpr int A_COL0 = NBUF * BN;
    static constexpr int STAGES = (TMEM_COLS - A_COL0) / 32 > 8 ? 8 : (TMEM_COLS - A_COL0) / 32;
    static constexpr int CTAS_PER_SM = DUAL ? 2 : 1;
    // registers are granted in blocks of 8 per thread: bound the pair of CTAs to 64 registers per thread
    static constexpr int BOUND_THREADS = DUAL ? 512 : THREADS;
    static_assert(A_COL0 + STAGES * 32 <= TMEM_COLS, "tensor memory budget");
    static_assert(STAGES >= G, "a producer group must not lap the ring (parity waits)");
    static constexpr int W_TILE_BYTES = BN * ROWB;           // one K stage of the expanded weights
    static constexpr int BITS_BYTES = PF * PROD_THREADS * 16;
};

struct WsLayout {
    int ktiles;       // 128-bit K stages
    int row_kt;       // > 0: producers work tile by tile (all row_kt stages of a row at once), see the producers
    int bits_bytes;   // staging ring of the packed words
    int smem;         // dynamic shared memory in bytes
};

template <int BN, int G, bool DUAL, int TEAMS = 1>
__host__ __device__ inline WsLayout ws_layout(int kwords, int mode)
{
    using C = Cfg<BN, G, DUAL, TEAMS>;
    WsLayout l;
    l.ktiles = (kwords + 3) >> 2;
    // Short K: a producer group takes whole tiles in turn instead of single stages, so the per-tile work
    // (row coordinates, tap mask, bookkeeping) is done once per row and tile.  A group then runs up to
    // (G - 1) * ktiles + 1 ring slots ahead of the slot it waits for; the parity waits need the ring
    // to be at least that deep.
    l.row_kt = (l.ktiles <= 3 && C::STAGES >= (G - 1) * l.ktiles + 1) ? l.ktiles : 0;
    l.bits_bytes = C::BITS_BYTES * (l.row_kt ? l.row_kt : 1);
    l.smem = 1024 + l.ktiles * C::W_TILE_BYTES + l.bits_bytes + BN * 4 + l.ktiles * 32;
    if (mode == 2) l.smem += TEAMS * ID_RING_BYTES + 16;      // identity staging rings of the module epilogue
    if (mode == 0) l.smem += TEAMS * EPI_WARPS * I32_TILE_BYTES + 16;   // store staging tiles of the int32 epilogue
    // Tensor memory is shared out by the resident CTAs (all 512 columns, or 256 each for two): ask
    // for enough shared memory that no further CTA of this kernel fits on the SM (it would sit in
    // tcgen05.alloc until a neighbour exits).
    const int floor_bytes = DUAL ? 78 * 1024 : 120 * 1024;
    if (l.smem < floor_bytes) l.smem = floor_bytes;
    return l;
}

template <int BN, int G, bool DUAL, int MODE, int TEAMS = 1>
__global__ void __launch_bounds__(Cfg<BN, G, DUAL, TEAMS>::BOUND_THREADS, Cfg<BN, G, DUAL, TEAMS>::CTAS_PER_SM)
conv_tc_ws_kernel(const ConvProblem p)
{
    using C = Cfg<BN, G, DUAL, TEAMS>;
    static_assert(C::NBUF % TEAMS == 0, "a team's tiles must map to a fixed set of accumulator buffers");
    constexpr bool FUSED = MODE == 1, MODULE = MODE == 2;
    constexpr int NBUF = C::NBUF;
    constexpr int MAX_STAGES = 8;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * MAX_STAGES + 2 * 4];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const WsLayout L = ws_layout<BN, G, DUAL, TEAMS>(p.kwords, MODE);
    const int ktiles = L.ktiles;
    constexpr int STAGES = C::STAGES;
    const int m_tiles = (p.M - 1) / BM + 1;                  // M >= 1; no overflow for M close to 2^31
    // N slices: a CTA keeps the weights of one slice of BN output channels and walks row tiles mb, mb + mstride, ...
    // (the grid is a multiple of the slice count)
    const int n_tiles = (p.C_out + BN - 1) / BN;
    const int n0 = ((int)blockIdx.x % n_tiles) * BN;
    const int cn = min(BN, p.C_out - n0);                     // channels of this slice
    const int mb = (int)blockIdx.x / n_tiles;
    const int mstride = (int)gridDim.x / n_tiles;
    const int my_tiles = (mb < m_tiles) ? (m_tiles - 1 - mb) / mstride + 1 : 0;
    const int total_items = my_tiles * ktiles;

    // shared-memory map (all 1024-byte aligned where the MMA reads)
    const uint32_t wexp = (smem_u32(smem_raw) + 1023u) & ~1023u;          // [ktiles][BN rows][128 B]
    const uint32_t bits_ring = wexp + (uint32_t)ktiles * C::W_TILE_BYTES; // [PF][PROD_THREADS][16 B]
    const uint32_t colc_addr = bits_ring + (uint32_t)L.bits_bytes;                 // [BN] int32
    const uint32_t ktab_addr = colc_addr + BN * 4;                        // unit table: [ktiles * 4 / gw] x {word offset, tap bit}
    const uint32_t idring = (ktab_addr + (uint32_t)ktiles * 32u + 15u) & ~15u;   // module epilogue only: [ID_SLOTS][BM rows][80 B]
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

    // ---- one-off: expand the weight tile, per-channel constants, K-word table
    for (int idx = tid; idx < ktiles * BN; idx += C::THREADS) {
        const int kt = idx / BN, row = idx - kt * BN;
        const uint32_t row_addr = wexp + (uint32_t)kt * C::W_TILE_BYTES + (uint32_t)row * ROWB;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int kword = kt * 4 + e;
            const bool live = kword < p.kwords && row < cn;              // rows / K words beyond the problem: zero bytes
            const uint32_t w = live ? __ldg(p.w + (long)(n0 + row) * p.kwords + kword) : 0u;
            expand_store_w_signed(w, live, row_addr, row & 7, 2 * e);
        }
    }
    for (int c = tid; c < BN; c += C::THREADS) {
        int pop = 0;
        if (c < cn)
            for (int kw = 0; kw < p.kwords; ++kw) pop += __popc(__ldg(p.w + (long)(n0 + c) * p.kwords + kw));
        // The accumulators start from a per-channel constant instead of zero (the epilogue writes it back after
        // reading a buffer, every MMA accumulates), so with acc = 64 * S + cst:
        //   int32: acc >> 5 with cst = 32 * (K - 2*pop)        fused: acc >= 0 with cst = 32 * (K - 2*pop - thr)
        // (a threshold beyond +-(K + 1) decides like that bound; clamping keeps the constant inside int32)
        int cst = p.K - 2 * pop;
        if (FUSED) {
            int t = c < cn ? __ldg(p.thr + n0 + c) : 0;
            t = max(min(t, p.K + 1), -p.K - 1);
            cst -= t;
        }
        cst *= 32;
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(colc_addr + 4u * c), "r"(cst) : "memory");
    }
    const int gw = gather_width(p.cw);
    build_unit_table(p, ktab_addr, ktiles * (4 / gw), gw, tid, C::THREADS);
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
        // stage at a time through named barrier 1 + slot.  There is one issuer on purpose: the
        // producers' parity waits rely on the ring being consumed in order (a second issuer working on
        // the next tile lets a late slot fall two phases behind a waiting producer).
        constexpr uint32_t idesc = make_idesc(BN) | (1u << 10);                  // B operand: signed bytes
        const uint64_t desc0 = make_desc(0);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32);
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);             // warp-uniform copy for the issuer
        const uint32_t a_tmem0 = tmem_u + (uint32_t)C::A_COL0;                   // + slot * 32 columns
        const uint32_t b_lo0 = (uint32_t)desc0 | ((wexp & 0x3FFFFu) >> 4);       // + kt * (W_TILE_BYTES / 16)
        int s = 0, buf = 0;
        for (int ti = 0; ti < my_tiles; ++ti) {
            const uint32_t d_tmem = tmem_u + (uint32_t)(buf * BN);
            const uint32_t tfull = tfull_bar(buf);
            for (int kt = 0; kt < ktiles; ++kt) {
                const uint32_t a_t = a_tmem0 + (uint32_t)s * 32u;
                const uint32_t b_lo = b_lo0 + (uint32_t)kt * (C::W_TILE_BYTES >> 4);
                const int nk = p.kwords - 4 * kt;                 // 32 bits of K per instruction; skip the zero tail
                const uint32_t ebar = empty_bar(s);
                asm volatile("bar.sync %0, 64;" ::"r"(1 + s) : "memory");
                tc_fence_after();
                // per 32 bytes of K: 8 tensor-memory columns of A, +2 (16-byte units) in the B descriptor
                if (elect_one()) {
                    tc_mma_i8_ts(d_tmem, a_t, b_lo, desc_hi, idesc, 1u);      // always accumulates: the buffer holds the constants
                    if (nk > 1) tc_mma_i8_ts(d_tmem, a_t + 8u, b_lo + 2u, desc_hi, idesc, 1u);
                    if (nk > 2) tc_mma_i8_ts(d_tmem, a_t + 16u, b_lo + 4u, desc_hi, idesc, 1u);
                    if (nk > 3) tc_mma_i8_ts(d_tmem, a_t + 24u, b_lo + 6u, desc_hi, idesc, 1u);
                    tc_commit(ebar);
                    if (kt == ktiles - 1) tc_commit(tfull);
                }
                __syncwarp();
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
        uint32_t ring_phase = 0, buf_phase = 0;      // every accumulator buffer is handed over by its epilogue team, first after initialising it
        bool alive = true;
        for (int ti = 0; ti < my_tiles; ++ti) {
            if (lane == 0 && alive) alive = mbar_wait(tempty_bar(buf), buf_phase, abort_flag, p.err, ERR_MMA_TIMEOUT);
            for (int kt = 0; kt < ktiles; ++kt) {
                if (lane == 0 && alive) alive = mbar_wait(full_bar(s), ring_phase, abort_flag, p.err, ERR_MMA_TIMEOUT);
                // after a time-out: bar.sync, which pairs every release with one wait of the issuer (two bar.arrive in a
                // row on one barrier would complete it without the issuer)
                if (__shfl_sync(0xffffffffu, alive ? 1 : 0, 0)) asm volatile("bar.arrive %0, 64;" ::"r"(1 + s) : "memory");
                else asm volatile("bar.sync %0, 64;" ::"r"(1 + s) : "memory");
                if (++s == STAGES) { s = 0; ring_phase ^= 1u; }
            }
            if (++buf == NBUF) { buf = 0; buf_phase ^= 1u; }
        }
    } else if (warp <= EPI_WARPS * TEAMS) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;
        const int erow = quad * 32 + lane;
        const int team = (warp - 1) >> 2;                        // takes the tiles team, team + TEAMS, ...
        const uint32_t i32_tile = idring + (uint32_t)(team * EPI_WARPS + quad) * I32_TILE_BYTES;   // int32 epilogue (shares the place of the module's rings)
        bool alive = true;
        // module epilogue: chunk q of this thread's row sequence = (tile q / nch, chunk q % nch); its identity values
        // are staged ID_AHEAD chunks ahead in ring slot q % ID_SLOTS
        const int nch = (cn + 31) >> 5;
        const uint32_t id_warp = idring + (uint32_t)team * ID_RING_BYTES + (uint32_t)(quad * 32) * ID_ROW_BYTES;   // slot 0, the warp's first row
        int pf_ti = team, pf_ch = 0, pf_slot = 0, cur_slot = 0;
        auto prefetch_next = [&]() {
            if (pf_ti < my_tiles) {
                const long row0 = (long)(mb + pf_ti * mstride) * BM + quad * 32;
                module_prefetch(p, id_warp + (uint32_t)pf_slot * (BM * ID_ROW_BYTES), row0, n0 + pf_ch * 32, lane);
                if (++pf_ch == nch) { pf_ch = 0; pf_ti += TEAMS; }
            } else {
                cp_async_commit();
            }
            if (++pf_slot == ID_SLOTS) pf_slot = 0;
        };
        if (MODULE)
            for (int a = 0; a < ID_AHEAD; ++a) prefetch_next();
        // write the per-channel constants into 32 accumulator columns of this warp's rows (8 columns at a time:
        // the values are the same for every row)
        auto write_consts = [&](uint32_t t_chunk, int col0) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint4 a = ld_shared_v4(colc_addr + 4u * (col0 + 8 * q)), b = ld_shared_v4(colc_addr + 4u * (col0 + 8 * q + 4));
                const uint32_t c8[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                tc_st8_nowait(t_chunk + 8u * q, c8);
            }
        };
        // the team's accumulator buffers start out holding the constants
        for (int b = team; b < NBUF; b += TEAMS) {
            const uint32_t tb = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(b * BN);
#pragma unroll
            for (int ch = 0; ch < BN / 32; ++ch)
                if (ch * 32 < cn) write_consts(tb + (uint32_t)(ch * 32), ch * 32);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(b));
        }
        for (int ti = team; ti < my_tiles; ti += TEAMS) {
            const int buf = ti % NBUF;                            // tiles use the accumulator buffers in turn
            const uint32_t buf_phase = (uint32_t)(ti / NBUF) & 1u;
            const int m_tile = mb + ti * mstride;
            const int em = m_tile * BM + erow;
            if (alive) alive = mbar_wait(tfull_bar(buf), buf_phase, abort_flag, p.err, ERR_EPILOGUE_TIMEOUT);
            alive = __all_sync(0xffffffffu, alive && !*abort_flag);
            if (!alive) break;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BN);
            uint32_t words[BN / 32];
#pragma unroll
            for (int ch = 0; ch < BN / 32; ++ch) {
                const int col0 = ch * 32;
                words[ch] = 0;
                if (col0 < cn) {                                      // warp-uniform
                    uint32_t v[32];
                    tc_ld32(t_addr + (uint32_t)col0, v);
                    write_consts(t_addr + (uint32_t)col0, col0);      // the buffer's next tile starts from the constants again
                    if (FUSED) {
                        // bit = (v >= 0): the sign bits are shifted in, last column first
                        uint32_t acc = 0;
#pragma unroll
                        for (int i = 31; i >= 0; --i) acc = __funnelshift_l(v[i], acc, 1);
                        words[ch] = ~acc;
                    } else if (MODULE) {
                        int dot[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) dot[i] = (int)v[i] >> 5;
                        prefetch_next();
                        cp_async_wait<ID_AHEAD>();                    // this chunk's copy has landed
                        words[ch] = module_chunk(p, dot, id_warp + (uint32_t)cur_slot * (BM * ID_ROW_BYTES), (long)em - lane, n0 + col0, lane);
                        if (++cur_slot == ID_SLOTS) cur_slot = 0;
                    } else if ((p.C_out & 3) == 0 && (n0 + col0 + 32 <= p.C_out)) {
                        // full chunk (warp-uniform): staged, the warp stores whole 128-byte rows
                        int o[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = (int)v[i] >> 5;
                        const long row0 = (long)em - lane;
                        store_int32_block(static_cast<int32_t *>(p.out) + row0 * p.C_out + n0 + col0, p.C_out, o, i32_tile, row0, p.M, lane);
                    } else if (em < p.M) {
                        int32_t *dst = static_cast<int32_t *>(p.out) + (long)em * p.C_out + n0 + col0;
                        const bool vec = (p.C_out & 3) == 0 && (n0 + col0 + 32 <= p.C_out);
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            int4 o;
                            o.x = (int)v[4 * i4 + 0] >> 5;
                            o.y = (int)v[4 * i4 + 1] >> 5;
                            o.z = (int)v[4 * i4 + 2] >> 5;
                            o.w = (int)v[4 * i4 + 3] >> 5;
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
            tc_wait_st();                     // the constants are back in the buffer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
            if ((FUSED || (MODULE && p.out != nullptr)) && em < p.M) {
                const int owords = p.C_out >> 5, swords = cn >> 5;      // words of a row, of this slice
                uint32_t *dst = static_cast<uint32_t *>(p.out) + (long)em * owords + (n0 >> 5);
                if (BN == 128 && swords == 4 && (owords & 3) == 0) {
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(words[0], words[1], words[2], words[3]);
                } else if (BN >= 64 && swords == 2 && (owords & 1) == 0) {
                    *reinterpret_cast<uint2 *>(dst) = make_uint2(words[0], words[1]);
                } else {
#pragma unroll
                    for (int ch = 0; ch < BN / 32; ++ch)
                        if (ch < swords) dst[ch] = words[ch];
                }
            }
        }
        if (MODULE) cp_async_wait<0>();
    } else {
        // ------------------------------------------------------------------ producers
        // Group g takes items g, g + G, ... of the CTA's flattened (tile, stage) list.  Per item a
        // thread copies its row's 128 bits of K into its staging slot (PF items ahead), then expands
        // the oldest staged item into the ring slot of tensor memory.
        const int ptid = tid - C::FIRST_PRODUCER_THREAD;
        const int grp = ptid >> 7;                               // group = 4 consecutive warps
        const int quad = warp & 3;                               // tensor-memory lane quadrant this warp may write
        const int row = quad * 32 + lane;                        // the four warps of a group cover rows 0..127
        constexpr uint32_t SLOT_BYTES = C::PROD_THREADS * 16u;
        const uint32_t bits0 = bits_ring + (uint32_t)ptid * 16u, bits_end = bits0 + PF * SLOT_BYTES;
        const uint32_t st_addr0 = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)C::A_COL0;
        const uint32_t lane0 = lane == 0 ? 1u : 0u;
        const TileStep step = make_tile_step(p, (uint32_t)(BM * mstride));

        auto produce = [&](auto gw_tag) {
            constexpr int GW = decltype(gw_tag)::value;
            constexpr uint32_t TAB_STAGE = (4 / GW) * 8u;        // table bytes per stage
            // ---- load cursor
            RowCursor rc;
            rc.m = (uint32_t)mb * BM + (uint32_t)row;
            row_locate(p, rc);
            int l_kt = grp;
            int l_left = total_items > grp ? (total_items - grp + G - 1) / G : 0;
            while (l_kt >= ktiles) { l_kt -= ktiles; row_step(p, step, rc); }
            row_window(p, step, rc);
            uint32_t l_dst = bits0;
            auto issue = [&]() {
                gather_stage<GW>(p.x, rc, ktab_addr + (uint32_t)l_kt * TAB_STAGE, l_dst);
                l_dst += SLOT_BYTES;
                if (l_dst == bits_end) l_dst = bits0;
                --l_left;
                l_kt += G;
                if (l_kt >= ktiles) {
                    do { l_kt -= ktiles; row_step(p, step, rc); } while (l_kt >= ktiles);
                    row_window(p, step, rc);
                }
            };
#pragma unroll 1
            for (int n = 0; n < PF - 1; ++n) {
                if (l_left > 0) issue();
                cp_async_commit();
            }
            // ---- expand cursor
            uint32_t c_src = bits0;
            int s = grp;                          // ring slot (G <= STAGES) and its parity
            uint32_t phase = 1;                   // first pass through the ring: slots are free
#pragma unroll 1
            for (int it = grp; it < total_items; it += G) {
                if (l_left > 0) issue();
                cp_async_commit();
                cp_async_wait<PF - 1>();
                const uint4 bits = ld_shared_v4(c_src);
                c_src += SLOT_BYTES;
                if (c_src == bits_end) c_src = bits0;
                if (!mbar_wait_warp(empty_bar(s), phase, abort_flag, p.err, ERR_PRODUCER_TIMEOUT)) break;
                tc_fence_after();     // the MMAs that read this slot are complete (their commit released it)
                // expanded row -> 32 columns of this lane: column 8*e + j = word j of K word e (bytes 0 or 2^j, 64 for j = 7)
                uint32_t v[32];
                const uint32_t wds[4] = {bits.x, bits.y, bits.z, bits.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) expand_a(wds[e], &v[8 * e]);
                tc_st32(st_addr0 + (uint32_t)s * 32u, v);
                tc_fence_before();
                __syncwarp();
                mbar_arrive_pred(full_bar(s), lane0);
                s += G;
                if (s >= STAGES) { s -= STAGES; phase ^= 1u; }
            }
            cp_async_wait<0>();
        };
        // ---- short K: this group's items are the tiles grp, grp + G, ...; all stages of a row are staged
        // together (PF tiles ahead) and expanded one ring slot after the other
        auto produce_rows = [&](auto gw_tag, auto kt_tag) {
            constexpr int GW = decltype(gw_tag)::value;
            constexpr int KT = decltype(kt_tag)::value;
            constexpr uint32_t TAB_STAGE = (4 / GW) * 8u;
            constexpr uint32_t TSLOT_BYTES = SLOT_BYTES * KT;     // one staged tile: [KT][PROD_THREADS][16 B]
            const uint32_t tend = bits0 + PF * TSLOT_BYTES;
            const int nk_last = p.kwords - 4 * (KT - 1);          // K words of the row's last stage (1..4)
            const TileStep gstep = make_tile_step(p, (uint32_t)(BM * mstride * G));
            RowCursor rc;
            rc.m = (uint32_t)(mb + grp * mstride) * BM + (uint32_t)row;
            row_locate(p, rc);
            row_window(p, gstep, rc);
            int l_left = my_tiles > grp ? (my_tiles - grp + G - 1) / G : 0;
            uint32_t l_dst = bits0;
            auto issue = [&]() {
#pragma unroll
                for (int kt = 0; kt < KT; ++kt)
                    gather_stage<GW>(p.x, rc, ktab_addr + (uint32_t)kt * TAB_STAGE, l_dst + (uint32_t)kt * SLOT_BYTES,
                                     kt < KT - 1 ? 4 : (nk_last + GW - 1) / GW);
                l_dst += TSLOT_BYTES;
                if (l_dst == tend) l_dst = bits0;
                --l_left;
                row_step(p, gstep, rc);
                row_window(p, gstep, rc);
            };
#pragma unroll 1
            for (int n = 0; n < PF - 1; ++n) {
                if (l_left > 0) issue();
                cp_async_commit();
            }
            uint32_t c_src = bits0;
            int s = grp * KT;                     // ring slot of the tile's first stage and its parity
            uint32_t phase = 1;
            while (s >= STAGES) { s -= STAGES; phase ^= 1u; }
#pragma unroll 1
            for (int ti = grp; ti < my_tiles; ti += G) {
                if (l_left > 0) issue();
                cp_async_commit();
                cp_async_wait<PF - 1>();
                bool alive = true;
#pragma unroll
                for (int kt = 0; kt < KT; ++kt) {
                    const uint4 bits = ld_shared_v4(c_src + (uint32_t)kt * SLOT_BYTES);
                    if (alive && !mbar_wait_warp(empty_bar(s), phase, abort_flag, p.err, ERR_PRODUCER_TIMEOUT)) alive = false;
                    if (alive) {
                        tc_fence_after();
                        expand_store_stage(st_addr0 + (uint32_t)s * 32u, bits, kt < KT - 1 ? 4 : nk_last);
                        tc_fence_before();
                        __syncwarp();
                        mbar_arrive_pred(full_bar(s), lane0);
                    }
                    if (++s == STAGES) { s = 0; phase ^= 1u; }
                }
                if (!alive) break;
                c_src += TSLOT_BYTES;
                if (c_src == tend) c_src = bits0;
                s += (G - 1) * KT;                // the other groups' tiles
                while (s >= STAGES) { s -= STAGES; phase ^= 1u; }
            }
            cp_async_wait<0>();
        };
        auto rows_by_kt = [&](auto gw_tag) {
            if (L.row_kt == 1) produce_rows(gw_tag, IntC<1>{});
            else if (L.row_kt == 2) produce_rows(gw_tag, IntC<2>{});
            else produce_rows(gw_tag, IntC<3>{});
        };
        if (L.row_kt) {
            if (gw == 4) rows_by_kt(IntC<4>{});
            else if (gw == 2) rows_by_kt(IntC<2>{});
            else rows_by_kt(IntC<1>{});
        } else if (gw == 4) produce(IntC<4>{});
        else if (gw == 2) produce(IntC<2>{});
        else produce(IntC<1>{});
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
    }
}

template <int BN, int G, bool DUAL, int TEAMS = 1>
int launch_ws(const ConvProblem &p0, cudaStream_t stream)
{
    ConvProblem p = p0;
    p.err = device_error_word();
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    using C = Cfg<BN, G, DUAL, TEAMS>;
    const WsLayout L = ws_layout<BN, G, DUAL, TEAMS>(p.kwords, p.mode);
    const long m_tiles = ((long)p.M + BM - 1) / BM;
    const long slots = (long)sms * C::CTAS_PER_SM;
    const long n_tiles = (p.C_out + BN - 1) / BN;
    long per_slice = slots / n_tiles;                         // CTAs that share one slice of the weights
    if (per_slice < 1) return BCNN_ERR_UNSUPPORTED;
    if (per_slice > m_tiles) per_slice = m_tiles;
    const unsigned grid = (unsigned)(per_slice * n_tiles);
    void (*k)(const ConvProblem) = p.mode == 2 ? conv_tc_ws_kernel<BN, G, DUAL, 2, TEAMS>
                                   : (p.mode == 1 ? conv_tc_ws_kernel<BN, G, DUAL, 1, TEAMS> : conv_tc_ws_kernel<BN, G, DUAL, 0, TEAMS>);
    // the attribute is a property of the kernel, not of the launch: always the configuration's limit, so
    // that a captured launch stays valid whatever later calls with other shapes ask for
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, DUAL ? 113 * 1024 : MAX_SMEM - 1024) != cudaSuccess) return BCNN_ERR_CUDA;
    k<<<grid, C::THREADS, L.smem, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

// The expanded weights, the packed-word staging ring and the tables must fit in shared memory
// (in half of it when two CTAs share an SM).
template <int BN, int G, bool DUAL, int TEAMS = 1>
bool fits(const ConvProblem &p)
{
    return ws_layout<BN, G, DUAL, TEAMS>(p.kwords, p.mode).smem <= (DUAL ? 113 * 1024 : MAX_SMEM - 1024);
}

}  // namespace

bool conv_tc_ws_supports(const ConvProblem &p)
{
    if (p.mode != 0 && (p.C_out % 32 != 0)) return false;
    if (p.kh * p.kw > 31 || p.K > (1 << 16)) return false;
    // rows address the input by 32-bit word offsets
    if ((long)p.B * p.H * p.W * p.cw >= (1L << 31)) return false;
    if (p.C_out <= 32) return fits<32, 4, false>(p);
    if (p.C_out <= 64) return fits<64, 4, false>(p);
    if (fits<128, 4, false>(p) || fits<128, 2, false>(p)) return p.C_out <= 128 * 64;
    // wider layers whose 128-channel slice of the weights does not fit: 64-channel slices
    return p.C_out > 128 && p.C_out <= 64 * 64 && fits<64, 4, false>(p);
}

int launch_conv_tc_ws(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_tc_ws_supports(p)) return BCNN_ERR_UNSUPPORTED;
    // module epilogue: bound by the epilogue warps, so two teams of them, one producer group and two CTAs per SM;
    // layers wider than 64 channels run as 64-channel slices (two accumulator buffers are needed for two teams)
    if (p.mode == 2) {
        if (p.C_out <= 32 && fits<32, 1, true, 2>(p)) return launch_ws<32, 1, true, 2>(p, stream);
        if (p.C_out > 32 && fits<64, 1, true, 2>(p)) return launch_ws<64, 1, true, 2>(p, stream);
        if (p.C_out > 32 && p.C_out <= 32 * 64 && fits<32, 1, true, 2>(p)) return launch_ws<32, 1, true, 2>(p, stream);   // long K: 32-channel slices
    }
    // narrow layers: the per-stage cost of issuing MMAs exceeds their execution time, so two CTAs
    // per SM (two issuers) when the resident weights leave room for it
    if (p.C_out <= 32) return fits<32, 2, true>(p) ? launch_ws<32, 2, true>(p, stream) : launch_ws<32, 4, false>(p, stream);
    if (p.C_out <= 64) return fits<64, 2, true>(p) ? launch_ws<64, 2, true>(p, stream) : launch_ws<64, 4, false>(p, stream);
    // C_out > 128: slices of 128 (or 64) output channels, each CTA keeps one slice's weights
    if (fits<128, 2, true>(p)) return launch_ws<128, 2, true>(p, stream);
    if (fits<128, 4, false>(p)) return launch_ws<128, 4, false>(p, stream);
    if (fits<128, 2, false>(p)) return launch_ws<128, 2, false>(p, stream);     // long K: fewer producer groups, smaller staging ring
    return fits<64, 2, true>(p) ? launch_ws<64, 2, true>(p, stream) : launch_ws<64, 4, false>(p, stream);
}

}  // namespace bcnn
