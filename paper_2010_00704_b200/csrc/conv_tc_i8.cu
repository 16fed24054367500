// Streaming tcgen05 engine of the binary implicit GEMM (kind::i8): wide layers (C_out >= 256),
// long K, and the plain GEMMs.  Arithmetic as in the other tensor-core engines: sign bits are
// expanded to bytes on chip (activations {0, 2^j}, weights {0, 2^(7-j)}; byte 4j+i of a 32-bit
// group carries bit j+8i), every product of two set bits is 128, accumulators are int32 in
// tensor memory and   sum a*g = K - 2*popc(A) - 2*popc(G) + 4*popc(A and G).
//
// Persistent, warp-specialised; each CTA walks a static list of 128 x BN tiles.
//   warp 0          issuer: tcgen05.mma / commit only, waits on named barriers only (a memory
//                   instruction after tensor-core instructions would stall it)
//   warps 1-4       epilogue: tcgen05.ld, threshold + pack (or int32), hand the accumulator back
//   G = 2 producer groups, each 4 activation warps + BN/32 weight warps, one thread per tile
//                   row; the groups take the ring's stages alternately so that one group gathers
//                   while the other expands.  Packed words are staged with cp.async (16 bytes per
//                   row and stage, zero-fill out of range).
//                     activation rows -> TENSOR memory (tcgen05.st, 32 columns per stage): the
//                       MMA takes A from tensor memory, so shared memory carries only weights
//                     weight rows     -> shared memory, 128-byte-swizzled K-major tiles
//   last warp       control: does the issuer's mbarrier waits and releases it stage by stage
// Tensor memory (512 columns): BN = 256: one accumulator + 5 ring stages; BN = 128: two
// accumulators + 8 ring stages.  Row / column popcounts are taken from the words as they are
// expanded; each group leaves its partial constants for a tile in shared-memory slots.
// Every mbarrier wait is bounded and reports through the device error word.
#include "tc_common.cuh"

namespace bcnn {

namespace {

using namespace tc;

constexpr int EPI_WARPS = 4;
constexpr int G = 2;                      // producer groups
constexpr int PF = 3;                     // packed-word stages in flight per producer thread
constexpr int MAX_SMEM = 227 * 1024 - 512; // dynamic shared memory available beside the static part

constexpr int ERR_PRODUCER_TIMEOUT = 101;
constexpr int ERR_MMA_TIMEOUT = 102;
constexpr int ERR_EPILOGUE_TIMEOUT = 103;

template <int BN> struct Cfg {
    static constexpr int NBUF = BN == 256 ? 1 : 2;                       // accumulator buffers
    static constexpr int A_COL0 = NBUF * BN;                              // first column of the activation ring
    static constexpr int STAGES = BN == 256 ? 5 : 8;
    static constexpr int GROUP_WARPS = 4 + BN / 32;
    static constexpr int GROUP_THREADS = 32 * GROUP_WARPS;
    static constexpr int PROD_THREADS = G * GROUP_THREADS;
    static constexpr int FIRST_PRODUCER_WARP = 1 + EPI_WARPS;
    static constexpr int CONTROL_WARP = FIRST_PRODUCER_WARP + G * GROUP_WARPS;
    static constexpr int THREADS = 32 * (CONTROL_WARP + 1);
    static constexpr int W_BYTES = BN * ROWB;                             // one ring stage of weights
    static constexpr int BITS_BYTES = PF * PROD_THREADS * 16;
    static constexpr int SLOTS = STAGES + NBUF + 2;                       // per-tile constant slots
    static constexpr int SLOT_INTS = G * (BM + BN);
    static constexpr int CONST_BYTES = SLOTS * SLOT_INTS * 4;
    static_assert(A_COL0 + STAGES * 32 <= 512, "tensor memory budget");
    static_assert(STAGES >= G, "a producer group must not lap the ring (parity waits)");
};

template <int BN>
__host__ __device__ inline int smem_bytes(int ktab_words, int mode = 1)
{
    using C = Cfg<BN>;
    // module epilogue: + the identity staging ring; int32 output of the 128-wide tiles: + the store staging tiles
    // (both only used where they fit: 128-wide tiles)
    return 1024 + C::STAGES * C::W_BYTES + C::BITS_BYTES + C::CONST_BYTES + ktab_words * 4 +
           (mode == 2 ? ID_RING_BYTES + 16 : 0) + (mode == 0 && BN == 128 ? EPI_WARPS * I32_TILE_BYTES + 16 : 0);
}

template <int BN, int MODE>
__global__ void __launch_bounds__(Cfg<BN>::THREADS, 1)
conv_tc_i8_kernel(const ConvProblem p, const int ktab_words)
{
    using C = Cfg<BN>;
    constexpr bool FUSED = MODE == 1, MODULE = MODE == 2;
    constexpr int NBUF = C::NBUF;
    constexpr int STAGES = C::STAGES;
    constexpr int SLOTS = C::SLOTS;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * 8 + 2 * 2];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int ktiles = (p.kwords + 3) >> 2;
    const int m_tiles = (p.M - 1) / BM + 1;                  // M >= 1; no overflow for M close to 2^31
    const int n_tiles = (p.C_out + BN - 1) / BN;
    const int total_tiles = m_tiles * n_tiles;
    const int my_tiles = ((int)blockIdx.x < total_tiles) ? (total_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int total_items = my_tiles * ktiles;

    const uint32_t wring = (smem_u32(smem_raw) + 1023u) & ~1023u;         // [STAGES][BN rows][128 B]
    const uint32_t bits_ring = wring + STAGES * C::W_BYTES;               // [PF][PROD_THREADS][16 B]
    const uint32_t consts = bits_ring + C::BITS_BYTES;                    // [SLOTS][G][BM + BN] int32
    const uint32_t ktab_addr = consts + C::CONST_BYTES;                   // unit table of the gather: {word offset, tap bit}
    const uint32_t idring = (ktab_addr + (uint32_t)ktab_words * 4u + 15u) & ~15u;   // module epilogue only: [ID_SLOTS][BM rows][80 B]
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (8 + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (16 + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (18 + b); };
    volatile int *abort_flag = &abort_flag_smem;

    if (tid == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(full_bar(s), C::GROUP_WARPS);      // every warp of the group that owns the stage
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
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    const int gwidth = gather_width(p.cw);
    build_unit_table(p, ktab_addr, ktiles * (4 / gwidth), gwidth, tid, C::THREADS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;

    if (warp == 0) {
        // ------------------------------------------------------------------ issuer (no memory instructions)
        constexpr uint32_t idesc = make_idesc(BN);
        const uint64_t desc0 = make_desc(0);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32);
        const uint32_t b_lo0 = (uint32_t)desc0 | ((wring & 0x3FFFFu) >> 4);      // + slot * (W_BYTES / 16)
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);             // warp-uniform copy for the issuer
        const uint32_t a_tmem0 = tmem_u + (uint32_t)C::A_COL0;                   // + slot * 32 columns
        int s = 0, buf = 0;
        for (int ti = 0; ti < my_tiles; ++ti) {
            const uint32_t d_tmem = tmem_u + (uint32_t)(buf * BN);
            const uint32_t tfull = tfull_bar(buf);
            for (int kt = 0; kt < ktiles; ++kt) {
                const uint32_t a_t = a_tmem0 + (uint32_t)s * 32u;
                const uint32_t b_lo = b_lo0 + (uint32_t)s * (C::W_BYTES >> 4);
                const int nk = p.kwords - 4 * kt;                 // 32 bits of K per instruction; skip the zero tail
                const uint32_t ebar = empty_bar(s);
                asm volatile("bar.sync %0, 64;" ::"r"(1 + s) : "memory");
                tc_fence_after();
                // per 32 bytes of K: 8 tensor-memory columns of A, +2 (16-byte units) in the B descriptor
                if (elect_one()) {
                    tc_mma_i8_ts(d_tmem, a_t, b_lo, desc_hi, idesc, kt > 0 ? 1u : 0u);
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
        // A stage is released (bar.arrive on 1 + slot) once its ring slot is full and, for a tile's
        // first stage, once the accumulator buffer is free.  The slot being full implies that the
        // issuer is past the previous use of the same named barrier.  After a time-out the remaining
        // stages are released without waiting so that the issuer always terminates.
        int s = 0, buf = 0;
        uint32_t ring_phase = 0, buf_phase = 1;      // first use of every accumulator buffer: free
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
    } else if (warp <= EPI_WARPS) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;                 // tensor-memory lane quadrant this warp may read
        const int erow = quad * 32 + lane;
        bool alive = true;
        int buf = 0;
        uint32_t buf_phase = 0;
        // module epilogue: the identity values of this thread's row are staged ID_AHEAD live chunks ahead (a chunk is
        // live when its first channel exists), in ring slot (live chunk number) % ID_SLOTS
        const uint32_t id_warp = idring + (uint32_t)(quad * 32) * ID_ROW_BYTES;   // slot 0, the warp's first row
        // int32 output, 128-wide tiles: per-warp staging tile behind the (possibly unused) identity ring
        const uint32_t i32_tile = idring + (uint32_t)quad * I32_TILE_BYTES;     // (shares the place of the module's ring)
        int pf_ti = 0, pf_ch = 0, pf_slot = 0, cur_slot = 0;
        auto prefetch_next = [&]() {
            bool queued = false;
            while (pf_ti < my_tiles && !queued) {
                const int t = (int)blockIdx.x + pf_ti * (int)gridDim.x;
                const int nt = t / m_tiles, mt = t - nt * m_tiles;
                const int n = nt * BN + pf_ch * 32;
                if (n < p.C_out) {
                    module_prefetch(p, id_warp + (uint32_t)pf_slot * (BM * ID_ROW_BYTES), (long)mt * BM + quad * 32, n, lane);
                    queued = true;
                }
                if (++pf_ch == BN / 32) { pf_ch = 0; ++pf_ti; }
            }
            if (!queued) cp_async_commit();
            if (++pf_slot == ID_SLOTS) pf_slot = 0;
        };
        if (MODULE)
            for (int a = 0; a < ID_AHEAD; ++a) prefetch_next();
        for (int ti = 0; ti < my_tiles; ++ti) {
            const int tile = (int)blockIdx.x + ti * (int)gridDim.x;
            const int n_tile = tile / m_tiles, m_tile = tile - n_tile * m_tiles;
            const int m0 = m_tile * BM, n0 = n_tile * BN;
            const int em = m0 + erow;
            // which producer groups took part in this tile (each leaves partial constants): both,
            // unless the tile is a single stage
            const int first_group = (ti * ktiles) & 1;
            const bool two = ktiles >= 2;
            const uint32_t slot = consts + (uint32_t)((ti % SLOTS) * C::SLOT_INTS * 4);
            const uint32_t part0 = slot + (uint32_t)(first_group * (BM + BN) * 4);
            const uint32_t part1 = slot + (uint32_t)((first_group ^ 1) * (BM + BN) * 4);
            if (alive) alive = mbar_wait(tfull_bar(buf), buf_phase, abort_flag, p.err, ERR_EPILOGUE_TIMEOUT);
            alive = __all_sync(0xffffffffu, alive && !*abort_flag);
            if (!alive) break;
            tc_fence_after();
            int rowc, rowc1 = 0;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(rowc) : "r"(part0 + 4u * erow) : "memory");
            if (two) asm volatile("ld.shared.b32 %0, [%1];" : "=r"(rowc1) : "r"(part1 + 4u * erow) : "memory");
            rowc += rowc1;
            const uint32_t c0_addr = part0 + 4u * BM, c1_addr = part1 + 4u * BM;
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
                        // bit = (v + rowc + colc >= 0); sign bits are shifted in, last column first
                        uint32_t acc = 0;
#pragma unroll
                        for (int i4 = 7; i4 >= 0; --i4) {
                            uint4 cc = ld_shared_v4(c0_addr + 4u * (col0 + 4 * i4));
                            if (two) {
                                const uint4 c2 = ld_shared_v4(c1_addr + 4u * (col0 + 4 * i4));
                                cc.x += c2.x; cc.y += c2.y; cc.z += c2.z; cc.w += c2.w;
                            }
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 3] + rowc + (int)cc.w), acc, 1);
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 2] + rowc + (int)cc.z), acc, 1);
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 1] + rowc + (int)cc.y), acc, 1);
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 0] + rowc + (int)cc.x), acc, 1);
                        }
                        words[ch] = ~acc;
                    } else if (MODULE) {
                        int dot[32];
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            uint4 cc = ld_shared_v4(c0_addr + 4u * (col0 + 4 * i4));
                            if (two) {
                                const uint4 c2 = ld_shared_v4(c1_addr + 4u * (col0 + 4 * i4));
                                cc.x += c2.x; cc.y += c2.y; cc.z += c2.z; cc.w += c2.w;
                            }
                            dot[4 * i4 + 0] = (int)(v[4 * i4 + 0] >> 5) + rowc + (int)cc.x;
                            dot[4 * i4 + 1] = (int)(v[4 * i4 + 1] >> 5) + rowc + (int)cc.y;
                            dot[4 * i4 + 2] = (int)(v[4 * i4 + 2] >> 5) + rowc + (int)cc.z;
                            dot[4 * i4 + 3] = (int)(v[4 * i4 + 3] >> 5) + rowc + (int)cc.w;
                        }
                        prefetch_next();
                        cp_async_wait<ID_AHEAD>();                    // this chunk's copy has landed
                        words[ch] = module_chunk(p, dot, id_warp + (uint32_t)cur_slot * (BM * ID_ROW_BYTES), (long)em - lane, n0 + col0, lane);
                        if (++cur_slot == ID_SLOTS) cur_slot = 0;
                    } else if (BN == 128 && (p.C_out & 3) == 0 && (n0 + col0 + 32 <= p.C_out)) {
                        // full chunk (warp-uniform): staged, the warp stores whole 128-byte rows
                        int o[32];
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            uint4 cc = ld_shared_v4(c0_addr + 4u * (col0 + 4 * i4));
                            if (two) {
                                const uint4 c2 = ld_shared_v4(c1_addr + 4u * (col0 + 4 * i4));
                                cc.x += c2.x; cc.y += c2.y; cc.z += c2.z; cc.w += c2.w;
                            }
                            o[4 * i4 + 0] = (int)(v[4 * i4 + 0] >> 5) + rowc + (int)cc.x;
                            o[4 * i4 + 1] = (int)(v[4 * i4 + 1] >> 5) + rowc + (int)cc.y;
                            o[4 * i4 + 2] = (int)(v[4 * i4 + 2] >> 5) + rowc + (int)cc.z;
                            o[4 * i4 + 3] = (int)(v[4 * i4 + 3] >> 5) + rowc + (int)cc.w;
                        }
                        const long row0 = (long)em - lane;
                        store_int32_block(static_cast<int32_t *>(p.out) + row0 * p.C_out + n0 + col0, p.C_out, o, i32_tile, row0, p.M, lane);
                    } else if (em < p.M) {
                        int32_t *dst = static_cast<int32_t *>(p.out) + (long)em * p.C_out + n0 + col0;
                        const bool vec = (p.C_out & 3) == 0 && (n0 + col0 + 32 <= p.C_out);
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            uint4 cc = ld_shared_v4(c0_addr + 4u * (col0 + 4 * i4));
                            if (two) {
                                const uint4 c2 = ld_shared_v4(c1_addr + 4u * (col0 + 4 * i4));
                                cc.x += c2.x; cc.y += c2.y; cc.z += c2.z; cc.w += c2.w;
                            }
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
            // all reads of this accumulator buffer are complete: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
            if (++buf == NBUF) { buf = 0; buf_phase ^= 1u; }
            if ((FUSED || (MODULE && p.out != nullptr)) && em < p.M) {
                const int owords = p.C_out >> 5;
                uint32_t *dst = static_cast<uint32_t *>(p.out) + (long)em * owords + (n0 >> 5);
                if ((owords & 3) == 0 && n0 + BN <= p.C_out) {
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
        if (MODULE) cp_async_wait<0>();
    } else {
        // ------------------------------------------------------------------ producers
        const int pw = warp - C::FIRST_PRODUCER_WARP;            // producer warp index
        const int grp = pw / C::GROUP_WARPS, wi = pw - grp * C::GROUP_WARPS;
        const bool is_a = wi < 4;
        // activation warps are matched to tensor-memory lane quadrants (a warp may only touch
        // lanes 32 * (warp % 4) ...): the first four warps of a group have four distinct residues
        const int quad = warp & 3;
        const int row = is_a ? quad * 32 + lane : (wi - 4) * 32 + lane;   // row of the A or of the W tile
        const int ptid = tid - 32 * C::FIRST_PRODUCER_WARP;
        const int crow = is_a ? row : BM + row;                  // index into a constants part
        constexpr uint32_t SLOT_BYTES = C::PROD_THREADS * 16u;
        const uint32_t bits0 = bits_ring + (uint32_t)ptid * 16u, bits_end = bits0 + PF * SLOT_BYTES;
        const uint32_t st_addr0 = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)C::A_COL0;
        const uint32_t lane0 = lane == 0 ? 1u : 0u;
        const bool w16 = (p.kwords & 3) == 0;
        const TileStep step = make_tile_step(p, (uint32_t)BM * gridDim.x);

        // this thread's items: grp, grp + G, ... of the CTA's flattened (tile, stage) list
        // ---- load cursor: tile (n_tile, m_tile) and, per role, the activation row or the weight row
        int l_kt = grp;
        int l_left = total_items > grp ? (total_items - grp + G - 1) / G : 0;
        int l_n = (int)blockIdx.x / m_tiles, l_m = (int)blockIdx.x - l_n * m_tiles;
        RowCursor rc;
        rc.m = (uint32_t)l_m * BM + (uint32_t)row;
        rc.base = 0;
        rc.mask = 0;
        const uint32_t *wrow = p.w;
        bool wok = false;
        if (is_a) row_locate(p, rc);
        auto next_tile = [&]() {             // the CTA's next tile: gridDim.x further along (n_tile, m_tile)
            l_m += (int)gridDim.x;
            if (l_m < m_tiles) {
                if (is_a) row_step(p, step, rc);
            } else {
                do { l_m -= m_tiles; ++l_n; } while (l_m >= m_tiles);
                if (is_a) {
                    rc.m = (uint32_t)l_m * BM + (uint32_t)row;
                    row_locate(p, rc);
                }
            }
        };
        auto tile_ready = [&]() {            // per-tile values of the row after the cursor moved
            if (is_a) {
                row_window(p, step, rc);
            } else {
                const int n = l_n * BN + row;
                wok = n < p.C_out;
                wrow = p.w + (long)(wok ? n : 0) * p.kwords;
            }
        };
        while (l_kt >= ktiles) { l_kt -= ktiles; next_tile(); }
        tile_ready();
        uint32_t l_dst = bits0;
        auto issue_load = [&]() {
            if (is_a) {
                if (gwidth == 4) gather_stage<4>(p.x, rc, ktab_addr + (uint32_t)l_kt * 8u, l_dst);
                else if (gwidth == 2) gather_stage<2>(p.x, rc, ktab_addr + (uint32_t)l_kt * 16u, l_dst);
                else gather_stage<1>(p.x, rc, ktab_addr + (uint32_t)l_kt * 32u, l_dst);
            } else if (w16) {
                cp_async_zfill<16>(l_dst, wok ? wrow + l_kt * 4 : p.w, wok ? 16u : 0u);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int kword = l_kt * 4 + e;
                    const bool ok = wok && kword < p.kwords;
                    cp_async_zfill<4>(l_dst + 4u * e, ok ? wrow + kword : p.w, ok ? 4u : 0u);
                }
            }
            l_dst += SLOT_BYTES;
            if (l_dst == bits_end) l_dst = bits0;
            --l_left;
            l_kt += G;
            if (l_kt >= ktiles) {
                do { l_kt -= ktiles; next_tile(); } while (l_kt >= ktiles);
                tile_ready();
            }
        };

#pragma unroll 1
        for (int i = 0; i < PF - 1; ++i) {
            if (l_left > 0) issue_load();
            cp_async_commit();
        }

        // ---- expand cursor
        uint32_t c_src = bits0;
        int c_ti = 0, c_kt = grp, pop = 0;
        int s = grp;                          // ring slot (G <= STAGES) and its parity
        uint32_t phase = 1;                   // first pass through the ring: slots are free
#pragma unroll 1
        for (int it = grp; it < total_items; it += G) {
            if (l_left > 0) issue_load();
            cp_async_commit();
            cp_async_wait<PF - 1>();
            const uint4 bits = ld_shared_v4(c_src);
            c_src += SLOT_BYTES;
            if (c_src == bits_end) c_src = bits0;
            while (c_kt >= ktiles) { c_kt -= ktiles; ++c_ti; }
            if (!mbar_wait_warp(empty_bar(s), phase, abort_flag, p.err, ERR_PRODUCER_TIMEOUT)) break;
            pop += __popc(bits.x) + __popc(bits.y) + __popc(bits.z) + __popc(bits.w);
            if (c_kt + G >= ktiles) {
                // this group's last stage of the tile: leave its partial constants for the epilogue.
                //   fused: bit = acc - 64*pa - 32*(thr - K + 2*pg) >= 0      int32: (acc >> 5) - 2*pa + K - 2*pg
                // the term that does not depend on the popcounts goes with the group of the tile's first stage
                const bool first_group = ((c_ti * ktiles) & 1) == grp;
                int cst = FUSED ? -64 * pop : -2 * pop;
                if (!is_a && first_group) {
                    const int tile = (int)blockIdx.x + c_ti * (int)gridDim.x;
                    const int n = (tile / m_tiles) * BN + row;
                    // (a threshold beyond +-(K + 1) decides like that bound; clamping keeps the constant inside int32)
                    const int thr_n = max(min((FUSED && n < p.C_out) ? __ldg(p.thr + n) : 0, p.K + 1), -p.K - 1);
                    cst += FUSED ? -32 * (thr_n - p.K) : p.K;
                }
                const uint32_t part = consts + (uint32_t)(((c_ti % SLOTS) * C::SLOT_INTS + grp * (BM + BN) + crow) * 4);
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(part), "r"(cst) : "memory");
                pop = 0;
            }
            if (is_a) {
                tc_fence_after();     // the MMAs that read this slot are complete (their commit released it)
                // expanded row -> 32 columns of this lane: column 8*e + j = word j of K word e (bytes 0 or 2^j)
                uint32_t v[32];
                const uint32_t wds[4] = {bits.x, bits.y, bits.z, bits.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[8 * e + j] = wds[e] & (0x01010101u << j);
                tc_st32(st_addr0 + (uint32_t)s * 32u, v);
                tc_fence_before();
            } else {
                const uint32_t row_addr = wring + (uint32_t)s * C::W_BYTES + (uint32_t)row * ROWB;
                const int xr = row & 7;
                expand_store_w(bits.x, row_addr, xr, 0);
                expand_store_w(bits.y, row_addr, xr, 2);
                expand_store_w(bits.z, row_addr, xr, 4);
                expand_store_w(bits.w, row_addr, xr, 6);
                fence_async_proxy();  // generic-proxy stores -> visible to the MMA (async proxy)
            }
            __syncwarp();
            mbar_arrive_pred(full_bar(s), lane0);
            s += G;
            if (s >= STAGES) { s -= STAGES; phase ^= 1u; }
            c_kt += G;
        }
        cp_async_wait<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

int ktab_words_for(const ConvProblem &p)
{
    return ((p.kwords + 3) >> 2) * 8;        // at most four units of two words per 128-bit stage
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
    const int ktw = ktab_words_for(p);
    const int smem = smem_bytes<BN>(ktw, p.mode);
    if (smem > MAX_SMEM) return BCNN_ERR_UNSUPPORTED;
    void (*k)(const ConvProblem, const int) = p.mode == 2 ? conv_tc_i8_kernel<BN, 2> : (p.mode == 1 ? conv_tc_i8_kernel<BN, 1> : conv_tc_i8_kernel<BN, 0>);
    // the attribute is a property of the kernel, not of the launch: always the limit, so that a captured
    // launch stays valid whatever later calls with other shapes ask for
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM) != cudaSuccess) return BCNN_ERR_CUDA;
    k<<<grid, Cfg<BN>::THREADS, smem, stream>>>(p, ktw);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace

bool conv_tc_i8_supports(const ConvProblem &p)
{
    if (p.mode != 0 && (p.C_out % 32 != 0)) return false;
    if (p.kh * p.kw > 31) return false;                       // one validity bit per tap
    if ((long)p.B * p.H * p.W * p.cw >= (1L << 31)) return false;     // rows address the input by 32-bit word offsets
    if (smem_bytes<256>(ktab_words_for(p)) > MAX_SMEM) return false;   // the K-word table of the gather must fit
    // the epilogue constants (about 3K << 5) must stay below 2^31
    return p.K <= (1 << 20);
}

int launch_conv_tc_i8(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_tc_i8_supports(p)) return BCNN_ERR_UNSUPPORTED;
    // 256-wide tiles have a single accumulator buffer (tensor memory also holds the activation
    // ring), so their epilogue is not overlapped: worth it only when the K loop is long
    // (the module epilogue's staging ring only fits beside the 128-wide tiles' weight ring)
    // (int32 output up to K = 4608: the 128-wide tiles' staged stores, whole 128-byte rows, outweigh their extra expansion)
    if (p.C_out > 128 && p.kwords >= 24 && p.mode != 2 && !(p.mode == 0 && p.kwords <= 144)) {
        // ... unless the narrower tiles fill the last wave so much better that they win anyway: a 128-wide tile
        // costs about 0.6 of a 256-wide one (measured on the K = 2304 and K = 4608 layers)
        int dev = 0, sms = 148;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const long m_tiles = ((long)p.M + BM - 1) / BM;
        const long waves256 = (m_tiles * ((p.C_out + 255) / 256) + sms - 1) / sms;
        const long waves128 = (m_tiles * ((p.C_out + 127) / 128) + sms - 1) / sms;
        if (10 * waves256 <= 6 * waves128) return launch_bn<256>(p, stream);
        return launch_bn<128>(p, stream);
    }
    return launch_bn<128>(p, stream);
}

}  // namespace bcnn
