// Streaming tcgen05 engine on PREPARED weights: wide layers and long K (C_out > 128, the plain GEMMs).
//
// The weights of a layer never change between calls, yet the streaming engine (conv_tc_i8.cu) expands the same weight
// bits to bytes again for every 128-row tile: with 256-wide tiles two thirds of its producer warps do nothing else,
// and the MMA issuer waits for them five sixths of the time.  Here the expansion is done ONCE per layer by
// bcnn_prepare_weights into a caller-owned buffer (the weight matrix as signed bytes, K-major, rows padded to 128
// and K to 128; plus K - 2 popc(W_n) per row), and the kernel's weight operand arrives by TMA: one
// cp.async.bulk.tensor per ring stage (a 128-byte x BN-row box, 128-byte swizzle - exactly the shared-memory tile
// the MMA descriptor describes) issued by a loader warp, completing on the stage's mbarrier.  No warp touches a
// weight byte.
//
// Arithmetic: the weight-stationary engine's signed scheme (activation bytes {0, 2^j}, weight bytes +-2^(6-j), every
// product +-64): accumulator = 64 S,  sum a*g = 2 S + K - 2 popc(G):
//   int32 output:  (acc >> 5) + cst_n              cst_n = K - 2 popc(G_n)   (from the prepared buffer)
//   packed output: acc + 32 (cst_n - thr_n) >= 0   thr clamped to +-(K + 1)
// so there are no per-row constants, and the per-column ones are added by the epilogue from a small table.
//
//   warp 0        issuer (tcgen05.mma / commit only; waits on named barriers only)
//   warps 1-4     epilogue: build the tile's column table, tcgen05.ld, add + sign bits (or int32), store
//   G groups of 4 activation warps: implicit-im2col gather (cp.async), expansion, tcgen05.st into the ring in tensor memory
//   loader warp   weight tiles by TMA into the ring in shared memory
//   control warp  the issuer's mbarrier waits
// Every mbarrier wait is bounded and reports through the device error word.
#include "tc_common.cuh"
#include <cuda.h>

namespace bcnn {

namespace {

using namespace tc;

constexpr int EPI_WARPS = 4;
constexpr int G = 2;                      // activation producer groups
constexpr int PF = 3;                     // packed-word stages in flight per producer thread
constexpr int MAX_SMEM = 227 * 1024 - 512;

constexpr int ERR_PRODUCER_TIMEOUT = 131;
constexpr int ERR_MMA_TIMEOUT = 132;
constexpr int ERR_EPILOGUE_TIMEOUT = 133;
constexpr int ERR_LOADER_TIMEOUT = 134;

template <int BN> struct Cfg {
    static constexpr int NBUF = BN == 256 ? 1 : 2;                       // accumulator buffers
    static constexpr int A_COL0 = NBUF * BN;                              // first column of the activation ring
    static constexpr int STAGES = BN == 256 ? 5 : 8;
    static constexpr int PROD_THREADS = G * BM;
    static constexpr int FIRST_PRODUCER_WARP = 1 + EPI_WARPS;
    static constexpr int LOADER_WARP = FIRST_PRODUCER_WARP + 4 * G;
    static constexpr int CONTROL_WARP = LOADER_WARP + 1;
    static constexpr int THREADS = 32 * (CONTROL_WARP + 1);
    static constexpr int W_BYTES = BN * ROWB;                             // one ring stage of weights
    static constexpr int BITS_BYTES = PF * PROD_THREADS * 16;
    static constexpr int TABLE_BYTES = EPI_WARPS * BN * 4;                // one column table per epilogue warp
    static_assert(A_COL0 + STAGES * 32 <= 512, "tensor memory budget");
    static_assert(STAGES >= G, "a producer group must not lap the ring (parity waits)");
};

template <int BN>
__host__ __device__ inline int smem_bytes(int ktab_words, int mode)
{
    using C = Cfg<BN>;
    return 1024 + C::STAGES * C::W_BYTES + C::BITS_BYTES + C::TABLE_BYTES + ktab_words * 4 + 16 +
           (mode == 0 ? EPI_WARPS * I32_TILE_BYTES + 16 : 0);
}

template <int BN, int MODE>
__global__ void __launch_bounds__(Cfg<BN>::THREADS, 1)
conv_tc_pre_kernel(const ConvProblem p, const int32_t *cst, const __grid_constant__ CUtensorMap wmap, const int ktab_words)
{
    using C = Cfg<BN>;
    constexpr bool FUSED = MODE == 1;
    constexpr int NBUF = C::NBUF;
    constexpr int STAGES = C::STAGES;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * 8 + 2 * 2];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int ktiles = (p.kwords + 3) >> 2;
    const int m_tiles = (p.M - 1) / BM + 1;
    const int n_tiles = (p.C_out + BN - 1) / BN;
    const int total_tiles = m_tiles * n_tiles;
    const int my_tiles = ((int)blockIdx.x < total_tiles) ? (total_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int total_items = my_tiles * ktiles;

    const uint32_t wring = (smem_u32(smem_raw) + 1023u) & ~1023u;         // [STAGES][BN rows][128 B], written by TMA
    const uint32_t bits_ring = wring + STAGES * C::W_BYTES;               // [PF][PROD_THREADS][16 B]
    const uint32_t tables = bits_ring + C::BITS_BYTES;                    // [EPI_WARPS][BN] int32 column constants
    const uint32_t ktab_addr = tables + C::TABLE_BYTES;                   // unit table of the gather: {word offset, tap bit}
    const uint32_t i32_tiles = (ktab_addr + (uint32_t)ktab_words * 4u + 15u) & ~15u;   // int32 output: store staging tiles
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (8 + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (16 + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (18 + b); };
    volatile int *abort_flag = &abort_flag_smem;

    if (tid == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(full_bar(s), 4 + 1);           // the four activation warps of the stage's group + the loader's arrive (+ its bytes)
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
        constexpr uint32_t idesc = make_idesc(BN) | (1u << 10);                  // B operand: signed bytes
        const uint64_t desc0 = make_desc(0);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32);
        const uint32_t b_lo0 = (uint32_t)desc0 | ((wring & 0x3FFFFu) >> 4);      // + slot * (W_BYTES / 16)
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
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
        // A stage is released (bar.arrive on 1 + slot) once its ring slot is full (activations expanded, weights
        // landed) and, for a tile's first stage, once the accumulator buffer is free.  After a time-out the
        // remaining stages are released by bar.sync, which pairs every release with one wait of the issuer.
        int s = 0, buf = 0;
        uint32_t ring_phase = 0, buf_phase = 1;      // first use of every accumulator buffer: free
        bool alive = true;
        for (int ti = 0; ti < my_tiles; ++ti) {
            if (lane == 0 && alive) alive = mbar_wait(tempty_bar(buf), buf_phase, abort_flag, p.err, ERR_MMA_TIMEOUT);
            for (int kt = 0; kt < ktiles; ++kt) {
                if (lane == 0 && alive) alive = mbar_wait(full_bar(s), ring_phase, abort_flag, p.err, ERR_MMA_TIMEOUT);
                if (__shfl_sync(0xffffffffu, alive ? 1 : 0, 0)) asm volatile("bar.arrive %0, 64;" ::"r"(1 + s) : "memory");
                else asm volatile("bar.sync %0, 64;" ::"r"(1 + s) : "memory");
                if (++s == STAGES) { s = 0; ring_phase ^= 1u; }
            }
            if (++buf == NBUF) { buf = 0; buf_phase ^= 1u; }
        }
    } else if (warp == C::LOADER_WARP) {
        // ------------------------------------------------------------------ loader: weight tiles by TMA
        // item (tile, stage) -> ring slot item % STAGES; box = 128 bytes of K x BN rows at (kt * 128, n_tile * BN)
        int s = 0;
        uint32_t phase = 1;                           // first pass through the ring: slots are free
        int issued = 0;
        for (int ti = 0; ti < my_tiles; ++ti) {
            const int tile = (int)blockIdx.x + ti * (int)gridDim.x;
            const int n_row0 = (tile / m_tiles) * BN;
            bool ok = true;
            for (int kt = 0; kt < ktiles; ++kt) {
                ok = mbar_wait_warp(empty_bar(s), phase, abort_flag, p.err, ERR_LOADER_TIMEOUT);
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t dst = wring + (uint32_t)s * C::W_BYTES;
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full_bar(s)), "r"((uint32_t)C::W_BYTES) : "memory");
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(&wmap)), "r"(kt * ROWB), "r"(n_row0), "r"(full_bar(s)) : "memory");
                }
                __syncwarp();
                ++issued;
                if (++s == STAGES) { s = 0; phase ^= 1u; }
            }
            if (!ok) break;
        }
        // after a time-out elsewhere: copies still in flight must land before the CTA's shared memory goes away
        if (*abort_flag) {
            const int first = issued > STAGES ? issued - STAGES : 0;
            for (int it = first; it < issued; ++it)
                mbar_wait_warp(full_bar(it % STAGES), (uint32_t)(it / STAGES) & 1u, abort_flag, nullptr, 0);
        }
    } else if (warp <= EPI_WARPS) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;                 // tensor-memory lane quadrant this warp may read
        const int erow = quad * 32 + lane;
        const uint32_t i32_tile = i32_tiles + (uint32_t)quad * I32_TILE_BYTES;
        bool alive = true;
        int buf = 0;
        uint32_t buf_phase = 0;
        for (int ti = 0; ti < my_tiles; ++ti) {
            const int tile = (int)blockIdx.x + ti * (int)gridDim.x;
            const int n_tile = tile / m_tiles, m_tile = tile - n_tile * m_tiles;
            const int m0 = m_tile * BM, n0 = n_tile * BN;
            const int em = m0 + erow;
            // this tile's column constants, built while its MMAs run; every warp keeps its own table, so the four
            // warps need no barrier among themselves
            const uint32_t table = tables + (uint32_t)(quad * BN * 4);
            for (int c = lane; c < BN; c += 32) {
                const int n = n0 + c;
                int v = 0;
                if (n < p.C_out) {
                    v = __ldg(cst + n);
                    if (FUSED) {
                        int t = __ldg(p.thr + n);
                        t = max(min(t, p.K + 1), -p.K - 1);       // beyond that bound the decision is constant
                        v = 32 * (v - t);
                    }
                }
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(table + 4u * c), "r"(v) : "memory");
            }
            __syncwarp();
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
                if (n0 + col0 < p.C_out) {             // warp-uniform
                    uint32_t v[32];
                    tc_ld32(t_addr + (uint32_t)col0, v);
                    if (FUSED) {
                        // bit = (v + colc >= 0); sign bits are shifted in, last column first
                        uint32_t acc = 0;
#pragma unroll
                        for (int i4 = 7; i4 >= 0; --i4) {
                            const uint4 cc = ld_shared_v4(table + 4u * (col0 + 4 * i4));
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 3] + (int)cc.w), acc, 1);
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 2] + (int)cc.z), acc, 1);
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 1] + (int)cc.y), acc, 1);
                            acc = __funnelshift_l((uint32_t)((int)v[4 * i4 + 0] + (int)cc.x), acc, 1);
                        }
                        words[ch] = ~acc;
                    } else {
                        int o[32];
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            const uint4 cc = ld_shared_v4(table + 4u * (col0 + 4 * i4));
                            o[4 * i4 + 0] = ((int)v[4 * i4 + 0] >> 5) + (int)cc.x;
                            o[4 * i4 + 1] = ((int)v[4 * i4 + 1] >> 5) + (int)cc.y;
                            o[4 * i4 + 2] = ((int)v[4 * i4 + 2] >> 5) + (int)cc.z;
                            o[4 * i4 + 3] = ((int)v[4 * i4 + 3] >> 5) + (int)cc.w;
                        }
                        if ((p.C_out & 3) == 0 && (n0 + col0 + 32 <= p.C_out)) {
                            // full chunk (warp-uniform): staged, the warp stores whole 128-byte rows
                            const long row0 = (long)em - lane;
                            store_int32_block(static_cast<int32_t *>(p.out) + row0 * p.C_out + n0 + col0, p.C_out, o, i32_tile, row0, p.M, lane);
                        } else if (em < p.M) {
                            int32_t *dst = static_cast<int32_t *>(p.out) + (long)em * p.C_out + n0 + col0;
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (n0 + col0 + i < p.C_out) dst[i] = o[i];
                        }
                    }
                }
            }
            // all reads of this accumulator buffer are complete: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
            if (++buf == NBUF) { buf = 0; buf_phase ^= 1u; }
            if (FUSED && em < p.M) {
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
    } else {
        // ------------------------------------------------------------------ activation producers
        // Group g takes items g, g + G, ... of the CTA's flattened (tile, stage) list: a thread copies its row's 128
        // bits of K into its staging slot (PF items ahead), then expands the oldest staged item into the ring slot.
        const int ptid = tid - 32 * C::FIRST_PRODUCER_WARP;
        const int grp = ptid >> 7;
        const int quad = warp & 3;                               // tensor-memory lane quadrant this warp may write
        const int row = quad * 32 + lane;
        constexpr uint32_t SLOT_BYTES = C::PROD_THREADS * 16u;
        const uint32_t bits0 = bits_ring + (uint32_t)ptid * 16u, bits_end = bits0 + PF * SLOT_BYTES;
        const uint32_t st_addr0 = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)C::A_COL0;
        const uint32_t lane0 = lane == 0 ? 1u : 0u;
        const TileStep step = make_tile_step(p, (uint32_t)BM * gridDim.x);

        int l_kt = grp;
        int l_left = total_items > grp ? (total_items - grp + G - 1) / G : 0;
        int l_n = (int)blockIdx.x / m_tiles, l_m = (int)blockIdx.x - l_n * m_tiles;
        RowCursor rc;
        rc.m = (uint32_t)l_m * BM + (uint32_t)row;
        rc.base = 0;
        rc.mask = 0;
        row_locate(p, rc);
        auto next_tile = [&]() {             // the CTA's next tile: gridDim.x further along (n_tile, m_tile)
            l_m += (int)gridDim.x;
            if (l_m < m_tiles) {
                row_step(p, step, rc);
            } else {
                do { l_m -= m_tiles; ++l_n; } while (l_m >= m_tiles);
                rc.m = (uint32_t)l_m * BM + (uint32_t)row;
                row_locate(p, rc);
            }
        };
        while (l_kt >= ktiles) { l_kt -= ktiles; next_tile(); }
        row_window(p, step, rc);
        uint32_t l_dst = bits0;
        auto issue_load = [&]() {
            if (gwidth == 4) gather_stage<4>(p.x, rc, ktab_addr + (uint32_t)l_kt * 8u, l_dst);
            else if (gwidth == 2) gather_stage<2>(p.x, rc, ktab_addr + (uint32_t)l_kt * 16u, l_dst);
            else gather_stage<1>(p.x, rc, ktab_addr + (uint32_t)l_kt * 32u, l_dst);
            l_dst += SLOT_BYTES;
            if (l_dst == bits_end) l_dst = bits0;
            --l_left;
            l_kt += G;
            if (l_kt >= ktiles) {
                do { l_kt -= ktiles; next_tile(); } while (l_kt >= ktiles);
                row_window(p, step, rc);
            }
        };
#pragma unroll 1
        for (int i = 0; i < PF - 1; ++i) {
            if (l_left > 0) issue_load();
            cp_async_commit();
        }
        uint32_t c_src = bits0;
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
            // expanded row -> 32 columns of this lane: column 8*e + j = word j of K word e
            uint32_t v[32];
            const uint32_t wds[4] = {bits.x, bits.y, bits.z, bits.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) expand_a(wds[e], &v[8 * e]);
            if (!mbar_wait_warp(empty_bar(s), phase, abort_flag, p.err, ERR_PRODUCER_TIMEOUT)) break;
            tc_fence_after();     // the MMAs that read this slot are complete (their commit released it)
            tc_st32(st_addr0 + (uint32_t)s * 32u, v);
            tc_fence_before();
            __syncwarp();
            mbar_arrive_pred(full_bar(s), lane0);
            s += G;
            if (s >= STAGES) { s -= STAGES; phase ^= 1u; }
        }
        cp_async_wait<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// One weight word -> its 32 signed bytes (see expand_store_w_signed in tc_common.cuh: magnitude 2^(6-j), 1 for j = 7),
// written as two 16-byte pieces of the row; K-major rows of k_pad bytes, padded rows and K words are zero.
__global__ void __launch_bounds__(256)
prepare_weights_kernel(const uint32_t *w, uint8_t *wexp, int32_t *cst, int N, int kwords, int n_pad, int k_pad)
{
    const int kw_pad = k_pad / 32;
    const long total = (long)n_pad * kw_pad;
    for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
        const int kw = (int)(i % kw_pad), n = (int)(i / kw_pad);
        const bool live = n < N && kw < kwords;
        const uint32_t word = live ? __ldg(w + (long)n * kwords + kw) : 0u;
        const uint32_t nr = ~__byte_perm(__brev(word), 0u, 0x0123u);
        uint32_t o[8];
#pragma unroll
        for (int j = 0; j < 7; ++j)
            o[j] = live ? (nr & (0x01010101u << (7 - j))) * ((2u << j) - 1u) + (0x01010101u << (6 - j)) : 0u;
        o[7] = live ? (nr & 0x01010101u) * 0xFEu + 0x01010101u : 0u;
        uint4 *dst = reinterpret_cast<uint4 *>(wexp + (long)n * k_pad + (long)kw * 32);
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
    for (long n = (long)blockIdx.x * blockDim.x + threadIdx.x; n < n_pad; n += (long)gridDim.x * blockDim.x) {
        int pop = 0;
        if (n < N)
            for (int kw = 0; kw < kwords; ++kw) pop += __popc(__ldg(w + n * kwords + kw));
        cst[n] = n < N ? kwords * 32 - 2 * pop : 0;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

int ktab_words_for(const ConvProblem &p) { return ((p.kwords + 3) >> 2) * 8; }

template <int BN>
int launch_bn(const ConvProblem &p0, const PreparedWeights &pw, cudaStream_t stream)
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
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return BCNN_ERR_CUDA;
    CUtensorMap wmap;
    const cuuint64_t dims[2] = {(cuuint64_t)pw.k_pad, (cuuint64_t)pw.n_pad};
    const cuuint64_t strides[1] = {(cuuint64_t)pw.k_pad};
    const cuuint32_t box[2] = {(cuuint32_t)ROWB, (cuuint32_t)BN};
    const cuuint32_t estr[2] = {1, 1};
    if (encode(&wmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t *>(pw.wexp), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return BCNN_ERR_CUDA;
    void (*k)(const ConvProblem, const int32_t *, const CUtensorMap, const int) = p.mode == 1 ? conv_tc_pre_kernel<BN, 1> : conv_tc_pre_kernel<BN, 0>;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM) != cudaSuccess) return BCNN_ERR_CUDA;
    k<<<grid, Cfg<BN>::THREADS, smem, stream>>>(p, pw.cst, wmap, ktw);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace

void prepared_layout(int C_out, int K, PreparedWeights &pw, size_t &bytes)
{
    pw.n_pad = (C_out + 127) / 128 * 128;
    pw.k_pad = (K + 127) / 128 * 128;
    const size_t wbytes = (size_t)pw.n_pad * pw.k_pad;          // a multiple of 16384
    bytes = wbytes + (size_t)pw.n_pad * 4;
    pw.wexp = nullptr;
    pw.cst = nullptr;
}

int launch_prepare_weights(const uint32_t *w, void *prepared, int C_out, int K, cudaStream_t stream)
{
    PreparedWeights pw;
    size_t bytes;
    prepared_layout(C_out, K, pw, bytes);
    uint8_t *wexp = static_cast<uint8_t *>(prepared);
    int32_t *cst = reinterpret_cast<int32_t *>(wexp + (size_t)pw.n_pad * pw.k_pad);
    const long total = (long)pw.n_pad * (pw.k_pad / 32);
    const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
    prepare_weights_kernel<<<blocks, 256, 0, stream>>>(w, wexp, cst, C_out, K / 32, pw.n_pad, pw.k_pad);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

// ---- the variant that allocates nothing -------------------------------------------------------------------------
// Some callers cannot hand the library a buffer for the prepared weights because they cannot allocate device memory
// at all at the point where they call: code that runs inside somebody else's memory plan (an inference server whose
// arena is sized before the model's layers are known, a plug-in that only ever receives its input and output
// tensors), or code running while allocation is forbidden or would synchronise the device.  For them the prepared
// form lives in this array: it is part of the library's image, so every GPU that loads the library holds these
// STATIC_PREPARED_BYTES until the process exits.  The host-side name of a __device__ array is only a stand-in; the
// kernels need its device address, fetched once per device with cudaGetSymbolAddress.
constexpr size_t STATIC_PREPARED_BYTES = (size_t)4 << 20;
static __device__ __align__(256) unsigned char g_static_prepared[STATIC_PREPARED_BYTES];

size_t static_prepared_capacity() { return STATIC_PREPARED_BYTES; }

// Device address of the array on the current device (nullptr on failure); looked up on a device's first call.
static void *static_prepared_address()
{
    static void *cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cache[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_prepared) != cudaSuccess) return nullptr;
        cache[dev] = ptr;
    }
    return cache[dev];
}

int launch_conv_tc_pre_static(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_tc_pre_supports(p)) return BCNN_ERR_UNSUPPORTED;
    PreparedWeights pw;
    size_t bytes = 0;
    prepared_layout(p.C_out, p.K, pw, bytes);
    if (bytes > STATIC_PREPARED_BYTES) return BCNN_ERR_WORKSPACE;
    void *scratch = static_prepared_address();
    if (!scratch) return BCNN_ERR_CUDA;
    // the expansion rewrites every byte of the layout it uses (padding rows and K words as zeros), so nothing of an
    // earlier call's contents is ever read
    const int st = launch_prepare_weights(p.w, scratch, p.C_out, p.K, stream);
    if (st != BCNN_OK) return st;
    return launch_conv_tc_pre(p, scratch, stream);
}

bool conv_tc_pre_supports(const ConvProblem &p)
{
    if (p.mode != 0 && p.mode != 1) return false;
    if (p.mode == 1 && (p.C_out % 32 != 0)) return false;
    if (p.kh * p.kw > 31) return false;                       // one validity bit per tap
    if ((long)p.B * p.H * p.W * p.cw >= (1L << 31)) return false;     // rows address the input by 32-bit word offsets
    if (smem_bytes<256>(ktab_words_for(p), p.mode) > MAX_SMEM) return false;
    return p.K <= (1 << 20);                                  // 64 K + 32 (2 K + 1) stays far below 2^31
}

int launch_conv_tc_pre(const ConvProblem &p, const void *prepared, cudaStream_t stream)
{
    if (!conv_tc_pre_supports(p)) return BCNN_ERR_UNSUPPORTED;
    PreparedWeights pw;
    size_t bytes;
    prepared_layout(p.C_out, p.K, pw, bytes);
    pw.wexp = static_cast<const uint8_t *>(prepared);
    pw.cst = reinterpret_cast<const int32_t *>(pw.wexp + (size_t)pw.n_pad * pw.k_pad);
    // 256-wide tiles have a single accumulator buffer (their epilogue is not overlapped): worth it when the K loop is
    // long and the narrower tiles do not fill the last wave so much better (as in the streaming engine)
    if (p.C_out > 128 && p.kwords >= 24) {
        int dev = 0, sms = 148;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const long m_tiles = ((long)p.M + BM - 1) / BM;
        const long waves256 = (m_tiles * ((p.C_out + 255) / 256) + sms - 1) / sms;
        const long waves128 = (m_tiles * ((p.C_out + 127) / 128) + sms - 1) / sms;
        if (10 * waves256 <= 6 * waves128) return launch_bn<256>(p, pw, stream);
    }
    return launch_bn<128>(p, pw, stream);
}

}  // namespace bcnn
