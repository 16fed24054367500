// Wide pointwise engine: binary 1x1 convolutions (stride 1, no padding) and plain GEMMs with K = 256 or 512 bits and
// 128, 256 or 512 output channels, packed output - the deeper binary 1x1 convolutions of the paper's network (Section
// 4.2.1; Table 1: 256 and 512 channels at 56 x 56 ... 14 x 14).  A 128-row tile of such a layer is only 8 or 16 words of
// K per row and a few hundred tensor-pipe cycles per 128 output channels: the engines that cut the output channels
// into slices and walk the rows once per slice expand every activation row once per slice and pay a pipeline's
// start-up per slice and tile.
//
// Here a tile's activations are expanded ONCE and multiplied against all the weight slices the CTA keeps in shared
// memory (RS slices of 128 output channels, expanded once per CTA: all of a K = 256 layer, one slice of a K = 512
// layer - then the CTAs form C_out / 128 groups, one per slice, and each group walks all row tiles).
//   * A row tile is a contiguous block of x (128 rows x K / 8 bytes): one bulk asynchronous copy (cp.async.bulk) per tile
//     into a ring in shared memory, two loader warps taking alternate tiles.
//   * Tensor memory: two accumulators and a ring of activation UNITS of eight K words (64 columns); a tile is one unit
//     (K = 256) or two (K = 512, filled by two producer groups).  Four producer groups of four warps (thread = row: two
//     16-byte shared-memory loads, 64 logic operations, two tensor-memory stores).
//   * A tile's output channels are cut into PARTS of AW channels: 128 for K = 256 (three units = three tiles fit beside
//     the accumulators), 64 for K = 512 (five units = two and a half tiles).  Two issuer warps walk the tiles in order
//     and take alternate parts, each with its own accumulator and epilogue group: per part an issuer waits for its
//     accumulator, issues the constant MMA (the per-channel constants of up to four slices sit side by side in one
//     operand tile) and the K / 32 MMAs, and commits on the part's "done" barrier.  One issuer's waits, fence and commit
//     between two parts take about as long as a short part's MMAs run (measured: one issuer kept the tensor pipe 47 %
//     busy); with two, one's MMAs run during the other's bookkeeping.
//   * The producers that reuse a unit wait for the last part of each issuer of the tile that used it.
// Arithmetic as in the other tcgen05 engines: activation bytes {0, 2^j}, signed weight bytes, every product +-64,
// accumulator = 32 (dot - threshold), output bit = (accumulator >= 0).  K = 256: |accumulator| < 2^15, packed 16-bit
// loads and byte-permute sign gathering (the weight rows are laid out in that gathering's column order).
// "Done" numbers d = tile * parts + part use barrier d % 64.  A parity wait is only right while the waiter starts waiting
// for completion k after k - 1 and before k + 1: the epilogue group of d takes its barrier's completions in turn, and
// its issuer cannot get past part d + 2 (it needs the accumulator of d back), let alone to d + 64; the producers that
// wait for d are those of a tile at most three tiles later, which both issuers issue before the tile of d + 64 (a tile
// has at most eight parts).
// Every mbarrier wait is bounded and reports through the device error word.
#include "tc_slot.cuh"

namespace bcnn {

namespace {

using namespace tc;

constexpr int ERR_PN_LOADER_TIMEOUT = 151;       // loader: no free ring stage
constexpr int ERR_PN_PRODUCER_TIMEOUT = 152;     // producer: the tile's rows did not arrive
constexpr int ERR_PN_ISSUER_TIMEOUT = 153;       // issuer: a tile's activations were not filled
constexpr int ERR_PN_EPILOGUE_TIMEOUT = 154;     // epilogue: a slice's MMAs did not complete
constexpr int ERR_PN_UNIT_TIMEOUT = 155;         // producer: the unit's previous MMAs did not complete
constexpr int ERR_PN_ACC_TIMEOUT = 156;          // issuer: an accumulator was not handed back

constexpr int NGRP = 2;                   // loader / epilogue groups
constexpr int NPG = 4;                    // producer groups of four warps
constexpr int RD = 4;                     // row tiles in a loader's ring
constexpr int CONST_COLS = 8;
constexpr int UWORDS = 8;                 // K words per unit
constexpr int U_COLS = 8 * UWORDS;
constexpr int BN = 128;                   // output channels per weight slice (rows of a weight tile)
constexpr int NB = 64, NAF = 8;
constexpr int NISS = 2;                   // issuer warps (parts alternate)
constexpr int MAX_NACC = 4;
constexpr int C_COL = 448;                 // accumulators and units share the columns below (7 x 64)
static_assert(C_COL + CONST_COLS <= 512, "tensor memory budget");
constexpr int FIRST_LOADER_WARP = 2, FIRST_PRODUCER_WARP = 4, FIRST_EPILOGUE_WARP = 4 + 4 * NPG;
constexpr int WARPS = 4 + 4 * NPG + 4 * NGRP;
constexpr int THREADS = 32 * WARPS;
constexpr int W_TILE_BYTES = BN * ROWB;   // one 128-bit stage of one slice's expanded weights

struct PnPlan {
    int rs;            // resident slices per CTA (1, 2 or 4)
    int ng;            // CTA groups = slices / rs
    int m_tiles;
};

// UPT: units per tile = K / 256; AW: accumulator columns = output channels per part (128 for K = 256, 64 for K = 512).
template <int UPT, int AW>
__global__ void __launch_bounds__(THREADS, 1)
conv_tc_pn_kernel(const ConvProblem p, const PnPlan plan)
{
    constexpr int KWORDS = UWORDS * UPT, KT = KWORDS / 4;
    constexpr bool PACK16 = UPT == 1;
    constexpr int TILE_BYTES = BM * KWORDS * 4;
    constexpr int NBARS = 2 * NGRP * RD + NAF + NB + MAX_NACC;
    // an accumulator per issuer / epilogue group.  K = 256: parts of 128 channels (nine MMAs of 64 columns would be 288
    // tensor-pipe cycles, less than the issuer's and the epilogue's fixed work per part) and three units = three tiles;
    // K = 512: parts of 64 channels and five units = two and a half tiles
    constexpr int NACC = 2, NUNIT = (C_COL - NACC * AW) / U_COLS;           // 3 units beside 2 x 128 columns, 5 beside 2 x 64
    constexpr int A_COL0 = NACC * AW;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[NBARS];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int RS = plan.rs, PARTS = (BN / AW) * plan.rs;   // resident slices, parts (AW channels) per tile
    // CTA group cg keeps the slices cg * RS .. cg * RS + RS - 1; the CTAs of a group share the row tiles
    const int cg = (int)blockIdx.x % plan.ng, idx = (int)blockIdx.x / plan.ng, per_group = (int)gridDim.x / plan.ng;
    const int my_tiles = idx < plan.m_tiles ? (plan.m_tiles - 1 - idx) / per_group + 1 : 0;
    auto row_tile = [&](int n) { return idx + n * per_group; };

    const uint32_t wexp = (smem_u32(smem_raw) + 1023u) & ~1023u;          // [RS][KT][128 rows][128 B] expanded weights
    const uint32_t cexp = wexp + (uint32_t)(RS * KT) * W_TILE_BYTES;      // [128 rows][128 B]: 32-byte piece s = constants of slice s
    const uint32_t ring = cexp + W_TILE_BYTES;                            // [NGRP][RD] row tiles
    const uint32_t bar0 = smem_u32(bars);
    auto load_full = [&](int gr, int s) { return bar0 + 8u * (gr * RD + s); };
    auto load_empty = [&](int gr, int s) { return bar0 + 8u * (NGRP * RD + gr * RD + s); };
    auto a_full = [&](int s) { return bar0 + 8u * (2 * NGRP * RD + s); };
    auto tile_done = [&](int s) { return bar0 + 8u * (2 * NGRP * RD + NAF + s); };
    auto acc_free = [&](int s) { return bar0 + 8u * (2 * NGRP * RD + NAF + NB + s); };
    volatile int *abort_flag = &abort_flag_smem;

    if (tid == 0) {
        for (int s = 0; s < NGRP * RD; ++s) {
            mbar_init(load_full(0, s), 1);              // the loader's arrive (+ the copy's bytes)
            mbar_init(load_empty(0, s), 4 * UPT);       // the producer warps that read the stage
        }
        for (int s = 0; s < NAF; ++s) mbar_init(a_full(s), 4 * UPT);    // the producer warps that fill the tile's units
        for (int s = 0; s < NB; ++s) mbar_init(tile_done(s), 1);        // the issuer's commit
        for (int s = 0; s < MAX_NACC; ++s) mbar_init(acc_free(s), 4);   // the four warps of the epilogue group that reads it
        abort_flag_smem = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // The loader warps start now: the first row tiles arrive while the other warps expand the weights (these kernels
    // run for 10 - 40 us; the weights' expansion and the first copy's latency are 1.5 - 2 us each).  The other warps meet
    // at a named barrier of their own; everybody meets again at the end.
    const bool is_loader = warp >= FIRST_LOADER_WARP && warp < FIRST_PRODUCER_WARP;
    auto sync_workers = [&]() { asm volatile("bar.sync 1, %0;" ::"r"(THREADS - 64) : "memory"); };
    if (!is_loader) {
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // ---- one-off: the resident slices' expanded weights and constants; MMA row `row` of slice s carries channel ch
    for (int i = tid < 64 ? tid : tid - 64; i < RS * (KT + 1) * BN; i += THREADS - 64) {   // (threads 64 .. 127 are the loaders)
        const int row = i % BN, kt = (i / BN) % (KT + 1), s = i / (BN * (KT + 1));
        const int ch = (cg * RS + s) * BN + (PACK16 ? (row & ~31) + channel_of_column(row & 31) : row);
        const bool have = ch < p.C_out;
        const int xr = row & 7;
        if (kt < KT) {
            const uint32_t row_addr = wexp + (uint32_t)(s * KT + kt) * W_TILE_BYTES + (uint32_t)row * ROWB;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t w = have ? __ldg(p.w + (long)ch * KWORDS + kt * 4 + e) : 0u;
                expand_store_w_signed(w, have, row_addr, xr, 2 * e);
            }
        } else {
            // cst = 32 * c, c = K - 2 popc(G) - thr (thr clamped to +-(K + 1)); the constant activation tile's bytes are
            // all 32, so the 32 signed bytes add up to c: c / 32 everywhere, one more unit of c's sign in |c % 32|
            int pop = 0;
            if (have)
                for (int e = 0; e < KWORDS; ++e) pop += __popc(__ldg(p.w + (long)ch * KWORDS + e));
            int t = have ? __ldg(p.thr + ch) : 0;
            t = max(min(t, p.K + 1), -p.K - 1);
            const int c = have ? p.K - 2 * pop - t : 0;
            const int base = c / 32, rem = c - 32 * base, unit = rem < 0 ? -1 : 1, nrem = rem < 0 ? -rem : rem;
            uint32_t cw[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                uint32_t word = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) word |= (uint32_t)((base + ((4 * q + b) < nrem ? unit : 0)) & 0xFF) << (8 * b);
                cw[q] = word;
            }
            const uint32_t crow = cexp + (uint32_t)row * ROWB;
            st_shared_v4(crow + (uint32_t)(((2 * s) ^ xr) << 4), cw[0], cw[1], cw[2], cw[3]);
            st_shared_v4(crow + (uint32_t)(((2 * s + 1) ^ xr) << 4), cw[4], cw[5], cw[6], cw[7]);
        }
    }
    fence_async_proxy();
    tc_fence_before();
    sync_workers();
    tc_fence_after();
    // the constant activation tile: every byte 32
    if (warp >= FIRST_PRODUCER_WARP && warp < FIRST_PRODUCER_WARP + 4) {
        const uint32_t c8[8] = {0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u};
        tc_st8_nowait(tmem_base_smem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)C_COL, c8);
        tc_wait_st();
    }
    tc_fence_before();
    sync_workers();
    tc_fence_after();
    }
    const uint32_t tmem_base = is_loader ? 0u : tmem_base_smem;

    if (warp < NISS) {
        // ------------------------------------------------------------------ MMA issuer of the parts d = warp (mod 2), in order.
        // (One issuer's waits, fence and commit between two parts take about as long as a part's MMAs run: with two
        // issuers one's MMAs run during the other's bookkeeping.)
        constexpr uint32_t idesc = make_idesc(AW) | (1u << 10);                  // B operand: signed bytes
        constexpr uint32_t HALF_DESC = (uint32_t)(64 * ROWB) >> 4;               // rows 64 .. 127 of a weight tile
        const uint64_t desc0 = make_desc(wexp);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32), b_lo = (uint32_t)desc0;
        const uint32_t c_lo = (uint32_t)make_desc(cexp);
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t c_t = tmem_u + (uint32_t)C_COL;
        bool ok = true;
        for (int n = 0; n < my_tiles && ok; ++n) {
            if (!pw_wait(a_full(n % NAF), (uint32_t)(n / NAF) & 1u, abort_flag, p.err, ERR_PN_ISSUER_TIMEOUT)) break;
            for (int j = warp; j < PARTS; j += NISS) {
                const int d = n * PARTS + j;                                      // "done" number
                const int acc = d % NACC;
                const int s = AW == BN ? j : j >> 1, hf = AW == BN ? 0 : j & 1;   // part j = rows hf * 64 .. of slice s
                if (d >= NACC) {                  // the epilogue has read the accumulator's previous contents
                    ok = pw_wait(acc_free(acc), (uint32_t)(d / NACC - 1) & 1u, abort_flag, p.err, ERR_PN_ACC_TIMEOUT);
                    if (!ok) break;
                }
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t d_t = tmem_u + (uint32_t)(acc * AW);
                    const uint32_t w_lo = b_lo + (uint32_t)(s * KT) * (W_TILE_BYTES >> 4) + (uint32_t)hf * HALF_DESC;
                    tc_mma_i8_ts(d_t, c_t, c_lo + (uint32_t)hf * HALF_DESC + 2u * s, desc_hi, idesc, 0u);   // accumulator = the constants
#pragma unroll
                    for (int h = 0; h < UPT; ++h) {
                        const uint32_t a_t = tmem_u + (uint32_t)(A_COL0 + ((n * UPT + h) % NUNIT) * U_COLS);
#pragma unroll
                        for (int t = 0; t < UWORDS; ++t) {
                            const int e = h * UWORDS + t;
                            tc_mma_i8_ts(d_t, a_t + 8u * t, w_lo + (uint32_t)((e >> 2) * (W_TILE_BYTES >> 4) + 2 * (e & 3)), desc_hi, idesc, 1u);
                        }
                    }
                    tc_commit(tile_done(d % NB));
                }
                __syncwarp();
            }
        }
    } else if (warp < FIRST_PRODUCER_WARP) {
        // ------------------------------------------------------------------ loader of group warp - 2: one row tile per bulk copy
        const int grp = warp - FIRST_LOADER_WARP;
        int stage = 0;
        uint32_t phase = 1;                       // first pass through the ring: the stages are free
        int issued = 0;
        for (int n = grp; n < my_tiles; n += NGRP) {
            if (!pw_wait<256>(load_empty(grp, stage), phase, abort_flag, p.err, ERR_PN_LOADER_TIMEOUT)) break;
            if (lane == 0) {
                const long row0 = (long)row_tile(n) * BM;
                const long rows = min((long)BM, (long)p.M - row0);                // rows beyond M keep whatever the stage held
                const uint32_t bytes = (uint32_t)rows * KWORDS * 4u;              // a multiple of 32
                const uint32_t dst = ring + (uint32_t)(grp * RD + stage) * TILE_BYTES;
                const uint32_t *src = p.x + row0 * KWORDS;
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(load_full(grp, stage)), "r"(bytes) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(dst), "l"(src), "r"(bytes), "r"(load_full(grp, stage)) : "memory");
            }
            __syncwarp();
            ++issued;
            if (++stage == RD) { stage = 0; phase ^= 1u; }
        }
        // after a time-out elsewhere: copies still in flight must land before the CTA's shared memory goes away
        if (*abort_flag) {
            const int first = issued > RD ? issued - RD : 0;
            for (int q = first; q < issued; ++q)
                pw_wait(load_full(grp, q % RD), (uint32_t)(q / RD) & 1u, abort_flag, nullptr, 0);
        }
    } else if (warp >= FIRST_EPILOGUE_WARP) {
        // ------------------------------------------------------------------ epilogue group (warp - first) / 4: "done" numbers d = group (mod 2)
        const int quad = warp & 3;
        const int grp = (warp - FIRST_EPILOGUE_WARP) >> 2;
        const int r = quad * 32 + lane;                           // row of the tile
        const uint32_t t_lane0 = tmem_base + ((uint32_t)(quad * 32) << 16);
        const int owords = p.C_out >> 5;
        const int total = my_tiles * PARTS;
        for (int d = grp; d < total; d += 2) {
            const int n = d / PARTS, j = d - n * PARTS, acc = d % NACC;
            const uint32_t t_lane = t_lane0 + (uint32_t)(acc * AW);
            if (!pw_wait<64>(tile_done(d % NB), (uint32_t)(d / NB) & 1u, abort_flag, p.err, ERR_PN_EPILOGUE_TIMEOUT)) break;
            tc_fence_after();
            uint32_t words[AW / 32];
            if constexpr (PACK16) {
                uint32_t rr[AW / 64][32];
#pragma unroll
                for (int h = 0; h < AW / 64; ++h) tc_ld64_pack16(t_lane + (uint32_t)(h * 64), rr[h]);
                tc_wait_ld();
#pragma unroll
                for (int h = 0; h < AW / 64; ++h) pin_regs(rr[h]);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_free(acc));
#pragma unroll
                for (int h = 0; h < AW / 64; ++h) {
                    words[2 * h] = sign_word(rr[h]);
                    words[2 * h + 1] = sign_word(rr[h] + 16);
                }
            } else {
#pragma unroll
                for (int ch = 0; ch < AW / 32; ++ch) {
                    uint32_t v[32];
                    tc_ld32(t_lane + (uint32_t)(ch * 32), v);
                    if (ch == AW / 32 - 1) {                              // the accumulator's last columns are in registers
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(acc_free(acc));
                    }
                    // bit i = (v[i] >= 0): sign bits shifted in, last column first; two chains of 16
                    uint32_t hi = 0, lo = 0;
#pragma unroll
                    for (int i = 15; i >= 0; --i) {
                        hi = __funnelshift_l(v[16 + i], hi, 1);
                        lo = __funnelshift_l(v[i], lo, 1);
                    }
                    words[ch] = ~__byte_perm(lo, hi, 0x5410);
                }
            }
            const long m = (long)row_tile(n) * BM + r;
            if (m < p.M) {
                uint32_t *dst = static_cast<uint32_t *>(p.out) + m * owords + (cg * PARTS + j) * (AW / 32);
                if constexpr (AW == 128) *reinterpret_cast<uint4 *>(dst) = make_uint4(words[0], words[1], words[2 % (AW / 32)], words[3 % (AW / 32)]);
                else *reinterpret_cast<uint2 *>(dst) = make_uint2(words[0], words[1]);
            }
        }
    } else {
        // ------------------------------------------------------------------ producer group (warp - first) / 4
        // thread = row of the tile = tensor-memory lane.  The group fills unit h (K words 8 h .. 8 h + 7) of the tiles
        // n0, n0 + step, ...
        const int quad = warp & 3;
        const int grp = (warp - FIRST_PRODUCER_WARP) >> 2;
        const int h = UPT == 2 ? (grp & 1) : 0;
        const int n0 = UPT == 2 ? (grp >> 1) : grp, step = UPT == 2 ? NPG / 2 : NPG;
        const int r = quad * 32 + lane;
        const uint32_t my_off = (uint32_t)(r * KWORDS * 4 + h * UWORDS * 4);
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)A_COL0;
        const uint32_t lane0 = lane == 0 ? 1u : 0u;
        for (int n = n0; n < my_tiles; n += step) {
            const int lg = n & 1, stage = (n >> 1) % RD;
            if (!pw_wait<64>(load_full(lg, stage), (uint32_t)((n >> 1) / RD) & 1u, abort_flag, p.err, ERR_PN_PRODUCER_TIMEOUT)) break;
            const uint32_t src = ring + (uint32_t)(lg * RD + stage) * TILE_BYTES + my_off;
            const uint4 q0 = ld_shared_v4(src), q1 = ld_shared_v4(src + 16u);
            __syncwarp();
            mbar_arrive_pred(load_empty(lg, stage), lane0);        // the stage may be refilled
            // the first four words are expanded before the wait for the unit
            uint32_t v[32];
            expand_a(q0.x, &v[0]); expand_a(q0.y, &v[8]); expand_a(q0.z, &v[16]); expand_a(q0.w, &v[24]);
            // the MMAs of the tile that used this ring position last have read it (nothing to wait for the first time round)
            const int u = n * UPT + h;
            if (u >= NUNIT) {
                const int dm = (u - NUNIT) / UPT * PARTS + PARTS - 1;         // that tile's last "done" numbers: one per issuer
                if (PARTS >= 2 && !pw_wait<64>(tile_done((dm - 1) % NB), (uint32_t)((dm - 1) / NB) & 1u, abort_flag, p.err, ERR_PN_UNIT_TIMEOUT)) break;
                if (!pw_wait<64>(tile_done(dm % NB), (uint32_t)(dm / NB) & 1u, abort_flag, p.err, ERR_PN_UNIT_TIMEOUT)) break;
            }
            tc_fence_after();
            const uint32_t taddr = t_lane + (uint32_t)((u % NUNIT) * U_COLS);
            tc_st32_nowait(taddr, v);
            uint32_t v4[32];
            expand_a(q1.x, &v4[0]); expand_a(q1.y, &v4[8]); expand_a(q1.z, &v4[16]); expand_a(q1.w, &v4[24]);
            tc_st32_nowait(taddr + 32u, v4);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            mbar_arrive_pred(a_full(n % NAF), lane0);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// resident slices per CTA: all of a K = 256 layer (up to four: 128 KB); one of a K = 512 layer (two would fit, but
// measured, four groups of 37 SMs with one slice each beat two groups with two: 20.5 against 23.5 us on 512 x 512 at
// M = 50176 - half the weights to expand at the start, and the row tiles divide more evenly)
int pn_resident_slices(int kwords, int slices) { return kwords == 8 ? slices : 1; }

template <int UPT, int AW>
int launch_pn(const ConvProblem &p0, cudaStream_t stream)
{
    constexpr int KWORDS = UWORDS * UPT, KT = KWORDS / 4, TILE_BYTES = BM * KWORDS * 4;
    ConvProblem p = p0;
    p.err = device_error_word();
    PnPlan plan;
    const int slices = p.C_out / BN;
    plan.rs = pn_resident_slices(KWORDS, slices);
    plan.ng = slices / plan.rs;
    plan.m_tiles = (p.M - 1) / BM + 1;
    const int smem = 1024 + (plan.rs * KT + 1) * W_TILE_BYTES + NGRP * RD * TILE_BYTES + 128;
    if (smem > 227 * 1024 - 1024) return BCNN_ERR_UNSUPPORTED;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int per_group = sms / plan.ng;
    if (per_group > plan.m_tiles) per_group = plan.m_tiles;
    if (per_group < 1) per_group = 1;
    void (*k)(const ConvProblem, const PnPlan) = conv_tc_pn_kernel<UPT, AW>;
    const int ask = smem < 120 * 1024 ? 120 * 1024 : smem;          // one CTA per SM (it takes all of tensor memory)
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 1024) != cudaSuccess) return BCNN_ERR_CUDA;
    k<<<(unsigned)(per_group * plan.ng), THREADS, ask, stream>>>(p, plan);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace

bool conv_tc_pn_supports(const ConvProblem &p)
{
    if (p.mode != 1) return false;                               // packed output only
    if (!(p.kh == 1 && p.kw == 1 && p.stride == 1 && p.pad == 0)) return false;
    if (p.kwords != 8 && p.kwords != 16) return false;           // K = 256 or 512
    return p.C_out == 128 || p.C_out == 256 || p.C_out == 512;
}

int launch_conv_tc_pn(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_tc_pn_supports(p)) return BCNN_ERR_UNSUPPORTED;
    return p.kwords == 8 ? launch_pn<1, 128>(p, stream) : launch_pn<2, 64>(p, stream);
}

}  // namespace bcnn
