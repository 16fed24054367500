// Short-K 3x3 engine: binary 3x3 convolutions (stride 1 or 2) on 32 or 64 input channels with up to 128 output
// channels, packed output - the stem / down-sampling shaped layers and the first 3x3 layers of the backbone, where a
// 128-row tile is nine or eighteen 32-bit words of K per row and the weight-stationary engine spends most of its
// instructions on the gather (a table look-up, a mask test and a 4-byte cp.async per K word).
//
// The implicit im2col is done by TMA:
//   * an output tile is a TH x TW = 8 x 16 patch of output pixels of one image (128 rows of the patch matrix);
//   * its input halo - ((TH-1) s + 3) rows x ((TW-1) s + 3) pixels x C_in bits - arrives by ONE tiled TMA copy
//     (cp.async.bulk.tensor.3d over the packed input seen as [B][H][W * C_in / 32 words]) into a ring in shared
//     memory.  Out-of-image rows and pixels are the copy's zero fill = the -1 padding: no tap masks anywhere.  The
//     copy's first word must be 16-byte aligned, so the box starts up to three pixels left of the halo (XOFF);
//   * a producer thread (= one output pixel) reads its nine pixels' words from the halo tile at compile-time offsets,
//     expands them and stores them to tensor memory: per K word one shared-memory load and the eight logic operations.
// Arithmetic as in the pointwise engine (conv_tc_pw.cu): unsigned activation bytes {0, 2^j} against signed weight bytes,
// every product +-64, the per-channel constant written by a first MMA against a constant activation tile.
//
// One commit per tile.  Tensor memory holds NACC accumulators and a ring of NUNIT activation UNITS: the nine taps of
// 32 input channels of one tile (72 columns).  A tile is one unit for C_in = 32 and two for C_in = 64 (K order: channel
// word, then tap).  An issuer warp walks tiles in order: it waits until the tile's units are full and its accumulator
// free, issues the tile's MMAs and ONE commit on the tile's "done" barrier, which the epilogue (accumulator ready) and
// the producers (units free again) wait on: with the producers ahead the MMAs of consecutive tiles queue back to back.
// Four producer groups of four warps fill ONE unit of every tile they take:
//   * C_in = 64 (tiles of 640+ tensor-pipe cycles, one issuer): groups 2 j and 2 j + 1 fill the two units of the tiles
//     n = j (mod 2).  The ring holds five (six) units = two and a half (three) tiles, so a tile's first unit reuses
//     columns that were free one tile earlier than those of its second unit: only half of a tile's stores have to fit
//     into the time of one tile's MMAs;
//   * C_in = 32 (tiles of 160 - 320 tensor-pipe cycles, bound by instruction issue): group j fills the tiles
//     n = j (mod 4), and two issuer warps take alternate tiles (one issuer's waits and commit would be the bound); the
//     ring then has an even number of units, so that a unit's next user belongs to the same issuer.
// Two loader warps and two epilogue groups take alternate tiles.
// The "done" barriers form a ring of NB = 8 (tile n -> barrier n % 8), a multiple of NACC and more than the tiles in
// flight.  K = 288: |accumulator| <= 32 (2 K + 1) < 2^15, so the epilogue reads packed 16-bit halves and gathers sign
// bits with byte permutes; K = 576: 32-bit accumulators, sign bits shifted in.
// A parity wait on an mbarrier is only right while the waiter starts waiting for completion k after completion k - 1 and
// before completion k + 1.  Tile n's "done" is completion n / 8 of its barrier; its waiters are the epilogue of tile n
// and the producers of the tiles (at most four ahead) that reuse its units.  Every one of them has seen an earlier tile
// of the same issuer done within the last eight (an issuer's tiles complete in order), and tile n + 8 cannot be issued
// before they are through: its issuer first issues the reusing tiles (the same issuer), which need those units filled,
// and, NB being a multiple of NACC, tile n + 8 needs the accumulator of tile n back from the epilogue.
// Every mbarrier wait is bounded and reports through the device error word.
#include "tc_slot.cuh"
#include <cuda.h>

namespace bcnn {

namespace {

using namespace tc;

constexpr int ERR_C3_LOADER_TIMEOUT = 141;       // loader: no free ring stage
constexpr int ERR_C3_PRODUCER_TIMEOUT = 142;     // producer: the tile's halo did not arrive
constexpr int ERR_C3_ISSUER_TIMEOUT = 143;       // issuer: a tile's activations were not filled
constexpr int ERR_C3_EPILOGUE_TIMEOUT = 144;     // epilogue: the tile's MMAs did not complete
constexpr int ERR_C3_UNIT_TIMEOUT = 145;         // producer: the unit's previous MMAs did not complete
constexpr int ERR_C3_ACC_TIMEOUT = 146;          // issuer: an accumulator was not handed back

constexpr int TH = 8, TW = 16;            // output tile (TH * TW = 128 = tensor-memory lanes)
constexpr int NGRP = 2;                   // loader / epilogue groups (alternate tiles)
constexpr int NPG = 4;                    // producer groups of four warps
constexpr int RD = 6;                     // halo tiles in a loader's ring
constexpr int CONST_COLS = 8;
constexpr int TAPS = 9;
constexpr int U_COLS = 8 * TAPS;          // columns of a unit
constexpr int NB = 8;                     // ring of "tile done" barriers
constexpr int NAF = 4;                    // ring of "tile full" barriers (at most four tiles are being filled)
constexpr int MAX_NUNIT = 6, MAX_NACC = 4;

// CW: words per input pixel (1, 2) = units per tile; BN: accumulator columns per tile (32, 64, 128 >= C_out).
template <int CW, int BN> struct C3Cfg {
    static constexpr int KW = TAPS * CW;                    // words of K per row
    static constexpr int KT = (KW + 3) / 4;                 // 128-byte stages of the expanded weights
    // 128 output channels run as two halves of 64 against the same activation units: the accumulator of one half is
    // read by its epilogue group while the other half's MMAs run (one 128-column accumulator would leave room for
    // neither a second one nor enough units)
    static constexpr int NH = BN == 128 ? 2 : 1;            // halves
    static constexpr int AW = BN / NH;                      // accumulator columns
    static constexpr int NACC = NH == 2 ? 2 : (CW == 1 && BN == 32 ? 4 : 2);   // accumulators (NH == 2: one per half)
    static constexpr int NISS = CW == 2 || NH == 2 ? 1 : 2; // issuer warps
    static constexpr bool PACK16 = CW == 1;
    static constexpr int NU0 = (512 - CONST_COLS - NACC * AW) / U_COLS;
    static constexpr int NU1 = NU0 > MAX_NUNIT ? MAX_NUNIT : NU0;
    static constexpr int NUNIT = CW == 1 ? (NU1 > 4 ? 4 : NU1 / 2 * 2) : NU1;   // 4 (C_in 32); 6, 5, 5 (C_in 64)
    static constexpr int A_COL0 = NACC * AW;
    static constexpr int C_COL = A_COL0 + NUNIT * U_COLS;   // the constant activation tile
    static_assert(C_COL + CONST_COLS <= 512, "tensor memory budget");
    static_assert(NUNIT >= 2 * CW && (NUNIT + CW - 1) / CW <= NAF && NB % NACC == 0 && NACC <= MAX_NACC && NACC % NISS == 0 &&
                  (NISS == 1 || NUNIT % NISS == 0), "barrier rings");
    // warps: 0 (and 1) issuers, 2 and 3 loaders, then the producer groups, then the epilogue groups (groups start at
    // multiples of four: warp % 4 is the tensor-memory lane quadrant of a warp)
    static constexpr int FIRST_LOADER_WARP = 2;
    static constexpr int FIRST_PRODUCER_WARP = 4;
    static constexpr int FIRST_EPILOGUE_WARP = 4 + 4 * NPG;
    static constexpr int WARPS = 4 + 4 * NPG + 4 * NGRP;
    static constexpr int THREADS = 32 * WARPS;
    static constexpr int W_TILE_BYTES = BN * ROWB;
};

struct C3Geom {
    int stride, xoff;        // XOFF: pixels between the box's first pixel and the halo's
    int wbw, hb;             // box: words per row, rows
    int stage_bytes;         // hb * wbw * 4 rounded up to 128
    int tiles_x, tiles_y;    // tiles per image row / column of tiles
    int total_tiles;
};

C3Geom c3_geometry(const ConvProblem &p)
{
    C3Geom g;
    g.stride = p.stride;
    const int A = 4 / p.cw;                                  // pixels per 16 bytes
    g.xoff = (A - p.pad % A) % A;
    const int wpx = ((TW - 1) * p.stride + 3 + g.xoff + A - 1) / A * A;
    g.wbw = wpx * p.cw;
    g.hb = (TH - 1) * p.stride + 3;
    g.stage_bytes = (g.hb * g.wbw * 4 + 127) / 128 * 128;
    g.tiles_x = (p.OW + TW - 1) / TW;
    g.tiles_y = (p.OH + TH - 1) / TH;
    g.total_tiles = p.B * g.tiles_x * g.tiles_y;
    return g;
}

template <int CW, int BN>
int c3_smem_bytes(const C3Geom &g)
{
    using C = C3Cfg<CW, BN>;
    return 1024 + (C::KT + 1) * C::W_TILE_BYTES + NGRP * RD * g.stage_bytes + 128;
}

template <int CW, int BN>
__global__ void __launch_bounds__(C3Cfg<CW, BN>::THREADS, 1)
conv_tc_c3_kernel(const ConvProblem p, const C3Geom g, const __grid_constant__ CUtensorMap xmap)
{
    using C = C3Cfg<CW, BN>;
    constexpr int KW = C::KW, KT = C::KT, NACC = C::NACC, NUNIT = C::NUNIT, NH = C::NH, AW = C::AW;
    constexpr int NBARS = 2 * NGRP * RD + NAF + NB + MAX_NACC;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[NBARS];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    // this CTA's tiles: blockIdx.x + n * gridDim.x, n = 0, 1, ...; tile n belongs to loader / epilogue group n % 2, uses
    // accumulator n % NACC, "full" barrier n % NAF, "done" barrier n % NB (two halves: both epilogue groups, accumulator =
    // half, "done" barrier (2 n + half) % NB); its unit h is the CTA's unit number n * CW + h,
    // in ring position (n * CW + h) % NUNIT
    const int my_tiles = (int)blockIdx.x < g.total_tiles ? (g.total_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int cn = min(BN, p.C_out);

    const uint32_t wexp = (smem_u32(smem_raw) + 1023u) & ~1023u;          // [KT][BN rows][128 B] expanded weights
    const uint32_t cexp = wexp + KT * C::W_TILE_BYTES;                    // [BN rows][128 B] constant bytes (first 32 of a row)
    const uint32_t ring = cexp + C::W_TILE_BYTES;                         // [NGRP][RD] halo tiles
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
            mbar_init(load_empty(0, s), 4 * CW);        // the producer warps that read the stage
        }
        for (int s = 0; s < NAF; ++s) mbar_init(a_full(s), 4 * CW);     // the producer warps that fill the tile's units
        for (int s = 0; s < NB; ++s) mbar_init(tile_done(s), 1);        // the issuer's commit
        for (int s = 0; s < MAX_NACC; ++s) mbar_init(acc_free(s), 4);   // the four epilogue warps of the tile's group
        abort_flag_smem = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // ---- one-off: expanded weights and the constant bytes.  K position e of the MMAs = channel word e / 9, tap e % 9
    // (global weight word tap * CW + channel word) -> stage e / 4, 32-byte piece e % 4; MMA row `row` carries channel ch
    for (int idx = tid; idx < (KT + 1) * BN; idx += C::THREADS) {
        const int kt = idx / BN, row = idx - kt * BN;
        const int ch = C::PACK16 ? (row & ~31) + channel_of_column(row & 31) : row;
        const bool have = ch < cn;
        const int xr = row & 7;
        if (kt < KT) {
            const uint32_t row_addr = wexp + (uint32_t)kt * C::W_TILE_BYTES + (uint32_t)row * ROWB;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int kpos = kt * 4 + e;
                const bool live = kpos < KW && have;
                const uint32_t w = live ? __ldg(p.w + (long)ch * KW + (kpos % TAPS) * CW + kpos / TAPS) : 0u;
                expand_store_w_signed(w, live, row_addr, xr, 2 * e);
            }
        } else {
            // cst = 32 * c, c = K - 2 popc(G) - thr (thr clamped to +-(K + 1)); the constant activation tile's bytes are
            // all 32, so the row's 32 signed bytes add up to c: c / 32 everywhere, one more unit of c's sign in |c % 32|
            int pop = 0;
            if (have)
                for (int e = 0; e < KW; ++e) pop += __popc(__ldg(p.w + (long)ch * KW + e));
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
            st_shared_v4(crow + (uint32_t)((0 ^ xr) << 4), cw[0], cw[1], cw[2], cw[3]);
            st_shared_v4(crow + (uint32_t)((1 ^ xr) << 4), cw[4], cw[5], cw[6], cw[7]);
        }
    }
    fence_async_proxy();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;
    // the constant activation tile: every byte 32
    if (warp >= C::FIRST_PRODUCER_WARP && warp < C::FIRST_PRODUCER_WARP + 4) {
        const uint32_t c8[8] = {0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u};
        tc_st8_nowait(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)C::C_COL, c8);
        tc_wait_st();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    // tile index -> image and the tile's first output pixel
    auto tile_origin = [&](int tile, int &b, int &oh0, int &ow0) {
        const unsigned per_img = (unsigned)(g.tiles_x * g.tiles_y);
        b = (int)((unsigned)tile / per_img);
        const unsigned rem = (unsigned)tile - (unsigned)b * per_img;
        const unsigned ty = rem / (unsigned)g.tiles_x;
        oh0 = (int)ty * TH;
        ow0 = (int)(rem - ty * (unsigned)g.tiles_x) * TW;
    };
    auto tile_of = [&](int n) { return (int)blockIdx.x + n * (int)gridDim.x; };

    if (warp < C::NISS) {
        // ------------------------------------------------------------------ MMA issuer of tiles n = warp (mod NISS), in order
        constexpr uint32_t idesc = make_idesc(AW) | (1u << 10);                  // B operand: signed bytes
        constexpr uint32_t HALF_DESC = (uint32_t)(AW * ROWB) >> 4;               // weight rows of the second half
        const uint64_t desc0 = make_desc(wexp);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32), b_lo = (uint32_t)desc0;
        const uint32_t c_lo = (uint32_t)make_desc(cexp);
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t c_t = tmem_u + (uint32_t)C::C_COL;
        bool ok = true;
        for (int n = warp; n < my_tiles && ok; n += C::NISS) {
            if (!pw_wait(a_full(n % NAF), (uint32_t)(n / NAF) & 1u, abort_flag, p.err, ERR_C3_ISSUER_TIMEOUT)) break;
#pragma unroll
            for (int hf = 0; hf < NH; ++hf) {
                // the epilogue has read the accumulator's previous tile
                const int acc = NH == 2 ? hf : n % NACC;
                const int prev = NH == 2 ? n - 1 : n / NACC - 1;                 // completion of acc_free to wait for
                if (prev >= 0) {
                    ok = pw_wait(acc_free(acc), (uint32_t)prev & 1u, abort_flag, p.err, ERR_C3_ACC_TIMEOUT);
                    if (!ok) break;
                }
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t d_t = tmem_u + (uint32_t)(acc * AW);
                    tc_mma_i8_ts(d_t, c_t, c_lo + hf * HALF_DESC, desc_hi, idesc, 0u);   // accumulator = the per-channel constants
#pragma unroll
                    for (int h = 0; h < CW; ++h) {
                        const uint32_t a_t = tmem_u + (uint32_t)(C::A_COL0 + ((n * CW + h) % NUNIT) * U_COLS);
#pragma unroll
                        for (int t = 0; t < TAPS; ++t) {
                            const int e = h * TAPS + t;
                            tc_mma_i8_ts(d_t, a_t + 8u * t, b_lo + hf * HALF_DESC + (uint32_t)((e >> 2) * (C::W_TILE_BYTES >> 4) + 2 * (e & 3)),
                                         desc_hi, idesc, 1u);
                        }
                    }
                    tc_commit(tile_done((n * NH + hf) % NB));
                }
                __syncwarp();
            }
        }
    } else if (warp < C::FIRST_LOADER_WARP) {
        // (idle)
    } else if (warp < C::FIRST_PRODUCER_WARP) {
        // ------------------------------------------------------------------ loader of group warp - 2: one halo tile per TMA copy
        const int grp = warp - C::FIRST_LOADER_WARP;
        int stage = 0;
        uint32_t phase = 1;                       // first pass through the ring: the stages are free
        int issued = 0;
        for (int n = grp; n < my_tiles; n += NGRP) {
            if (!pw_wait<256>(load_empty(grp, stage), phase, abort_flag, p.err, ERR_C3_LOADER_TIMEOUT)) break;
            if (lane == 0) {
                const uint32_t dst = ring + (uint32_t)(grp * RD + stage) * (uint32_t)g.stage_bytes;
                int b, oh0, ow0;
                tile_origin(tile_of(n), b, oh0, ow0);
                const int x = (ow0 * g.stride - p.pad - g.xoff) * CW;        // words; a multiple of 4 by construction
                const int y = oh0 * g.stride - p.pad;
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(load_full(grp, stage)), "r"((uint32_t)(g.hb * g.wbw * 4)) : "memory");
                asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                             ::"r"(dst), "l"(reinterpret_cast<uint64_t>(&xmap)), "r"(x), "r"(y), "r"(b), "r"(load_full(grp, stage)) : "memory");
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
    } else if (warp >= C::FIRST_EPILOGUE_WARP) {
        // ------------------------------------------------------------------ epilogue group (warp - first) / 4
        const int quad = warp & 3;
        const int grp = (warp - C::FIRST_EPILOGUE_WARP) >> 2;
        const int r = quad * 32 + lane;                           // row of the tile = output pixel (r / TW, r % TW)
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16);
        const int owords = p.C_out >> 5;
        // NH == 1: the group takes alternate tiles; NH == 2: the group takes its half (64 channels) of every tile
        for (int n = NH == 2 ? 0 : grp; n < my_tiles; n += NH == 2 ? 1 : NGRP) {
            const int acc = NH == 2 ? grp : n % NACC;
            const int d = NH == 2 ? 2 * n + grp : n;                              // the tile's (half's) "done" number
            const int ch0 = NH == 2 ? 2 * grp : 0;                                // first output word of this accumulator
            if (!pw_wait<C::NISS == 1 ? 64 : 128>(tile_done(d % NB), (uint32_t)(d / NB) & 1u, abort_flag, p.err, ERR_C3_EPILOGUE_TIMEOUT)) break;
            tc_fence_after();
            uint32_t words[AW / 32];
            if constexpr (C::PACK16) {
                constexpr int NR = AW == 32 ? 16 : 32;                       // registers per load
                constexpr int NL = AW == 32 ? 1 : AW / 64;                   // loads
                uint32_t rr[NL][NR];
                if constexpr (AW == 32) {
                    tc_ld32_pack16(t_lane + (uint32_t)(acc * AW), rr[0]);
                } else {
#pragma unroll
                    for (int h = 0; h < NL; ++h) tc_ld64_pack16(t_lane + (uint32_t)(acc * AW + h * 64), rr[h]);
                }
                tc_wait_ld();
#pragma unroll
                for (int h = 0; h < NL; ++h) pin_regs(rr[h]);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_free(acc));
                if constexpr (AW == 32) {
                    words[0] = sign_word(rr[0]);
                } else {
#pragma unroll
                    for (int h = 0; h < NL; ++h) {
                        words[2 * h] = sign_word(rr[h]);
                        words[2 * h + 1] = sign_word(rr[h] + 16);
                    }
                }
            } else {
#pragma unroll
                for (int ch = 0; ch < AW / 32; ++ch) {
                    uint32_t v[32];
                    tc_ld32(t_lane + (uint32_t)(acc * AW + ch * 32), v);
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
            int b, oh0, ow0;
            tile_origin(tile_of(n), b, oh0, ow0);
            const int oh = oh0 + (r >> 4), ow = ow0 + (r & 15);
            if (oh < p.OH && ow < p.OW) {
                uint32_t *dst = static_cast<uint32_t *>(p.out) + (((long)b * p.OH + oh) * p.OW + ow) * owords + ch0;
                if (AW == 64 && (owords & 1) == 0) {                  // (an even word count keeps the pair 8-byte aligned)
                    *reinterpret_cast<uint2 *>(dst) = make_uint2(words[0], words[1 % (AW / 32)]);
                } else {
#pragma unroll
                    for (int ch = 0; ch < AW / 32; ++ch)
                        if (ch0 + ch < owords) dst[ch] = words[ch];
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ producer group (warp - first) / 4
        // thread = output pixel (ty, tx) of the tile = tensor-memory lane; its nine input pixels sit at rows
        // ty * s + kr, pixels tx * s + XOFF + kt of the halo tile.  The group fills unit h (channel word h of the nine
        // taps) of the tiles n0, n0 + step, ...
        const int quad = warp & 3;
        const int grp = (warp - C::FIRST_PRODUCER_WARP) >> 2;
        const int h = CW == 2 ? (grp & 1) : 0;
        const int n0 = CW == 2 ? (grp >> 1) : grp, step = CW == 2 ? NPG / 2 : NPG;
        const int r = quad * 32 + lane;
        const uint32_t my_off = (uint32_t)((((r >> 4) * g.stride) * g.wbw + ((r & 15) * g.stride + g.xoff) * CW + h) * 4);
        const uint32_t row_pitch = (uint32_t)(g.wbw * 4);
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)C::A_COL0;
        const uint32_t lane0 = lane == 0 ? 1u : 0u;
        for (int n = n0; n < my_tiles; n += step) {
            const int lg = n & 1, stage = (n >> 1) % RD;
            uint32_t wds[TAPS];
            if (!pw_wait<64>(load_full(lg, stage), (uint32_t)((n >> 1) / RD) & 1u, abort_flag, p.err, ERR_C3_PRODUCER_TIMEOUT)) break;
            const uint32_t src = ring + (uint32_t)(lg * RD + stage) * (uint32_t)g.stage_bytes + my_off;
#pragma unroll
            for (int tap = 0; tap < TAPS; ++tap)
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(wds[tap]) : "r"(src + (uint32_t)(tap / 3) * row_pitch + (uint32_t)((tap % 3) * CW * 4)) : "memory");
            __syncwarp();
            mbar_arrive_pred(load_empty(lg, stage), lane0);        // the stage may be refilled
            // the first four words are expanded before the wait for the unit
            uint32_t v[32];
#pragma unroll
            for (int e = 0; e < 4; ++e) expand_a(wds[e], &v[8 * e]);
            // the MMAs of the tile that used this ring position last have read it (nothing to wait for the first time round)
            const int u = n * CW + h;
            if (u >= NUNIT) {
                const int dm = (u - NUNIT) / CW * NH + NH - 1;                    // that tile's last "done" number
                if (!pw_wait<64>(tile_done(dm % NB), (uint32_t)(dm / NB) & 1u, abort_flag, p.err, ERR_C3_UNIT_TIMEOUT)) break;
            }
            tc_fence_after();
            const uint32_t taddr = t_lane + (uint32_t)((u % NUNIT) * U_COLS);
            tc_st32_nowait(taddr, v);
            {
                uint32_t v4[32];
#pragma unroll
                for (int e = 0; e < 4; ++e) expand_a(wds[4 + e], &v4[8 * e]);
                tc_st32_nowait(taddr + 32u, v4);
                uint32_t v8[8];
                expand_a(wds[8], v8);
                tc_st8_nowait(taddr + 64u, v8);
            }
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn c3_encode_fn()
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

template <int CW, int BN>
int launch_c3(const ConvProblem &p0, cudaStream_t stream)
{
    using C = C3Cfg<CW, BN>;
    ConvProblem p = p0;
    p.err = device_error_word();
    const C3Geom g = c3_geometry(p);
    const int smem = c3_smem_bytes<CW, BN>(g);
    if (smem > 227 * 1024 - 1024) return BCNN_ERR_UNSUPPORTED;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    EncodeTiledFn encode = c3_encode_fn();
    if (!encode) return BCNN_ERR_CUDA;
    // the packed input as [B][H][W * CW] 32-bit words; box = wbw words x hb rows of one image; zero fill outside
    CUtensorMap xmap;
    const cuuint64_t dims[3] = {(cuuint64_t)p.W * CW, (cuuint64_t)p.H, (cuuint64_t)p.B};
    const cuuint64_t strides[2] = {(cuuint64_t)p.W * CW * 4, (cuuint64_t)p.H * p.W * CW * 4};
    const cuuint32_t box[3] = {(cuuint32_t)g.wbw, (cuuint32_t)g.hb, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint32_t *>(p.x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return BCNN_ERR_CUDA;
    const unsigned grid = (unsigned)(g.total_tiles < sms ? g.total_tiles : sms);
    void (*k)(const ConvProblem, const C3Geom, const CUtensorMap) = conv_tc_c3_kernel<CW, BN>;
    const int ask = smem < 120 * 1024 ? 120 * 1024 : smem;          // one CTA per SM (it takes all of tensor memory)
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 1024) != cudaSuccess) return BCNN_ERR_CUDA;
    k<<<grid, C::THREADS, ask, stream>>>(p, g, xmap);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace

bool conv_tc_c3_supports(const ConvProblem &p)
{
    if (p.mode != 1) return false;                               // packed output only
    if (p.kh != 3 || p.kw != 3 || p.stride < 1 || p.stride > 2 || p.pad > 1) return false;
    if (p.cw != 1 && p.cw != 2) return false;
    if (p.C_out % 32 != 0 || p.C_out > 128) return false;
    if ((p.W * p.cw) % 4 != 0) return false;                     // image rows must be 16-byte multiples (TMA strides)
    if ((reinterpret_cast<uintptr_t>(p.x) & 15u) != 0) return false;   // TMA base address
    const long tiles = (long)p.B * ((p.OH + TH - 1) / TH) * ((p.OW + TW - 1) / TW);
    return tiles < (1L << 30);                                   // tile numbers are 32-bit on the device
}

int launch_conv_tc_c3(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_tc_c3_supports(p)) return BCNN_ERR_UNSUPPORTED;
    if (p.cw == 1) {
        if (p.C_out <= 32) return launch_c3<1, 32>(p, stream);
        if (p.C_out <= 64) return launch_c3<1, 64>(p, stream);
        return launch_c3<1, 128>(p, stream);
    }
    if (p.C_out <= 32) return launch_c3<2, 32>(p, stream);
    if (p.C_out <= 64) return launch_c3<2, 64>(p, stream);
    return launch_c3<2, 128>(p, stream);
}

}  // namespace bcnn
