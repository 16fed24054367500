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
// The CTA runs TWO independent pipelines (slots); tiles alternate between them.  A slot owns a loader warp with a ring
// of halo tiles, four producer warps, an issuer warp, four epilogue warps and its share of tensor memory: NACC
// accumulators and a ring of NU activation UNITS of UW words of K (8 columns per word).  A tile's K is cut into
// UPT = ceil(9 C_in / 32 / UW) units.  The producers fill units in order, the issuer multiplies a unit as soon as it is
// full and hands it back with a commit, the last unit's commit also hands the accumulator to the epilogue; so inside a
// slot the expansion of the next unit (or tile) runs under the MMAs of this one, and the epilogue of a tile under the
// MMAs of the next (NACC = 2).  An issuer that waits right behind its own MMAs stalls until they drain; the other
// slot's MMAs fill that gap.
// K = 288 or 576 makes |accumulator| exceed 16 bits, so the epilogue reads 32-bit accumulators and shifts sign bits in.
// A parity wait on an mbarrier is only right while the waiter starts waiting for completion k after completion k - 1 and
// before completion k + 1: every barrier here has one group of waiters that takes its completions in turn.
// Every mbarrier wait is bounded and reports through the device error word.
#include "tc_slot.cuh"
#include <cuda.h>

namespace bcnn {

namespace {

using namespace tc;

constexpr int ERR_C3_LOADER_TIMEOUT = 141;       // loader: no free ring stage
constexpr int ERR_C3_PRODUCER_TIMEOUT = 142;     // producer: the tile's halo did not arrive
constexpr int ERR_C3_ISSUER_TIMEOUT = 143;       // issuer: a unit was not filled
constexpr int ERR_C3_EPILOGUE_TIMEOUT = 144;     // epilogue: the tile's MMAs did not complete
constexpr int ERR_C3_UNIT_TIMEOUT = 145;         // producer: a unit's previous MMAs did not complete
constexpr int ERR_C3_ACC_TIMEOUT = 146;          // issuer: an accumulator was not handed back

constexpr int TH = 8, TW = 16;            // output tile (TH * TW = 128 = tensor-memory lanes)
constexpr int NSLOT = 2;
constexpr int RD = 6;                     // halo tiles in a slot's ring
constexpr int CONST_COLS = 8;
constexpr int MAX_NU = 3, MAX_NACC = 2;

// CW: words per input pixel (1, 2); BN: accumulator columns per tile (32, 64, 128 >= C_out).
template <int CW, int BN> struct C3Cfg {
    static constexpr int KW = 9 * CW;                       // words of K per row
    static constexpr int KT = (KW + 3) / 4;                 // 128-byte stages of the expanded weights
    static constexpr int NACC = BN == 128 ? 1 : 2;          // accumulators per slot
    static constexpr int UW = BN == 32 ? 9 : 5;             // words per unit
    static constexpr int NU = BN == 32 ? 2 : 3;             // units in a slot's ring
    static constexpr int UPT = (KW + UW - 1) / UW;          // units per tile
    static constexpr int U_COLS = 8 * UW;
    static constexpr int SLOT_COLS = NACC * BN + NU * U_COLS;
    static constexpr int C_COL = NSLOT * SLOT_COLS;         // the constant activation tile
    static_assert(C_COL + CONST_COLS <= 512, "tensor memory budget");
    static_assert(NU <= MAX_NU && NACC <= MAX_NACC, "barrier table");
    // warps: 0, 1 issuers; 2, 3 loaders; then per slot four producer warps, then per slot four epilogue warps
    // (groups start at multiples of four: warp % 4 is the tensor-memory lane quadrant of a warp)
    static constexpr int FIRST_LOADER_WARP = 2;
    static constexpr int FIRST_PRODUCER_WARP = 4;
    static constexpr int FIRST_EPILOGUE_WARP = 4 + 4 * NSLOT;
    static constexpr int WARPS = 4 + 8 * NSLOT;
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
    return 1024 + (C::KT + 1) * C::W_TILE_BYTES + NSLOT * RD * g.stage_bytes + 128;
}

// tensor-memory stores of n expanded words (8 columns each) starting at taddr, no wait
template <int N>
__device__ __forceinline__ void store_words(uint32_t taddr, const uint32_t *wds)
{
#pragma unroll
    for (int e4 = 0; e4 + 4 <= N; e4 += 4) {
        uint32_t v[32];
#pragma unroll
        for (int e = 0; e < 4; ++e) expand_a(wds[e4 + e], &v[8 * e]);
        tc_st32_nowait(taddr + 8u * e4, v);
    }
#pragma unroll
    for (int e = N / 4 * 4; e < N; ++e) {
        uint32_t v[8];
        expand_a(wds[e], v);
        tc_st8_nowait(taddr + 8u * e, v);
    }
}

template <int CW, int BN>
__global__ void __launch_bounds__(C3Cfg<CW, BN>::THREADS, 1)
conv_tc_c3_kernel(const ConvProblem p, const C3Geom g, const __grid_constant__ CUtensorMap xmap)
{
    using C = C3Cfg<CW, BN>;
    constexpr int KW = C::KW, KT = C::KT, NACC = C::NACC, UW = C::UW, NU = C::NU, UPT = C::UPT;
    constexpr int BARS_PER_SLOT = 2 * RD + 2 * MAX_NU + 2 * MAX_NACC;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[NSLOT * BARS_PER_SLOT];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    // this CTA's tiles: blockIdx.x + q * gridDim.x; tile q belongs to slot q % 2, the slot's n-th tile is q = 2 n + slot
    const int my_tiles = (int)blockIdx.x < g.total_tiles ? (g.total_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int cn = min(BN, p.C_out);

    const uint32_t wexp = (smem_u32(smem_raw) + 1023u) & ~1023u;          // [KT][BN rows][128 B] expanded weights
    const uint32_t cexp = wexp + KT * C::W_TILE_BYTES;                    // [BN rows][128 B] constant bytes (first 32 of a row)
    const uint32_t ring = cexp + C::W_TILE_BYTES;                         // [NSLOT][RD] halo tiles
    const uint32_t bar0 = smem_u32(bars);
    auto load_full = [&](int sl, int s) { return bar0 + 8u * (sl * BARS_PER_SLOT + s); };
    auto load_empty = [&](int sl, int s) { return bar0 + 8u * (sl * BARS_PER_SLOT + RD + s); };
    auto a_full = [&](int sl, int s) { return bar0 + 8u * (sl * BARS_PER_SLOT + 2 * RD + s); };
    auto a_empty = [&](int sl, int s) { return bar0 + 8u * (sl * BARS_PER_SLOT + 2 * RD + MAX_NU + s); };
    auto acc_full = [&](int sl, int s) { return bar0 + 8u * (sl * BARS_PER_SLOT + 2 * RD + 2 * MAX_NU + s); };
    auto acc_free = [&](int sl, int s) { return bar0 + 8u * (sl * BARS_PER_SLOT + 2 * RD + 2 * MAX_NU + MAX_NACC + s); };
    volatile int *abort_flag = &abort_flag_smem;

    if (tid == 0) {
        for (int sl = 0; sl < NSLOT; ++sl) {
            for (int s = 0; s < RD; ++s) {
                mbar_init(load_full(sl, s), 1);         // the loader's arrive (+ the copy's bytes)
                mbar_init(load_empty(sl, s), 4);        // the slot's four producer warps
            }
            for (int s = 0; s < MAX_NU; ++s) {
                mbar_init(a_full(sl, s), 4);            // the slot's four producer warps
                mbar_init(a_empty(sl, s), 1);           // the issuer's commit
            }
            for (int s = 0; s < MAX_NACC; ++s) {
                mbar_init(acc_full(sl, s), 1);          // the issuer's commit
                mbar_init(acc_free(sl, s), 4);          // the slot's four epilogue warps
            }
        }
        abort_flag_smem = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // ---- one-off: expanded weights (K word e -> stage e / 4, 32-byte piece e % 4) and the constant bytes
    for (int idx = tid; idx < (KT + 1) * BN; idx += C::THREADS) {
        const int kt = idx / BN, row = idx - kt * BN;
        const bool have = row < cn;
        const int xr = row & 7;
        if (kt < KT) {
            const uint32_t row_addr = wexp + (uint32_t)kt * C::W_TILE_BYTES + (uint32_t)row * ROWB;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int kword = kt * 4 + e;
                const bool live = kword < KW && have;
                const uint32_t w = live ? __ldg(p.w + (long)row * KW + kword) : 0u;
                expand_store_w_signed(w, live, row_addr, xr, 2 * e);
            }
        } else {
            // cst = 32 * c, c = K - 2 popc(G) - thr (thr clamped to +-(K + 1)); the constant activation tile's bytes are
            // all 32, so the row's 32 signed bytes add up to c: c / 32 everywhere, one more unit of c's sign in |c % 32|
            int pop = 0;
            if (have)
                for (int e = 0; e < KW; ++e) pop += __popc(__ldg(p.w + (long)row * KW + e));
            int t = have ? __ldg(p.thr + row) : 0;
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
    auto slot_tiles = [&](int slot) { return (my_tiles + 1 - slot) / 2; };
    auto tile_of = [&](int slot, int n) { return (int)blockIdx.x + (2 * n + slot) * (int)gridDim.x; };

    if (warp < NSLOT) {
        // ------------------------------------------------------------------ MMA issuer of slot `warp`
        const int slot = warp;
        constexpr uint32_t idesc = make_idesc(BN) | (1u << 10);                  // B operand: signed bytes
        const uint64_t desc0 = make_desc(wexp);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32), b_lo = (uint32_t)desc0;
        const uint32_t c_lo = (uint32_t)make_desc(cexp);
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0) + (uint32_t)(slot * C::SLOT_COLS);
        const uint32_t c_t = tmem_u - (uint32_t)(slot * C::SLOT_COLS) + (uint32_t)C::C_COL;
        const int nt = slot_tiles(slot);
        int ust = 0, acc = 0;
        uint32_t uphase = 0, aphase = 0;          // parity of the unit ring's / the accumulators' current round
        bool ok = true;
        for (int n = 0; n < nt && ok; ++n) {
            const uint32_t d_t = tmem_u + (uint32_t)(acc * BN);
#pragma unroll
            for (int h = 0; h < UPT; ++h) {
                ok = pw_wait(a_full(slot, ust), uphase, abort_flag, p.err, ERR_C3_ISSUER_TIMEOUT);
                if (!ok) break;
                if (h == 0 && n >= NACC) {       // the epilogue has read the accumulator's previous tile
                    ok = pw_wait(acc_free(slot, acc), aphase ^ 1u, abort_flag, p.err, ERR_C3_ACC_TIMEOUT);
                    if (!ok) break;
                }
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t a_t = tmem_u + (uint32_t)(NACC * BN + ust * C::U_COLS);
                    if (h == 0) tc_mma_i8_ts(d_t, c_t, c_lo, desc_hi, idesc, 0u);   // accumulator = the per-channel constants
#pragma unroll
                    for (int e = h * UW; e < (h + 1) * UW && e < KW; ++e)
                        tc_mma_i8_ts(d_t, a_t + 8u * (e - h * UW), b_lo + (uint32_t)((e >> 2) * (C::W_TILE_BYTES >> 4) + 2 * (e & 3)), desc_hi, idesc, 1u);
                    tc_commit(a_empty(slot, ust));
                    if (h == UPT - 1) tc_commit(acc_full(slot, acc));
                }
                __syncwarp();
                if (++ust == NU) { ust = 0; uphase ^= 1u; }
            }
            if (++acc == NACC) { acc = 0; aphase ^= 1u; }
        }
    } else if (warp < C::FIRST_PRODUCER_WARP) {
        // ------------------------------------------------------------------ loader of slot warp - 2: one halo tile per TMA copy
        const int slot = warp - C::FIRST_LOADER_WARP;
        const int nt = slot_tiles(slot);
        int stage = 0;
        uint32_t phase = 1;                       // first pass through the ring: the stages are free
        int issued = 0;
        for (int n = 0; n < nt; ++n) {
            if (!pw_wait(load_empty(slot, stage), phase, abort_flag, p.err, ERR_C3_LOADER_TIMEOUT)) break;
            if (lane == 0) {
                const uint32_t dst = ring + (uint32_t)(slot * RD + stage) * (uint32_t)g.stage_bytes;
                int b, oh0, ow0;
                tile_origin(tile_of(slot, n), b, oh0, ow0);
                const int x = (ow0 * g.stride - p.pad - g.xoff) * CW;        // words; a multiple of 4 by construction
                const int y = oh0 * g.stride - p.pad;
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(load_full(slot, stage)), "r"((uint32_t)(g.hb * g.wbw * 4)) : "memory");
                asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                             ::"r"(dst), "l"(reinterpret_cast<uint64_t>(&xmap)), "r"(x), "r"(y), "r"(b), "r"(load_full(slot, stage)) : "memory");
            }
            __syncwarp();
            ++issued;
            if (++stage == RD) { stage = 0; phase ^= 1u; }
        }
        // after a time-out elsewhere: copies still in flight must land before the CTA's shared memory goes away
        if (*abort_flag) {
            const int first = issued > RD ? issued - RD : 0;
            for (int q = first; q < issued; ++q)
                pw_wait(load_full(slot, q % RD), (uint32_t)(q / RD) & 1u, abort_flag, nullptr, 0);
        }
    } else if (warp >= C::FIRST_EPILOGUE_WARP) {
        // ------------------------------------------------------------------ epilogue of slot (warp - first) / 4
        const int quad = warp & 3;
        const int slot = (warp - C::FIRST_EPILOGUE_WARP) >> 2;
        const int r = quad * 32 + lane;                           // row of the tile = output pixel (r / TW, r % TW)
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(slot * C::SLOT_COLS);
        const int owords = p.C_out >> 5;
        const int nt = slot_tiles(slot);
        int acc = 0;
        uint32_t aphase = 0;
        for (int n = 0; n < nt; ++n) {
            if (!pw_wait(acc_full(slot, acc), aphase, abort_flag, p.err, ERR_C3_EPILOGUE_TIMEOUT)) break;
            tc_fence_after();
            uint32_t words[BN / 32];
#pragma unroll
            for (int ch = 0; ch < BN / 32; ++ch) {
                words[ch] = 0;
                if (ch * 32 < cn) {                                   // warp-uniform
                    uint32_t v[32];
                    tc_ld32(t_lane + (uint32_t)(acc * BN + ch * 32), v);
                    if ((ch + 1) * 32 >= cn) {                        // the accumulator's last columns are in registers
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(acc_free(slot, acc));
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
            tile_origin(tile_of(slot, n), b, oh0, ow0);
            const int oh = oh0 + (r >> 4), ow = ow0 + (r & 15);
            if (oh < p.OH && ow < p.OW) {
                uint32_t *dst = static_cast<uint32_t *>(p.out) + (((long)b * p.OH + oh) * p.OW + ow) * owords;
                if (BN == 128 && owords == 4) {
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(words[0], words[1 % (BN / 32)], words[2 % (BN / 32)], words[3 % (BN / 32)]);
                } else if (BN >= 64 && owords == 2) {
                    *reinterpret_cast<uint2 *>(dst) = make_uint2(words[0], words[1 % (BN / 32)]);
                } else {
#pragma unroll
                    for (int ch = 0; ch < BN / 32; ++ch)
                        if (ch < owords) dst[ch] = words[ch];
                }
            }
            if (++acc == NACC) { acc = 0; aphase ^= 1u; }
        }
    } else {
        // ------------------------------------------------------------------ producers of slot (warp - first) / 4
        // thread = output pixel (ty, tx) of the tile = tensor-memory lane; its nine input pixels sit at rows
        // ty * s + kr, pixels tx * s + XOFF + kt of the halo tile
        const int quad = warp & 3;
        const int slot = (warp - C::FIRST_PRODUCER_WARP) >> 2;
        const int r = quad * 32 + lane;
        const uint32_t my_off = (uint32_t)((((r >> 4) * g.stride) * g.wbw + ((r & 15) * g.stride + g.xoff) * CW) * 4);
        const uint32_t row_pitch = (uint32_t)(g.wbw * 4);
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(slot * C::SLOT_COLS + NACC * BN);
        const uint32_t lane0 = lane == 0 ? 1u : 0u;
        const int nt = slot_tiles(slot);
        int stage = 0, ust = 0, units = 0;
        uint32_t lphase = 0, uphase = 0;
        bool ok = true;
        for (int n = 0; n < nt && ok; ++n) {
            uint32_t wds[KW];
            if (!pw_wait(load_full(slot, stage), lphase, abort_flag, p.err, ERR_C3_PRODUCER_TIMEOUT)) break;
            const uint32_t src = ring + (uint32_t)(slot * RD + stage) * (uint32_t)g.stage_bytes + my_off;
#pragma unroll
            for (int kr = 0; kr < 3; ++kr)
#pragma unroll
                for (int kt = 0; kt < 3; ++kt) {
                    const uint32_t a = src + (uint32_t)kr * row_pitch + (uint32_t)(kt * CW * 4);
                    if constexpr (CW == 2) {
                        asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(wds[(kr * 3 + kt) * 2]), "=r"(wds[(kr * 3 + kt) * 2 + 1]) : "r"(a) : "memory");
                    } else {
                        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(wds[kr * 3 + kt]) : "r"(a) : "memory");
                    }
                }
            __syncwarp();
            mbar_arrive_pred(load_empty(slot, stage), lane0);       // the stage may be refilled
            if (++stage == RD) { stage = 0; lphase ^= 1u; }
#pragma unroll
            for (int h = 0; h < UPT; ++h) {
                // the MMAs of the unit's previous use have read it (nothing to wait for the first time round the ring)
                if (units >= NU) {
                    ok = pw_wait(a_empty(slot, ust), uphase ^ 1u, abort_flag, p.err, ERR_C3_UNIT_TIMEOUT);
                    if (!ok) break;
                }
                tc_fence_after();
                constexpr int LAST = KW - (UPT - 1) * UW;           // words of the tile's last unit
                const uint32_t taddr = t_lane + (uint32_t)(ust * C::U_COLS);
                if (h < UPT - 1) store_words<UW>(taddr, &wds[h * UW]);
                else store_words<LAST>(taddr, &wds[(UPT - 1) * UW]);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                mbar_arrive_pred(a_full(slot, ust), lane0);
                ++units;
                if (++ust == NU) { ust = 0; uphase ^= 1u; }
            }
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
