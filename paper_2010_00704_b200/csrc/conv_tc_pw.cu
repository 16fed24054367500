// Pointwise engine: binary 1x1 convolutions (stride 1, no padding) and plain GEMMs with a short K (32..128 bits)
// and up to 128 output channels, packed output.  These layers move 8..32 bytes per output row and are bound by
// memory, not by the tensor pipe: the binary 1x1 convolution is the only binary operator of the paper's own network
// (Section 4.2.1; Table 1), at resolutions up to 224 x 224.
//
// Arithmetic as in the weight-stationary engine (conv_tc_ws.cu): sign bits expanded to bytes on chip, unsigned
// activation bytes {0, 2^j} against signed weight bytes +-2^(6-j), int32 accumulators in tensor memory, and with
// S = sum over set activation bits of the weight signs:  sum a*g = 2 S + K - 2 popc(G),  accumulator = 64 S + cst,
// cst = 32 (K - 2 popc(G) - threshold), output bit = (accumulator >= 0).
//
// What differs is everything around the MMAs; a row of the patch matrix is simply KW consecutive words of x.
//   * Work is cut into CHUNKS of T tiles (T * 128 rows) and BLOCKS of G consecutive chunks; a CTA takes whole
//     blocks.  A block is one contiguous range of x and arrives by ONE bulk asynchronous copy (cp.async.bulk,
//     6 - 12 KB, completion on an mbarrier) into a ring in shared memory, issued by a loader warp: issuing a bulk
//     copy costs the warp about 400 cycles whatever its size, and the bytes in flight per SM do not depend on how
//     many threads are waiting.
//   * Tensor memory is cut into NSLOT slots of T tiles (accumulator + expanded activation tile each).  Every slot is
//     a pipeline of its own - one issuer warp, one producer group and one epilogue group of four warps - and takes
//     the chunks slot, slot + NSLOT, ...  Per chunk there is ONE hand-over in each direction: the producers expand
//     all T tiles (ld.shared, 8 logic operations per word, tcgen05.st) and arrive once; the issuer issues all MMAs
//     back to back and commits once; the epilogue reads the T accumulators and hands the slot back as soon as
//     they are in registers.  An issuer only ever waits for MMAs that completed a whole slot cycle ago, so it can
//     do its own mbarrier waits.  (An issuer that waits right behind its own MMAs stalls until they drain: with one
//     issuer for all slots that was about 700 cycles per chunk and the whole kernel's bound; two buffers per slot
//     fed by one issuer stall the same way on the second commit.)
//   * The per-channel constant is the accumulator's starting value, and an MMA writes it: the first MMA of a tile
//     (not accumulating) multiplies a constant activation tile (every byte 32, written once) with 32 signed bytes
//     per channel that add up to cst / 32.  Nobody ever stores constants into tensor memory, so the epilogue only
//     reads.
//   * The epilogue loads accumulators as packed 16-bit halves (tcgen05.ld .pack::16b: |accumulator| < 2^15 for
//     K <= 128), two columns per register, and gathers sign bits with byte permutes in sign-replication mode: one
//     PRMT + one LOP3 per four columns instead of one shift per column.  Bit s of byte B of an output word then
//     comes from accumulator column 2s (B = 0), 2s + 1 (B = 1), 16 + 2s (B = 2), 17 + 2s (B = 3) of its 32-column
//     block; the weight rows are laid out in that order (channel_of_column), which costs nothing.
// Parity waits on an mbarrier are only right while the waiter starts waiting for completion k after completion k - 1
// and before completion k + 1; binding every role of a slot to that slot, and giving every slot the same number of
// chunks in every block (G is a multiple of NSLOT), gives every waiter each completion of its barriers in turn.
// Every mbarrier wait is bounded and reports through the device error word; the loader waits for its copies in
// flight before the CTA ends after a time-out.
#include "tc_slot.cuh"

namespace bcnn {

namespace {

using namespace tc;

constexpr int ERR_PW_LOADER_TIMEOUT = 121;       // loader: no free ring stage
constexpr int ERR_PW_PRODUCER_TIMEOUT = 122;     // producer: the chunk's rows did not arrive
constexpr int ERR_PW_ISSUER_TIMEOUT = 123;       // issuer: the slot's rows were not expanded
constexpr int ERR_PW_EPILOGUE_TIMEOUT = 124;     // epilogue: the chunk's MMAs did not complete
constexpr int ERR_PW_SLOT_TIMEOUT = 125;         // producer: the slot's previous MMAs did not complete
constexpr int ERR_PW_ACC_TIMEOUT = 126;          // issuer: the slot's accumulators were not handed back

constexpr int MAX_BLOCKS = 16;            // stages of the shared-memory ring (one block each)
constexpr int RING_BYTES = 96 * 1024;
constexpr int BLOCK_BYTES_TARGET = 12 * 1024;
constexpr int CONST_COLS = 8;             // the constant activation tile: 32 bytes per row

// tiles (accumulator + expanded activations) that fit in tensor memory beside the constant tile, cut into three slots
// where that leaves whole tiles (3, 6..12 tiles), else two (4, 5 tiles)
__host__ __device__ constexpr int pw_tiles(int kw, int bn) { return (512 - CONST_COLS) / (bn + 8 * kw); }
__host__ __device__ constexpr int pw_nslot(int kw, int bn) { return (pw_tiles(kw, bn) >= 6 || pw_tiles(kw, bn) == 3) ? 3 : 2; }
__host__ __device__ constexpr int pw_t(int kw, int bn)
{
    return pw_tiles(kw, bn) / pw_nslot(kw, bn) > 4 ? 4 : pw_tiles(kw, bn) / pw_nslot(kw, bn);
}

// KW: words of K per row (1..4); BN: accumulator columns per tile (32, 64, 128 >= C_out).
template <int KW, int BN> struct PwCfg {
    static constexpr int T = pw_t(KW, BN);                  // tiles per chunk
    static constexpr int NSLOT = pw_nslot(KW, BN);
    static constexpr int TILES = NSLOT * T;
    static constexpr int A_COL0 = TILES * BN;               // accumulators first, then the expanded activation tiles
    static constexpr int A_COLS = 8 * KW;
    static constexpr int C_COL = A_COL0 + TILES * A_COLS;   // the constant activation tile
    static_assert(C_COL + CONST_COLS <= 512, "tensor memory budget");
    static_assert(T >= 1 && T <= 4 && NSLOT >= 2 && NSLOT <= 3, "slot shape");
    static constexpr int CHUNK_ROWS = T * BM;
    static constexpr int CHUNK_BYTES = CHUNK_ROWS * KW * 4;
    // chunks per block: a multiple of the slots (every slot has the same share of every block), about 12 KB
    static constexpr int G0 = BLOCK_BYTES_TARGET / (NSLOT * CHUNK_BYTES);
    static constexpr int G = NSLOT * (G0 < 1 ? 1 : G0);
    static constexpr int BLOCK_ROWS = G * CHUNK_ROWS;
    static constexpr int BLOCK_BYTES = G * CHUNK_BYTES;
    static constexpr int NBLK = RING_BYTES / BLOCK_BYTES > MAX_BLOCKS ? MAX_BLOCKS : RING_BYTES / BLOCK_BYTES;
    static_assert(NBLK >= 4, "ring depth");
    // warps: 0..NSLOT-1 issuers (one per slot), 3 loader, then per slot four producer warps, then per slot four
    // epilogue warps (groups start at multiples of four: warp % 4 is the tensor-memory lane quadrant of a warp)
    static constexpr int LOADER_WARP = 3;
    static constexpr int FIRST_PRODUCER_WARP = 4;
    static constexpr int FIRST_EPILOGUE_WARP = 4 + 4 * NSLOT;
    static constexpr int WARPS = 4 + 8 * NSLOT;
    static constexpr int THREADS = 32 * WARPS;
    static constexpr int W_BYTES = BN * ROWB;               // expanded weights: [BN rows][128 B], 32 * KW bytes used per row
    static constexpr int SMEM = 1024 + 2 * W_BYTES + NBLK * BLOCK_BYTES + 64;
    static constexpr int SMEM_ASK = SMEM < 120 * 1024 ? 120 * 1024 : SMEM;     // one CTA per SM (it takes all of tensor memory)
};

template <int KW, int BN>
__global__ void __launch_bounds__(PwCfg<KW, BN>::THREADS, 1)
conv_tc_pw_kernel(const ConvProblem p)
{
    using C = PwCfg<KW, BN>;
    constexpr int T = C::T, NSLOT = C::NSLOT, G = C::G, NBLK = C::NBLK;

    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * MAX_BLOCKS + 3 * 3];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag_smem;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    // this CTA's blocks: blockIdx.x, blockIdx.x + gridDim.x, ...; its j-th chunk (chunk j % G of its block j / G)
    // belongs to slot j % NSLOT.  Only the last block of all can be short; it is the last one of its CTA.
    const long n_blocks = ((long)p.M + C::BLOCK_ROWS - 1) / C::BLOCK_ROWS;
    const int my_blocks = (long)blockIdx.x < n_blocks ? (int)((n_blocks - 1 - blockIdx.x) / gridDim.x) + 1 : 0;
    int my_chunks = my_blocks * G;
    if (my_blocks > 0 && (long)blockIdx.x + (long)(my_blocks - 1) * gridDim.x == n_blocks - 1) {
        const long rows_last = (long)p.M - (n_blocks - 1) * C::BLOCK_ROWS;
        my_chunks -= G - (int)((rows_last + C::CHUNK_ROWS - 1) / C::CHUNK_ROWS);
    }
    // first row of this CTA's chunk j
    auto chunk_row0 = [&](int j) { return ((long)blockIdx.x + (long)(j / G) * gridDim.x) * C::BLOCK_ROWS + (long)(j % G) * C::CHUNK_ROWS; };
    const int cn = min(BN, p.C_out);

    const uint32_t wexp = (smem_u32(smem_raw) + 1023u) & ~1023u;          // [BN rows][128 B] expanded weights
    const uint32_t cexp = wexp + C::W_BYTES;                              // [BN rows][128 B] constant bytes (first 32 of a row)
    const uint32_t ring = cexp + C::W_BYTES;                              // [NBLK][BLOCK_ROWS][KW words]
    const uint32_t bar0 = smem_u32(bars);
    auto load_full = [&](int s) { return bar0 + 8u * s; };
    auto load_empty = [&](int s) { return bar0 + 8u * (MAX_BLOCKS + s); };
    auto a_full = [&](int s) { return bar0 + 8u * (2 * MAX_BLOCKS + s); };
    auto mma_done = [&](int s) { return bar0 + 8u * (2 * MAX_BLOCKS + 3 + s); };
    auto acc_free = [&](int s) { return bar0 + 8u * (2 * MAX_BLOCKS + 6 + s); };
    volatile int *abort_flag = &abort_flag_smem;

    if (tid == 0) {
        for (int s = 0; s < MAX_BLOCKS; ++s) {
            mbar_init(load_full(s), 1);             // the loader's arrive (+ the copy's bytes)
            mbar_init(load_empty(s), 4 * G);        // four producer warps for each of the block's chunks
        }
        for (int s = 0; s < 3; ++s) {
            mbar_init(a_full(s), 4);                // the slot's four producer warps
            mbar_init(mma_done(s), 1);              // the slot's issuer (commit)
            mbar_init(acc_free(s), 4);              // the slot's four epilogue warps
        }
        abort_flag_smem = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // ---- one-off: expanded weights and constant bytes; MMA row `row` carries channel 32 * (row / 32) + channel_of_column(row % 32)
    for (int row = tid; row < BN; row += C::THREADS) {
        const int ch = (row & ~31) + channel_of_column(row & 31);
        const bool have = ch < cn;
        const uint32_t row_addr = wexp + (uint32_t)row * ROWB;
        int pop = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool live = e < KW && have;
            const uint32_t w = live ? __ldg(p.w + (long)ch * KW + e) : 0u;
            pop += __popc(w);
            expand_store_w_signed(w, live, row_addr, row & 7, 2 * e);
        }
        // cst = 32 * c, c = K - 2 popc(G) - thr with thr clamped to +-(K + 1) (beyond that bound the decision is
        // constant); the constant tile's bytes are all 32, so the row's 32 signed bytes must add up to c:
        // c / 32 everywhere and one more unit of c's sign in the first |c % 32| of them
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
        const int xr = row & 7;
        st_shared_v4(crow + (uint32_t)((0 ^ xr) << 4), cw[0], cw[1], cw[2], cw[3]);
        st_shared_v4(crow + (uint32_t)((1 ^ xr) << 4), cw[4], cw[5], cw[6], cw[7]);
    }
    fence_async_proxy();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;
    // the constant activation tile: every byte 32 (one producer group writes its four lane quadrants)
    if (warp >= C::FIRST_PRODUCER_WARP && warp < C::FIRST_PRODUCER_WARP + 4) {
        const uint32_t c8[8] = {0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u, 0x20202020u};
        tc_st8_nowait(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)C::C_COL, c8);
        tc_wait_st();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (warp < NSLOT) {
        // ------------------------------------------------------------------ MMA issuer of slot `warp`
        const int slot = warp;
        constexpr uint32_t idesc = make_idesc(BN) | (1u << 10);                  // B operand: signed bytes
        const uint64_t desc0 = make_desc(wexp);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32), b_lo = (uint32_t)desc0;
        const uint32_t c_lo = (uint32_t)make_desc(cexp);
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t c_t = tmem_u + (uint32_t)C::C_COL;
        uint32_t phase = 0;
        for (int j = slot; j < my_chunks; j += NSLOT) {
            // the epilogue has read the slot's previous accumulators (nothing to wait for the first time round)
            if (j >= NSLOT && !pw_wait(acc_free(slot), phase ^ 1u, abort_flag, p.err, ERR_PW_ACC_TIMEOUT)) break;
            if (!pw_wait(a_full(slot), phase, abort_flag, p.err, ERR_PW_ISSUER_TIMEOUT)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int t = 0; t < T; ++t) {
                    const uint32_t d_t = tmem_u + (uint32_t)((slot * T + t) * BN);
                    const uint32_t a_t = tmem_u + (uint32_t)(C::A_COL0 + (slot * T + t) * C::A_COLS);
                    tc_mma_i8_ts(d_t, c_t, c_lo, desc_hi, idesc, 0u);            // accumulator = the per-channel constants
#pragma unroll
                    for (int e = 0; e < KW; ++e)
                        tc_mma_i8_ts(d_t, a_t + 8u * e, b_lo + 2u * e, desc_hi, idesc, 1u);
                }
                tc_commit(mma_done(slot));
            }
            __syncwarp();
            phase ^= 1u;
        }
    } else if (warp == C::LOADER_WARP) {
        // ------------------------------------------------------------------ loader
        // One bulk copy per block into ring stage b % NBLK.  A last block whose byte count is not a multiple of 16
        // is copied by the warp with plain loads instead.  Rows beyond M are never read from x; whatever the stage
        // holds there is expanded and multiplied, and the epilogue does not store those rows.
        int stage = 0;
        uint32_t phase = 1;                       // first pass through the ring: the stages are free
        int issued = 0;
        for (int b = 0; b < my_blocks; ++b) {
            const long row0 = ((long)blockIdx.x + (long)b * gridDim.x) * C::BLOCK_ROWS;
            const long rows = min((long)C::BLOCK_ROWS, (long)p.M - row0);
            const uint32_t bytes = (uint32_t)rows * KW * 4u;
            if (!pw_wait(load_empty(stage), phase, abort_flag, p.err, ERR_PW_LOADER_TIMEOUT)) break;
            const uint32_t dst = ring + (uint32_t)stage * C::BLOCK_BYTES;
            const uint32_t *src = p.x + row0 * KW;
            if ((bytes & 15u) == 0u) {
                if (lane == 0) {
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(load_full(stage)), "r"(bytes) : "memory");
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(dst), "l"(src), "r"(bytes), "r"(load_full(stage)) : "memory");
                }
            } else {
                for (uint32_t i = lane; i < bytes / 4u; i += 32)
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(dst + 4u * i), "r"(__ldg(src + i)) : "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(load_full(stage));
            }
            __syncwarp();
            ++issued;
            if (++stage == NBLK) { stage = 0; phase ^= 1u; }
        }
        // after a time-out elsewhere: copies still in flight must land before the CTA's shared memory goes away
        if (*abort_flag) {
            const int first = issued > NBLK ? issued - NBLK : 0;
            for (int b = first; b < issued; ++b)
                pw_wait(load_full(b % NBLK), (uint32_t)(b / NBLK) & 1u, abort_flag, nullptr, 0);
        }
    } else if (warp >= C::FIRST_EPILOGUE_WARP) {
        // ------------------------------------------------------------------ epilogue of slot (warp - first) / 4
        const int quad = warp & 3;
        const int slot = (warp - C::FIRST_EPILOGUE_WARP) >> 2;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(slot * T * BN);
        const int owords = p.C_out >> 5;
        uint32_t phase = 0;
        for (int j = slot; j < my_chunks; j += NSLOT) {
            const long row_w = chunk_row0(j) + quad * 32 + lane;                 // this thread's row in tile 0
            if (!pw_wait(mma_done(slot), phase, abort_flag, p.err, ERR_PW_EPILOGUE_TIMEOUT)) break;
            tc_fence_after();
            phase ^= 1u;
            // all of the chunk's accumulators -> registers, one wait, and the slot goes back to the issuer before
            // any bit is gathered
            constexpr int NR = BN == 32 ? 16 : 32;                       // registers per load
            constexpr int NL = BN == 32 ? 1 : BN / 64;                   // loads per tile
            uint32_t r[T * NL][NR];
#pragma unroll
            for (int t = 0; t < T; ++t) {
                if constexpr (BN == 32) {
                    tc_ld32_pack16(t_lane + (uint32_t)(t * BN), r[t]);
                } else {
#pragma unroll
                    for (int h = 0; h < NL; ++h) tc_ld64_pack16(t_lane + (uint32_t)(t * BN + h * 64), r[t * NL + h]);
                }
            }
            tc_wait_ld();
#pragma unroll
            for (int q = 0; q < T * NL; ++q) pin_regs(r[q]);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_free(slot));
#pragma unroll
            for (int t = 0; t < T; ++t) {
                uint32_t words[BN / 32];
                if constexpr (BN == 32) {
                    words[0] = sign_word(r[t]);
                } else {
#pragma unroll
                    for (int h = 0; h < NL; ++h) {
                        words[2 * h] = sign_word(r[t * NL + h]);
                        words[2 * h + 1] = sign_word(r[t * NL + h] + 16);
                    }
                }
                const long m = row_w + (long)t * BM;
                if (m < p.M) {
                    uint32_t *dst = static_cast<uint32_t *>(p.out) + m * owords;
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
            }
        }
    } else if (warp >= C::FIRST_PRODUCER_WARP) {
        // ------------------------------------------------------------------ producers of slot (warp - first) / 4
        // thread = row of a tile = tensor-memory lane
        const int quad = warp & 3;
        const int slot = (warp - C::FIRST_PRODUCER_WARP) >> 2;
        const int row = quad * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(C::A_COL0 + slot * T * C::A_COLS);
        const uint32_t lane0 = lane == 0 ? 1u : 0u;
        uint32_t phase = 0;
        for (int j = slot; j < my_chunks; j += NSLOT) {
            const int blk = j / G, stage = blk % NBLK;
            if (!pw_wait(load_full(stage), (uint32_t)(blk / NBLK) & 1u, abort_flag, p.err, ERR_PW_PRODUCER_TIMEOUT)) break;
            const uint32_t src = ring + (uint32_t)stage * C::BLOCK_BYTES + (uint32_t)(j % G) * C::CHUNK_BYTES + (uint32_t)row * (KW * 4u);
            uint32_t wds[T][KW];
#pragma unroll
            for (int t = 0; t < T; ++t) {
                const uint32_t a = src + (uint32_t)t * (BM * KW * 4u);
                if constexpr (KW == 4) {
                    const uint4 q = ld_shared_v4(a);
                    wds[t][0] = q.x; wds[t][1] = q.y; wds[t][2] = q.z; wds[t][3] = q.w;
                } else if constexpr (KW == 2) {
                    asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(wds[t][0]), "=r"(wds[t][1]) : "r"(a) : "memory");
                } else {
#pragma unroll
                    for (int e = 0; e < KW; ++e)
                        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(wds[t][e]) : "r"(a + 4u * e) : "memory");
                }
            }
            __syncwarp();
            mbar_arrive_pred(load_empty(stage), lane0);           // (the stage may be refilled once all its chunks have been read)
            // expanded rows in registers first; only the stores wait for the slot
            uint32_t v[T][8 * KW];
#pragma unroll
            for (int t = 0; t < T; ++t)
#pragma unroll
                for (int e = 0; e < KW; ++e) expand_a(wds[t][e], &v[t][8 * e]);
            // the MMAs of the slot's previous chunk have read its activation columns
            if (j >= NSLOT && !pw_wait(mma_done(slot), phase ^ 1u, abort_flag, p.err, ERR_PW_SLOT_TIMEOUT)) break;
            tc_fence_after();
#pragma unroll
            for (int t = 0; t < T; ++t) {
                const uint32_t taddr = t_lane + (uint32_t)(t * C::A_COLS);
                if constexpr (KW == 4) {
                    tc_st32_nowait(taddr, v[t]);
                } else {
#pragma unroll
                    for (int e = 0; e < KW; ++e) {
                        const uint32_t (&v8)[8] = *reinterpret_cast<const uint32_t (*)[8]>(&v[t][8 * e]);
                        tc_st8_nowait(taddr + 8u * e, v8);
                    }
                }
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            mbar_arrive_pred(a_full(slot), lane0);
            phase ^= 1u;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

template <int KW, int BN>
int launch_pw(const ConvProblem &p0, cudaStream_t stream)
{
    using C = PwCfg<KW, BN>;
    ConvProblem p = p0;
    p.err = device_error_word();
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long n_blocks = ((long)p.M + C::BLOCK_ROWS - 1) / C::BLOCK_ROWS;
    const unsigned grid = (unsigned)(n_blocks < sms ? n_blocks : sms);
    void (*k)(const ConvProblem) = conv_tc_pw_kernel<KW, BN>;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_ASK) != cudaSuccess) return BCNN_ERR_CUDA;
    k<<<grid, C::THREADS, C::SMEM_ASK, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

template <int KW>
int launch_pw_kw(const ConvProblem &p, cudaStream_t stream)
{
    if (p.C_out <= 32) return launch_pw<KW, 32>(p, stream);
    if (p.C_out <= 64) return launch_pw<KW, 64>(p, stream);
    return launch_pw<KW, 128>(p, stream);
}

}  // namespace

bool conv_tc_pw_supports(const ConvProblem &p)
{
    if (p.mode != 1) return false;                               // packed output only
    if (!(p.kh == 1 && p.kw == 1 && p.stride == 1 && p.pad == 0)) return false;
    if (p.kwords < 1 || p.kwords > 4) return false;              // K <= 128: accumulators fit 16 bits
    return p.C_out % 32 == 0 && p.C_out <= 128;
}

int launch_conv_tc_pw(const ConvProblem &p, cudaStream_t stream)
{
    if (!conv_tc_pw_supports(p)) return BCNN_ERR_UNSUPPORTED;
    switch (p.kwords) {
    case 1: return launch_pw_kw<1>(p, stream);
    case 2: return launch_pw_kw<2>(p, stream);
    case 3: return launch_pw_kw<3>(p, stream);
    default: return launch_pw_kw<4>(p, stream);
    }
}

}  // namespace bcnn
