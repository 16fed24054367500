// Device helpers shared by the tcgen05 engines: mbarrier waits with a bound and back-off,
// tcgen05 instruction wrappers (MMA from shared / tensor memory, commit, ld, st, fences),
// cp.async staging, shared-memory descriptors and the bit -> byte expansions.
#pragma once
#include "bcnn_common.cuh"
#include <cuda_fp16.h>

namespace bcnn {
namespace tc {

constexpr int BM = 128;                   // rows of an output tile = tensor-memory lanes
constexpr int ROWB = 128;                 // bytes of one expanded row per stage (= 128 bits of K)
constexpr uint32_t WAIT_LIMIT = 1u << 17; // polls before a wait gives up
// upper bound (ns) for which one try_wait may suspend the thread
constexpr uint32_t SUSPEND_HINT_NS = 20000;
constexpr uint32_t SLEEP_NS = 100;

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
// slots, so after a first failed poll the waiter sleeps between polls.  The polling loop is kept
// out of line: the common case is one successful try_wait.
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err, int code,
                                                   uint32_t limit = WAIT_LIMIT)
{
    for (uint32_t it = 0; it < limit; ++it) {
        __nanosleep(SLEEP_NS);
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    if (err) atomicCAS(err, 0, code);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err, int code,
                                          uint32_t limit = WAIT_LIMIT)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, err, code, limit);
}
// Whole-warp wait: one try_wait per lane and a vote in the common case.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err, int code,
                                               uint32_t limit = WAIT_LIMIT)
{
    bool ok = mbar_try_wait(bar, parity);
    if (__all_sync(0xffffffffu, ok)) return true;
    if (!ok) ok = mbar_wait_slow(bar, parity, abort_flag, err, code, limit);
    return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void mbar_arrive_pred(uint32_t bar, uint32_t pred)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "@q mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}"
        ::"r"(bar), "r"(pred) : "memory");
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
// Single-thread forms (the caller has already elected one lane).
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred = 0;
    asm volatile("{\n\t.reg .b32 rx;\n\t.reg .pred px;\n\telect.sync rx|px, 0xffffffff;\n\tselp.u32 %0, 1, 0, px;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void tc_mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi,
                                             uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], db, %4, {%6, %6, %6, %6}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(0u)
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
// Same without the completion wait, for several stores followed by one tc_wait_st().
__device__ __forceinline__ void tc_st32_nowait(uint32_t taddr, const uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr),
          "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
// 8 columns (one K word) of this warp's 32 lanes <- 8 registers.
__device__ __forceinline__ void tc_st8_nowait(uint32_t taddr, const uint32_t (&v)[8])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
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
// Weights take the value 2^(7-j) where the activation byte is 2^j: reverse the bits of each byte once
// (bit j+8i -> bit (7-j)+8i), after which every output word is again a single AND.
__device__ __forceinline__ void expand_store_w(uint32_t w, uint32_t row_addr, int xr, int c)
{
    const uint32_t r = __byte_perm(__brev(w), 0u, 0x0123u);
    st_shared_v4(row_addr + (uint32_t)(((c) ^ xr) << 4),
                 r & 0x80808080u, r & 0x40404040u, r & 0x20202020u, r & 0x10101010u);
    st_shared_v4(row_addr + (uint32_t)(((c + 1) ^ xr) << 4),
                 r & 0x08080808u, r & 0x04040404u, r & 0x02020202u, r & 0x01010101u);
}

// Activation word -> 8 words for the signed-weight scheme: word j holds bits j, j+8, j+16, j+24 as bytes
// 2^j for j <= 6; bit 7 goes to 64 as well (its weight magnitude is 1 where bit 6's is 1 too, see below).
__device__ __forceinline__ void expand_a(uint32_t w, uint32_t *v)
{
#pragma unroll
    for (int j = 0; j < 7; ++j) v[j] = w & (0x01010101u << j);
    v[7] = (w >> 1) & 0x40404040u;
}
// Weight word -> signed bytes matching expand_a: magnitude 2^(6-j) for j <= 6 and 1 for j = 7, sign = the weight's
// sign (bit set: +), so that every product with a set activation byte is +-64.  `live` false writes zeros.
// The bits of each byte are reversed once (bit j -> bit 7-j) and inverted; in word j the flag "weight is -" then
// sits at bit 7-j of every byte, exactly the lowest bit of the two's-complement pattern of -2^(6-j) above the
// magnitude bit: flag * (2^(j+1) - 1) sets bits 7-j..7, adding the magnitude bit 6-j completes the byte (no
// carries between bytes: every byte stays below 256).  Word 7 (magnitude 1): flag at bit 0, * 0xFE, + 1.
__device__ __forceinline__ void expand_store_w_signed(uint32_t w, bool live, uint32_t row_addr, int xr, int c)
{
    const uint32_t nr = ~__byte_perm(__brev(w), 0u, 0x0123u);
    uint32_t o[8];
#pragma unroll
    for (int j = 0; j < 7; ++j)
        o[j] = live ? (nr & (0x01010101u << (7 - j))) * ((2u << j) - 1u) + (0x01010101u << (6 - j)) : 0u;
    o[7] = live ? (nr & 0x01010101u) * 0xFEu + 0x01010101u : 0u;
    st_shared_v4(row_addr + (uint32_t)(((c) ^ xr) << 4), o[0], o[1], o[2], o[3]);
    st_shared_v4(row_addr + (uint32_t)(((c + 1) ^ xr) << 4), o[4], o[5], o[6], o[7]);
}

// Expand the first nk (1..4) K words of a 128-bit stage into this lane's tensor-memory row (8 columns per word)
// and wait for the stores.  A partial stage stores only its words: the MMAs skip the rest.
__device__ __forceinline__ void expand_store_stage(uint32_t taddr, const uint4 &bits, int nk)
{
    const uint32_t wds[4] = {bits.x, bits.y, bits.z, bits.w};
    if (nk >= 4) {
        uint32_t v[32];
#pragma unroll
        for (int e = 0; e < 4; ++e) expand_a(wds[e], &v[8 * e]);
        tc_st32_nowait(taddr, v);
    } else {
#pragma unroll
        for (int e = 0; e < 3; ++e)
            if (e < nk) {                                   // warp-uniform
                uint32_t v[8];
                expand_a(wds[e], v);
                tc_st8_nowait(taddr + 8u * e, v);
            }
    }
    tc_wait_st();
}

// ---- implicit-im2col gather -----------------------------------------------------------------------
// K is cut into units of GW words that never straddle a tap: GW = 4 (one 16-byte copy) when a pixel
// is a multiple of four words, 2 when it is even, else 1.  The unit table holds, per unit, the word
// offset from the row's top-left input pixel and the tap's bit (0 for the zero padding of K beyond
// kwords); a row carries the word offset of its top-left input pixel and the mask of its taps that
// fall inside the image, so one unit costs a mask test, an add and a copy with zero fill.
__host__ __device__ __forceinline__ int gather_width(int cw) { return (cw & 3) == 0 ? 4 : ((cw & 1) == 0 ? 2 : 1); }

template <int V> struct IntC { static constexpr int value = V; };

__device__ __forceinline__ void build_unit_table(const ConvProblem &p, uint32_t tab_addr, int units, int gw, int tid, int nthreads)
{
    for (int u = tid; u < units; u += nthreads) {
        const int kword = u * gw;
        uint32_t off = 0, bit = 0;
        if (kword < p.kwords) {
            const int tap = kword / p.cw, cj = kword - tap * p.cw;
            const int r = tap / p.kw, t = tap - r * p.kw;
            off = (uint32_t)((r * p.W + t) * p.cw + cj);
            bit = 1u << tap;
        }
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(tab_addr + 8u * u), "r"(off), "r"(bit) : "memory");
    }
}

// Advance of a CTA from one of its row tiles to the next: a constant number of rows, split once into
// whole images, output rows and output columns, so that a row's coordinates follow by carries.
struct TileStep {
    uint32_t rows;
    int db, doh, dow;
    uint32_t pat;            // bit r*kw for every kernel row r
    bool pointwise;          // 1x1, stride 1, no padding: row m reads input pixel m, no coordinates needed
};
__device__ __forceinline__ TileStep make_tile_step(const ConvProblem &p, uint32_t rows)
{
    TileStep s;
    const uint32_t ohw = (uint32_t)(p.OH * p.OW);
    s.rows = rows;
    s.db = (int)(rows / ohw);
    const uint32_t rem = rows - (uint32_t)s.db * ohw;
    s.doh = (int)(rem / (uint32_t)p.OW);
    s.dow = (int)(rem - (uint32_t)s.doh * (uint32_t)p.OW);
    s.pat = 0;
    for (int r = 0; r < p.kh; ++r) s.pat |= 1u << (r * p.kw);
    s.pointwise = p.kh == 1 && p.kw == 1 && p.stride == 1 && p.pad == 0;
    return s;
}
struct RowCursor {
    uint32_t m;              // row of the implicit patch matrix
    int b, oh, ow;
    int base;                // word offset of the top-left input pixel (may be negative)
    uint32_t mask;           // taps inside the image; 0 for rows beyond M
};
__device__ __forceinline__ void row_locate(const ConvProblem &p, RowCursor &rc)
{
    const uint32_t ohw = (uint32_t)(p.OH * p.OW);
    rc.b = (int)exact_div(rc.m, p.ohw_mul, p.ohw_shift);
    const uint32_t rem = rc.m - (uint32_t)rc.b * ohw;
    rc.oh = (int)exact_div(rem, p.ow_mul, p.ow_shift);
    rc.ow = (int)(rem - (uint32_t)rc.oh * (uint32_t)p.OW);
}
__device__ __forceinline__ void row_step(const ConvProblem &p, const TileStep &s, RowCursor &rc)
{
    rc.m += s.rows;
    if (s.pointwise) return;
    rc.ow += s.dow;
    if (rc.ow >= p.OW) { rc.ow -= p.OW; ++rc.oh; }
    rc.oh += s.doh;
    if (rc.oh >= p.OH) { rc.oh -= p.OH; ++rc.b; }
    rc.b += s.db;
}
__device__ __forceinline__ uint32_t low_bits(int n) { return (1u << n) - 1u; }   // 0 <= n <= 31
__device__ __forceinline__ void row_window(const ConvProblem &p, const TileStep &s, RowCursor &rc)
{
    if (s.pointwise) {                                      // warp-uniform
        rc.base = (int)(rc.m * (uint32_t)p.cw);
        rc.mask = rc.m < (uint32_t)p.M ? 1u : 0u;
        return;
    }
    const int ih0 = rc.oh * p.stride - p.pad, iw0 = rc.ow * p.stride - p.pad;
    rc.base = ((rc.b * p.H + ih0) * p.W + iw0) * p.cw;
    // taps t with 0 <= iw0 + t < W and r with 0 <= ih0 + r < H (an empty range gives an empty mask)
    const int clo = min(max(-iw0, 0), p.kw), chi = max(min(p.W - iw0, p.kw), 0);
    const int rlo = min(max(-ih0, 0), p.kh), rhi = max(min(p.H - ih0, p.kh), 0);
    const uint32_t cols = low_bits(chi) & ~low_bits(clo);
    const uint32_t rows = s.pat & low_bits(rhi * p.kw) & ~low_bits(rlo * p.kw);
    rc.mask = rc.m < (uint32_t)p.M ? cols * rows : 0u;
}
template <int BYTES>
__device__ __forceinline__ void cp_async_zfill(uint32_t dst, const void *src, uint32_t nbytes)
{
    if (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(nbytes) : "memory");
    else if (BYTES == 8)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(nbytes) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(nbytes) : "memory");
}
// One 128-bit stage (4 / GW units, table entries at `tab`) of the row `rc` -> 16 bytes at `dst`.  Only the
// first `nunits` units are copied (warp-uniform; the zero tail of K beyond the last word needs no copy when
// nobody reads it).
template <int GW>
__device__ __forceinline__ void gather_stage(const uint32_t *x, const RowCursor &rc, uint32_t tab, uint32_t dst, int nunits = 4)
{
    constexpr int U = 4 / GW;
    uint32_t ent[2 * U];
    if (U == 1) {
        asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(ent[0]), "=r"(ent[1]) : "r"(tab));
    } else {
#pragma unroll
        for (int h = 0; h < U / 2; ++h)
            asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(ent[4 * h]), "=r"(ent[4 * h + 1]), "=r"(ent[4 * h + 2]), "=r"(ent[4 * h + 3]) : "r"(tab + 16u * h));
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (u >= nunits) break;
        const bool ok = (rc.mask & ent[2 * u + 1]) != 0u;
        const int idx = ok ? rc.base + (int)ent[2 * u] : 0;
        cp_async_zfill<GW * 4>(dst + (uint32_t)(u * GW * 4), x + idx, ok ? (uint32_t)(GW * 4) : 0u);
    }
}

// int32 output of one accumulator chunk: 32 rows (one per lane) x 32 consecutive columns.  A lane storing its own
// row touches 32 rows x 16 bytes per instruction; staged through shared memory the warp stores 4 rows x 128
// contiguous bytes per instruction instead.  `warp_tile`: I32_TILE_BYTES of shared memory owned by this warp;
// `dst0` points at (row0, first column), `ldc` is the row pitch in elements (a multiple of 4, 16-byte aligned rows).
// All 32 lanes must call it.
constexpr int I32_ROW_BYTES = 144;                         // 128 + 16: conflict-free both ways
constexpr int I32_TILE_BYTES = 32 * I32_ROW_BYTES;
__device__ __forceinline__ void store_int32_block(int32_t *dst0, long ldc, const int (&o)[32], uint32_t warp_tile,
                                                  long row0, long M, int lane)
{
    const uint32_t mine = warp_tile + (uint32_t)(lane * I32_ROW_BYTES);
#pragma unroll
    for (int i4 = 0; i4 < 8; ++i4)
        st_shared_v4(mine + 16u * i4, (uint32_t)o[4 * i4], (uint32_t)o[4 * i4 + 1], (uint32_t)o[4 * i4 + 2], (uint32_t)o[4 * i4 + 3]);
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = (lane >> 3) + 4 * i;
        const uint4 v = ld_shared_v4(warp_tile + (uint32_t)(r * I32_ROW_BYTES + (lane & 7) * 16));
        if (row0 + r < M) *reinterpret_cast<uint4 *>(dst0 + (long)r * ldc + 4 * (lane & 7)) = v;
    }
    __syncwarp();
}

// Convolution-module epilogue (Section 4.2.1).
//
// Identity staging: an epilogue thread owns one output row and walks its 32-channel chunks in order.  The 64 bytes of
// fp16 identity values of a chunk are copied with cp.async into the row's slot of a small ring in shared memory,
// ID_AHEAD chunks before they are needed (across tile boundaries), so the loads are in flight while the MMAs run
// and while earlier chunks are computed.  Rows are ID_ROW_BYTES apart (64 + 16: conflict-free 16-byte accesses
// across a warp, both one row per lane and four lanes per row).
// (A variant that turns each 32 x 32 block through shared memory so that a lane owns a channel - parameters in
// registers, contiguous 64-byte requests, warp votes for the sign words - was measured at 0.55x the speed of this
// one: its 2-byte accesses and 32 votes per block cost more than the strided 16-byte accesses here.)
constexpr int ID_AHEAD = 2;
constexpr int ID_SLOTS = ID_AHEAD + 1;
constexpr int ID_ROW_BYTES = 80;
constexpr int ID_RING_BYTES = ID_SLOTS * BM * ID_ROW_BYTES;      // 30720

// Queue the copy of one chunk for the 32 rows of this warp (always commits a group, empty when there is nothing to
// copy).  The warp copies cooperatively: lane l fetches 16-byte part l % 4 of rows l / 4 + 8 i, so that one
// instruction touches 8 rows x 64 contiguous bytes instead of 32 rows x 16 bytes; `warp_slot` is the slot of the
// warp's first row, `row0` that row.  After cp.async.wait_group a __syncwarp makes all lanes' copies visible.
__device__ __forceinline__ void module_prefetch(const ConvProblem &p, uint32_t warp_slot, long row0, int n0, int lane)
{
    if (p.identity) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = (lane >> 2) + 8 * i;
            const long row = row0 + r;
            const bool ok = row < p.M;
            cp_async16(warp_slot + (uint32_t)(r * ID_ROW_BYTES + (lane & 3) * 16),
                       p.identity + (ok ? row * p.C_out + n0 + 8 * (lane & 3) : 0), ok);
        }
    }
    cp_async_commit();
}

// One chunk: 32 consecutive output channels n0 .. n0+31 of the warp's 32 output rows, lane = row.
//   t = dot * scale + shift;  u = t + identity;  r = u >= 0 ? u : slope * u;  y = fp16(r);  bit = (y + next_bias >= 0)
// one fp32 operation per step, each rounded to nearest (no fused multiply-add), the sign taken of the stored
// fp16 value.  Reads the identity values from the row's staging slot, writes the 32 fp16 values back into the
// same slot, from where the warp stores them cooperatively (same 8 rows x 64 bytes per instruction), and returns
// the 32 sign bits of the lane's row (bit i = channel n0 + i).  The channel count is a multiple of 32, so every
// 8-channel group is 16-byte aligned.  All 32 lanes must call it.
template <bool HAS_ID, bool HAS_NB>
__device__ __forceinline__ uint32_t module_chunk_t(const ConvProblem &p, const int (&dot)[32], uint32_t slot_addr, int n0)
{
    uint32_t bits = 0;
#pragma unroll
    for (int g = 0; g < 4; ++g) {                           // 8 channels per group
        uint4 idv = make_uint4(0u, 0u, 0u, 0u);
        if (HAS_ID) idv = ld_shared_v4(slot_addr + 16u * g);
        const uint32_t idw[4] = {idv.x, idv.y, idv.z, idv.w};
        uint32_t ow[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int n = n0 + 8 * g + 4 * h;
            const float4 sc = __ldg(reinterpret_cast<const float4 *>(p.bn_scale + n));
            const float4 sh = __ldg(reinterpret_cast<const float4 *>(p.bn_shift + n));
            const float4 sl = __ldg(reinterpret_cast<const float4 *>(p.slope + n));
            float4 nb = make_float4(0.f, 0.f, 0.f, 0.f);
            if (HAS_NB) nb = __ldg(reinterpret_cast<const float4 *>(p.next_bias + n));
            const float scs[4] = {sc.x, sc.y, sc.z, sc.w}, shs[4] = {sh.x, sh.y, sh.z, sh.w};
            const float sls[4] = {sl.x, sl.y, sl.z, sl.w}, nbs[4] = {nb.x, nb.y, nb.z, nb.w};
#pragma unroll
            for (int q = 0; q < 2; ++q) {                   // two channels at a time: paired fp16 <-> fp32 conversions
                const int c = 8 * g + 4 * h + 2 * q;
                const float2 idf = __half22float2(*reinterpret_cast<const __half2 *>(&idw[2 * h + q]));
                float r[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    float t = __fmul_rn(__int2float_rn(dot[c + e]), scs[2 * q + e]);
                    t = __fadd_rn(t, shs[2 * q + e]);
                    const float u = HAS_ID ? __fadd_rn(t, e ? idf.y : idf.x) : t;
                    r[e] = (u >= 0.0f) ? u : __fmul_rn(sls[2 * q + e], u);
                }
                const __half2 y2 = __floats2half2_rn(r[0], r[1]);      // round to nearest even, element-wise
                ow[2 * h + q] = *reinterpret_cast<const uint32_t *>(&y2);
                const float2 yf = __half22float2(y2);
                bits |= (__fadd_rn(yf.x, nbs[2 * q]) >= 0.0f ? 1u : 0u) << c;
                bits |= (__fadd_rn(yf.y, nbs[2 * q + 1]) >= 0.0f ? 1u : 0u) << (c + 1);
            }
        }
        st_shared_v4(slot_addr + 16u * g, ow[0], ow[1], ow[2], ow[3]);
    }
    return bits;
}
__device__ __forceinline__ uint32_t module_chunk(const ConvProblem &p, const int (&dot)[32], uint32_t warp_slot,
                                                 long row0, int n0, int lane)
{
    const uint32_t slot_addr = warp_slot + (uint32_t)(lane * ID_ROW_BYTES);
    __syncwarp();                                           // the cooperative copies of all lanes have landed
    uint32_t bits;
    if (p.identity) bits = p.next_bias ? module_chunk_t<true, true>(p, dot, slot_addr, n0) : module_chunk_t<true, false>(p, dot, slot_addr, n0);
    else bits = p.next_bias ? module_chunk_t<false, true>(p, dot, slot_addr, n0) : module_chunk_t<false, false>(p, dot, slot_addr, n0);
    __syncwarp();                                           // the rows of all lanes are staged
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = (lane >> 2) + 8 * i;
        const long row = row0 + r;
        const uint4 v = ld_shared_v4(warp_slot + (uint32_t)(r * ID_ROW_BYTES + (lane & 3) * 16));
        if (row < p.M) *reinterpret_cast<uint4 *>(p.y_real + row * p.C_out + n0 + 8 * (lane & 3)) = v;
    }
    __syncwarp();                                           // the slot may be refilled
    return bits;
}

}  // namespace tc
}  // namespace bcnn
