// Helpers of the slot-pipeline engines (conv_tc_pw.cu, conv_tc_c3.cu): tensor-memory loads that do not wait, the
// register pin that keeps uses behind the wait, the short-sleep bounded mbarrier wait, and the sign-bit gathering
// from packed 16-bit accumulator halves.
#pragma once
#include "tc_common.cuh"

namespace bcnn {
namespace tc {

// 64 accumulator columns of this warp's 32 rows as packed 16-bit halves: register i = columns 2i (low) and 2i + 1.
// The loads below do NOT wait: several are issued in a row, then tc_wait_ld(), then pin_regs() on every destination
// array - an empty volatile asm that takes the registers as read-write operands, so that no use of them can be
// scheduled ahead of the wait.
__device__ __forceinline__ void tc_ld64_pack16(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.pack::16b.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
// 32 columns -> 16 registers.
__device__ __forceinline__ void tc_ld32_pack16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.pack::16b.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void pin_regs(uint32_t (&v)[16])
{
    asm volatile("" : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                      "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]) :: "memory");
}
__device__ __forceinline__ void pin_regs(uint32_t (&v)[32])
{
    asm volatile("" : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                      "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                      "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
                      "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31]) :: "memory");
}

// Waits of this engine: hand-overs are on the critical path of a slot's cycle, so the waiter sleeps only briefly
// between polls (a failed try_wait returns at once: measured, polling without any sleep more than doubled the
// instructions the SM executes; the shared helpers' 100 ns is a fifth of a slot's cycle here).
// Bounded by elapsed clock cycles (about two seconds), checked every 64 polls together with the CTA's abort flag.
constexpr long long PW_WAIT_CYCLES = 4000000000LL;
constexpr uint32_t PW_SLEEP_NS = 32;
template <uint32_t SLEEP = PW_SLEEP_NS>
static __device__ __noinline__ bool pw_wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err, int code)
{
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        __nanosleep(SLEEP);
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > PW_WAIT_CYCLES) break;
        }
    }
    *abort_flag = 1;
    if (err) atomicCAS(err, 0, code);
    return false;
}
// whole-warp wait (every lane polls; the verdict is a vote).  SLEEP: nanoseconds between polls - short for hand-overs on
// a pipeline's critical path, longer for roles with slack (a polling warp takes issue slots from the warps that work).
template <uint32_t SLEEP = PW_SLEEP_NS>
__device__ __forceinline__ bool pw_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err, int code)
{
    bool ok = mbar_try_wait(bar, parity);
    if (__all_sync(0xffffffffu, ok)) return true;
    if (!ok) ok = pw_wait_slow<SLEEP>(bar, parity, abort_flag, err, code);
    return __all_sync(0xffffffffu, ok);
}

// Output word of a 32-column block from its 16 packed registers: bit = (accumulator >= 0).  PRMT in sign-replication
// mode turns the two halves of two registers into four bytes 0x00 / 0xFF; step s keeps bit s of every byte.
__device__ __forceinline__ uint32_t sign_word(const uint32_t *r)
{
    uint32_t w = 0;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        uint32_t d;
        asm("prmt.b32 %0, %1, %2, 0xFDB9;" : "=r"(d) : "r"(r[s]), "r"(r[8 + s]));    // sign bytes of r[s].b1, r[s].b3, r[8+s].b1, r[8+s].b3
        w |= ~d & (0x01010101u << s);
    }
    return w;
}

// Accumulator column c of a 32-column block holds this channel of the block (the order sign_word gathers bits in).
__host__ __device__ constexpr int channel_of_column(int c)
{
    return c < 16 ? ((c & 1) ? 8 + (c >> 1) : (c >> 1)) : ((c & 1) ? 24 + ((c - 16) >> 1) : 16 + ((c - 16) >> 1));
}

// 32 accumulator columns (32-bit) of this warp's 32 rows, without the completion wait.
__device__ __forceinline__ void tc_ld32_nowait(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}

}  // namespace tc
}  // namespace bcnn
