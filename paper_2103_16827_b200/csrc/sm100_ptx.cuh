// Thin inline-PTX wrappers for sm_100a: mbarrier, TMA tile loads, tcgen05 (TMEM alloc, MMA,
// commit, load) and the shared-memory / instruction descriptors of the int8 MMA.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "qasr_internal.h"

namespace qasr {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

// ---- mbarrier ----------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait: gives up after `limit_ns` of wall time (two seconds unless the caller says otherwise),
// raises the sticky device status and the CTA-wide abort flag, and returns false. Callers then leave
// their loops and fall through to the common teardown.
// Each poll is a try_wait that may suspend the thread for up to about a microsecond, so a waiting
// warp costs few issue slots.
constexpr uint32_t kWaitPollsHardCap = 1u << 30;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
#ifndef QASR_WAIT_HINT_NS
#define QASR_WAIT_HINT_NS 1000u
#endif
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(QASR_WAIT_HINT_NS)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned* status, unsigned long long limit_ns = kWaitLimitNs,
                                          unsigned sleep_ns = 20) {
    if (mbar_test(bar, parity)) return true;
    // Bound: limit_ns of wall time (checked every 64 polls), with a hard cap on the poll count
    // that the default limit cannot reach sooner than that.
    unsigned long long t_start = 0;
    for (uint32_t it = 0; it < kWaitPollsHardCap; ++it) {
        if (mbar_try(bar, parity)) return true;
        __nanosleep(sleep_ns);      // a waiting warp leaves its issue slots to the warps that work
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t_start == 0) t_start = now;
            if (now - t_start > limit_ns) break;
        }
    }
    *abort_flag = 1;
    atomicOr(status, QASR_STATUS_TIMEOUT);
    return false;
}

// One lane of a converged warp, the same one on every call. A warp that runs its loop as a whole and
// lets only the elected lane issue keeps its loop state (stage counters, descriptors, barrier addresses)
// in warp-uniform form, which the single-lane form under `if (lane == 0)` does not.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// ---- programmatic dependent launch ---------------------------------------------------------
// launch_dependents lets the next kernel of the stream start its prologue while this one still runs;
// wait blocks until every kernel this one depends on has completed and its writes are visible.
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- TMA tile loads (each CTA fetches its own tiles) ----------------------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---- tcgen05: tensor memory ------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// mbarrier arrives once all tcgen05 operations issued so far by this thread have completed.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], int8 x int8 -> int32, K = 32 per instruction.
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Each lane reads 16 consecutive 32-bit columns of its own TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
// Waits for the TMEM loads issued so far. The destination registers are passed through the
// statement so that no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[16]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :
                 : "memory");
}

// ---- descriptors -----------------------------------------------------------------------------
// Shared-memory matrix descriptor: start address, leading/stride byte offsets (all >> 4),
// descriptor version 1 at bit 46, swizzle mode in bits 61..63.
constexpr uint64_t SWIZZLE_128B = 2, SWIZZLE_64B = 4, SWIZZLE_32B = 6;
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint64_t swizzle) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (swizzle << 61);
}
// Instruction descriptor of kind::i8: signed 8-bit A and B, int32 accumulator, M x N tile.
// a_mn / b_mn: 0 = K-major operand, 1 = MN-major operand.
__host__ __device__ __forceinline__ uint32_t idesc_i8(int M, int N, int a_mn, int b_mn) {
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Two int32 values saturated to int8 and packed above/below each other (b -> byte 0, a -> byte 1,
// the low half of c -> bytes 2..3).
__device__ __forceinline__ uint32_t pack_sat_s8(int a, int b, uint32_t c) {
    uint32_t d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// Four int32 values -> four saturated int8 in one word, v0 in the lowest byte.
__device__ __forceinline__ uint32_t pack4_sat_s8(int v0, int v1, int v2, int v3) {
    return pack_sat_s8(v1, v0, pack_sat_s8(v3, v2, 0u));
}

// High word of the 64-bit sum a * b + c. Written as a carry chain of the two 32-bit halves, which the assembler
// turns into one multiply-add that takes the 64-bit addend; `mad.wide.s32` with a 64-bit addend comes out as a
// wide multiply followed by a two-instruction 64-bit add (counted per opcode on a B200: 3 instead of 1 per value).
__device__ __forceinline__ int mad_hi64(int a, int b, long long c) {
    int lo, hi;
    asm("{mad.lo.cc.s32 %0, %2, %3, %4;\n\tmadc.hi.s32 %1, %2, %3, %5;}"
        : "=r"(lo), "=r"(hi) : "r"(a), "r"(b), "r"((int)c), "r"((int)(c >> 32)));
    return hi;
}
// Byte B of a word, sign-extended: one prmt whose selector replicates the byte's sign over the upper three bytes.
template <int B>
__device__ __forceinline__ int sext_byte(uint32_t w) {
    uint32_t d;
    asm("prmt.b32 %0, %1, 0, %2;" : "=r"(d) : "r"(w), "n"(B | ((8 | B) << 4) | ((8 | B) << 8) | ((8 | B) << 12)));
    return (int)d;
}
// max(byte, 0) on four packed int8: the sign of every byte replicated over the byte, then cleared.
__device__ __forceinline__ uint32_t relu4_s8(uint32_t w) {
    uint32_t sign;
    asm("prmt.b32 %0, %1, 0, 0xba98;" : "=r"(sign) : "r"(w));
    return w & ~sign;
}

}  // namespace ptx
}  // namespace qasr
