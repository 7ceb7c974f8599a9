// Device-side helpers shared by the kernels: mbarrier wrappers, the bounded wait, and the codes a
// kernel may leave in the plan's status word.
#pragma once

#include <cstdint>

// Codes of the device status word (first int32 of the index buffer).  The first code recorded wins
// (atomicCAS from 0); cpa_plan_status maps them to a cpa_status.
constexpr int32_t kStatusWaitGaveUp = 1;   // a bounded wait ran out           -> CPA_ETIMEOUT
constexpr int32_t kStatusNoSpace = 2;      // an append found no page/slot left -> CPA_ENOSPC

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" :: "r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait: at most `limit` tries (each try suspends the thread for a short, hardware-defined
// time).  When the limit is hit the wait records kStatusWaitGaveUp in `status`, sets `dead` and
// returns; with `dead` set every later wait returns at once, so a kernel that lost one barrier
// runs to its end instead of hanging.  Returns true when the phase completed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, bool& dead, int32_t* status, uint32_t limit) {
    if (dead) return false;
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (++spins > limit) {
            dead = true;
            atomicCAS(status, 0, kStatusWaitGaveUp);
            return false;
        }
    }
    return true;
}
// The last look at a barrier before a thread leaves a kernel whose waits gave up: a copy that was
// issued against it may still be in flight into this CTA's shared memory, and the CTA must not end
// under it.  Records nothing; the status word already says that the launch's results are void.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity, uint32_t limit) {
    for (uint32_t spins = 0; spins <= limit; ++spins)
        if (mbar_try_wait(bar, parity)) return;
}
