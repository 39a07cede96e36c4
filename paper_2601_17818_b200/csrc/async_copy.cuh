// Shared-memory barriers (mbarrier), bounded waits on them and bulk asynchronous copies into shared memory: the
// plumbing shared by the kernels that stage data through shared memory with the copy engine (gram.cu, delta_pass.cu).
// Every wait is bounded: when the limit runs out the caller's CTA-wide abort flag is raised and the wait returns
// false; the kernel then leaves in an orderly way and reports VITCOP_ERR_TIMEOUT.
#pragma once

#include "internal.cuh"

namespace vitcop {

constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // bounded waits: after 2 s (default) give up and leave
constexpr unsigned long long kDrainLimitNs = 20000000ull;    // bounded waits for this CTA's own copies / MMAs after giving up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false (after raising `abort_flag`) when the time limit is hit or another role gave up.
// limit_ns == 0 gives up at once, whatever the barrier's state (failure-handling tests use it to send one role of
// a CTA down the give-up path while the others have work in flight).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns) {
    if (limit_ns != 0ull) {
        if (mbar_try_wait(bar, parity)) return true;
        const unsigned long long t0 = global_ns();
        for (uint32_t it = 1;; ++it) {
            if (mbar_try_wait(bar, parity)) return true;
            if ((it & 63u) == 0u) {
                if (*abort_flag) return false;
                if (global_ns() - t0 > limit_ns) break;
            }
        }
    }
    *abort_flag = 1;
    return false;
}
// Bounded wait without side effects, used while leaving after a timeout.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
    const unsigned long long t0 = global_ns();
    while (!mbar_try_wait(bar, parity))
        if (global_ns() - t0 > kDrainLimitNs) break;
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
                 : "memory");
}
}  // namespace vitcop
