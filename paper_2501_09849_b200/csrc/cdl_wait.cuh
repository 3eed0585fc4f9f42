// Bounded mbarrier waits and the timeout record of the status block (device code shared by the tensor-core
// kernels).  No wait in this library spins without a limit: a wait that runs out returns false, the kernel writes
// a record into its status block and winds down through its normal exit path.
#pragma once
#include <stdint.h>

#include "cdl_internal.h"

namespace cdl {

// Upper bound, in nanoseconds, on how long one try_wait may keep its thread suspended while the phase is pending:
// a suspended poller leaves the issue slots of its scheduler to the warps that share it.
constexpr unsigned int kTryWaitHintNs = 20000;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kTryWaitHintNs)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// The same poll without a suspend-time hint (the time it may stay suspended is then the implementation's own): it
// costs about half of the hinted form when the phase is already complete, which is what the single threads that
// drive a pipeline mostly find, so they try this once before they go into the bounded wait.
__device__ __forceinline__ bool mbar_try_wait_now(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Records an expired wait in a status block: two tag words first, then the code itself, so that a reader takes
// the block for a record only when all three words are there (stale memory of a recycled allocation is not).
__device__ __forceinline__ void record_timeout(int *status)
{
    status[1] = (int)kStatusTag1;
    status[2] = (int)kStatusTag2;
    __threadfence();
    atomicExch(status, CDL_ERR_TIMEOUT);
}
// Bounded wait: false when the barrier did not complete within limit_ns or another thread already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, unsigned long long limit_ns)
{
    for (int fast = 0; fast < 64; ++fast)
        if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag != 0) return false;
        if (global_ns() - t0 > limit_ns) return false;
    }
}

}  // namespace cdl
