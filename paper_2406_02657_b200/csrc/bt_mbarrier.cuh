// Shared-memory barrier helpers of the kernels that move data with the copy engine (bulk copies and
// TMA tensor copies complete on an mbarrier).  Internal to the library.
#pragma once

#include <stdint.h>

namespace bt {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Suspends the thread for a short, implementation-defined time when the phase is not complete.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
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
// Non-blocking test: far cheaper than try_wait when the phase has already completed (the usual case).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
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
// Wait bounded by a number of polls (each poll suspends briefly): false when the limit runs out.
__device__ __forceinline__ bool mbar_wait_polls(uint32_t bar, uint32_t parity, uint32_t poll_limit)
{
    if (mbar_test_wait(bar, parity)) return true;
    for (uint32_t it = 0; it < poll_limit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}


__device__ __forceinline__ uint64_t global_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Wait bounded in wall time (limit_ns; the clock is looked at every 64 polls) and in polls (spin_limit),
// for kernels whose threads wait on one another: *abort_flag is a shared-memory word that a thread sets
// when its own wait runs out and that every waiting thread of the CTA watches, so that one failed wait
// winds the whole CTA down.  Returns false when the limit ran out here or another thread gave up.
__device__ __forceinline__ bool mbar_wait_walltime(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t spin_limit,
                                                   uint64_t limit_ns)
{
    if (mbar_test_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    for (uint32_t it = 0; it < spin_limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            const uint64_t now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) break;
        }
    }
    *abort_flag = 1;
    return false;
}

}  // namespace bt
