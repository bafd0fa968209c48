// The bounded mbarrier wait of the one-CTA kernels, and the shared-memory flag helpers it uses.
#pragma once
#include <stdint.h>

#include "ksa_ptx.cuh"

namespace ksa {

__device__ __forceinline__ uint32_t ld_shared_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_shared_u32(uint32_t addr, uint32_t v)
{
    asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

constexpr long long kWaitLimitCycles = 1ll << 31;       // about a second

// Bounded wait.  Returns false if the wait gave up or the CTA is aborting.  On giving up it records `code` in the
// status word (first one wins) and raises the CTA's abort flag, so that every other role leaves its loop too.
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, uint32_t abort_addr, int32_t* status, int code,
                                             long long limit_cycles = kWaitLimitCycles)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (ld_shared_u32(abort_addr) != 0u) return false;
            if (clock64() - t0 > limit_cycles) {
                atomicCAS(status, 0, code);
                st_shared_u32(abort_addr, 1u);
                return false;
            }
        }
    }
}

}  // namespace ksa
