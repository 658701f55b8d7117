// mbarrier helpers shared by the warp-specialised kernels (tensor-core prefill kernels, streaming kernels):
// init / arrive / expect-tx / try-wait, and the BOUNDED wait every role uses.  A wait never spins without limit:
// after `budget` SM clock ticks it raises the CTA's abort flag and the sticky status EXMOE_ERR_TIMEOUT and returns
// false; every other waiter of the CTA sees the flag within 16 polls and returns false too, so that all roles
// leave their loops and the kernel ends with the context intact (exercised by exmoe_debug_wait_timeout).
#pragma once
#include <stdint.h>
#include <cuda_runtime.h>
#include "../../include/exmoe.h"

namespace exmoe {

constexpr long long kWaitBudget = 2000000000ll;   // clock64 ticks (~1 s) before a wait gives up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait; returns false when the CTA is aborting (and raises the abort on expiry)
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          long long budget = kWaitBudget) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned polls = 0;
    while (!mbar_try(bar, parity)) {
        if ((++polls & 15u) == 0) {                    // the bookkeeping of the bound is amortised over 16 polls
            if (*abort_flag) return false;
            if (clock64() - t0 > budget) {
                *abort_flag = 1;
                atomicExch(status, EXMOE_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

}  // namespace exmoe
