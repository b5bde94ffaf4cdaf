// Bounded waits on shared-memory mbarriers, shared by every kernel of the library that waits for a TMA copy or a
// tensor-core commit.  No wait in the library spins without a limit: after `cap` polls the waiting thread raises the
// CTA's abort flag (after which every wait of the CTA returns at once) and the context's device status word
// (kFlagTimeout, reported by fdkv_device_status as FDKV_ERR_TIMEOUT), and the kernel runs to its end without the data.
#pragma once

#include <cstdint>

#include "fdkv_internal.h"

namespace fdkv {

constexpr uint32_t kWaitCap = 1u << 22;  // polls before a wait gives up (seconds, where a copy lands within microseconds)

__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}

// Waits for the phase with the given parity of the barrier at shared-memory address `bar`.
__device__ __forceinline__ void mbar_wait_bounded(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, int32_t* status,
                                                  uint32_t cap = kWaitCap) {
    if (mbar_try_wait(bar, parity)) return;  // the common case: one poll, no look at the abort flag
    if (*abort_flag) return;
    for (uint32_t i = 0; i < cap; ++i) {
        if (mbar_try_wait(bar, parity)) return;
        if ((i & 255u) == 255u && *abort_flag) return;
    }
    *abort_flag = 1;
    atomicMax(status, (int32_t)kFlagTimeout);
}

}  // namespace fdkv
