// Bounded waits of the tcgen05 kernels: no wait on an mbarrier spins forever.
#pragma once

#include <cstdint>

#include "mom.h"
#include "tc_ptx.cuh"

namespace mom {

constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s: far beyond any legitimate wait

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait: false when the limit was reached (records the failure) or another role gave up.  CLUSTER: the barrier's
// arrivals come from threads of the peer CTA too, whose writes the waiter then reads (acquire at cluster scope).
template <bool CLUSTER = false>
__device__ __forceinline__ bool wait_barrier(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status, int detail,
                                             unsigned long long limit_ns = WAIT_LIMIT_NS) {
    unsigned long long start = 0;
    for (uint32_t i = 0;; ++i) {
        if (CLUSTER ? ptx::mbar_try_wait_cluster(bar, parity) : ptx::mbar_try_wait(bar, parity)) return true;
        if ((i & 63) == 63) {
            if (*abort_flag) return false;
            const unsigned long long now = global_ns();
            if (start == 0) start = now;
            else if (now - start > limit_ns) break;
        }
    }
    if (atomicCAS(status, 0, (int)MOM_ERR_DEVICE_TIMEOUT) == 0) status[1] = detail;
    *abort_flag = 1;
    __threadfence_block();
    return false;
}

}  // namespace mom
