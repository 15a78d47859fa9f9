// Self-check of the bounded wait used by the persistent kernels.
#pragma once
#include "persistent.cuh"

namespace ef21 {

// One-block self-check of the bounded wait: spins on a word that nobody writes and must come back
// with EF21_ERR_TIMEOUT in the status word instead of hanging.
__global__ void bounded_wait_selftest_kernel(const unsigned long long* never_written, unsigned* status,
                                             unsigned spin_limit) {
    unsigned spins = 0;
    while (true) {
        const unsigned long long w = ld_relaxed_u64(never_written);
        if ((unsigned)(w >> 48) == 0xffffu) break;
        if (++spins > spin_limit) { record_error(status, 5u); break; }
    }
}

}  // namespace ef21
