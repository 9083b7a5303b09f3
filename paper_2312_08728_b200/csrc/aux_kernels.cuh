// Two small kernels beside the step kernels: the wait that must run out (error-path test) and the shuffle written
// out as a table (parity test of the permutation).
#pragma once

#include "glm_kernel.cuh"

namespace bmgdk {

// Waits, with the step kernel's protocol, for a packet tag that nobody writes: the wait must run out of its
// budget, record BMGD_ERR_TIMEOUT in the status word, raise the abort flag and return.  For testing the error path.
__global__ void wait_probe_kernel(const unsigned long long* packet, uint32_t tag, unsigned long long timeout_ns, int* status) {
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    bool aborted = false;
    while (!aborted) {
        if ((uint32_t)(ld_packet(packet) >> 32) == tag) break;
        if ((++spins & 0x3FFu) == 0u) {
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > timeout_ns || ((volatile int*)status)[1] != 0) {
                atomicCAS(status, 0, kStatusTimeout);
                atomicExch(status + 1, 1);
                aborted = true;
            }
        }
    }
}

// Writes out[j] = pi(j) for one (seed, chain, round): the shuffle exactly as the step kernel uses it.
__global__ void perm_kernel(unsigned long long seed, uint32_t chain, uint32_t round, uint32_t N0, uint32_t* out) {
    const FeistelDomain dom = make_domain(N0);
    const RoundKeys rk = round_keys(seed, chain, round);
    for (unsigned long long j = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; j < N0;
         j += (unsigned long long)gridDim.x * blockDim.x)
        out[j] = perm_index((uint32_t)j, dom, rk);
}

}  // namespace bmgdk
