// Barrier over all CTAs of a cooperatively launched (hence co-resident) grid, with a bounded wait.
#pragma once

#include "sample_select.cuh"

namespace profk {

constexpr uint32_t SPIN_LIMIT = 1u << 24;   // polls (each ~100 ns apart) before a wait gives up

// Sense-free generation barrier over all CTAs of a co-resident grid.  Returns false when
// the wait gave up (or an earlier one did); the caller then leaves the kernel.
__device__ __forceinline__ bool grid_barrier(WsHeader* h, uint32_t& gen) {
    __shared__ uint32_t s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t ok = 1;
        __threadfence();
        const uint32_t arrived = atomicAdd(&h->bar_count, 1u);
        if (arrived == gridDim.x - 1) {
            atomicExch(&h->bar_count, 0u);
            __threadfence();
            atomicAdd(&h->bar_gen, 1u);
        } else {
            uint32_t polls = 0;
            while (*((volatile uint32_t*)&h->bar_gen) == gen) {
                __nanosleep(64);
                if (++polls > SPIN_LIMIT) { atomicExch(&h->error, 1u); ok = 0; break; }
            }
        }
        __threadfence();
        if (*((volatile uint32_t*)&h->error) != 0) ok = 0;
        s_ok = ok;
    }
    __syncthreads();
    gen += 1;
    return s_ok != 0;
}

}  // namespace profk
