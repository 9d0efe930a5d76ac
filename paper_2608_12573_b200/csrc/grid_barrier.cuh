// Barrier over all CTAs of a cooperatively launched (hence co-resident) grid, with a bounded wait.
#pragma once

#include "sample_select.cuh"

namespace profk {

constexpr uint32_t SPIN_LIMIT = 1u << 24;   // polls (each ~100 ns apart) before a wait gives up

// Sense-free generation barrier over `members` co-resident CTAs that share the words *count (zero before
// the first use, and again after every completed barrier) and *generation (any value).  `gen` is the caller's
// copy of the generation, read before its first arrival.  Returns false when the wait gave up (or an earlier
// one did, anywhere in the grid); the caller then leaves the kernel.  `limit` is the number of polls a wait may take.
__device__ __forceinline__ bool cta_group_barrier(uint32_t* count, uint32_t* generation, uint32_t* error, uint32_t members,
                                                  uint32_t& gen, uint32_t limit = SPIN_LIMIT) {
    __shared__ uint32_t s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t ok = 1;
        __threadfence();
        const uint32_t arrived = atomicAdd(count, 1u);
        if (arrived == members - 1) {
            atomicExch(count, 0u);
            __threadfence();
            atomicAdd(generation, 1u);
        } else {
            uint32_t polls = 0;
            while (*((volatile uint32_t*)generation) == gen) {
                __nanosleep(64);
                if (++polls > limit) { atomicExch(error, 1u); ok = 0; break; }
            }
        }
        __threadfence();
        if (*((volatile uint32_t*)error) != 0) ok = 0;
        s_ok = ok;
    }
    __syncthreads();
    gen += 1;
    return s_ok != 0;
}

// The same over all CTAs of the grid, on the workspace header's words.
__device__ __forceinline__ bool grid_barrier(WsHeader* h, uint32_t& gen) {
    return cta_group_barrier(&h->bar_count, &h->bar_gen, &h->error, gridDim.x, gen);
}

}  // namespace profk
