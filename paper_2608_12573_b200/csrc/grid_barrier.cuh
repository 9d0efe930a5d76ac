// Barrier over all CTAs of a cooperatively launched (hence co-resident) grid, with a bounded wait.
#pragma once

#include "sample_select.cuh"

namespace profk {

constexpr uint32_t SPIN_LIMIT = 1u << 24;   // polls (each ~50-100 ns apart) before a wait gives up

// Barrier over `members` co-resident CTAs on one counter.  The counter only grows: a CTA arrives with an atomic add
// and waits until the count reaches the next multiple of `members` above the value its own arrival found.  There is
// no second word, no reset and nobody who releases the others: the barrier is over one poll after the last arrival
// has landed in L2.  *count must be a multiple of `members` when the first CTA arrives -- it is zero at the start of
// a call, and every completed barrier adds `members` -- so the kernels of a call that share a counter all have the
// same number of members.  Returns false when the wait gave up (or an earlier one did, anywhere in the grid); the
// caller then leaves the kernel.  `limit` is the number of polls a wait may take.
__device__ __forceinline__ bool cta_group_barrier(uint32_t* count, uint32_t* error, uint32_t members, uint32_t limit = SPIN_LIMIT) {
    __shared__ uint32_t s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t ok = 1;
        __threadfence();
        const uint32_t old = atomicAdd(count, 1u);
        const uint32_t target = old - old % members + members;
        // (a CTA that gave up anywhere has set the error word: looked at now and then, so that the others follow it
        // out instead of waiting their own limits out)
        uint32_t polls = 0;
        while ((int32_t)(*((volatile uint32_t*)count) - target) < 0) {
            __nanosleep(32);
            if (++polls > limit) { atomicExch(error, 1u); ok = 0; break; }
            if ((polls & 1023u) == 0 && *((volatile uint32_t*)error) != 0) { ok = 0; break; }
        }
        __threadfence();
        s_ok = ok;
    }
    __syncthreads();
    return s_ok != 0;
}

// The same over all CTAs of the grid, on the workspace header's counter.
__device__ __forceinline__ bool grid_barrier(WsHeader* h) {
    return cta_group_barrier(&h->bar_count, &h->error, gridDim.x);
}

}  // namespace profk
