// Building blocks shared by the kernels that finish a call (Section 3, "Refinement"): block
// scans, bitonic sorts, a most-significant-digit radix select over 64-bit candidate records
// held in memory, and the ordered write of a row's output.
//
// Candidate records are 64-bit integers whose ascending order is "value descending, index
// ascending", so the exact top-k of a set of records is "its k smallest records, sorted".
#pragma once

#include "sample_select.cuh"

namespace profk {

constexpr int RF_BITS = 12;                 // digit width of the general select
constexpr int RF_BINS = 1 << RF_BITS;
constexpr uint32_t RF_EDGE_CAP = 1024;      // boundary bins up to this size are ranked directly

enum : uint32_t { ROW_OK = 0, ROW_RECALL = 1, ROW_OVERFLOW = 2, ROW_DIRECT = 3, ROW_RECALL_REFILTERED = 4, ROW_OVERFLOW_REFILTERED = 5 };

__device__ __forceinline__ uint64_t shr64(uint64_t x, int s) { return s >= 64 ? 0ull : (x >> s); }

// Block-wide inclusive scan for any block size that is a multiple of 32 (<= 1024).
__device__ __forceinline__ uint32_t block_scan_any(uint32_t v, uint32_t* warp_sums) {
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t n = __shfl_up_sync(FULL_MASK, v, d);
        if (lane >= (unsigned)d) v += n;
    }
    if (lane == 31) warp_sums[warp] = v;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < nwarps ? warp_sums[lane] : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t n = __shfl_up_sync(FULL_MASK, w, d);
            if (lane >= (unsigned)d) w += n;
        }
        warp_sums[lane] = w;
    }
    __syncthreads();
    if (warp > 0) v += warp_sums[warp - 1];
    __syncthreads();   // warp_sums may be reused right away
    return v;
}

// Ascending bitonic sort of P = 2^j records in shared memory by the whole CTA.
__device__ __forceinline__ void bitonic_sort_shared(uint64_t* a, uint32_t P) {
    for (uint32_t size = 2; size <= P; size <<= 1) {
        for (uint32_t stride = size >> 1; stride > 0; stride >>= 1) {
            for (uint32_t i = threadIdx.x; i < (P >> 1); i += blockDim.x) {
                const uint32_t lo = 2 * i - (i & (stride - 1));
                const uint32_t hi = lo + stride;
                const bool ascending = (lo & size) == 0;
                const uint64_t x = a[lo], y = a[hi];
                if ((x > y) == ascending) { a[lo] = y; a[hi] = x; }
            }
            __syncthreads();
        }
    }
}

// Shared state of one select.
struct SelectShared {
    alignas(16) uint32_t hist[RF_BINS];   // bin counts, then running cursors
    alignas(16) uint32_t start[RF_BINS];  // first position of every bin
    uint64_t edge[RF_EDGE_CAP];      // records of the boundary bin (general select only)
    uint32_t warp_sums[32];
    uint32_t digit, before, cnt, fill, n_edge, crowded;
    unsigned long long or_bits, limit;
};

// Records read from memory (shared or global): every thread visits whole-warp rounds.
struct MemRecords {
    const uint64_t* recs;
    uint32_t n;
    template <typename F> __device__ __forceinline__ void for_each(F&& f) const {
        const uint32_t n_round = (n + 31u) & ~31u;
        for (uint32_t i = threadIdx.x; i < n_round; i += blockDim.x) f(i < n ? recs[i] : 0ull, i < n);
    }
};

// General select: finds limit = the need-th smallest record (records are distinct) by radix
// passes and compacts the records <= limit into sortbuf.  sh.or_bits = OR over (record XOR
// first); sh.fill and sh.n_edge must be zero.  All threads call it.
template <typename Src>
__device__ __forceinline__ void select_smallest(const Src& src, uint64_t first, uint32_t need, uint64_t* sortbuf,
                                                uint32_t sort_cap, SelectShared& sh) {
    const unsigned tid = threadIdx.x, nthr = blockDim.x, lane = lane_id();
    const int top = 64 - __clzll((long long)sh.or_bits);       // bits >= top are common to all records
    uint64_t prefix = shr64(first, top);
    uint64_t limit = ~0ull;
    for (int done = 0; done < top;) {
        const int shift = top - done - RF_BITS > 0 ? top - done - RF_BITS : 0;
        const int width = top - done - shift;
        const uint32_t nbins = 1u << width;
        for (uint32_t i = tid; i < nbins; i += nthr) sh.hist[i] = 0;
        __syncthreads();
        src.for_each([&](uint64_t rec, bool valid) {
            if (valid && shr64(rec, shift + width) == prefix) atomicAdd(&sh.hist[(uint32_t)(rec >> shift) & (nbins - 1)], 1u);
        });
        __syncthreads();
        const uint32_t per = (RF_BINS + nthr - 1) / nthr;
        uint32_t sum = 0;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t bin = tid * per + j;
            sum += bin < nbins ? sh.hist[bin] : 0;
        }
        uint32_t before = block_scan_any(sum, sh.warp_sums) - sum;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t bin = tid * per + j;
            const uint32_t c = bin < nbins ? sh.hist[bin] : 0;
            if (before < need && need <= before + c) { sh.digit = bin; sh.before = before; sh.cnt = c; }
            before += c;
        }
        __syncthreads();
        prefix = (prefix << width) | sh.digit;
        need -= sh.before;
        const uint32_t in_bin = sh.cnt;
        done += width;
        __syncthreads();
        if (in_bin == need || done >= top) { limit = ((prefix + 1) << shift) - 1; break; }
        if (in_bin <= RF_EDGE_CAP) {
            // collect the boundary bin and rank its records: the need-th smallest is the limit
            src.for_each([&](uint64_t rec, bool valid) {
                if (valid && shr64(rec, shift) == prefix) {
                    const uint32_t pos = atomicAdd(&sh.n_edge, 1u);
                    if (pos < RF_EDGE_CAP) sh.edge[pos] = rec;
                }
            });
            __syncthreads();
            for (uint32_t i = tid; i < in_bin; i += nthr) {
                const uint64_t mine = sh.edge[i];
                uint32_t rank = 0;
                for (uint32_t j = 0; j < in_bin; ++j) rank += sh.edge[j] < mine;
                if (rank == need - 1) sh.limit = mine;
            }
            __syncthreads();
            limit = sh.limit;
            break;
        }
    }
    // compact the winners (one shared-memory atomic per warp and visit)
    src.for_each([&](uint64_t rec, bool valid) {
        const bool take = valid && rec <= limit;
        const unsigned bal = __ballot_sync(FULL_MASK, take);
        if (bal) {
            uint32_t base = 0;
            if (lane == 0) base = atomicAdd(&sh.fill, (uint32_t)__popc(bal));
            base = __shfl_sync(FULL_MASK, base, 0);
            const uint32_t pos = base + __popc(bal & ((1u << lane) - 1u));
            if (take && pos < sort_cap) sortbuf[pos] = rec;
        }
    });
    __syncthreads();
}

// Ascending bitonic sort of P records (P a power of two, 32 <= P <= 1024), one per thread of
// the first P threads.  Exchanges at distance < 32 are warp shuffles; only the longer ones
// go through shared memory (scratch holds P records) with a named barrier over those P
// threads, so the rest of the CTA does not take part.
__device__ __forceinline__ uint64_t bitonic_sort_first_threads(uint64_t v, uint32_t P, uint64_t* scratch) {
    const unsigned tid = threadIdx.x;
    for (uint32_t size = 2; size <= P; size <<= 1) {
        const bool ascending = (tid & size) == 0;
        for (uint32_t stride = size >> 1; stride > 0; stride >>= 1) {
            uint64_t other;
            if (stride >= 32) {
                scratch[tid] = v;
                asm volatile("bar.sync 1, %0;" ::"r"(P) : "memory");
                other = scratch[tid ^ stride];
                asm volatile("bar.sync 1, %0;" ::"r"(P) : "memory");
            } else {
                other = __shfl_xor_sync(FULL_MASK, v, stride);
            }
            const bool lower = (tid & stride) == 0;
            const bool keep_min = lower == ascending;
            v = (keep_min == (other < v)) ? other : v;
        }
    }
    return v;
}

template <typename T>
__device__ __forceinline__ void write_output(T* out_vals, int64_t* out_idx, uint32_t k, uint64_t row, uint32_t j, uint64_t rec) {
    out_vals[row * (uint64_t)k + j] = Elem<T>::from_key(record_key(rec));
    out_idx[row * (uint64_t)k + j] = (int64_t)record_idx(rec);
}

// Orders the m records in sortbuf (all threads have passed a barrier since they were written)
// and writes the first kk of them as row `row` of the output.
template <typename T>
__device__ __forceinline__ void sort_and_write(uint64_t* sortbuf, uint32_t m, uint32_t kk, uint32_t k, uint64_t row,
                                               T* out_vals, int64_t* out_idx) {
    const unsigned tid = threadIdx.x, nthr = blockDim.x;
    if (m <= nthr) {
        uint32_t P = 32;
        while (P < m) P <<= 1;
        const uint64_t v0 = tid < m ? sortbuf[tid] : ~0ull;
        __syncthreads();                                    // sortbuf doubles as the exchange scratch
        if (tid < P) {
            const uint64_t v = bitonic_sort_first_threads(v0, P, sortbuf);
            if (tid < kk) write_output(out_vals, out_idx, k, row, tid, v);
        }
    } else {
        uint32_t P = 1;
        while (P < m) P <<= 1;
        for (uint32_t i = m + tid; i < P; i += nthr) sortbuf[i] = ~0ull;
        __syncthreads();
        bitonic_sort_shared(sortbuf, P);
        for (uint32_t j = tid; j < kk; j += nthr) write_output(out_vals, out_idx, k, row, j, sortbuf[j]);
    }
}

}  // namespace profk
