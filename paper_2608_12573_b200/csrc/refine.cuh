// Stage 4 (Section 3, "Refinement"): exact top-k of the candidate buffer, written out in
// the order "value descending, index ascending".
//
// Candidate records are 64-bit integers whose ascending order is exactly that order, so
// refinement is "the k smallest records, sorted".  One CTA per row: the records are staged
// in shared memory when they fit, a most-significant-digit radix select (11 bits per pass,
// starting at the first bit in which the records differ) cuts them down to k, and a
// bitonic sort in shared memory orders the k winners.
#pragma once

#include "sample_select.cuh"

namespace profk {

constexpr int RF_BINS = 2048;

template <typename T> struct RefineParams {
    const RowCtl* ctl;
    const uint64_t* buf;     // rows x capacity records
    uint32_t capacity;
    uint32_t k;
    uint32_t stage_cap;      // records that fit the shared-memory staging area
    uint32_t sort_cap;       // power of two >= k: size of the shared-memory sort area
    T* out_vals;             // rows x k
    int64_t* out_idx;        // rows x k
    int use_pdl;
};

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

template <typename T>
__global__ void refine_kernel(const RefineParams<T> p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* sortbuf = reinterpret_cast<uint64_t*>(smem_raw);                 // sort_cap records
    uint64_t* staged = sortbuf + p.sort_cap;                                   // stage_cap records
    __shared__ uint32_t hist[RF_BINS];
    __shared__ uint32_t warp_sums[32];
    __shared__ uint32_t s_digit, s_before, s_cnt, s_fill;
    __shared__ unsigned long long s_or;

    const unsigned tid = threadIdx.x, nthr = blockDim.x;
    const uint64_t row = blockIdx.x;
    if (p.use_pdl) pdl_wait();

    uint32_t n = p.ctl[row].n_final;
    if (n > p.capacity) n = p.capacity;
    const uint32_t kk = n < p.k ? n : p.k;          // real outputs; the rest is padding (relaxed mode)
    const uint64_t* src = p.buf + row * (uint64_t)p.capacity;

    const bool use_stage = n <= p.stage_cap && n > p.sort_cap;
    if (use_stage) {
        for (uint32_t i = tid; i < n; i += nthr) staged[i] = src[i];
        __syncthreads();
    }
    const uint64_t* recs = use_stage ? staged : src;

    uint32_t m;   // records to sort
    if (n > p.sort_cap) {
        // ---- radix select: limit = the kk-th smallest record ----
        if (tid == 0) { s_or = 0ull; s_fill = 0; }
        __syncthreads();
        const uint64_t first = recs[0];
        uint64_t diff = 0;
        for (uint32_t i = tid; i < n; i += nthr) diff |= recs[i] ^ first;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) diff |= __shfl_xor_sync(FULL_MASK, diff, d);
        if (lane_id() == 0 && diff) atomicOr(&s_or, (unsigned long long)diff);
        __syncthreads();
        const int top = 64 - __clzll((long long)s_or);      // bits >= top are common to all records (s_or != 0: n >= 2)
        uint64_t prefix = shr64(first, top);
        uint32_t need = kk;
        uint64_t limit = ~0ull;
        for (int done = 0; done < top;) {
            const int shift = top - done - 11 > 0 ? top - done - 11 : 0;
            const int width = top - done - shift;
            const uint32_t nbins = 1u << width;
            for (uint32_t i = tid; i < nbins; i += nthr) hist[i] = 0;
            __syncthreads();
            for (uint32_t i = tid; i < n; i += nthr) {
                const uint64_t rec = recs[i];
                if (shr64(rec, shift + width) == prefix) atomicAdd(&hist[(uint32_t)(rec >> shift) & (nbins - 1)], 1u);
            }
            __syncthreads();
            const uint32_t per = (RF_BINS + nthr - 1) / nthr;
            uint32_t sum = 0;
            for (uint32_t j = 0; j < per; ++j) {
                const uint32_t bin = tid * per + j;
                sum += bin < nbins ? hist[bin] : 0;
            }
            uint32_t before = block_scan_any(sum, warp_sums) - sum;
            for (uint32_t j = 0; j < per; ++j) {
                const uint32_t bin = tid * per + j;
                const uint32_t c = bin < nbins ? hist[bin] : 0;
                if (before < need && need <= before + c) { s_digit = bin; s_before = before; s_cnt = c; }
                before += c;
            }
            __syncthreads();
            prefix = (prefix << width) | s_digit;
            need -= s_before;
            const bool whole_bin = s_cnt == need;
            done += width;
            __syncthreads();
            if (whole_bin || done >= top) { limit = ((prefix + 1) << shift) - 1; break; }
        }
        // ---- compact the kk winners into the sort area ----
        for (uint32_t i = tid; i < n; i += nthr) {
            const uint64_t rec = recs[i];
            if (rec <= limit) {
                const uint32_t pos = atomicAdd(&s_fill, 1u);
                if (pos < p.sort_cap) sortbuf[pos] = rec;
            }
        }
        m = kk;
    } else {
        for (uint32_t i = tid; i < n; i += nthr) sortbuf[i] = src[i];
        m = n;
    }

    uint32_t P = 1;
    while (P < m) P <<= 1;
    for (uint32_t i = m + tid; i < P; i += nthr) sortbuf[i] = ~0ull;
    __syncthreads();
    bitonic_sort_shared(sortbuf, P);

    T* ov = p.out_vals + row * (uint64_t)p.k;
    int64_t* oi = p.out_idx + row * (uint64_t)p.k;
    for (uint32_t j = tid; j < p.k; j += nthr) {
        if (j < kk) {
            const uint64_t rec = sortbuf[j];
            ov[j] = Elem<T>::from_key(record_key(rec));
            oi[j] = (int64_t)record_idx(rec);
        } else {
            ov[j] = Elem<T>::from_bits(Elem<T>::NEG_INF_BITS);
            oi[j] = -1;
        }
    }
}

}  // namespace profk
