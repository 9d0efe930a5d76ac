// Stage 4 (Section 3, "Refinement"): the count check and the exact top-k of the candidate
// buffer, written out in the order "value descending, index ascending".
//
// Candidate records are 64-bit integers whose ascending order is exactly that order, so
// refinement is "the k smallest records, sorted".  One CTA per row.  The CTA first takes the
// paper's check -- fewer than k candidates, or more than the buffer holds, means the row is
// left to the exact-selection kernel that follows.  Otherwise the records (held in registers
// when they fit) are binned by their key's distance above tau into 4096 logarithmic bins; a scan of the
// bin counts gives every bin its first output position and finds the bin that holds the k-th
// best record; the records of that bin and of all better bins are grouped by bin in shared
// memory, and each of them finds its final position by ranking itself inside its (small) bin.
// No sort is needed.  When a bin is too crowded for that (many equal values) a
// most-significant-digit radix select plus a bitonic sort does the same job.
#pragma once

#include "sample_select.cuh"

namespace profk {

constexpr int RF_BITS = 12;                 // digit width of the general select
constexpr int RF_BINS = 1 << RF_BITS;
constexpr uint32_t RF_EDGE_CAP = 1024;      // boundary bins up to this size are ranked directly

enum : uint32_t { ROW_OK = 0, ROW_RECALL = 1, ROW_OVERFLOW = 2, ROW_DIRECT = 3 };

template <typename T> struct RefineParams {
    RowCtl* ctl;
    WsHeader* header;
    const uint64_t* buf;     // row r's records start at buf + r * buf_stride
    uint64_t buf_stride;
    uint32_t capacity;
    uint32_t k;
    uint32_t k_accept;
    uint32_t stage_cap;      // records the general select may stage in shared memory (0 = read them from the buffer)
    uint32_t sort_cap;       // power of two >= k: records the sort area holds (the area has RF_EDGE_CAP more)
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

template <typename T>
__global__ void __launch_bounds__(1024) refine_kernel(const RefineParams<T> p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* sortbuf = reinterpret_cast<uint64_t*>(smem_raw);                 // sort_cap + RF_EDGE_CAP records
    uint64_t* staged = sortbuf + p.sort_cap + RF_EDGE_CAP;                     // stage_cap records
    __shared__ SelectShared sh;

    const unsigned tid = threadIdx.x, nthr = blockDim.x, lane = lane_id();
    const uint64_t row = blockIdx.x;
    if (tid == 0) { sh.or_bits = 0ull; sh.fill = 0; sh.n_edge = 0; sh.crowded = 0; }
    for (uint32_t i = tid; i < RF_BINS; i += nthr) sh.hist[i] = 0;
    __syncthreads();
    pdl_launch_dependents();                 // the exact-selection kernel may be staged behind this one
    if (p.use_pdl) pdl_wait();
    PROFK_STAMP(1, 0);

    // The first batch of records (8 per thread, kept in registers) is requested at once, together with
    // the row's control block: which of them are real is known when the survivor count arrives.
    const uint64_t* src = p.buf + row * p.buf_stride;
    uint64_t r[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const uint32_t i = u * nthr + tid;
        r[u] = i < p.capacity ? src[i] : ~0ull;
    }

    // ---- the count check of stage 4 ----
    const RowCtl ctl = p.ctl[row];
    const uint32_t R = ctl.count;
    const uint32_t status = R > p.capacity ? ROW_OVERFLOW : R < p.k_accept ? ROW_RECALL : ROW_OK;
    if (tid == 0) {
        p.ctl[row].status = status;
        p.ctl[row].n_final = status ? p.k : R;
        if (status) atomicAdd(&p.header->n_failed, 1u);
    }
    if (status != ROW_OK) return;            // the exact-selection kernel takes this row

    const uint32_t n = R;
    const uint32_t kk = n < p.k ? n : p.k;          // real outputs; the rest is padding (relaxed mode)
    for (uint32_t j = kk + tid; j < p.k; j += nthr) {       // relaxed mode: padding after a short buffer
        p.out_vals[row * (uint64_t)p.k + j] = Elem<T>::from_bits(Elem<T>::NEG_INF_BITS);
        p.out_idx[row * (uint64_t)p.k + j] = -1;
    }

    // ---- bin the records by the distance d of their key above tau, on a logarithmic scale: the bin is
    //      the exponent and the top seven mantissa bits of d as a float (monotone in d, 32 x 128 = 4096
    //      bins, fine where the records are dense -- just above tau -- and coarse where they are rare).
    //      Bin 0 holds the largest keys. ----
    const uint32_t tau_key = Elem<T>::key(Elem<T>::from_bits(ctl.tau_bits));
    const uint32_t nbatch = (n + 8 * nthr - 1) / (8 * nthr);   // one batch = 8 records per thread
    auto load_batch = [&](uint32_t b) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t i = (b * 8 + u) * nthr + tid;
            r[u] = i < n ? src[i] : ~0ull;
        }
    };
    auto valid = [&](uint32_t b, int u) { return (b * 8 + u) * nthr + tid < n; };
    auto bin_of = [&](uint64_t rec) {
        const uint32_t key = record_key(rec);
        const uint32_t d = key > tau_key ? key - tau_key : 0u;
        const uint32_t f = __float_as_uint((float)d);           // 0 for d = 0, exponent >= 127 otherwise
        const uint32_t level = f > (127u << 23) ? (f >> 16) - (127u << 7) : 0u;     // 0 .. 4095
        return (uint32_t)(RF_BINS - 1) - level;
    };
    PROFK_STAMP(1, 1);

    for (uint32_t b = 0; b < nbatch; ++b) {
        if (b > 0) load_batch(b);
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (valid(b, u)) atomicAdd(&sh.hist[bin_of(r[u])], 1u);
    }
    __syncthreads();

    // ---- scan the bin counts: first position of every bin, and the bin of the kk-th best record ----
    if (nthr * 4 == RF_BINS) {
        // four bins per thread, read and written as one 16-byte vector; two barriers in all
        const uint4 c = reinterpret_cast<const uint4*>(sh.hist)[tid];
        const uint32_t sum = c.x + c.y + c.z + c.w;
        uint32_t incl = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t v = __shfl_up_sync(FULL_MASK, incl, d);
            if (lane >= (unsigned)d) incl += v;
        }
        if (lane == 31) sh.warp_sums[tid >> 5] = incl;
        __syncthreads();
        uint32_t w = sh.warp_sums[lane];                       // every warp scans the 32 warp totals itself
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t v = __shfl_up_sync(FULL_MASK, w, d);
            if (lane >= (unsigned)d) w += v;
        }
        const uint32_t warp_before = __shfl_sync(FULL_MASK, w, (tid >> 5) ? (tid >> 5) - 1 : 0);
        const uint32_t b0 = incl - sum + ((tid >> 5) ? warp_before : 0u);
        const uint32_t b1 = b0 + c.x, b2 = b1 + c.y, b3 = b2 + c.z;
        const uint32_t before[4] = {b0, b1, b2, b3}, cnt[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (before[j] < kk && kk <= before[j] + cnt[j]) { sh.digit = tid * 4 + j; sh.before = before[j]; sh.cnt = cnt[j]; }
            if (before[j] < kk && cnt[j] > RF_EDGE_CAP) sh.crowded = 1;
        }
        reinterpret_cast<uint4*>(sh.start)[tid] = make_uint4(b0, b1, b2, b3);
        reinterpret_cast<uint4*>(sh.hist)[tid] = make_uint4(b0, b1, b2, b3);     // the bins' write cursors
    } else {
        const uint32_t per = (RF_BINS + nthr - 1) / nthr;
        uint32_t sum = 0;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t bin = tid * per + j;
            sum += bin < RF_BINS ? sh.hist[bin] : 0;
        }
        uint32_t before = block_scan_any(sum, sh.warp_sums) - sum;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t bin = tid * per + j;
            if (bin < RF_BINS) {
                const uint32_t c = sh.hist[bin];
                if (before < kk && kk <= before + c) { sh.digit = bin; sh.before = before; sh.cnt = c; }
                if (before < kk && c > RF_EDGE_CAP) sh.crowded = 1;         // a bin that matters is too full to rank
                sh.start[bin] = before;
                sh.hist[bin] = before;                                      // becomes the bin's write cursor
                before += c;
            }
        }
    }
    __syncthreads();
    PROFK_STAMP(1, 2);

    if (!sh.crowded) {
        // ---- group the records of the boundary bin and of all better bins by bin ----
        const uint32_t edge_bin = sh.digit;
        const uint32_t n_grouped = sh.before + sh.cnt;                      // < kk + RF_EDGE_CAP
        for (uint32_t b = 0; b < nbatch; ++b) {
            if (nbatch > 1) load_batch(b);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (valid(b, u)) {
                    const uint32_t bin = bin_of(r[u]);
                    if (bin <= edge_bin) sortbuf[atomicAdd(&sh.hist[bin], 1u)] = r[u];
                }
            }
        }
        __syncthreads();
        PROFK_STAMP(1, 3);
        // ---- every grouped record ranks itself inside its bin: that is its place in the output ----
        for (uint32_t s = tid; s < n_grouped; s += nthr) {
            const uint64_t mine = sortbuf[s];
            const uint32_t bin = bin_of(mine);
            const uint32_t first = sh.start[bin], last = sh.hist[bin];
            uint32_t pos = first;
            for (uint32_t j = first; j < last; ++j) pos += sortbuf[j] < mine;
            if (pos < kk) write_output(p.out_vals, p.out_idx, p.k, row, pos, mine);
        }
        PROFK_STAMP(1, 4);
        return;
    }

    // ---- crowded bins (many equal values): general select, then sort ----
    uint32_t m;
    if (n <= p.sort_cap) {
        for (uint32_t i = tid; i < n; i += nthr) sortbuf[i] = src[i];
        m = n;
        __syncthreads();
    } else {
        const bool use_stage = n <= p.stage_cap;
        const uint64_t first = src[0];
        uint64_t diff = 0;
        for (uint32_t i = tid; i < n; i += nthr) {
            const uint64_t rec = src[i];
            diff |= rec ^ first;
            if (use_stage) staged[i] = rec;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) diff |= __shfl_xor_sync(FULL_MASK, diff, d);
        if (lane == 0 && diff) atomicOr(&sh.or_bits, (unsigned long long)diff);
        __syncthreads();
        MemRecords mem{use_stage ? staged : src, n};
        select_smallest(mem, first, kk, sortbuf, p.sort_cap, sh);
        m = kk;
    }
    sort_and_write<T>(sortbuf, m, kk, p.k, row, p.out_vals, p.out_idx);
}

}  // namespace profk
