// Exact replacement of failed rows by the whole grid (Section 3, "Refinement": "if fewer than k
// candidates are collected, or if the buffer overflows ..., falls back to an exact top-k
// computation on the full input"), for the calls whose refine kernel does not do it itself:
// many rows, where one cluster per row would be mostly idle CTAs, and large selections.  The
// decision is taken on the device: the refine kernel checks every row's survivor count and
// leaves the rows that failed to this kernel, which returns at once when there are none.  For
// each failed row it selects the exact top-k of the whole row into the row's candidate buffer
// and, for selections small enough, orders it and writes the row's output.
//
// The exact selection is a most-significant-digit radix select over 64-bit candidate records
// (value key, then index), 11 bits per pass, run by the whole grid with a grid barrier after
// each pass.  The kernel is launched cooperatively so that all CTAs are co-resident; every
// wait is bounded and reports through the workspace header.
#pragma once

#include "grid_barrier.cuh"
#include "refine.cuh"
#include "rowscan.cuh"
#include "sample_select.cuh"

namespace profk {

constexpr int FB_THREADS = 1024;
constexpr int FB_UNROLL = 4;
constexpr int FB_BINS = 2048;
constexpr int FB_PASSES = 6;                // 5 x 11 bits + 9 bits = 64


template <typename T> struct FallbackParams {
    const T* in;
    uint64_t N;
    uint64_t rows;
    uint32_t k;
    uint32_t capacity;
    RowCtl* ctl;
    WsHeader* header;
    uint32_t* ghist;          // FB_PASSES x FB_BINS global histogram
    uint64_t* buf;            // row r's records start at buf + r * buf_stride
    uint64_t buf_stride;
    int sort_rows;            // 1 = order and write the repaired rows here; 0 = a later kernel does (large k)
    uint64_t tiles_per_row;
    int use_pdl;              // 1 = launched as a programmatic dependent of the refine kernel
    T* out_vals;              // rows x k
    int64_t* out_idx;         // rows x k
    // Many failed rows at once (a batch in direct mode, a batch of tie-flooded rows) are dealt out one per CTA
    // instead: each CTA runs the exact selection of exact_select.cuh on its own.  Null = always row by row.
    uint64_t* cta_records;    // gridDim.x x (k + XS_EDGE) records of scratch
    uint32_t* cta_counters;   // gridDim.x counters
    uint32_t sort_cap;        // power of two >= k: records the dynamic shared memory holds
    int parallel;             // 1 = the one-row-per-CTA mode may be used (its scratch is there, or none is needed)
    // The second filtering pass (second_chance.cuh) of a row that failed the check, taken by the whole grid before the
    // exact selection: when the rows are repaired one after the other by the kernel below, and by the fused
    // large-selection kernels for their single row.
    SampleInfo sample;        // sample.keys == null: none
    uint4* thr2;              // rows threshold records of that pass
};

static_assert(FB_BINS <= RF_BINS, "the grid-wide selection's histogram lives in SelectShared::hist");
constexpr uint32_t FB_PARALLEL_MIN = 8;     // from this many failed rows on, one CTA per row beats the grid per row

// Visits every element of `row` that falls to this CTA (tiles blockIdx.x, +gridDim.x, ...):
// f(record, valid) is called by all 32 lanes of each warp together.
template <typename T, typename F>
__device__ __forceinline__ void for_each_record(const FallbackParams<T>& p, uint64_t row, F&& f) {
    using V = typename Elem<T>::vec_t;
    constexpr int VEC = Elem<T>::VEC;
    constexpr uint32_t TILE_VECTORS = FB_THREADS * FB_UNROLL;
    const RowView<T> rv = row_view(p.in, p.N, row);
    for (uint64_t tile = blockIdx.x; tile < p.tiles_per_row; tile += gridDim.x) {
        V v[FB_UNROLL];
        bool inside[FB_UNROLL];
#pragma unroll
        for (int u = 0; u < FB_UNROLL; ++u)
            v[u] = load_row_vector(rv, p.N, tile * TILE_VECTORS + (uint64_t)u * FB_THREADS + threadIdx.x, &inside[u]);
#pragma unroll
        for (int u = 0; u < FB_UNROLL; ++u) {
            const uint64_t q = tile * TILE_VECTORS + (uint64_t)u * FB_THREADS + threadIdx.x;
            const int64_t i0 = (int64_t)(q * VEC) - (int64_t)rv.mis;
#pragma unroll
            for (int l = 0; l < VEC; ++l) {
                const int64_t i = i0 + l;
                const bool valid = inside[u] && i >= 0 && i < (int64_t)p.N;
                f(make_record(Elem<T>::key(vec_elem(v[u], l)), (uint32_t)i), valid);
            }
        }
    }
}

// Exact selection of the k smallest records of `row` by the whole grid (FB_THREADS threads per CTA, all CTAs
// co-resident): a most-significant-digit radix select over the row's elements as 64-bit records, 11 bits per pass,
// a grid barrier after each, then one more read of the row that appends the k winners to the row's buffer (counter:
// the row's `collect` word, zero on entry).  Called by every thread of every CTA.  Returns false when a bounded wait gave up (the caller leaves the kernel); on a true
// return the last barrier has been passed and the k records are in p.buf + row * p.buf_stride, in no particular order.
template <typename T>
__device__ __noinline__ bool grid_exact_select_row(const FallbackParams<T>& p, uint64_t row, uint32_t* sh_hist,
                                                   uint32_t* warp_sums) {
    __shared__ uint32_t s_digit, s_before, s_cnt;
    const unsigned tid = threadIdx.x, lane = lane_id();
    if (!grid_barrier(p.header)) return false;          // a previous row's histogram reads are over
    for (uint32_t i = blockIdx.x * FB_THREADS + tid; i < FB_PASSES * FB_BINS; i += gridDim.x * FB_THREADS)
        p.ghist[i] = 0;
    if (!grid_barrier(p.header)) return false;

    uint64_t prefix = 0;       // selected high bits, right-aligned
    uint32_t need = p.k;       // rank (from the smallest record) inside the prefix class
    uint64_t limit = ~0ull;    // records <= limit are the answer
    for (int pass = 0; pass < FB_PASSES; ++pass) {
        const int shift = pass < 5 ? 53 - 11 * pass : 0;
        const int width = pass < 5 ? 11 : 9;
        const uint32_t nbins = 1u << width;
        for (uint32_t i = tid; i < nbins; i += FB_THREADS) sh_hist[i] = 0;
        __syncthreads();
        for_each_record(p, row, [&](uint64_t rec, bool valid) {
            const bool in_class = valid && (pass == 0 || (rec >> (shift + width)) == prefix);
            const uint32_t digit = in_class ? (uint32_t)(rec >> shift) & (nbins - 1) : 0xFFFFFFFFu;
            const unsigned peers = __match_any_sync(FULL_MASK, digit);
            if (in_class && lane == (unsigned)(__ffs(peers) - 1)) atomicAdd(&sh_hist[digit], __popc(peers));
        });
        __syncthreads();
        uint32_t* gh = p.ghist + pass * FB_BINS;
        for (uint32_t i = tid; i < nbins; i += FB_THREADS) {
            const uint32_t c = sh_hist[i];
            if (c) atomicAdd(&gh[i], c);
        }
        if (!grid_barrier(p.header)) return false;

        // Every CTA finds the bin that holds the need-th smallest record of the class.
        constexpr int PER = FB_BINS / FB_THREADS;                   // bins per thread
        uint32_t c[PER], sum = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const uint32_t bin = tid * PER + j;
            c[j] = bin < nbins ? __ldcg(&gh[bin]) : 0;
            sum += c[j];
        }
        uint32_t before = block_inclusive_scan(sum, warp_sums) - sum;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (before < need && need <= before + c[j]) { s_digit = tid * PER + j; s_before = before; s_cnt = c[j]; }
            before += c[j];
        }
        __syncthreads();
        prefix = (prefix << width) | s_digit;
        need -= s_before;
        const bool whole_bin = (s_cnt == need);
        __syncthreads();
        if (whole_bin || pass == FB_PASSES - 1) {
            limit = ((prefix + 1) << shift) - 1;        // wraps to all-ones when the class is the last one
            break;
        }
    }

    // ---- collect the k records <= limit into the row's buffer ----
    uint64_t* dst = p.buf + row * p.buf_stride;
    uint32_t* counter = &p.ctl[row].collect;
    const unsigned lt_mask = (1u << lane) - 1u;
    for_each_record(p, row, [&](uint64_t rec, bool valid) {
        const bool take = valid && rec <= limit;
        const unsigned bal = __ballot_sync(FULL_MASK, take);
        if (bal) {
            unsigned base = 0;
            if (lane == 0) base = atomicAdd(counter, __popc(bal));
            base = __shfl_sync(FULL_MASK, base, 0);
            const unsigned pos = base + __popc(bal & lt_mask);
            if (take && pos < p.capacity) dst[pos] = rec;
        }
    });
    return grid_barrier(p.header);
}

// The second filtering pass (second_chance.cuh) of a row that failed the count check with `status`, by the whole grid:
// every CTA selects the plan's tighter (overflow) or looser (too few candidates) sample rank from the kept keys for
// itself, the grid filters the row once more into the row's buffer (from its start; counter: the row's `pad` word, zero
// on entry), one grid barrier, and every CTA takes the same count check.  Returns 1 when the row passed it: the buffer
// holds *R2 records, k <= *R2 <= capacity, *key2 is the order key of the threshold used, and the row's control block
// says so; 0 when no second pass applies (no keys kept, no such rank in the plan) or the row failed again; -1 when a
// bounded wait gave up (the caller leaves the kernel).  Called by every thread of every CTA (FB_THREADS threads).
template <typename T>
__device__ __noinline__ int grid_second_chance_row(const FallbackParams<T>& p, uint64_t row, uint32_t status, SelectShared& sh,
                                                   uint32_t* R2_out, uint32_t* key2_out) {
    const SampleInfo& sm = p.sample;
    if (sm.keys == nullptr) return 0;
    const uint32_t rung = status == ROW_OVERFLOW ? sm.r_tight : status == ROW_RECALL ? sm.r_loose : 0u;
    if (rung == 0) return 0;
    const unsigned tid = threadIdx.x;
    uint32_t key2, j2;
    // (every CTA for itself; a tighter rank lies among the keys at or above the first pass's threshold)
    kth_sample_record<T>(sm.keys + row * sm.S, sm.S, rung, sh, &key2, &j2,
                         status == ROW_OVERFLOW ? Elem<T>::key(Elem<T>::from_bits(__ldcg(&p.ctl[row].tau_bits))) : 0u);
    const uint32_t idx2 = sm.by_record ? sample_element_index(j2, row, sm.seed, sm.q, sm.rem, sm.S, sm.inv_s) : 0xFFFFFFFFu;
    const T tau2 = Elem<T>::from_key(key2);
    if (tid == 0) {
        const uint32_t top = Elem<T>::KEY_BITS == 32 ? 0xFFFFFFFFu : 0xFFFFu;
        p.thr2[row] = make_uint4(Elem<T>::bits(tau2), Elem<T>::bits(Elem<T>::from_key(key2 == top ? key2 : key2 + 1u)), idx2, 0u);
    }
    __syncthreads();
    FilterParams<T> fp = {};
    fp.in = p.in; fp.N = p.N; fp.rows = row + 1; fp.tau = nullptr; fp.capacity = p.capacity;
    fp.buf = p.buf; fp.buf_stride = p.buf_stride;
    fp.counts = &p.ctl[0].pad; fp.count_stride = sizeof(RowCtl) / 4;
    fp.thr = p.thr2;
    refilter_tiles<T, FB_THREADS>(fp, (uint32_t)row, 0, p.tiles_per_row, blockIdx.x, gridDim.x, tau2);
    if (!grid_barrier(p.header)) return -1;
    const uint32_t R2 = __ldcg(&p.ctl[row].pad);
    if (R2 < p.k || R2 > p.capacity) return 0;                 // (the same decision in every CTA)
    if (blockIdx.x == 0 && tid == 0) {
        p.ctl[row].status = status == ROW_OVERFLOW ? ROW_OVERFLOW_REFILTERED : ROW_RECALL_REFILTERED;
        p.ctl[row].count = R2;
        p.ctl[row].tau_bits = Elem<T>::bits(tau2);
        p.ctl[row].tau_idx = idx2;
    }
    *R2_out = R2;
    *key2_out = key2;
    return 1;
}

template <typename T>
__global__ void __launch_bounds__(FB_THREADS) fallback_kernel(const FallbackParams<T> p) {
    __shared__ SelectShared sh;                 // the per-CTA selection's state; its arrays also serve the grid-wide one
    uint32_t* sh_hist = sh.hist;                // FB_BINS <= RF_BINS words
    uint32_t* warp_sums = sh.warp_sums;
    __shared__ uint32_t flag_masks[FB_THREADS / 32];

    const unsigned tid = threadIdx.x, lane = lane_id(), warp = tid >> 5;
    pdl_launch_dependents();
    if (p.use_pdl) pdl_wait();

    // The count check was taken by the refine kernel (or, in direct mode, every row was marked by
    // the initialisation kernel): in the common case no row failed and this kernel is one load long.
    const uint32_t n_failed = __ldcg(&p.header->n_failed);
    if (n_failed == 0) return;

    if (p.parallel && n_failed >= FB_PARALLEL_MIN) {
        // ---- many rows: each CTA takes failed rows of its own (no grid barrier is reached) ----
        extern __shared__ __align__(16) unsigned char fb_smem[];
        uint64_t* sortbuf = reinterpret_cast<uint64_t*>(fb_smem);
        const uint32_t slots = p.k + XS_EDGE;
        uint64_t* recs = p.cta_records + (uint64_t)blockIdx.x * slots;
        const uint64_t tiles = tiles_per_row<T>(p.N, FB_THREADS * XS_UNROLL);
        for (uint64_t row = blockIdx.x; row < p.rows; row += gridDim.x) {
            const uint32_t status = __ldcg(&p.ctl[row].status);
            if (status == ROW_OK) continue;
            const uint32_t tau_key = Elem<T>::key(Elem<T>::from_bits(__ldcg(&p.ctl[row].tau_bits)));
            if (p.sort_rows) {
                exact_select_cluster<T>(p.in, p.N, row, p.k, 0, tiles, recs, p.cta_counters + blockIdx.x, sh, 1u, 0u,
                                        status == ROW_OVERFLOW, tau_key);
                finish_from_segments<T>(recs, slots, p.k, p.sort_cap, sortbuf, sh, row, p.out_vals, p.out_idx);
            } else {
                // large selections: exactly the k best records into the row's buffer, for the kernel that orders them
                exact_select_cluster<T>(p.in, p.N, row, p.k, 0, tiles, p.buf + row * p.buf_stride, &p.ctl[row].collect, sh, 1u, 0u,
                                        status == ROW_OVERFLOW, tau_key, 0u);
            }
            __syncthreads();
        }
        return;
    }


    for (uint64_t chunk = 0; chunk < p.rows; chunk += FB_THREADS) {
        // ---- FB_THREADS rows at a time; every CTA reads the same status words ----
        const uint64_t r = chunk + tid;
        const bool failed = r < p.rows && __ldcg(&p.ctl[r].status) != ROW_OK;
        const unsigned m = __ballot_sync(FULL_MASK, failed);
        if (lane == 0) flag_masks[warp] = m;
        __syncthreads();

        for (unsigned w = 0; w < FB_THREADS / 32; ++w) {
            unsigned mask = flag_masks[w];
            while (mask) {
                const unsigned b = __ffs(mask) - 1;
                mask &= mask - 1;
                const uint64_t row = chunk + w * 32 + b;

                // ---- first another filtering pass with the plan's tighter / looser sample rank, if it names one ----
                {
                    uint32_t R2 = 0, key2 = 0;
                    const int again = grid_second_chance_row<T>(p, row, __ldcg(&p.ctl[row].status), sh, &R2, &key2);
                    if (again < 0) return;
                    if (again == 1) {
                        if (p.sort_rows && blockIdx.x == 0) {      // (large selections: the kernel behind this one orders the row)
                            extern __shared__ __align__(16) unsigned char fb_smem[];
                            finish_from_segments<T>(p.buf + row * p.buf_stride, R2, p.k, p.sort_cap, reinterpret_cast<uint64_t*>(fb_smem), sh,
                                                    row, p.out_vals, p.out_idx);
                            __syncthreads();
                        }
                        continue;
                    }
                }
                // ---- exact selection of the k smallest records of `row` into the row's buffer ----
                if (!grid_exact_select_row<T>(p, row, sh_hist, warp_sums)) return;
                uint64_t* dst = p.buf + row * p.buf_stride;

                // ---- order the k records and write the row's output (first CTA; the others move on
                //      and meet it again at the next row's barrier) ----
                if (p.sort_rows && blockIdx.x == 0) {
                    extern __shared__ __align__(16) unsigned char fb_smem[];
                    uint64_t* sortbuf = reinterpret_cast<uint64_t*>(fb_smem);
                    for (uint32_t i = tid; i < p.k; i += FB_THREADS) sortbuf[i] = __ldcg(&dst[i]);
                    __syncthreads();
                    sort_and_write<T>(sortbuf, p.k, p.k, p.k, row, p.out_vals, p.out_idx);
                    __syncthreads();
                }
            }
        }
        __syncthreads();   // flag_masks is rewritten by the next chunk
    }
}

}  // namespace profk
