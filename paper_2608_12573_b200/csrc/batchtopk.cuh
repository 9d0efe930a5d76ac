// Flattened BatchTopK (Section 5, "Application: BatchTopK sparse autoencoders"): the B x d_dict pre-activations are
// one row of N = B * d_dict elements, the K = B * k largest are kept and all others become zero.  The consumer wants
// the kept SET -- as a list of (value, index) pairs in any order, as a bit mask, or scattered into a dense array of
// zeros -- not an ordered list, so after the filtering scan nothing has to be sorted: it is enough to find the K-th
// best candidate record and to emit every record up to it.
//
// One cooperative kernel (one CTA per SM, all co-resident, bounded grid barriers) does stage 4 in that form:
//   * the count check of Section 3, "Refinement"; a row that fails it is replaced on the spot by the exact selection
//     of the whole row (grid_exact_select_row), which leaves exactly K records -- all of them kept;
//   * otherwise a histogram select over the R candidate records in the bins of bins.cuh (distance D below the largest
//     record the filter can have kept, on a logarithmic scale: 2^18 fine bins in global memory, 512 coarse ones).
//     Level 0 is counted by the filter kernel itself as it appends the records (its HIST build), so this kernel starts
//     with the histogram made and no grid barrier at all when only the pairs are wanted; a call whose filter did not
//     count (or whose row was filtered a second time) counts here: fine bins with global atomics, coarse bins through
//     shared memory, ONE grid barrier.  Every CTA then scans the coarse bins and the 512 fine bins of the one that
//     holds the K-th best record; if that bin is crowded (many equal values: its records differ only in the index)
//     the next levels bin its D range linearly, 18 bits at a time, until at most BK_EDGE records are left in the
//     boundary class;
//   * the emit pass: every record of a better class is kept; the boundary class is copied to a short list, and the CTA
//     that finishes last (a ticket; nobody waits) ranks that list and keeps its best `need` records as well.  Kept records are appended to the pair list (one atomic per CTA
//     and pass), set their bit in the mask and are written to the dense array, which the kernel has zeroed before.
#pragma once

#include "fallback.cuh"

namespace profk {

constexpr int BK_THREADS = FB_THREADS;          // the exact selection it may call is written for this CTA size
constexpr int BK_BITS = BIN_BITS;
constexpr uint32_t BK_BINS = BIN_COUNT;
// the flag words after the bins: [0] pairs appended, [1] records in the boundary list, [2] CTAs done emitting
constexpr uint32_t BK_EDGE = 1024;              // a boundary class up to this size is ranked directly
constexpr uint32_t BK_COARSE = BIN_COARSE;
constexpr uint32_t BK_PER_COARSE = BIN_PER_COARSE;
static_assert(BK_COARSE <= BK_THREADS && BK_PER_COARSE <= BK_THREADS, "one thread per coarse bin, then per fine bin of one coarse bin");
constexpr uint32_t BK_WAIT_LIMIT = 1u << 22;    // polls of the "all CTAs have zeroed their share of the bins" counter
constexpr int BK_MAX_LEVELS = 6;                // 12 + 18 * 3 > 64 bits: more levels than any input needs

template <typename T> struct BatchTopkParams {
    FallbackParams<T> fb;        // the row (rows == 1), K, capacity, control block, header, histogram area, buffer
    uint32_t* bins;              // BIN_ROW_WORDS words: fine bins, flags, coarse bins
    int hist_ready;              // 1 = the filter kernel counted the records it appended in them (all else zero); 0 = nobody has touched them
    uint64_t* edge;              // BK_EDGE records: the boundary class
    uint32_t parts;              // 1, or FILTER_PARTS: the filter appended to that many parts of the buffer
    uint32_t part_cap;
    const uint32_t* part_counts;
    T* sel_vals;                 // K values of the kept elements, any order (null = not wanted); with sel_idx
    int64_t* sel_idx;            // K indices, same order
    uint32_t* mask;              // ceil(N / 32) words, bit i & 31 of word i >> 5 = element i is kept (null = not wanted)
    T* dense;                    // N elements: the kept values at their positions, zero elsewhere; may be the input itself
    int use_pdl;
    int direct;                  // 1 = no threshold / filter ran: the row is selected exactly
};

// Zeroes n elements at p (aligned to the element size only) with 16-byte stores where the address allows.
template <typename E>
__device__ __forceinline__ void bk_zero_fill(E* p, uint64_t n, uint64_t gid, uint64_t gthreads) {
    const uintptr_t a = (uintptr_t)p;
    const uint64_t head_bytes = (16 - (a & 15)) & 15;
    uint64_t head = head_bytes / sizeof(E);
    if (head > n) head = n;
    const uint64_t body = (n - head) * sizeof(E) / 16;                   // whole 16-byte vectors
    const uint64_t tail0 = head + body * (16 / sizeof(E));
    for (uint64_t i = gid; i < head; i += gthreads) p[i] = E{};
    uint4* v = reinterpret_cast<uint4*>(p + head);
    for (uint64_t i = gid; i < body; i += gthreads) v[i] = make_uint4(0u, 0u, 0u, 0u);
    for (uint64_t i = tail0 + gid; i < n; i += gthreads) p[i] = E{};
}

template <typename T>
__global__ void __launch_bounds__(BK_THREADS, 1) batchtopk_emit_kernel(const BatchTopkParams<T> p) {
    __shared__ SelectShared sh;                  // hist / start / warp_sums serve the scans here and the exact selection
    __shared__ uint32_t s_seg, s_seg_before, s_bin, s_bin_before, s_bin_count;
    __shared__ uint32_t s_warp_count[BK_THREADS / 32];

    const unsigned tid = threadIdx.x, lane = lane_id(), warp = tid >> 5;
    const unsigned nctas = gridDim.x, cta = blockIdx.x;
    const uint64_t gid = (uint64_t)cta * BK_THREADS + tid, gthreads = (uint64_t)nctas * BK_THREADS;
    const FallbackParams<T>& fb = p.fb;
    uint32_t* flags = p.bins + BIN_COUNT;
    uint32_t* coarse = flags + BIN_FLAGS;

    // Prologue, before the wait for the filter kernel: the workspace's bins and flags (nobody else uses them).
    // Each CTA then reports in through the header's `done` word (zeroed by the call's first kernel, long finished): the
    // histogram pass below needs every CTA's share to be zero, and by then all have reported -- a wait that does not wait.
    // (Not when the filter kernel counts in them: then the threshold kernels have cleared them.)
    if (!p.hist_ready) {
        for (uint64_t b = gid; b < BIN_ROW_WORDS; b += gthreads) p.bins[b] = 0;
        __threadfence();
        __syncthreads();
        if (tid == 0) atomicAdd(&fb.header->done, 1u);
    }
    pdl_launch_dependents();
    if (p.use_pdl) pdl_wait();

    // ---- the count check of stage 4 (the same in every CTA) ----
    const uint32_t K = fb.k;
    uint32_t pcount[FILTER_PARTS] = {};           // the records are pcount[j] at buf + j * part_cap
    uint32_t status;
    if (p.direct) {
        status = ROW_DIRECT;
    } else {
        uint32_t R = __ldcg(&fb.ctl[0].count);
        bool part_full = false;
        if (p.parts > 1) {                        // partitioned append: the row's count is the sum of its parts'
            uint64_t sum = 0;
#pragma unroll
            for (int j = 0; j < (int)FILTER_PARTS; ++j) {
                const uint32_t c = __ldcg(&p.part_counts[j * FILTER_PART_STRIDE]);
                part_full |= c > p.part_cap;
                pcount[j] = c < p.part_cap ? c : p.part_cap;
                sum += c;
            }
            R = sum > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)sum;
        } else {
            pcount[0] = R;
        }
        status = (R > fb.capacity || part_full) ? ROW_OVERFLOW : R < K ? ROW_RECALL : ROW_OK;
        if (cta == 0 && tid == 0) {
            if (p.parts > 1) fb.ctl[0].count = part_full && R <= fb.capacity ? fb.capacity + 1 : R;     // what the statistics report
            fb.ctl[0].status = status;
            fb.ctl[0].n_final = K;
            if (status) atomicAdd(&fb.header->n_failed, 1u);
        }
    }
    bool keep_all = false;                        // every record in the buffer is kept (it holds exactly K)
    uint32_t tau_key = 0;
    if (status != ROW_OK) {
        // A second filtering pass with the plan's tighter / looser sample rank first, if it names one ...
        uint32_t R2 = 0;
        const int again = p.direct ? 0 : grid_second_chance_row<T>(fb, 0, status, sh, &R2, &tau_key);
        if (again < 0) return;
        // ... else the exact replacement (Section 3, "Refinement"): the K best records of the whole row, into the buffer.
        if (again == 0 && !grid_exact_select_row<T>(fb, 0, sh.hist, sh.warp_sums)) return;
#pragma unroll
        for (int j = 0; j < (int)FILTER_PARTS; ++j) pcount[j] = 0;
        pcount[0] = again == 1 ? R2 : K;
        keep_all = again == 0;
    } else {
        tau_key = Elem<T>::key(Elem<T>::from_bits(__ldcg(&fb.ctl[0].tau_bits)));
    }
    uint32_t pend[FILTER_PARTS];                  // pend[j] = records in parts 0..j
    {
        uint32_t acc = 0;
#pragma unroll
        for (int j = 0; j < (int)FILTER_PARTS; ++j) { acc += pcount[j]; pend[j] = acc; }
    }
    const uint32_t total = pend[FILTER_PARTS - 1];
    const uint32_t iters = (uint32_t)((total + gthreads - 1) / gthreads);        // the same for every thread
    auto record_at = [&](uint64_t i) {
        uint32_t j = 0, before = 0;
#pragma unroll
        for (int q = 0; q < (int)FILTER_PARTS - 1; ++q)
            if (i >= pend[q]) { j = q + 1; before = pend[q]; }
        return (uint64_t)__ldcg(fb.buf + (uint64_t)j * p.part_cap + (i - before));
    };

    // The dense result and the mask start from zero.  (After the exact selection, which reads the input: the dense
    // array may be the input itself.)  The barriers below order these stores before the emit pass.
    if (p.mask) bk_zero_fill(p.mask, (fb.N + 31) / 32, gid, gthreads);
    if (p.dense) bk_zero_fill(p.dense, fb.N, gid, gthreads);

    // ---- the class of the K-th best record ----
    // D = distance of a record below `top`, the largest record the filter can have kept (tau's key, the last index);
    // D >= 0 for every kept record (their keys are >= tau's), larger D = better record.  A record holds the key above a
    // 32-bit index word of which a row only uses idx_bits bits; the unused bits are squeezed out of D, so that the bits
    // right below the key difference are real index bits: thousands of copies of one bf16 value then spread over the
    // logarithmic level's bins instead of crowding one (which costs further levels).
    const uint32_t top_hi = ~tau_key;
    const int idx_bits = index_bits(fb.N);
    auto dist = [&](uint64_t rec) { return record_dist(rec, top_hi, idx_bits); };
    uint64_t cls_lo = 0;          // the boundary class is cls_lo <= D < cls_lo + 2^cls_w ...
    int cls_w = 64;               // ... (64: every D)
    uint32_t need = K;            // ... and its `need` best records are kept, with every record of a better class
    bool whole = keep_all;        // the whole boundary class is kept: nothing to rank
    if (keep_all) need = 0;
    __shared__ uint32_t s_coarse[BK_COARSE];
    __shared__ uint32_t s_ok;
    // level 0 has been counted by the filter kernel (all of it: no record went in uncounted)
    const bool have_hist = p.hist_ready && status == ROW_OK && __ldcg(&flags[BIN_FLAG_UNCOUNTED]) == 0;
    if (keep_all) {
        // (the exact selection ended on a grid barrier, but the zero fill above came after it)
        if (!grid_barrier(fb.header)) return;
    } else if (have_hist) {
        // nothing to count; only the zero fill above has to be over everywhere before anybody emits
        if ((p.mask || p.dense) && !grid_barrier(fb.header)) return;
    } else if (p.hist_ready) {
        // the bins hold the counts of the first filtering pass, the buffer the records of the second: start again
        // (nobody has read the bins yet; the flags behind them are still zero)
        for (uint64_t b = gid; b < BIN_COUNT; b += gthreads) p.bins[b] = 0;
        for (uint64_t b = gid; b < BIN_COARSE; b += gthreads) coarse[b] = 0;
        if (!grid_barrier(fb.header)) return;
    } else {
        // every CTA has zeroed its share of the bins: reported before the wait for the filter kernel, so this returns at once
        if (tid == 0) {
            uint32_t ok = 1, polls = 0;
            while (*((volatile uint32_t*)&fb.header->done) < nctas) {
                __nanosleep(64);
                if (++polls > BK_WAIT_LIMIT) { atomicExch(&fb.header->error, 1u); ok = 0; break; }
            }
            __threadfence();
            s_ok = ok;
        }
        __syncthreads();
        if (!s_ok) return;
    }
    for (int level = 0; !whole && level < BK_MAX_LEVELS; ++level) {
        const int sh_bits = cls_w > BK_BITS ? cls_w - BK_BITS : 0;       // linear levels: D's bits below the bin
        auto bin_of = [&](uint64_t D, bool* in_class) {
            if (level == 0) { *in_class = true; return log_bin(D); }
            *in_class = D >= cls_lo && ((D - cls_lo) >> cls_w) == 0;
            return (uint32_t)((D - cls_lo) >> sh_bits) & (BK_BINS - 1);
        };
        // histogram, best records in the lowest bins: fine bins in global memory, coarse bins through shared memory
        if (!(level == 0 && have_hist)) {
            for (uint32_t c = tid; c < BK_COARSE; c += BK_THREADS) s_coarse[c] = 0;
            __syncthreads();
            for (uint64_t i = gid; i < total; i += gthreads) {
                bool in_class;
                const uint32_t f = BK_BINS - 1 - bin_of(dist(record_at(i)), &in_class);
                if (in_class) {
                    atomicAdd(&p.bins[f], 1u);
                    atomicAdd(&s_coarse[f / BK_PER_COARSE], 1u);
                }
            }
            __syncthreads();
            for (uint32_t c = tid; c < BK_COARSE; c += BK_THREADS) {
                const uint32_t n = s_coarse[c];
                if (n) atomicAdd(&coarse[c], n);
            }
            if (!grid_barrier(fb.header)) return;
        }
        // every CTA: the coarse bin, then the fine bin, of the need-th best record of the class
        {
            const uint32_t c = tid < BK_COARSE ? __ldcg(&coarse[tid]) : 0u;
            const uint32_t incl = block_inclusive_scan(c, sh.warp_sums);
            if (incl - c < need && need <= incl) { s_seg = tid; s_seg_before = incl - c; }
            __syncthreads();
        }
        {
            const uint32_t seg = s_seg, seg_before = s_seg_before;
            const uint32_t c = tid < BK_PER_COARSE ? __ldcg(&p.bins[seg * BK_PER_COARSE + tid]) : 0u;
            const uint32_t incl = block_inclusive_scan(c, sh.warp_sums);
            const uint32_t b0 = seg_before + incl - c;
            if (tid < BK_PER_COARSE && b0 < need && need <= b0 + c) { s_bin = seg * BK_PER_COARSE + tid; s_bin_before = b0; s_bin_count = c; }
            __syncthreads();
        }
        const uint32_t bin = BK_BINS - 1 - s_bin, in_bin = s_bin_count;
        need -= s_bin_before;
        if (level == 0) log_bin_range(bin, &cls_lo, &cls_w);
        else { cls_lo += (uint64_t)bin << sh_bits; cls_w = sh_bits; }
        __syncthreads();                           // the shared words are rewritten by the next level
        if (in_bin == need) { whole = true; break; }
        if (in_bin <= BK_EDGE) break;
        // crowded: one more level inside the class; the bins start from zero again
        if (!grid_barrier(fb.header)) return;                        // everybody has read this level's bins
        for (uint64_t b = gid; b < BK_BINS; b += gthreads) p.bins[b] = 0;
        for (uint64_t b = gid; b < BK_COARSE; b += gthreads) coarse[b] = 0;
        if (!grid_barrier(fb.header)) return;
    }
    // Kept outright: D >= keep_from.  Boundary list: cls_lo <= D < keep_from (empty when the whole class is kept).
    const bool top_class = cls_w >= 64 || cls_lo + (1ull << cls_w) < cls_lo;      // the class reaches the largest D there is
    const uint64_t keep_from = whole ? cls_lo : cls_lo + (1ull << (cls_w & 63));
    const uint32_t n_outright = K - (whole ? 0u : need);

    // ---- emit ----
    auto emit = [&](uint64_t rec, uint32_t pos) {
        const uint32_t idx = record_idx(rec);
        const T val = Elem<T>::from_key(record_key(rec));
        if (p.sel_idx) { p.sel_vals[pos] = val; p.sel_idx[pos] = (int64_t)idx; }
        if (p.mask) atomicOr(&p.mask[idx >> 5], 1u << (idx & 31u));
        if (p.dense) p.dense[idx] = val;
    };
    // Each thread takes up to EM records at a time (their loads in flight together); the CTA reserves room in the pair list
    // for all of them with one atomic.
    constexpr int EM = 4;
    for (uint32_t it0 = 0; it0 < iters; it0 += EM) {
        uint64_t rec[EM];
        bool valid[EM];
#pragma unroll
        for (int u = 0; u < EM; ++u) {
            const uint64_t i = (uint64_t)(it0 + u) * gthreads + gid;
            valid[u] = it0 + u < iters && i < total;
            rec[u] = valid[u] ? record_at(i) : 0ull;
        }
        unsigned keptm = 0, cnt = 0;               // bit u: record u is kept outright
#pragma unroll
        for (int u = 0; u < EM; ++u) {
            bool kept = false, boundary = false;
            if (valid[u]) {
                const uint64_t D = dist(rec[u]);
                kept = keep_all || (whole ? D >= keep_from : (!top_class && D >= keep_from));
                boundary = !kept && !whole && D >= cls_lo;
            }
            keptm |= kept ? 1u << u : 0u;
            cnt += kept ? 1u : 0u;
            const unsigned ebal = __ballot_sync(FULL_MASK, boundary);
            if (ebal) {
                uint32_t ebase = 0;
                if (lane == 0) ebase = atomicAdd(&flags[1], (uint32_t)__popc(ebal));
                ebase = __shfl_sync(FULL_MASK, ebase, 0);
                const uint32_t epos = ebase + __popc(ebal & ((1u << lane) - 1u));
                if (boundary && epos < BK_EDGE) p.edge[epos] = rec[u];
            }
        }
        uint32_t incl = cnt;                       // prefix of the counts over the warp, then over the CTA
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t v = __shfl_up_sync(FULL_MASK, incl, d);
            if (lane >= (unsigned)d) incl += v;
        }
        if (lane == 31) s_warp_count[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const uint32_t c = s_warp_count[lane];
            uint32_t wi = c;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t v = __shfl_up_sync(FULL_MASK, wi, d);
                if (lane >= (unsigned)d) wi += v;
            }
            uint32_t base = 0;
            if (lane == 31 && wi) base = atomicAdd(&flags[0], wi);
            base = __shfl_sync(FULL_MASK, base, 31);
            s_warp_count[lane] = base + wi - c;    // first position of the warp's records
        }
        __syncthreads();
        uint32_t pos = s_warp_count[warp] + incl - cnt;
#pragma unroll
        for (int u = 0; u < EM; ++u) {
            if ((keptm >> u) & 1u) {
                if (pos < n_outright) emit(rec[u], pos);
                ++pos;
            }
        }
        __syncthreads();                           // s_warp_count is rewritten by the next round
    }
    if (whole) return;

    // ---- the boundary class: the CTA that finishes last keeps its best `need` records ----
    __threadfence();                               // this thread's appends to the boundary list are out ...
    __syncthreads();                               // ... for every thread of the CTA
    if (tid == 0) s_ok = atomicAdd(&flags[2], 1u) == nctas - 1 ? 1u : 0u;
    __syncthreads();
    if (!s_ok) return;
    __threadfence();
    const uint32_t n_edge = min(__ldcg(&flags[1]), BK_EDGE);
    static_assert(BK_EDGE <= BK_THREADS && BK_EDGE <= RF_BINS && RF_EDGE_CAP >= BK_EDGE, "one thread, one bin and one slot per boundary record");
    // One more level in shared memory: the class's D range cut into BK_EDGE slices, best first.  Slices before the one
    // that holds the need-th best record are kept whole; of that slice -- a record or two as a rule -- the best are
    // found by comparing its records with one another.
    const int sl_shift = cls_w > 10 ? cls_w - 10 : 0;
    const uint64_t mine = tid < n_edge ? __ldcg(&p.edge[tid]) : 0ull;
    const uint32_t slice = tid < n_edge ? BK_EDGE - 1 - (uint32_t)(((dist(mine) - cls_lo) >> sl_shift) & (BK_EDGE - 1)) : 0u;
    sh.hist[tid] = 0;
    if (tid == 0) { sh.fill = 0; sh.n_edge = 0; }
    __syncthreads();
    if (tid < n_edge) atomicAdd(&sh.hist[slice], 1u);
    __syncthreads();
    {
        const uint32_t c = sh.hist[tid];
        const uint32_t incl = block_inclusive_scan(c, sh.warp_sums);
        if (incl - c < need && need <= incl) { s_bin = tid; s_bin_before = incl - c; }
        __syncthreads();
    }
    const uint32_t edge_slice = s_bin, edge_before = s_bin_before;
    uint64_t* list = sh.edge;                      // the records of that slice
    if (tid < n_edge) {
        if (slice < edge_slice) emit(mine, n_outright + atomicAdd(&sh.fill, 1u));
        else if (slice == edge_slice) list[atomicAdd(&sh.n_edge, 1u)] = mine;
    }
    __syncthreads();
    const uint32_t n_list = sh.n_edge;
    if (tid < n_edge && slice == edge_slice) {
        uint32_t rank = 0;
        for (uint32_t j = 0; j < n_list; ++j) rank += list[j] < mine;
        if (rank < need - edge_before) emit(mine, n_outright + edge_before + rank);
    }
}

}  // namespace profk
