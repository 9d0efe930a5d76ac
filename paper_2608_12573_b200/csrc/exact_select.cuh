// Exact replacement of a row that failed the count check (Section 3, "Refinement": with fewer
// than k candidates, or a buffer that overflowed, the row's answer is an exact top-k of the full
// input), run inside the refine kernel by the thread-block clusters that own the row.
//
// The row's elements are viewed as 64-bit candidate records (value key, then index), so the
// answer is "the k smallest records".  A most-significant-digit radix select finds the k-th
// smallest record: each pass histograms one digit (11 bits) of the records that share the
// digits chosen so far -- first the bits of the key, then, if many records have exactly the
// k-th key, the bits of the index -- every CTA over its own tiles; the CTAs' histograms are
// summed through distributed shared memory, and every CTA picks the digit for itself.  Once
// the first digit of the index is chosen, the records still in play lie in one contiguous range
// of the row, and later passes read only that range.  The passes stop as soon as the class that
// holds the k-th record is small (XS_EDGE records; for values without heavy ties that is after
// the first pass), and a last pass appends every record up to the end of that class -- the k
// smallest and a few more -- to a scratch area.
//
// A long row is cut into segments of whole tiles, one cluster per segment, so that all SMs read
// it; each cluster selects from its own segment, and whichever cluster finishes last (a ticket
// taken after its records are fenced) selects the k smallest of all segments' records, orders
// them and writes the row's output (refine.cuh).
//
// Only hardware cluster barriers are used, and no cluster waits for another: nothing here
// depends on CTAs being co-resident.
#pragma once

#include <cooperative_groups.h>

#include "rowscan.cuh"
#include "select_sort.cuh"

namespace profk {

constexpr int XS_BITS = 11;                 // digit width
constexpr uint32_t XS_BINS = 1u << XS_BITS;
constexpr int XS_UNROLL = 4;                // 16-byte vectors a thread has in flight
constexpr uint32_t XS_EDGE = 2048;          // a class of the k-th record this small is handed on whole
static_assert(XS_BINS <= RF_BINS, "the digit histogram lives in SelectShared::hist");

// Visits the vectors of tiles [tile_lo, tile_hi) of the row that fall to CTA `crank` of `csize`
// (tiles crank, crank + csize, ...): f(keys, i0, valid) is called by all 32 lanes of each warp
// together, with the keys of one vector's elements, the row index i0 of its first element (as a
// 32-bit word: it wraps for the elements before the row's start, which are not valid) and a mask
// whose bit l says whether element l lies inside the row.  A tile is blockDim.x * XS_UNROLL
// consecutive vectors.
template <typename T, typename F>
__device__ __forceinline__ void xs_for_each(const RowView<T>& rv, uint64_t N, uint64_t tile_lo, uint64_t tile_hi,
                                            unsigned crank, unsigned csize, F&& f) {
    using V = typename Elem<T>::vec_t;
    constexpr int VEC = Elem<T>::VEC;
    constexpr uint32_t FULL = (1u << VEC) - 1u;
    const uint64_t tile_vectors = (uint64_t)blockDim.x * XS_UNROLL;
    for (uint64_t tile = tile_lo + crank; tile < tile_hi; tile += csize) {
        V v[XS_UNROLL];
        bool inside[XS_UNROLL];
        const uint64_t q0 = tile * tile_vectors + threadIdx.x;
#pragma unroll
        for (int u = 0; u < XS_UNROLL; ++u) v[u] = load_row_vector(rv, N, q0 + (uint64_t)u * blockDim.x, &inside[u]);
#pragma unroll
        for (int u = 0; u < XS_UNROLL; ++u) {
            const int64_t i0 = (int64_t)((q0 + (uint64_t)u * blockDim.x) * VEC) - (int64_t)rv.mis;
            uint32_t valid = 0;
            if (inside[u]) {
                valid = FULL;
                if (i0 < 0 || i0 + VEC > (int64_t)N) {
                    valid = 0;
#pragma unroll
                    for (int l = 0; l < VEC; ++l)
                        if (i0 + l >= 0 && i0 + l < (int64_t)N) valid |= 1u << l;
                }
            }
            uint32_t keys[VEC];
#pragma unroll
            for (int l = 0; l < VEC; ++l) keys[l] = Elem<T>::key(vec_elem(v[u], l));
            f(keys, (uint32_t)i0, valid);
        }
    }
}

// Number of elements of the row that lie in tiles [tile_lo, tile_hi).
__device__ __forceinline__ uint64_t xs_elements_in_tiles(uint64_t N, uint32_t mis, uint64_t tile_elems, uint64_t tile_lo,
                                                         uint64_t tile_hi) {
    const uint64_t v_lo = tile_lo * tile_elems, v_hi = tile_hi * tile_elems;      // virtual coordinates: index + mis
    const uint64_t i_lo = v_lo > mis ? v_lo - mis : 0;
    const uint64_t i_hi = v_hi > mis ? (v_hi - mis < N ? v_hi - mis : N) : 0;
    return i_hi > i_lo ? i_hi - i_lo : 0;
}

// Writes a superset of the k smallest records (all records, if there are at most k) among the
// elements of row `row` that lie in tiles [seg_lo, seg_hi) to dst[0 .. k + edge), in any order: at most
// k + edge - 1 records (exactly the k smallest when edge is 0), the unused slots filled with all-ones (no
// record has that value).
// Returns after a cluster barrier: on return the records are in global memory.
// Called by all threads of all CTAs of the cluster (CTA `crank` of `csize`); *collect is a counter
// for this call alone.
//
// use_tau says that the row's buffer overflowed: at least k elements of the row are >= tau, so only
// those matter, and the flood is most likely made of copies of tau itself.  One pass then counts the
// elements above tau and histograms the index digit of the elements equal to tau; when the k-th
// record turns out to be one of the latter, its key is known and its first index digit chosen after
// that single pass.
//
// Kept out of line: the refine kernel's register budget is set by its common path (it has to fit beside
// the last CTAs of the filter kernel on an SM); this rare path takes its spills inside the call.
template <typename T>
__device__ __noinline__ void exact_select_cluster(const T* in, uint64_t N, uint64_t row, uint32_t k, uint64_t seg_lo,
                                                  uint64_t seg_hi, uint64_t* dst, uint32_t* collect, SelectShared& sh,
                                                  unsigned csize, unsigned crank, bool use_tau, uint32_t tau_key,
                                                  uint32_t edge = XS_EDGE) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    constexpr int VEC = Elem<T>::VEC;
    const unsigned tid = threadIdx.x, nthr = blockDim.x, lane = lane_id();
    // A cluster of one is launched as a plain CTA: its barrier is the CTA's own.
    auto sync_all = [&]() { if (csize > 1) cluster.sync(); else __syncthreads(); };
    const RowView<T> rv = row_view(in, N, row);
    const uint64_t tile_elems = (uint64_t)nthr * XS_UNROLL * VEC;
    const int idx_bits = N > 1 ? 64 - __clzll((long long)(N - 1)) : 1;      // bits an index occupies
    const uint64_t n_seg = xs_elements_in_tiles(N, rv.mis, tile_elems, seg_lo, seg_hi);
    const uint32_t slots = k + edge;
    if (crank == 0 && tid == 0) *collect = 0;          // ordered before the appends by the barriers below
    for (uint32_t i = crank * nthr + tid; i < slots; i += csize * nthr) dst[i] = ~0ull;      // so are these

    // The k-th smallest record is found digit by digit: first the bits of nk = ~key (ascending nk is
    // descending value), then, among the records with exactly that key, the bits of the index.  All of
    // it is 32-bit arithmetic; the 64-bit record appears only in the last pass.
    constexpr int KB = Elem<T>::KEY_BITS;
    constexpr uint32_t KMASK = KB == 32 ? 0xFFFFFFFFu : ((1u << (KB & 31)) - 1u);
    bool key_phase = true;
    int lo_sel = KB;                        // bits [lo_sel, top) of the current phase's word are chosen ...
    uint32_t chosen = 0;                    // ... and equal `chosen` (right-aligned)
    bool none_chosen = true;
    uint32_t kth_nk = 0;                    // nk of the k-th record, once all its bits are chosen
    uint32_t need = k;                      // rank (from the smallest record) inside the chosen class
    uint64_t tile_lo = seg_lo, tile_hi = seg_hi;
    uint64_t limit = ~0ull;                 // records <= limit are handed on; a segment of at most k elements goes whole
    bool found = n_seg <= (uint64_t)k;      // true once `limit` is final

    // Histogram of one pass.  Equal values come in long runs of whole warps of vectors with one digit:
    // those are counted in registers (the same in every lane).  Otherwise, element by element: the lanes
    // with a digit usually share it (index digits always do), which a vote settles; only a real mix
    // needs a match across the warp.
    uint32_t run_digit = 0xFFFFFFFFu, run_count = 0;
    auto run_add = [&](uint32_t d, uint32_t n) {
        if (d != run_digit) {
            if (lane == 0 && run_count) atomicAdd(&sh.hist[run_digit], run_count);
            run_digit = d;
            run_count = 0;
        }
        run_count += n;
    };
    auto run_flush = [&]() {
        if (lane == 0 && run_count) atomicAdd(&sh.hist[run_digit], run_count);
        run_digit = 0xFFFFFFFFu;
        run_count = 0;
    };
    auto count = [&](const uint32_t (&digit)[VEC]) {
        bool same = true;
#pragma unroll
        for (int l = 1; l < VEC; ++l) same = same && digit[l] == digit[0];
        const uint32_t d0 = __shfl_sync(FULL_MASK, digit[0], 0);
        if (__all_sync(FULL_MASK, same && digit[0] == d0)) {
            if (d0 != 0xFFFFFFFFu) run_add(d0, 32u * VEC);          // all-ones: a warp with nothing in the class
            return;
        }
#pragma unroll
        for (int l = 0; l < VEC; ++l) {
            const bool has = digit[l] != 0xFFFFFFFFu;
            const unsigned m = __ballot_sync(FULL_MASK, has);
            if (m == 0) continue;
            const uint32_t d = __shfl_sync(FULL_MASK, digit[l], __ffs(m) - 1);
            if (__all_sync(FULL_MASK, !has || digit[l] == d)) {
                run_add(d, (uint32_t)__popc(m));
            } else {
                const unsigned peers = __match_any_sync(FULL_MASK, digit[l]);
                if (has && lane == (unsigned)(__ffs(peers) - 1)) atomicAdd(&sh.hist[digit[l]], (uint32_t)__popc(peers));
            }
        }
    };
    // Sums the CTAs' histograms (complete on entry: call after sync_all) and finds the bin that holds the
    // need-th smallest record of the class: sh.digit, sh.before (records in lower bins), sh.cnt (in the
    // bin), sh.n_edge (in all bins).  Every CTA computes the same.
    auto merge_and_pick = [&](uint32_t nbins) {
        for (uint32_t bin = tid; bin < nbins; bin += nthr) {
            uint32_t sum = 0;
            if (csize > 1) {
                for (unsigned c = 0; c < csize; ++c) sum += cluster.map_shared_rank(sh.hist, c)[bin];
            } else {
                sum = sh.hist[bin];
            }
            sh.start[bin] = sum;
        }
        __syncthreads();
        const uint32_t per = (XS_BINS + nthr - 1) / nthr;
        uint32_t sum = 0;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t bin = tid * per + j;
            sum += bin < nbins ? sh.start[bin] : 0;
        }
        uint32_t before = block_scan_any(sum, sh.warp_sums) - sum;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t bin = tid * per + j;
            const uint32_t c = bin < nbins ? sh.start[bin] : 0;
            if (before < need && need <= before + c) { sh.digit = bin; sh.before = before; sh.cnt = c; }
            before += c;
        }
        if (tid == nthr - 1) sh.n_edge = before;
        __syncthreads();
    };
    // After a pass of the index phase the class is one contiguous range of indices.
    auto narrow_to_index_range = [&](int lo) {
        const uint64_t i_lo = (uint64_t)chosen << lo;
        const uint64_t i_end = i_lo + (1ull << lo) < N ? i_lo + (1ull << lo) : N;
        const uint64_t t_lo = (i_lo + rv.mis) / tile_elems, t_hi = (i_end - 1 + rv.mis) / tile_elems + 1;
        tile_lo = t_lo > seg_lo ? t_lo : seg_lo;
        tile_hi = t_hi < seg_hi ? t_hi : seg_hi;
    };
    auto limit_of_class = [&](int lo) {     // the largest record of the chosen class
        const uint32_t last = (uint32_t)((((uint64_t)chosen + 1ull) << lo) - 1ull);
        return key_phase ? ((uint64_t)(~KMASK | last) << 32) | 0xFFFFFFFFull : ((uint64_t)(~KMASK | kth_nk) << 32) | last;
    };

    bool synced = false;                    // a cluster barrier has ordered the resets above before the appends
    int hi = KB;
    if (use_tau && !found) {
        // ---- the buffer overflowed: count the elements above tau, histogram the first index digit of the
        //      elements equal to tau ----
        const uint32_t tau_nk = ~tau_key & KMASK;
        const int lo = idx_bits - XS_BITS > 0 ? idx_bits - XS_BITS : 0;
        const uint32_t nbins = 1u << (idx_bits - lo);
        for (uint32_t i = tid; i < nbins; i += nthr) sh.hist[i] = 0;
        if (tid == 0) sh.fill = 0;
        __syncthreads();
        uint32_t above = 0;
        xs_for_each(rv, N, seg_lo, seg_hi, crank, csize, [&](const uint32_t (&key)[VEC], uint32_t i0, uint32_t valid) {
            uint32_t digit[VEC];
#pragma unroll
            for (int l = 0; l < VEC; ++l) {
                const uint32_t nk = ~key[l] & KMASK;
                const bool ok = (valid >> l) & 1u;
                above += ok && nk < tau_nk;
                digit[l] = ok && nk == tau_nk ? (i0 + l) >> lo : 0xFFFFFFFFu;
            }
            count(digit);
        });
        run_flush();
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) above += __shfl_xor_sync(FULL_MASK, above, d);
        if (lane == 0 && above) atomicAdd(&sh.fill, above);
        sync_all();
        synced = true;
        uint32_t above_all = 0;
        if (csize > 1) {
            for (unsigned c = 0; c < csize; ++c) above_all += *cluster.map_shared_rank(&sh.fill, c);
        } else {
            above_all = sh.fill;
        }
        if (above_all < k) {                // the k-th record is not above tau: at best it equals tau
            need = k - above_all;
            merge_and_pick(nbins);
            const uint32_t equal_all = sh.n_edge, in_bin = sh.cnt, digit = sh.digit, before = sh.before;
            sync_all();                     // peers have read this CTA's counters
            key_phase = false;
            kth_nk = tau_nk;
            if (equal_all < need) {         // fewer than k elements >= tau in this segment: all of them go on
                limit = ((uint64_t)(~KMASK | tau_nk) << 32) | 0xFFFFFFFFull;
                found = true;
            } else {
                chosen = digit;
                none_chosen = false;
                lo_sel = lo;
                need -= before;
                if (in_bin - need < edge || in_bin == need || lo == 0) {
                    limit = limit_of_class(lo);
                    found = true;
                } else {
                    narrow_to_index_range(lo);
                    hi = lo;
                }
            }
        } else {
            sync_all();                     // peers have read this CTA's counters; the general passes start over
        }
    }

    while (!found) {
        const int lo = hi - XS_BITS > 0 ? hi - XS_BITS : 0;
        const uint32_t nbins = 1u << (hi - lo);
        for (uint32_t i = tid; i < nbins; i += nthr) sh.hist[i] = 0;
        __syncthreads();
        if (key_phase) {
            xs_for_each(rv, N, tile_lo, tile_hi, crank, csize, [&](const uint32_t (&key)[VEC], uint32_t, uint32_t valid) {
                uint32_t digit[VEC];
#pragma unroll
                for (int l = 0; l < VEC; ++l) {
                    const uint32_t nk = ~key[l] & KMASK;
                    const bool in_class = ((valid >> l) & 1u) && (none_chosen || (nk >> lo_sel) == chosen);
                    digit[l] = in_class ? (nk >> lo) & (nbins - 1) : 0xFFFFFFFFu;
                }
                count(digit);
            });
        } else {
            xs_for_each(rv, N, tile_lo, tile_hi, crank, csize, [&](const uint32_t (&key)[VEC], uint32_t i0, uint32_t valid) {
                uint32_t digit[VEC];
#pragma unroll
                for (int l = 0; l < VEC; ++l) {
                    const uint32_t idx = i0 + l;
                    const bool in_class = ((valid >> l) & 1u) && (~key[l] & KMASK) == kth_nk && (none_chosen || (idx >> lo_sel) == chosen);
                    digit[l] = in_class ? (idx >> lo) & (nbins - 1) : 0xFFFFFFFFu;
                }
                count(digit);
            });
        }
        run_flush();
        sync_all();                         // every CTA's histogram of this pass is complete
        synced = true;
        merge_and_pick(nbins);
        chosen = (none_chosen ? 0u : chosen << (lo_sel - lo)) | sh.digit;
        none_chosen = false;
        lo_sel = lo;
        need -= sh.before;
        const uint32_t in_bin = sh.cnt;
        sync_all();                         // peers have read this CTA's histogram; sh.digit may be rewritten

        // Stop when at most XS_EDGE - 1 records beyond the k-th would be taken along.
        if (in_bin - need < edge || in_bin == need || (!key_phase && lo == 0)) {
            limit = limit_of_class(lo);
            found = true;
        } else if (key_phase && lo == 0) {  // the key is known and widely shared: go on with the index
            key_phase = false;
            kth_nk = chosen;
            none_chosen = true;
            hi = idx_bits;                  // index bits above idx_bits are zero in every record
        } else {
            if (!key_phase) narrow_to_index_range(lo);
            hi = lo;
        }
    }
    if (!synced) sync_all();

    // ---- append the records <= limit ----
    const unsigned lt_mask = (1u << lane) - 1u;
    xs_for_each(rv, N, seg_lo, seg_hi, crank, csize, [&](const uint32_t (&key)[VEC], uint32_t i0, uint32_t valid) {
        uint32_t take = 0;
#pragma unroll
        for (int l = 0; l < VEC; ++l)
            if (((valid >> l) & 1u) && make_record(key[l], i0 + l) <= limit) take |= 1u << l;
        if (!__any_sync(FULL_MASK, take != 0)) return;
#pragma unroll
        for (int l = 0; l < VEC; ++l) {
            const bool mine = (take >> l) & 1u;
            const unsigned bal = __ballot_sync(FULL_MASK, mine);
            if (bal) {
                unsigned base = 0;
                if (lane == 0) base = atomicAdd(collect, (uint32_t)__popc(bal));
                base = __shfl_sync(FULL_MASK, base, 0);
                const unsigned pos = base + __popc(bal & lt_mask);
                if (mine && pos < slots) dst[pos] = make_record(key[l], i0 + l);
            }
        }
    });
    __threadfence();
    sync_all();
}

}  // namespace profk
