// A second filtering pass before the exact fallback (Section 3, "Refinement", sends a row that fails the count check
// to an exact top-k of the full input; the appendix, "Fallback as a Safety Mechanism", counts on that being rare).
// The sample outlives the failure: its keys are kept in the workspace, so a row whose buffer overflowed is filtered
// once more with the threshold of a tighter sample rank, a row with too few candidates with that of a looser one
// (profk_plan_t.r_tight / r_loose) -- one read of the row at streaming speed instead of the two to seven slower ones of
// the exact selection -- and only a row that fails the check again is selected exactly.
// The pieces here run inside the refine kernel's clusters: the selection of a sample rank from the stored keys by
// one CTA, and the filtering scan of a range of tiles.
#pragma once

#include "filter.cuh"
#include "select_sort.cuh"

namespace profk {

// What the refine kernel needs to know about the sample (keys == null: no second pass).
struct SampleInfo {
    const uint32_t* keys;    // rows x S order keys in sample order
    uint32_t S;
    uint64_t seed;
    uint64_t q;              // N / S
    uint32_t rem;            // N % S
    float inv_s;             // 1 / S
    int by_record;           // the threshold is a (value, index) record
    uint32_t r_tight, r_loose;
};

// The rank-th largest of the S sample keys at `keys`, as a record under (key descending, sample number ascending):
// its key and its sample number.  All threads of the CTA call it; uses sh.hist, sh.warp_sums, sh.digit, sh.before, sh.cnt.
template <typename T>
__device__ __noinline__ void kth_sample_record(const uint32_t* keys, uint32_t S, uint32_t rank, SelectShared& sh, uint32_t* key_out,
                                               uint32_t* j_out) {
    constexpr int KB = Elem<T>::KEY_BITS;
    const unsigned tid = threadIdx.x, nthr = blockDim.x;
    uint32_t prefix = 0, need = rank;
    int consumed = 0;
    while (consumed < KB) {
        const int width = KB - consumed < 11 ? KB - consumed : 11;
        const int shift = KB - consumed - width;
        const uint32_t nbins = 1u << width;
        for (uint32_t b = tid; b < nbins; b += nthr) sh.hist[b] = 0;
        __syncthreads();
        for (uint32_t i = tid; i < S; i += nthr) {
            const uint32_t k = __ldcg(&keys[i]);
            if (consumed == 0 || (k >> (KB - consumed)) == prefix) atomicAdd(&sh.hist[(k >> shift) & (nbins - 1)], 1u);
        }
        __syncthreads();
        // the digit of the need-th largest key of the class: bins from the top
        const uint32_t per = (nbins + nthr - 1) / nthr;
        uint32_t sum = 0;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t rb = tid * per + j;
            sum += rb < nbins ? sh.hist[nbins - 1 - rb] : 0;
        }
        uint32_t before = block_scan_any(sum, sh.warp_sums) - sum;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t rb = tid * per + j;
            const uint32_t c = rb < nbins ? sh.hist[nbins - 1 - rb] : 0;
            if (before < need && need <= before + c) { sh.digit = nbins - 1 - rb; sh.before = before; }
            before += c;
        }
        __syncthreads();
        prefix = (prefix << width) | sh.digit;
        need -= sh.before;
        consumed += width;
        __syncthreads();
    }
    // of the samples with exactly this key, the need-th in sample order
    uint32_t seen = 0;
    for (uint32_t base = 0; base < S; base += nthr) {
        const uint32_t i = base + tid;
        const uint32_t flag = i < S && __ldcg(&keys[i]) == prefix;
        const uint32_t in_run = (uint32_t)__syncthreads_count((int)flag);
        const uint32_t incl = block_scan_any(flag, sh.warp_sums);
        if (flag && seen + incl == need) sh.cnt = i;
        seen += in_run;
        if (seen >= need) break;
    }
    __syncthreads();
    *key_out = prefix;
    *j_out = sh.cnt;
    __syncthreads();
}

// The filtering scan over tiles tile_lo + crank, + csize, ... < tile_hi of `row` (a tile is THREADS * 4 vectors), with the
// threshold tau (fp.thr[row] holds its record): every element not below it is appended to the row's buffer through
// fp.counts.  The same fast test and slow path as the filter kernel's.
template <typename T, int THREADS>
__device__ __forceinline__ void refilter_tiles(const FilterParams<T>& fp, uint32_t row, uint64_t tile_lo, uint64_t tile_hi, unsigned crank,
                                               unsigned csize, T tau) {
    using V = typename Elem<T>::vec_t;
    constexpr int VEC = Elem<T>::VEC, UNROLL = 4;
    constexpr uint32_t TILE_VECTORS = THREADS * UNROLL, ALL_INSIDE = (1u << UNROLL) - 1u;
    const RowView<T> rv = row_view(fp.in, fp.N, row);
    bool full = false;                 // this warp has seen the buffer overflow: nothing more to append
    for (uint64_t tile = tile_lo + crank; tile < tile_hi && !full; tile += csize) {
        const uint64_t qbase = tile * TILE_VECTORS;
        V v[UNROLL];
        uint32_t inside_mask;
        if (qbase * VEC >= rv.mis && (qbase + TILE_VECTORS) * VEC <= fp.N + rv.mis) {
            const V* ptr = reinterpret_cast<const V*>(rv.aligned_base) + qbase + threadIdx.x;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) v[u] = ld_stream(ptr + u * THREADS);
            inside_mask = ALL_INSIDE;
        } else {
            inside_mask = 0;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                bool in;
                v[u] = load_row_vector(rv, fp.N, qbase + (uint64_t)u * THREADS + threadIdx.x, &in);
                inside_mask |= in ? 1u << u : 0u;
            }
        }
        bool hit = false;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) hit |= (((inside_mask >> u) & 1u) && vec_any_pass(v[u], tau));
        if (__any_sync(FULL_MASK, hit))
            full = filter_slow_path_direct<T, THREADS, UNROLL, false>(fp, v, inside_mask, row, qbase, rv.mis, tau) != 0xFFFFFFFFu;
    }
}

}  // namespace profk
