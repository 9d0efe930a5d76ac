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
// its key and its sample number.  All threads of the CTA call it (whole warps); uses sh.hist, sh.start, sh.edge,
// sh.warp_sums, sh.digit, sh.before, sh.cnt, sh.fill, sh.n_edge (the last two left zero).
// `lower` is a key with at least `rank` sample keys at or above it, if the caller knows one (the first pass's threshold
// when a tighter rank is wanted), else 0.
// Ranks up to the CTA's thread count -- all that the plans ask for -- are found without a histogram: a key that has
// `rank` keys at or above it bounds the answer from below (the caller's, or the rank-th largest of the threads' own
// maxima after one pass over the keys); the keys at or above the bound, a few times `rank` of them, are collected in
// shared memory and compared with one another.  (A radix select over all keys, the general path below, spends its
// first pass on shared-memory atomics into the handful of bins that the keys of a sample crowd: 94 us for 2^17 keys.)
template <typename T>
__device__ __noinline__ void kth_sample_record(const uint32_t* keys, uint32_t S, uint32_t rank, SelectShared& sh, uint32_t* key_out,
                                               uint32_t* j_out, uint32_t lower = 0) {
    {
        const unsigned tid = threadIdx.x, nthr = blockDim.x;
        constexpr int KU = 8;                    // loads in flight per thread
        if (rank <= nthr && nthr <= RF_BINS) {
            if (lower == 0) {
                // the threads' maxima, and the rank-th largest of them (ties by thread number)
                uint32_t mx = 0;
                for (uint32_t i0 = 0; i0 < S; i0 += KU * nthr) {
                    uint32_t kk[KU];
#pragma unroll
                    for (int u = 0; u < KU; ++u) {
                        const uint32_t i = i0 + u * nthr + tid;
                        kk[u] = i < S ? __ldcg(&keys[i]) : 0u;
                    }
#pragma unroll
                    for (int u = 0; u < KU; ++u) mx = kk[u] > mx ? kk[u] : mx;
                }
                sh.start[tid] = mx;
                __syncthreads();
                uint32_t above = 0;
                for (uint32_t j = 0; j < nthr; ++j) {
                    const uint32_t o = sh.start[j];
                    above += (o > mx) || (o == mx && j < tid);
                }
                if (above == rank - 1) sh.digit = mx;
                __syncthreads();
                lower = sh.digit;
                __syncthreads();
            }
            // collect the records at or above the bound: (key << 32) | ~(sample number), larger = better
            if (tid == 0) sh.fill = 0;
            __syncthreads();
            for (uint32_t i0 = 0; i0 < S; i0 += KU * nthr) {
                uint32_t kk[KU];
#pragma unroll
                for (int u = 0; u < KU; ++u) {
                    const uint32_t i = i0 + u * nthr + tid;
                    kk[u] = i < S ? __ldcg(&keys[i]) : 0u;
                }
#pragma unroll
                for (int u = 0; u < KU; ++u) {
                    const uint32_t i = i0 + u * nthr + tid;
                    if (i < S && kk[u] >= lower) {
                        const uint32_t slot = atomicAdd(&sh.fill, 1u);
                        if (slot < RF_EDGE_CAP) sh.edge[slot] = ((uint64_t)kk[u] << 32) | (uint64_t)(0xFFFFFFFFu - i);
                    }
                }
            }
            __syncthreads();
            const uint32_t ncand = sh.fill;
            __syncthreads();
            if (tid == 0) sh.fill = 0;
            if (ncand <= RF_EDGE_CAP) {
                for (uint32_t c = tid; c < ncand; c += nthr) {
                    const uint64_t mine = sh.edge[c];
                    uint32_t above = 0;
                    for (uint32_t j = 0; j < ncand; ++j) above += sh.edge[j] > mine;
                    if (above == rank - 1) { sh.digit = (uint32_t)(mine >> 32); sh.cnt = 0xFFFFFFFFu - (uint32_t)mine; }
                }
                __syncthreads();
                *key_out = sh.digit;
                *j_out = sh.cnt;
                __syncthreads();
                return;
            }
            __syncthreads();                     // more candidates than the list holds (a sample of equal keys): the general path
        }
    }
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
        // (whole warps together: the keys of a sample crowd a few bins of the first pass, and the lanes that meet in a
        // bin add once for all of them -- one shared-memory atomic per key took a 2^17-key sample 100 us a pass)
        // (eight loads in flight per thread: one at a time, a 2^17-key sample took 128 round trips to L2 a pass)
        constexpr int KU = 8;
        for (uint32_t i0 = 0; i0 < S; i0 += KU * nthr) {
            uint32_t kk[KU];
#pragma unroll
            for (int u = 0; u < KU; ++u) {
                const uint32_t i = i0 + u * nthr + tid;
                kk[u] = i < S ? __ldcg(&keys[i]) : 0u;
            }
#pragma unroll
            for (int u = 0; u < KU; ++u) {
                const uint32_t i = i0 + u * nthr + tid;
                const uint32_t k = kk[u];
                const bool in_class = i < S && (consumed == 0 || (k >> (KB - consumed)) == prefix);
                const uint32_t digit = in_class ? (k >> shift) & (nbins - 1) : 0xFFFFFFFFu;
                const unsigned peers = __match_any_sync(FULL_MASK, digit);
                if (in_class && lane_id() == (unsigned)(__ffs(peers) - 1)) atomicAdd(&sh.hist[digit], (uint32_t)__popc(peers));
            }
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
    // Of the samples with exactly this key, the need-th in sample order.  Sample i is looked at in round i / nthr by
    // thread i % nthr: every warp votes on its 32 samples of a round and notes the count; the counts, in (round, warp)
    // order, are scanned once, and the warp whose vote holds the need-th match votes again to find the lane.  (Up to
    // RF_BINS counts at a time: the rounds are taken in groups.)
    const unsigned lane = lane_id(), warp = tid >> 5, nwarps = nthr >> 5;
    const uint32_t rounds = (S + nthr - 1) / nthr, rounds_per_group = RF_BINS / nwarps;
    uint32_t seen = 0;
    for (uint32_t g0 = 0; g0 < rounds; g0 += rounds_per_group) {
        const uint32_t g1 = g0 + rounds_per_group < rounds ? g0 + rounds_per_group : rounds;
        for (uint32_t r0 = g0; r0 < g1; r0 += 8) {                        // (eight loads in flight)
            uint32_t kk[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t i = (r0 + u) * nthr + tid;
                kk[u] = (r0 + u < g1 && i < S) ? __ldcg(&keys[i]) : ~prefix;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t i = (r0 + u) * nthr + tid;
                const unsigned bal = __ballot_sync(FULL_MASK, r0 + u < g1 && i < S && kk[u] == prefix);
                if (lane == 0 && r0 + u < g1) sh.hist[(r0 + u - g0) * nwarps + warp] = (uint32_t)__popc(bal);
            }
        }
        __syncthreads();
        const uint32_t ncounts = (g1 - g0) * nwarps, per = (ncounts + nthr - 1) / nthr;
        uint32_t sum = 0;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t c = tid * per + j;
            sum += c < ncounts ? sh.hist[c] : 0u;
        }
        uint32_t before = seen + block_scan_any(sum, sh.warp_sums) - sum;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t c = tid * per + j;
            const uint32_t cnt = c < ncounts ? sh.hist[c] : 0u;
            if (before < need && need <= before + cnt) { sh.digit = c; sh.before = before; }
            before += cnt;
        }
        if (tid == nthr - 1) sh.n_edge = before;             // matches up to the end of this group
        __syncthreads();
        const uint32_t upto = sh.n_edge;
        if (need <= upto) {
            const uint32_t c = sh.digit, r = g0 + c / nwarps, off = need - sh.before;      // the off-th match of that vote
            if (warp == c % nwarps) {
                const uint32_t i = r * nthr + tid;
                const bool flag = i < S && __ldcg(&keys[i]) == prefix;
                const unsigned bal = __ballot_sync(FULL_MASK, flag);
                if (flag && (uint32_t)__popc(bal & ((2u << lane) - 1u)) == off) sh.cnt = i;
            }
            break;
        }
        seen = upto;
        __syncthreads();                                     // the counts are rewritten by the next group
    }
    __syncthreads();
    *key_out = prefix;
    *j_out = sh.cnt;
    __syncthreads();
    if (tid == 0) sh.n_edge = 0;                             // as the callers' kernels set it at their start
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
