// Stage 4 for large selections (k beyond what one CTA orders in shared memory; the flattened
// BatchTopK case of Section 5, "Application", selects K = B k = 131,072 values): the count
// check, then the k smallest candidate records in ascending order -- which is "value
// descending, index ascending" -- by the whole grid, launched cooperatively (one CTA per SM, all
// co-resident), one row after the other.
//
// Main path: the records are counted in the bins of bins.cuh (262144 bins in global memory on a
// logarithmic scale of the distance from the threshold record, 512 coarse bins over them; the
// filter kernel makes this histogram itself where it can), a scan over the coarse and then the
// fine bins turns the counts into first positions, the records are scattered into a second
// buffer grouped by bin, and every record of a bin that reaches into the first k positions
// ranks itself inside its bin -- a handful of comparisons -- to find its place in the output.
// Two grid barriers when the histogram comes with the buffer, three or four otherwise.
// Reserve path, taken when a bin is too crowded for that (very many equal records far from the threshold):
// a bitonic network over P = 2^j records in the row's buffer, exchanges below one tile
// (16384 records = 128 KB) in shared memory, the longer ones on the buffer in global memory.
// The steps of both paths are separated by grid barriers whose waits are bounded: a wait that gives
// up sets the workspace's error flag and the kernel returns.
#pragma once

#include "fallback.cuh"
#include "grid_barrier.cuh"
#include "refine.cuh"

namespace profk {

constexpr uint32_t BT_TILE = 16384;          // records per shared-memory tile
constexpr int BT_THREADS = 1024;
constexpr uint32_t LG_WAIT_LIMIT = 1u << 22;  // polls of the "all CTAs have zeroed their share of the bins" counter
constexpr uint32_t LG_CROWDED = 1024;        // a bin this full (among those that matter) sends the row to the reserve path

template <typename T> struct LargeParams {
    RowCtl* ctl;
    WsHeader* header;
    uint64_t* buf;           // row r: records at buf + r * 2 * row_stride, then row_stride records of scratch;
    uint64_t row_stride;     //        row_stride is a power of two >= capacity, >= BT_TILE
    uint32_t* bins;          // rows x BIN_ROW_WORDS words: bin counts / positions, then flags
    unsigned long long* slots;   // 2 words per CTA of the grid, then one per CTA: per-CTA minima / maxima and scan totals
    uint32_t groups;         // CTA groups the grid is cut into (<= WS_GROUPS; gridDim.x is a multiple of it)
    uint32_t parts;          // 1, or FILTER_PARTS: the filter appended to that many parts of the row's buffer (first phase only)
    uint32_t part_cap;       // records per part
    const uint32_t* part_counts;   // row r, part j: part_counts[(r * 8 + j) * 64]
    uint64_t rows;
    uint32_t capacity;
    uint32_t k;
    uint32_t k_accept;
    int phase;               // 0 = count check, then sort the rows that pass; 1 = sort the rows the exact selection repaired
    T* out_vals;             // rows x k
    int64_t* out_idx;        // rows x k
    int use_pdl;
    // A single row (fused == 1; one group of CTAs): a row that fails the count check, or a row in direct mode, is replaced
    // inside this kernel by the grid-wide exact selection and ordered right away -- one launch instead of three.
    // A few rows (fused == 2; phase 0, no direct mode): the groups order the rows that pass side by side; then the whole
    // grid meets at one barrier and, if some row failed, takes the failed rows one after the other as a single group --
    // second filtering pass or exact selection, then the ordering -- again in this one launch.
    int fused;
    FallbackParams<T> fb;    // what that selection needs (fused != 0 only)
    int idx_bits;            // bits an index of the row occupies (1 .. 32)
    int hist_ready;          // 1 = (fused) the filter kernel counted the records it appended in the row's bins; the rest of
                             // the row's BIN_ROW_WORDS words are zero.  0 = nobody has touched them
};

// All exchanges of the network with stride < BT_TILE, for one tile held in shared memory.
// `base` is the tile's first global position (directions depend on the global position);
// sizes run from size_lo to size_hi, each from stride min(size/2, BT_TILE/2) down to 1.
__device__ __forceinline__ void bitonic_tile_steps(uint64_t* tile, uint64_t base, uint64_t size_lo, uint64_t size_hi) {
    for (uint64_t size = size_lo; size <= size_hi; size <<= 1) {
        uint32_t stride = size / 2 < BT_TILE / 2 ? (uint32_t)(size / 2) : BT_TILE / 2;
        for (; stride > 0; stride >>= 1) {
            for (uint32_t i = threadIdx.x; i < BT_TILE / 2; i += BT_THREADS) {
                const uint32_t lo = 2 * i - (i & (stride - 1));
                const uint32_t hi = lo + stride;
                const bool ascending = ((base + lo) & size) == 0;
                const uint64_t x = tile[lo], y = tile[hi];
                if ((x > y) == ascending) { tile[lo] = y; tile[hi] = x; }
            }
            __syncthreads();
        }
    }
}

// Shared-memory state of the scan over the bins (refine_large_kernel).
struct ScanShared {
    uint32_t coarse[BIN_COARSE];     // records in the coarse bins before each one
    uint32_t ccount[BIN_COARSE];     // records in each coarse bin
    uint16_t listed[BIN_COARSE];     // the coarse bins that matter, in order
    uint32_t nlisted;                // how many are listed
    uint32_t scattered;              // positions the scatter fills: [0, scattered)
};

// The scan of one row's bins by one group of `nctas` CTAs (this one: `cta`); all BT_THREADS threads call it.  Every CTA
// sums the coarse bins before each of its own and lists the coarse bins that matter -- not empty, and starting below
// position kk: the fine bins of the others are never looked at, and their records stay where they are.  CTA c turns
// the counts of the fine bins of the c-th, (c + nctas)-th, ... listed coarse bin into first positions (bins[b]) and
// flags a crowded bin among them.  On return the lists are in shared memory for every thread of the block (the loop's
// block-wide scans come after the last write to them).
__device__ __noinline__ void scan_bins(uint32_t* bins, const uint32_t* coarse, uint32_t* flags, ScanShared& ss, uint32_t* s_warp,
                                       unsigned cta, unsigned nctas, uint32_t kk) {
    const unsigned tid = threadIdx.x;
    {
        const uint32_t c = tid < BIN_COARSE ? __ldcg(&coarse[tid]) : 0u;
        const uint32_t incl = block_inclusive_scan(c, s_warp);
        if (tid < BIN_COARSE) { ss.coarse[tid] = incl - c; ss.ccount[tid] = c; }
        const bool listed = c != 0 && incl - c < kk;
        if (tid == 0) ss.scattered = 0;
        __syncthreads();
        const uint32_t at = block_inclusive_scan(listed ? 1u : 0u, s_warp);
        if (listed) { ss.listed[at - 1] = (uint16_t)tid; atomicMax(&ss.scattered, incl); }   // (incl: the end of the last listed one)
        if (tid == BT_THREADS - 1) ss.nlisted = at;
        __syncthreads();
    }
    // (two coarse bins a round, one per half of the CTA; the counts of the first two rounds are loaded ahead)
    constexpr int SEG_PER_ROUND = BT_THREADS / BIN_PER_COARSE;
    constexpr int ROUNDS_AHEAD = 2;
    static_assert(SEG_PER_ROUND == 2, "a round of the scan covers two coarse bins");
    const uint32_t nlisted = ss.nlisted;
    const uint32_t half = tid / BIN_PER_COARSE, fine = tid % BIN_PER_COARSE;
    uint32_t ahead[ROUNDS_AHEAD];
#pragma unroll
    for (int a = 0; a < ROUNDS_AHEAD; ++a) {
        const uint32_t li = cta + (a * SEG_PER_ROUND + half) * nctas;
        ahead[a] = li < nlisted ? __ldcg(&bins[(uint32_t)ss.listed[li] * BIN_PER_COARSE + fine]) : 0u;
    }
    int turn = 0;
    for (uint32_t li0 = cta; li0 < nlisted; li0 += SEG_PER_ROUND * nctas, ++turn) {
        const uint32_t li = li0 + half * nctas;
        const bool mine = li < nlisted;
        const uint32_t seg = mine ? ss.listed[li] : 0u;
        const uint32_t b = seg * BIN_PER_COARSE + fine;
        uint32_t c = 0;
        if (turn < ROUNDS_AHEAD) {
#pragma unroll
            for (int a = 0; a < ROUNDS_AHEAD; ++a)
                if (a == turn) c = ahead[a];
        } else if (mine) {
            c = __ldcg(&bins[b]);
        }
        __syncthreads();                                             // s_warp of the round before
        // records of this round's first coarse bin: they precede the second half's bins in the block-wide scan
        const uint32_t first_total = ss.ccount[ss.listed[li0]];
        const uint32_t excl = block_inclusive_scan(c, s_warp) - c;
        if (mine) {
            const uint32_t before = ss.coarse[seg] + excl - (half ? first_total : 0u);
            if (before < kk && c > LG_CROWDED) atomicOr(&flags[0], 1u);
            bins[b] = before;                                        // first position; the scatter advances it to the end
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(BT_THREADS, 1) refine_large_kernel(const LargeParams<T> p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* tile = reinterpret_cast<uint64_t*>(smem_raw);          // BT_TILE records
    __shared__ unsigned long long s_max[32];
    __shared__ uint32_t s_warp[32];
    __shared__ ScanShared ss;
    uint32_t* const s_coarse = ss.coarse;
    static_assert(BIN_COARSE <= BT_THREADS && BIN_PER_COARSE <= BT_THREADS, "one thread per coarse bin, then per fine bin of one coarse bin");

    // The grid works as p.groups groups of CTAs (one for a single row); a group takes rows group, group + groups, ...
    // one after the other, all its CTAs on one row, with a barrier of its own.
    // (not constants: the repair round of fused == 2 regroups the grid into one group)
    unsigned ngroups = p.groups, nctas = gridDim.x / ngroups, group = blockIdx.x / nctas, cta = blockIdx.x % nctas;
    const unsigned tid = threadIdx.x;
    uint64_t gid = (uint64_t)cta * BT_THREADS + tid;                 // thread index inside the group
    uint64_t gthreads = (uint64_t)nctas * BT_THREADS;
    unsigned long long* slot_max = p.slots + gridDim.x + group * nctas;
    uint32_t* bar_count = &p.header->group_bar[group][0];
    auto barrier = [&]() { return cta_group_barrier(bar_count, &p.header->error, nctas); };

    // A single row whose filter did not count: the bins are cleared here, before the wait for the filter kernel, and each
    // CTA reports in through the header's `done` word (zeroed by the call's first kernel, long finished).
    bool clean_bins = p.fused == 1 && !p.hist_ready;
    if (clean_bins) {
        for (uint64_t b = gid; b < BIN_ROW_WORDS; b += gthreads) p.bins[b] = 0;
        __threadfence();
        __syncthreads();
        if (tid == 0) atomicAdd(&p.header->done, 1u);
    }
    pdl_launch_dependents();
    if (p.use_pdl) pdl_wait();

    for (int round = 0; round < 2; ++round) {
    if (round == 1) {
        // ---- fused == 2: the groups are through with the rows that passed; the whole grid, as one group, takes the rest ----
        if (p.fused != 2) break;
        if (!grid_barrier(p.header)) return;
        if (__ldcg(&p.header->n_failed) == 0) break;
        ngroups = 1; nctas = gridDim.x; group = 0; cta = blockIdx.x;
        gid = (uint64_t)cta * BT_THREADS + tid;
        gthreads = (uint64_t)nctas * BT_THREADS;
        slot_max = p.slots + gridDim.x;
        bar_count = &p.header->bar_count;          // (the counter of grid_barrier: the same members from here on)
    }
    for (uint64_t row = group; row < p.rows; row += ngroups) {
        // ---- is this row for this launch?  (the decision is the same in every CTA) ----
        const RowCtl ctl = p.ctl[row];
        uint32_t n;
        uint32_t nparts = 1, pcount[FILTER_PARTS] = {};      // the records are pcount[j] at G + j * part_cap
        uint32_t tau_key = Elem<T>::key(Elem<T>::from_bits(ctl.tau_bits));
        bool from_filter = false;        // the buffer is what a filtering pass with threshold tau_key left
        bool status_ok = false;          // ... the first one
        if (p.phase == 0) {
            uint32_t status;
            bool direct = false;
            if (round == 0) {
                uint32_t R = ctl.count;
                bool part_full = false;
                if (p.parts > 1) {                   // partitioned append: the row's count is the sum of its parts'
                    nparts = FILTER_PARTS;
                    uint64_t sum = 0;
#pragma unroll
                    for (int j = 0; j < (int)FILTER_PARTS; ++j) {
                        const uint32_t c = p.part_counts[(row * FILTER_PARTS + j) * FILTER_PART_STRIDE];
                        part_full |= c > p.part_cap;
                        pcount[j] = c < p.part_cap ? c : p.part_cap;
                        sum += c;
                    }
                    R = sum > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)sum;
                } else {
                    pcount[0] = R;
                }
                direct = ctl.status == ROW_DIRECT;                     // marked by the initialisation kernel: no filter ran
                status = direct ? ROW_DIRECT : (R > p.capacity || part_full) ? ROW_OVERFLOW : R < p.k_accept ? ROW_RECALL : ROW_OK;
                if (cta == 0 && tid == 0 && !direct) {
                    if (p.parts > 1) p.ctl[row].count = part_full && R <= p.capacity ? p.capacity + 1 : R;   // what the statistics report
                    p.ctl[row].status = status;
                    p.ctl[row].n_final = status ? p.k : R;
                    if (status) atomicAdd(&p.header->n_failed, 1u);
                }
                n = R;
                from_filter = status_ok = status == ROW_OK;
            } else {
                // (the status another group's CTA wrote before the barrier: read past this SM's L1)
                status = __ldcg(&p.ctl[row].status);
                if (status == ROW_OK) continue;                    // ordered in the first round
                n = 0;
            }
            if (status != ROW_OK) {
                if (p.fused == 0 || (p.fused == 2 && round == 0)) continue;   // the exact-selection kernel and the second phase, or the second round, take this row
                // first a second filtering pass with the plan's tighter / looser sample rank, if it names one (the tile in
                // shared memory, unused so far, holds that pass's selection state) ...
                uint32_t R2 = 0, key2 = 0;
                const int again = direct ? 0 : grid_second_chance_row<T>(p.fb, row, status, *reinterpret_cast<SelectShared*>(smem_raw), &R2, &key2);
                if (again < 0) return;
                // ... else the k best records of the whole row into the row's buffer; ordered below like any buffer
                if (again == 0 && !grid_exact_select_row<T>(p.fb, row, reinterpret_cast<uint32_t*>(tile), s_warp)) return;
                nparts = 1;
#pragma unroll
                for (int j = 0; j < (int)FILTER_PARTS; ++j) pcount[j] = 0;
                pcount[0] = n = again == 1 ? R2 : p.k;
                if (again == 1) { from_filter = true; tau_key = key2; }
            }
        } else {
            if (ctl.status == ROW_OK) continue;  // already written by the first phase
            if (ctl.status == ROW_OVERFLOW_REFILTERED || ctl.status == ROW_RECALL_REFILTERED) {
                n = ctl.count;                   // what a second filtering pass left (its threshold is in the control block)
                from_filter = true;
            } else {
                n = p.k;                         // the exact selection left exactly k records
            }
            pcount[0] = n;
        }
        const uint32_t kk = n < p.k ? n : p.k;
        uint64_t* G = p.buf + row * 2 * p.row_stride;
        uint64_t* G2 = G + p.row_stride;
        uint32_t* bins = p.bins + row * (uint64_t)BIN_ROW_WORDS;
        uint32_t* flags = bins + BIN_COUNT;                              // [0] = some bin that matters is crowded
        uint32_t* coarse = flags + BIN_FLAGS;
        // every record of the row once, spread over the grid's threads
        // (The parts are walked as one run of sum(pcount) positions: part by part, a part of 20 K records would
        // keep one thread in seven of the grid busy and cost a memory round trip of its own, eight per pass.)
        uint32_t pend[FILTER_PARTS];                                                // pend[j] = records in parts 0..j
        {
            uint32_t acc = 0;
#pragma unroll
            for (int j = 0; j < (int)FILTER_PARTS; ++j) { acc += pcount[j]; pend[j] = acc; }
        }
        auto record_at = [&](uint64_t i) {
            uint32_t j = 0, before = 0;
#pragma unroll
            for (int q = 0; q < (int)FILTER_PARTS - 1; ++q)
                if (i >= pend[q]) { j = q + 1; before = pend[q]; }
            return (unsigned long long)__ldcg(G + (uint64_t)j * p.part_cap + (i - before));
        };
        auto for_each_record = [&](auto&& f) {           // (two loads in flight per thread: a pass is one or two rounds long)
            const uint64_t total = pend[FILTER_PARTS - 1];
            for (uint64_t i = gid; i < total; i += 2 * gthreads) {
                const bool two = i + gthreads < total;
                const unsigned long long r0 = record_at(i), r1 = two ? record_at(i + gthreads) : 0ull;
                f(r0);
                if (two) f(r1);
            }
        };

        for (uint64_t j = kk + gid; j < p.k; j += gthreads) {            // relaxed mode: padding after a short buffer
            p.out_vals[row * (uint64_t)p.k + j] = Elem<T>::from_bits(Elem<T>::NEG_INF_BITS);
            p.out_idx[row * (uint64_t)p.k + j] = -1;
        }

        // ================= main path: bin, scan, scatter, rank inside bins =================
        // The bins of bins.cuh measure a record from the largest record the buffer can hold.  For a row that passed the
        // check that is the threshold's key with the last index (its histogram may have been made by the filter kernel);
        // for a row that was selected exactly, the largest record of the buffer: one pass and a barrier more.
        uint32_t top_hi;
        bool counted = false;            // the bins hold this buffer's histogram already
        if (from_filter) {
            top_hi = ~tau_key;
            counted = p.hist_ready && status_ok && __ldcg(&flags[BIN_FLAG_UNCOUNTED]) == 0;
        } else {
            unsigned long long hi = 0ull;
            for_each_record([&](unsigned long long rec) { hi = rec > hi ? rec : hi; });
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                const unsigned long long h2 = __shfl_xor_sync(FULL_MASK, hi, d);
                hi = h2 > hi ? h2 : hi;
            }
            if ((tid & 31) == 0) s_max[tid >> 5] = hi;
            __syncthreads();
            if (tid < 32) {
                hi = s_max[tid];
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) {
                    const unsigned long long h2 = __shfl_xor_sync(FULL_MASK, hi, d);
                    hi = h2 > hi ? h2 : hi;
                }
                if (tid == 0) slot_max[cta] = hi;
            }
            if (!barrier()) return;
            unsigned long long rmax = 0ull;
            for (unsigned c = tid & 31; c < nctas; c += 32) {
                const unsigned long long h2 = __ldcg(&slot_max[c]);
                rmax = h2 > rmax ? h2 : rmax;
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                const unsigned long long h2 = __shfl_xor_sync(FULL_MASK, rmax, d);
                rmax = h2 > rmax ? h2 : rmax;
            }
            top_hi = (uint32_t)(rmax >> 32);
        }
        const int ib = p.idx_bits;
        auto bin_of = [&](unsigned long long rec) { return record_bin(rec, top_hi, ib); };

        if (!counted) {
            if (clean_bins) {
                // every CTA zeroed its share of the bins before it waited for the filter kernel and reported in: by now all
                // have, so this returns at once
                if (tid == 0) {
                    uint32_t ok = 1, polls = 0;
                    while (*((volatile uint32_t*)&p.header->done) < gridDim.x) {
                        __nanosleep(64);
                        if (++polls > LG_WAIT_LIMIT) { atomicExch(&p.header->error, 1u); ok = 0; break; }
                    }
                    __threadfence();
                    s_warp[0] = ok;
                }
                __syncthreads();
                const uint32_t ok = s_warp[0];
                __syncthreads();
                if (!ok) return;
                clean_bins = false;
            } else {
                for (uint64_t b = gid; b < BIN_ROW_WORDS; b += gthreads)
                    if (b < BIN_COUNT + 1 || b >= BIN_COUNT + BIN_FLAGS) bins[b] = 0;      // the bins, the "crowded" flag, the coarse bins
                if (!barrier()) return;
            }
            // histogram: fine bins in global memory, coarse bins through shared memory
            for (uint32_t c = tid; c < BIN_COARSE; c += BT_THREADS) s_coarse[c] = 0;
            __syncthreads();
            for_each_record([&](unsigned long long rec) {
                const uint32_t b = bin_of(rec);
                atomicAdd(&bins[b], 1u);
                atomicAdd(&s_coarse[b / BIN_PER_COARSE], 1u);
            });
            __syncthreads();
            for (uint32_t c = tid; c < BIN_COARSE; c += BT_THREADS) {
                const uint32_t cn = s_coarse[c];
                if (cn) atomicAdd(&coarse[c], cn);
            }
            if (!barrier()) return;
        }

        // scan (out of line: its registers are its own): the coarse bins' first positions, the list of the coarse bins that
        // matter, and the first positions of their fine bins
        scan_bins(bins, coarse, flags, ss, s_warp, cta, nctas, kk);
        if (!barrier()) return;

        if (__ldcg(&flags[0]) == 0) {
            // scatter into the second buffer, grouped by bin: the records of the listed coarse bins
            for_each_record([&](unsigned long long rec) {
                const uint32_t b = bin_of(rec);
                if (s_coarse[b / BIN_PER_COARSE] < kk) G2[atomicAdd(&bins[b], 1u)] = rec;
            });
            if (!barrier()) return;
            // rank inside the bin: bin b now occupies [end of the bin before it, bins[b]); the first fine bin of a coarse bin
            // starts where the coarse bin does
            // (only positions below the end of the bin that holds position kk-1 matter; they are a prefix)
            uint64_t g_end = (uint64_t)kk + LG_CROWDED < n ? (uint64_t)kk + LG_CROWDED : n;
            g_end = g_end < ss.scattered ? g_end : ss.scattered;
            for (uint64_t g = gid; g < g_end; g += gthreads) {
                const unsigned long long rec = __ldcg(&G2[g]);
                const uint32_t b = bin_of(rec);
                const uint32_t first = b % BIN_PER_COARSE ? __ldcg(&bins[b - 1]) : s_coarse[b / BIN_PER_COARSE], last = __ldcg(&bins[b]);
                if (first < kk) {
                    uint32_t pos = first;
                    for (uint32_t j = first; j < last; ++j) pos += __ldcg(&G2[j]) < rec;
                    if (pos < kk) write_output(p.out_vals, p.out_idx, p.k, row, pos, rec);
                }
            }
            continue;                    // next row: its first barrier also orders this row's reads before any reuse
        }

        // ================= reserve path: bitonic network =================
        if (nparts > 1) {                        // it wants the records in one run: through the second buffer and back
            uint64_t first = 0;
            for (uint32_t j = 0; j < nparts; ++j) {
                const uint64_t* part = G + (uint64_t)j * p.part_cap;
                for (uint64_t i = gid; i < pcount[j]; i += gthreads) G2[first + i] = __ldcg(&part[i]);
                first += pcount[j];
            }
            if (!barrier()) return;
            for (uint64_t i = gid; i < n; i += gthreads) G[i] = __ldcg(&G2[i]);
            if (!barrier()) return;
        }
        uint64_t P = BT_TILE;
        while (P < n) P <<= 1;

        // ---- sort every tile (sizes 2 .. BT_TILE); positions beyond n hold all-ones padding ----
        const uint64_t tiles = P / BT_TILE;
        for (uint64_t t = cta; t < tiles; t += nctas) {
            const uint64_t base = t * BT_TILE;
            for (uint32_t i = tid; i < BT_TILE; i += BT_THREADS) tile[i] = base + i < n ? __ldcg(&G[base + i]) : ~0ull;
            __syncthreads();
            bitonic_tile_steps(tile, base, 2, BT_TILE);
            for (uint32_t i = tid; i < BT_TILE; i += BT_THREADS) G[base + i] = tile[i];
            __syncthreads();
        }
        if (!barrier()) return;

        // ---- merge: exchanges at distance >= BT_TILE on the buffer, the rest tile by tile ----
        for (uint64_t size = 2ull * BT_TILE; size <= P; size <<= 1) {
            for (uint64_t stride = size / 2; stride >= BT_TILE; stride >>= 1) {
                for (uint64_t q = gid; q < P / 2; q += gthreads) {
                    const uint64_t lo2 = 2 * q - (q & (stride - 1));
                    const uint64_t hi2 = lo2 + stride;
                    const bool ascending = (lo2 & size) == 0;
                    const uint64_t x = __ldcg(&G[lo2]), y = __ldcg(&G[hi2]);
                    if ((x > y) == ascending) { G[lo2] = y; G[hi2] = x; }
                }
                if (!barrier()) return;
            }
            for (uint64_t t = cta; t < tiles; t += nctas) {
                const uint64_t base = t * BT_TILE;
                for (uint32_t i = tid; i < BT_TILE; i += BT_THREADS) tile[i] = __ldcg(&G[base + i]);
                __syncthreads();
                bitonic_tile_steps(tile, base, size, size);
                for (uint32_t i = tid; i < BT_TILE; i += BT_THREADS) G[base + i] = tile[i];
                __syncthreads();
            }
            if (!barrier()) return;
        }

        for (uint64_t j = gid; j < kk; j += gthreads) write_output(p.out_vals, p.out_idx, p.k, row, (uint32_t)j, __ldcg(&G[j]));
    }
    }
}

}  // namespace profk
