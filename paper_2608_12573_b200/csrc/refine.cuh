// Stage 4 (Section 3, "Refinement"): the count check and the exact top-k of the candidate
// buffer, written out in the order "value descending, index ascending".
//
// Candidate records are 64-bit integers whose ascending order is exactly that order, so
// refinement is "the k smallest records, sorted".  One thread-block cluster per row; its first
// CTA does the refinement proper.  Every CTA first takes the paper's check -- fewer than k
// candidates, or more than the buffer holds, means the row is replaced by an exact top-k of the
// full input, which the whole cluster computes (exact_select.cuh); when the check passes, as it
// almost always does, the other CTAs leave at once.  The first CTA then bins the records (held
// in registers when they fit) by their key's distance above tau into 4096 logarithmic bins; a
// scan of the bin counts gives every bin its first output position and finds the bin that holds
// the k-th best record; the records of that bin and of all better bins are grouped by bin in
// shared memory, and each of them finds its final position by ranking itself inside its (small)
// bin.  No sort is needed.  When a bin is too crowded for that (many equal values) a
// most-significant-digit radix select plus a bitonic sort does the same job.
//
// In direct mode (a row too short for sampling to pay) there is no threshold and no buffer to
// refine: every row goes straight to the exact selection.
#pragma once

#include "exact_select.cuh"
#include "second_chance.cuh"
#include "select_sort.cuh"

namespace profk {

template <typename T> struct RefineParams {
    const T* in;             // rows x N input (read only by the exact selection)
    uint64_t N;
    RowCtl* ctl;
    WsHeader* header;
    uint64_t* buf;           // row r's records start at buf + r * buf_stride
    uint64_t buf_stride;
    uint32_t capacity;
    uint32_t k;
    uint32_t k_accept;
    uint32_t stage_cap;      // records the general select may stage in shared memory (0 = read them from the buffer)
    uint32_t sort_cap;       // power of two >= k: records the sort area holds (the area has RF_EDGE_CAP more)
    T* out_vals;             // rows x k
    int64_t* out_idx;        // rows x k
    int use_pdl;
    int direct;              // 1 = no threshold / filter ran: every row is selected exactly
    uint32_t cluster_size;   // CTAs per cluster; 1 = launched without a cluster dimension, and rows that fail the
                             // check are left to the exact-selection kernel that follows
    uint32_t clusters_per_row;   // segments a failed row is cut into for its exact selection, one cluster each
    uint64_t* xs_records;    // rows x clusters_per_row x (k + XS_EDGE) records selected from the segments
    uint32_t* xs_counters;   // rows x clusters_per_row append counters
    SampleInfo sample;       // the kept sample and the second-chance ranks (sample.keys == null: none; clusters only)
    uint4* thr2;             // rows threshold records of the second filtering pass
};

// Records selected from the segments of a row, read through L2 (other clusters wrote them); unused
// slots hold all-ones.
struct SegmentRecords {
    const uint64_t* recs;
    uint32_t n;
    template <typename F> __device__ __forceinline__ void for_each(F&& f) const {
        const uint32_t n_round = (n + 31u) & ~31u;
        for (uint32_t i = threadIdx.x; i < n_round; i += blockDim.x) {
            const uint64_t rec = i < n ? __ldcg(&recs[i]) : ~0ull;
            f(rec, rec != ~0ull);
        }
    }
};

// The k smallest of the n records at `recs` (slots that hold all-ones are empty; at least k are not, and
// recs[0] is one of them), ordered, as row `row` of the output.  One CTA; the records were written by other
// CTAs, fenced, and are read through L2.
template <typename T>
__device__ __forceinline__ void finish_from_segments(const uint64_t* recs, uint32_t n, uint32_t k, uint32_t sort_cap,
                                                     uint64_t* sortbuf, SelectShared& sh, uint64_t row, T* out_vals,
                                                     int64_t* out_idx) {
    const unsigned tid = threadIdx.x, nthr = blockDim.x, lane = lane_id();
    if (tid == 0) { sh.or_bits = 0ull; sh.fill = 0; sh.n_edge = 0; }
    __syncthreads();
    const uint64_t first = __ldcg(&recs[0]);
    uint64_t diff = 0;
    for (uint32_t i = tid; i < n; i += nthr) {
        const uint64_t rec = __ldcg(&recs[i]);
        if (rec != ~0ull) diff |= rec ^ first;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) diff |= __shfl_xor_sync(FULL_MASK, diff, d);
    if (lane == 0 && diff) atomicOr(&sh.or_bits, (unsigned long long)diff);
    __syncthreads();
    select_smallest(SegmentRecords{recs, n}, first, k, sortbuf, sort_cap, sh);
    sort_and_write<T>(sortbuf, k, k, k, row, out_vals, out_idx);
}

// Stage 4 proper: the k best of the R = ctl.count candidate records of `row`, in order, written to the output.  One CTA;
// sh.hist zero, sh.or_bits = sh.fill = sh.n_edge = sh.crowded = 0 on entry.  PRELOADED: r[] holds the first batch of
// records already (8 per thread, requested before the survivor count was known; slots beyond the capacity all ones).
template <typename T, bool PRELOADED>
__device__ __forceinline__ void refine_row(const RefineParams<T>& p, uint64_t row, const RowCtl& ctl, uint64_t (&r)[8], uint64_t* sortbuf,
                                           uint64_t* staged, SelectShared& sh) {
    const unsigned tid = threadIdx.x, nthr = blockDim.x, lane = lane_id();
    const uint64_t* src = p.buf + row * p.buf_stride;
    const uint32_t R = ctl.count;

    const uint32_t n = R;
    const uint32_t kk = n < p.k ? n : p.k;          // real outputs; the rest is padding (relaxed mode)
    for (uint32_t j = kk + tid; j < p.k; j += nthr) {       // relaxed mode: padding after a short buffer
        p.out_vals[row * (uint64_t)p.k + j] = Elem<T>::from_bits(Elem<T>::NEG_INF_BITS);
        p.out_idx[row * (uint64_t)p.k + j] = -1;
    }

    // ---- bin the records by the distance d of their key above tau, on a logarithmic scale: the bin is
    //      the exponent and the top seven mantissa bits of d as a float (monotone in d, 32 x 128 = 4096
    //      bins, fine where the records are dense -- just above tau -- and coarse where they are rare).
    //      Bin 0 holds the largest keys.  A CTA of 256 threads (the rows of a large batch, a thousand or two records
    //      each) takes five mantissa bits, 1024 bins: four bins per thread again, and a quarter of the scan. ----
    const uint32_t tau_key = Elem<T>::key(Elem<T>::from_bits(ctl.tau_bits));
    const uint32_t nbins = nthr == 256 ? RF_BINS / 4 : RF_BINS;
    const int bin_shift = nthr == 256 ? 18 : 16;
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
        const uint32_t level = f > (127u << 23) ? (f >> bin_shift) - (127u << (23 - bin_shift)) : 0u;     // 0 .. nbins - 1
        return (nbins - 1u) - level;
    };

    for (uint32_t b = 0; b < nbatch; ++b) {
        if (b > 0 || !PRELOADED) load_batch(b);
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (valid(b, u)) atomicAdd(&sh.hist[bin_of(r[u])], 1u);
    }
    __syncthreads();

    // ---- scan the bin counts: first position of every bin, and the bin of the kk-th best record ----
    if (nthr * 4 == nbins) {
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
        uint32_t w = lane < (nthr >> 5) ? sh.warp_sums[lane] : 0u;       // every warp scans the warps' totals itself
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
        const uint32_t per = (nbins + nthr - 1) / nthr;
        uint32_t sum = 0;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t bin = tid * per + j;
            sum += bin < nbins ? sh.hist[bin] : 0;
        }
        uint32_t before = block_scan_any(sum, sh.warp_sums) - sum;
        for (uint32_t j = 0; j < per; ++j) {
            const uint32_t bin = tid * per + j;
            if (bin < nbins) {
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
        // ---- every grouped record ranks itself inside its bin: that is its place in the output ----
        for (uint32_t s = tid; s < n_grouped; s += nthr) {
            const uint64_t mine = sortbuf[s];
            const uint32_t bin = bin_of(mine);
            const uint32_t first = sh.start[bin], last = sh.hist[bin];
            uint32_t pos = first;
            for (uint32_t j = first; j < last; ++j) pos += sortbuf[j] < mine;
            if (pos < kk) write_output(p.out_vals, p.out_idx, p.k, row, pos, mine);
        }
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

// The same out of line, for the one CTA that refines a row after a second filtering pass (second_chance_row): the refine
// kernel's own path keeps its registers.
template <typename T>
__device__ __noinline__ void refine_row_again(const RefineParams<T>& p, uint64_t row, uint64_t* sortbuf, uint64_t* staged, SelectShared& sh) {
    const unsigned tid = threadIdx.x, nthr = blockDim.x;
    __syncthreads();
    if (tid == 0) { sh.or_bits = 0ull; sh.fill = 0; sh.n_edge = 0; sh.crowded = 0; }
    for (uint32_t i = tid; i < RF_BINS; i += nthr) sh.hist[i] = 0;
    __syncthreads();
    const RowCtl ctl = p.ctl[row];               // the count and the threshold of the second pass (this CTA wrote them)
    uint64_t r[8];
    refine_row<T, false>(p, row, ctl, r, sortbuf, staged, sh);
}

// The second chance (second_chance.cuh) of a row that failed the count check, run by all clusters of the row, each over
// its own segment: the threshold of the plan's tighter (after an overflow) or looser (after too few candidates) sample
// rank is selected from the kept keys -- by every CTA for itself, nobody waits for anybody -- the segment is filtered with
// it into the row's buffer (counter: the row's `pad` word), and the cluster that finishes last takes the check
// k <= R' <= M on the new count.  Returns, the same in every CTA of a cluster: 0 = not the last cluster, or the last one
// and the row is answered (its first CTA refines it from the buffer like any row); 2 = the last cluster and the check
// failed again.
template <typename T>
__device__ __noinline__ int second_chance_row(const RefineParams<T>& p, uint64_t row, unsigned seg, unsigned crank, uint32_t rung,
                                              uint32_t failed_status, uint64_t* sortbuf, SelectShared& sh, uint32_t tau_key) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned tid = threadIdx.x, nthr = blockDim.x;
    const unsigned csize = p.cluster_size, nseg = p.clusters_per_row;
    const SampleInfo& sm = p.sample;
    uint32_t key2, j2;
    // (a tighter rank lies among the keys at or above the first pass's threshold)
    kth_sample_record<T>(sm.keys + row * sm.S, sm.S, rung, sh, &key2, &j2, failed_status == ROW_OVERFLOW ? tau_key : 0u);
    const uint32_t idx2 = sm.by_record ? sample_element_index(j2, row, sm.seed, sm.q, sm.rem, sm.S, sm.inv_s) : 0xFFFFFFFFu;
    const T tau2 = Elem<T>::from_key(key2);
    if (tid == 0) {                              // (every CTA of the row writes the same sixteen bytes)
        const uint32_t top = Elem<T>::KEY_BITS == 32 ? 0xFFFFFFFFu : 0xFFFFu;
        p.thr2[row] = make_uint4(Elem<T>::bits(tau2), Elem<T>::bits(Elem<T>::from_key(key2 == top ? key2 : key2 + 1u)), idx2, 0u);
    }
    __syncthreads();

    FilterParams<T> fp = {};
    fp.in = p.in; fp.N = p.N; fp.rows = row + 1; fp.tau = nullptr; fp.capacity = p.capacity;
    fp.buf = p.buf; fp.buf_stride = p.buf_stride;
    fp.counts = &p.ctl[0].pad; fp.count_stride = sizeof(RowCtl) / 4;
    fp.thr = p.thr2;
    const uint64_t tiles = tiles_per_row<T>(p.N, nthr * XS_UNROLL);
    const uint64_t seg_lo = tiles * seg / nseg, seg_hi = tiles * (seg + 1) / nseg;
    if (nthr == 512) refilter_tiles<T, 512>(fp, (uint32_t)row, seg_lo, seg_hi, crank, csize, tau2);
    else refilter_tiles<T, 1024>(fp, (uint32_t)row, seg_lo, seg_hi, crank, csize, tau2);
    __threadfence();
    cluster.sync();                              // the whole cluster's records and counts are out

    // the last cluster to get here sees all of them
    if (crank == 0 && tid == 0) {
        const uint32_t ticket = atomicAdd(&p.ctl[row].collect, 1u);
        uint32_t decision = 0;
        if (ticket == nseg - 1) {
            p.ctl[row].collect = 0;
            __threadfence();
            const uint32_t R2 = __ldcg(&p.ctl[row].pad);
            decision = (R2 >= p.k && R2 <= p.capacity) ? 1u : 2u;
            if (decision == 1u) {
                p.ctl[row].status = failed_status == ROW_OVERFLOW ? ROW_OVERFLOW_REFILTERED : ROW_RECALL_REFILTERED;
                p.ctl[row].count = R2;
                p.ctl[row].tau_bits = Elem<T>::bits(tau2);
                p.ctl[row].tau_idx = idx2;
            }
        }
        sh.crowded = decision;
    }
    cluster.sync();
    const uint32_t decision = *cluster.map_shared_rank(&sh.crowded, 0);
    cluster.sync();                              // the first CTA's word has been read by all: it may go on
    if (decision == 1u && crank == 0) refine_row_again<T>(p, row, sortbuf, sortbuf + p.sort_cap + RF_EDGE_CAP, sh);
    return decision == 2u ? 2 : 0;
}

// The exact top-k of the full row, for a row that failed the count check (Section 3, "Refinement").
// Cluster `seg` of the row's clusters selects the k smallest records (and a few more) of its segment of
// the row; the cluster that finishes last merges: the k smallest of all segments' records, ordered, are
// the row's output.  The ticket is the row's `collect` word, zero on entry and zero again on exit.
// When the plan names a second-chance rank for this kind of failure and the sample was kept, that comes first; the
// exact selection then runs only if the second pass fails too, by the one cluster that found out, over the whole row.
template <typename T>
__device__ __noinline__ void exact_row(const RefineParams<T>& p, uint64_t row, unsigned seg, unsigned crank, uint64_t* sortbuf,
                                       SelectShared& sh, uint32_t status, uint32_t tau_key) {
    const unsigned tid = threadIdx.x, nthr = blockDim.x;
    const unsigned csize = p.cluster_size, nseg = p.clusters_per_row;
    const bool overflowed = status == ROW_OVERFLOW;
    const uint64_t tiles = tiles_per_row<T>(p.N, nthr * XS_UNROLL);
    const uint32_t slots = p.k + XS_EDGE;                // per segment: a superset of its k smallest records
    const uint32_t rung = status == ROW_OVERFLOW ? p.sample.r_tight : status == ROW_RECALL ? p.sample.r_loose : 0u;
    if (rung != 0 && p.sample.keys != nullptr && csize > 1 && (nthr == 512 || nthr == 1024)) {
        if (second_chance_row<T>(p, row, seg, crank, rung, status, sortbuf, sh, tau_key) != 2) return;
        // failed again: this cluster alone selects from the whole row, into its own scratch
        const uint64_t* mine = p.xs_records + (row * nseg + seg) * (uint64_t)slots;
        exact_select_cluster<T>(p.in, p.N, row, p.k, 0, tiles, p.xs_records + (row * nseg + seg) * (uint64_t)slots,
                                p.xs_counters + row * nseg + seg, sh, csize, crank, false, 0u);
        if (crank != 0) return;
        finish_from_segments<T>(mine, slots, p.k, p.sort_cap, sortbuf, sh, row, p.out_vals, p.out_idx);
        return;
    }
    const uint64_t seg_lo = tiles * seg / nseg, seg_hi = tiles * (seg + 1) / nseg;
    const uint64_t* recs = p.xs_records + (row * nseg) * (uint64_t)slots;
    exact_select_cluster<T>(p.in, p.N, row, p.k, seg_lo, seg_hi, p.xs_records + (row * nseg + seg) * (uint64_t)slots,
                            p.xs_counters + row * nseg + seg, sh, csize, crank, overflowed, tau_key);
    if (crank != 0) return;

    // every thread of this cluster has fenced its records; the last cluster to get here sees them all
    if (tid == 0) {
        const uint32_t ticket = atomicAdd(&p.ctl[row].collect, 1u);
        const bool last = ticket == nseg - 1;
        if (last) { p.ctl[row].collect = 0; __threadfence(); }
        sh.cnt = last ? 1u : 0u;
    }
    __syncthreads();
    if (sh.cnt == 0) return;
    __syncthreads();                         // sh.cnt is rewritten by the select below

    finish_from_segments<T>(recs, nseg * slots, p.k, p.sort_cap, sortbuf, sh, row, p.out_vals, p.out_idx);
}

// Two builds of the kernel.  With up to 512 threads a refine CTA has to start beside the last CTAs
// of the filter kernel on an SM, and 48 registers per thread is what fits there; the (rare) exact
// selection then runs with spills.  A CTA of 1024 threads does not fit there anyway and gets the
// registers the exact selection wants.
template <typename T, int MAXREG>
__global__ void __maxnreg__(MAXREG) refine_kernel(const __grid_constant__ RefineParams<T> p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* sortbuf = reinterpret_cast<uint64_t*>(smem_raw);                 // sort_cap + RF_EDGE_CAP records
    uint64_t* staged = sortbuf + p.sort_cap + RF_EDGE_CAP;                     // stage_cap records
    __shared__ SelectShared sh;

    // CTAs of a row are consecutive: clusters_per_row clusters (along x) of cluster_size CTAs.
    const unsigned csize = p.cluster_size, nseg = p.clusters_per_row;
    const unsigned cta_in_row = blockIdx.x % (csize * nseg);
    const unsigned seg = cta_in_row / csize, crank = cta_in_row % csize;
    const bool refiner = cta_in_row == 0;            // the CTA that refines the row's buffer
    const unsigned tid = threadIdx.x, nthr = blockDim.x, lane = lane_id();
    const uint64_t row = blockIdx.x / (csize * nseg);
    if (refiner) {
        if (tid == 0) { sh.or_bits = 0ull; sh.fill = 0; sh.n_edge = 0; sh.crowded = 0; }
        for (uint32_t i = tid; i < RF_BINS; i += nthr) sh.hist[i] = 0;
        __syncthreads();
    }
    pdl_launch_dependents();
    if (p.use_pdl) pdl_wait();

    // The first batch of records (8 per thread, kept in registers) is requested at once, together with
    // the row's control block: which of them are real is known when the survivor count arrives.
    const uint64_t* src = p.buf + row * p.buf_stride;
    uint64_t r[8];
    if (refiner && !p.direct) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t i = u * nthr + tid;
            r[u] = i < p.capacity ? src[i] : ~0ull;
        }
    }

    // ---- the count check of stage 4 ----
    RowCtl ctl;
    uint32_t status;
    if (p.direct) {                          // the row's control block was set up by the initialisation kernel
        ctl.tau_bits = 0; ctl.count = 0;
        status = ROW_DIRECT;
    } else {
        ctl = p.ctl[row];
        status = ctl.count > p.capacity ? ROW_OVERFLOW : ctl.count < p.k_accept ? ROW_RECALL : ROW_OK;
        if (refiner && tid == 0) {
            p.ctl[row].status = status;
            p.ctl[row].n_final = status ? p.k : ctl.count;
            if (status) atomicAdd(&p.header->n_failed, 1u);
        }
    }
    if (status != ROW_OK) {
        if (csize == 1) return;              // the exact-selection kernel that follows takes this row
        exact_row<T>(p, row, seg, crank, sortbuf, sh, status, Elem<T>::key(Elem<T>::from_bits(ctl.tau_bits)));
        return;
    }
    if (!refiner) return;
    refine_row<T, true>(p, row, ctl, r, sortbuf, staged, sh);
}

}  // namespace profk
