// Stages 1 and 2 (Section 3, "Sampling" and "Threshold estimation"): gather S stratified
// Philox samples of a row and select the t-th largest as the threshold tau.
//
// One thread-block cluster handles one row.  Each CTA of the cluster gathers its share of
// the samples into shared memory as order keys.  The t-th largest key is then found by
//   * a short cut for small ranks (t <= 128): every CTA derives a lower bound L on the
//     answer from the maxima of 128 groups of its keys (the t-th largest group maximum has
//     at least t keys at or above it), sends only its keys >= L to the first CTA through
//     distributed shared memory (remote atomics and stores), and the first CTA ranks those
//     few candidates directly; for ranks up to 128 per CTA of the cluster the bound is the smallest over the
//     CTAs of their ceil(t / csize)-th largest group maxima, and the candidates are ranked by the whole cluster;
//   * otherwise (deeper ranks, or so many ties that the candidates do not fit) a radix select
//     whose per-digit histograms are summed across the cluster through distributed shared
//     memory.
// Only hardware cluster barriers are used -- no spinning on global memory.
#pragma once

#include <cooperative_groups.h>

#include <utility>

#include "common.cuh"

namespace profk {

namespace cg = cooperative_groups;

constexpr int SEL_THREADS = 1024;
constexpr int SEL_SMALL_THREADS = 256;  // CTA size of the variant for batches of rows with small samples
constexpr int SEL_BINS = 2048;        // 11-bit digits
constexpr int SEL_GROUPS = 128;       // groups of 8 lanes whose maxima bound the answer from below
constexpr uint32_t SEL_CAND_CAP = 4096;
#ifndef PROFK_SEL_WIDE_MIN
#define PROFK_SEL_WIDE_MIN 16
#endif
constexpr uint32_t SEL_WIDE_MIN = PROFK_SEL_WIDE_MIN;   // smallest rank for which a cluster exchanges its CTAs' bounds
constexpr uint32_t SEL_SPREAD_MIN = 128;    // more candidates than this are ranked by all CTAs of the cluster

// Per-row control block in the workspace.
struct RowCtl {
    uint32_t tau_bits;   // threshold (element bit pattern)
    uint32_t count;      // survivors appended by the filter (R, or something > capacity)
    uint32_t collect;    // records appended by the exact-selection path
    uint32_t status;     // PROFK_ROW_* (| 0x80000000 on a timeout)
    uint32_t n_final;    // records the refine step has to order
    uint32_t capacity;
    uint32_t tau_idx;    // index of the threshold record; 0xFFFFFFFF = the threshold is the value alone
    uint32_t pad;        // survivors appended by a second filtering pass (second_chance.cuh)
};
static_assert(sizeof(RowCtl) == 32, "RowCtl is 32 bytes");

constexpr int WS_GROUPS = 32;            // most CTA groups of the large-k refine

// Header of the workspace: state of the grid barrier used by the exact-selection kernel.
struct WsHeader {
    uint32_t bar_count;  // arrivals at the grid barrier since the start of the call (grid_barrier.cuh)
    uint32_t bar_gen;    // (unused)
    uint32_t error;      // non-zero = a bounded wait gave up
    uint32_t done;       // CTAs of the emit / large-refine kernel that have cleared their share of the bins
    uint32_t n_failed;   // rows whose count check failed
    uint32_t tile_counter;  // hands out the filter kernel's tiles
    uint32_t pad[58];
    uint32_t group_bar[WS_GROUPS][2];   // barriers of the CTA groups of the large-k refine: {arrivals, unused}
};
static_assert(sizeof(WsHeader) == 512, "WsHeader is 512 bytes");

template <typename T> struct SelectParams {
    const T* in;
    uint64_t N;
    uint32_t S;            // sample size
    uint32_t t;            // rank, 1-based, t-th largest
    uint64_t seed;
    uint32_t per_cta;      // samples per CTA of the cluster (even)
    uint64_t q;            // N / S
    uint32_t rem;          // N % S
    float inv_s;           // 1 / S
    T* tau;                // rows thresholds out (may be null when thr is given)
    uint4* thr;            // null, or rows threshold records for the filter: {bits of tau, bits of the next value in the total
                           // order, index of the threshold record (0xFFFFFFFF = the threshold is the value alone), 0}
    RowCtl* ctl;           // may be null (stand-alone use)
    WsHeader* header;      // may be null
    uint32_t capacity;
    uint32_t* sample_idx;  // may be null; rows x S
    const uint32_t* keys_in;   // null, or rows x S keys of the sample gathered by gather_kernel before this one
    uint32_t* part_counts;     // null, or the counters of the partitioned append (FILTER_PARTS per row, FILTER_PART_STRIDE words apart) to reset with the row's
    int by_record;             // 1 = the threshold is the t-th sampled record (value descending, index ascending), 0 = its value
    uint32_t* keys_store;      // null, or rows x S: the sample's keys are kept here for a second filtering pass (when this kernel gathers them itself)
    uint4* zero;               // null, or zero_vecs 16-byte vectors to clear for the kernels behind this one (the bins the filter counts in)
    uint32_t zero_vecs;
};

// floor(j * N / S) = j * (N / S) + floor(j * (N % S) / S).  The second quotient is below S
// (< 2^18), so a float estimate is within one of it and an integer check repairs it.
__device__ __forceinline__ uint64_t stratum_start(uint64_t j, uint64_t q, uint32_t rem, uint32_t S, float inv_s) {
    if (rem == 0) return j * q;
    const uint64_t x = j * (uint64_t)rem;
    int64_t e = (int64_t)((float)x * inv_s);
    int64_t r = (int64_t)x - e * (int64_t)S;
    while (r < 0) { --e; r += S; }
    while (r >= (int64_t)S) { ++e; r -= S; }
    return j * q + (uint64_t)e;
}

// Element index of sample j of `row`: the Philox draw of stratum j again (one block serves samples 2p and 2p + 1).
__device__ __forceinline__ uint32_t sample_element_index(uint32_t j, uint64_t row, uint64_t seed, uint64_t q, uint32_t rem, uint32_t S, float inv_s) {
    const Philox4 r = philox4x32_10(j >> 1, (uint32_t)row, (uint32_t)(row >> 32), 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
    const uint64_t b0 = stratum_start(j, q, rem, S, inv_s);
    const uint64_t b1 = stratum_start((uint64_t)j + 1, q, rem, S, inv_s);
    const uint64_t u = (j & 1u) ? (((uint64_t)r.w << 32) | r.z) : (((uint64_t)r.y << 32) | r.x);
    return (uint32_t)(b0 + __umul64hi(u, b1 - b0));
}

// Writes tau for one row: the key of the threshold and the number j of the sample that holds it.  Samples are
// stratified, so among samples "smaller index" and "smaller sample number" are the same order; the element
// index of sample j is drawn again here by the one thread that publishes.
template <typename T>
__device__ __forceinline__ void publish_threshold(const SelectParams<T>& p, uint64_t row, uint32_t tau_key, uint32_t j) {
    const T tau = Elem<T>::from_key(tau_key);
    if (p.tau) p.tau[row] = tau;
    if (p.ctl || p.thr) {
        if (p.ctl) p.ctl[row].tau_bits = Elem<T>::bits(tau);
        uint32_t idx = 0xFFFFFFFFu;
        if (p.by_record) idx = sample_element_index(j, row, p.seed, p.q, p.rem, p.S, p.inv_s);
        if (p.ctl) p.ctl[row].tau_idx = idx;
        if (p.thr) {
            const uint32_t top = Elem<T>::KEY_BITS == 32 ? 0xFFFFFFFFu : 0xFFFFu;
            const uint32_t next_key = tau_key == top ? tau_key : tau_key + 1u;
            p.thr[row] = make_uint4(Elem<T>::bits(tau), Elem<T>::bits(Elem<T>::from_key(next_key)), idx, 0u);
        }
    }
}

// Block-wide inclusive scan of one value per thread (blockDim.x == SEL_THREADS or fewer warps).
__device__ __forceinline__ uint32_t block_inclusive_scan(uint32_t v, uint32_t* warp_sums) {
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t n = __shfl_up_sync(FULL_MASK, v, d);
        if (lane >= (unsigned)d) v += n;
    }
    if (lane == 31) warp_sums[warp] = v;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = warp_sums[lane];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t n = __shfl_up_sync(FULL_MASK, w, d);
            if (lane >= (unsigned)d) w += n;
        }
        warp_sums[lane] = w;
    }
    __syncthreads();
    if (warp > 0) v += warp_sums[warp - 1];
    return v;
}

// Stage 1 on its own, over the whole GPU: the keys of the sampled elements of every row, in sample order.
// One thread per pair of samples.  For a long row every sample lies on a page of its own, and the address
// translations of a large sample take a 16-CTA cluster tens of microseconds; spread over all SMs they take a few.
constexpr int GATHER_THREADS = 256;

template <typename T> struct GatherParams {
    const T* in;
    uint64_t N;
    uint64_t rows;
    uint32_t S;
    uint64_t seed;
    uint64_t q;            // N / S
    uint32_t rem;          // N % S
    float inv_s;           // 1 / S
    uint32_t* keys_out;    // rows x S (a shard: the keys of its strata only, pairs * 2 of them)
    // A shard of one row (the whole row: pair_lo = 0, pairs = ceil(S / 2), base = 0): `in` points at element `base` of the
    // row and the kernel takes strata 2 * pair_lo ... 2 * (pair_lo + pairs) - 1, all of which lie inside the shard.
    uint64_t pair_lo;
    uint64_t pairs;
    uint64_t base;
    uint4* zero;           // null, or zero_vecs 16-byte vectors to clear for the kernels behind this one (the bins the filter counts in)
    uint32_t zero_vecs;
};

template <typename T>
__global__ void __launch_bounds__(GATHER_THREADS) gather_kernel(const GatherParams<T> p) {
    const uint64_t pairs = p.pairs;
    const uint64_t g = (uint64_t)blockIdx.x * GATHER_THREADS + threadIdx.x;
    const bool active = g < p.rows * pairs;
    const uint64_t row = active ? g / pairs : 0;
    const uint64_t j = active ? 2 * (p.pair_lo + g % pairs) : 0;     // even sample of the pair
    const bool second = active && j + 1 < p.S;
    const T* rowp = p.in + row * p.N - p.base;
    uint32_t idx0 = 0, idx1 = 0;
    if (active) {
        const Philox4 r = philox4x32_10((uint32_t)(j >> 1), (uint32_t)row, (uint32_t)(row >> 32), 0u,
                                        (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
        const uint64_t b0 = stratum_start(j, p.q, p.rem, p.S, p.inv_s);
        const uint64_t b1 = stratum_start(j + 1, p.q, p.rem, p.S, p.inv_s);
        idx0 = (uint32_t)(b0 + __umul64hi(((uint64_t)r.y << 32) | r.x, b1 - b0));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(rowp + idx0));
        if (second) {
            const uint64_t b2 = stratum_start(j + 2, p.q, p.rem, p.S, p.inv_s);
            idx1 = (uint32_t)(b1 + __umul64hi(((uint64_t)r.w << 32) | r.z, b2 - b1));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(rowp + idx1));
        }
    }
    pdl_wait();                  // the positions needed nothing; the values need the work queued before this kernel
    // Dependents are released only now, after the wait: the kernels behind this one read the input before their
    // own wait (which covers this kernel alone), so they must not start before whatever wrote the input has finished.
    pdl_launch_dependents();
    if (p.zero)        // (after the wait: the previous call's last kernel has read these words)
        for (uint64_t i = g; i < p.zero_vecs; i += (uint64_t)gridDim.x * GATHER_THREADS) p.zero[i] = make_uint4(0u, 0u, 0u, 0u);
    if (active) {
        const T v0 = rowp[idx0];
        const T v1 = second ? rowp[idx1] : v0;
        uint32_t* out = p.keys_out + row * p.S + (j - 2 * p.pair_lo);
        out[0] = Elem<T>::key(v0);
        if (second) out[1] = Elem<T>::key(v1);
    }
}

// THREADS = THREADS is the general kernel.  THREADS = SEL_SMALL_THREADS is for batches of rows with small
// samples (one CTA per row, at most SEL_CAND_CAP samples, rank at most THREADS / 8): four such CTAs share an
// SM, so four times as many rows are in flight in a kernel that is all latency; it has no radix path, because
// with so few samples all of them fit among the candidates.
template <typename T, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == SEL_THREADS ? 1 : 4) sample_select_kernel(const SelectParams<T> p) {
    constexpr int GROUPS = THREADS / 8;          // groups of 8 lanes whose maxima bound the answer from below
    constexpr bool GENERAL = THREADS == SEL_THREADS;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw);          // per_cta keys
    // Candidates (filled in the first CTA only), as records (key << 32) | ~(sample number): distinct, and their
    // descending order is (value descending, index ascending).  The radix path reuses the space for its histograms.
    __shared__ uint64_t cand[SEL_CAND_CAP];
    __shared__ uint32_t gmax[GROUPS];
    __shared__ uint32_t warp_sums[32];
    __shared__ uint32_t s_digit, s_before, s_ncand, s_lower, s_lmin;

    cg::cluster_group cluster = cg::this_cluster();
    const unsigned csize = cluster.num_blocks();
    const unsigned crank = cluster.block_rank();
    const uint64_t row = blockIdx.x / csize;
    const unsigned tid = threadIdx.x, lane = lane_id();

    if (tid == 0) { s_ncand = 0; s_lower = 0; s_lmin = 0xFFFFFFFFu; }
    __syncthreads();
    // Split barrier: "my candidate counter is zero".  Peers wait for it only after their gather,
    // by which time every CTA has long arrived.
    auto zeroed = cluster.barrier_arrive();

    // ---- stage 1: gather this CTA's share of the sample -------------------------------
    // Samples come in pairs: one Philox block (four words) serves samples 2p and 2p+1.
    const uint32_t j0 = crank * p.per_cta;
    const uint32_t j1 = min(p.S, j0 + p.per_cta);
    const uint32_t n_local = j1 > j0 ? j1 - j0 : 0;
    const uint32_t n_round = (n_local + 31u) & ~31u;                 // whole warps take part in ballots
    const T* rowp = p.in + row * p.N;
    uint32_t my_max = 0;
    constexpr int PB = 2;                                            // pairs per batch: 4 loads in flight per thread
    if (p.keys_in) {
        // the sample was gathered by the kernel before this one: take this CTA's share of its keys
        pdl_wait();
        const uint32_t* src = p.keys_in + row * p.S + j0;
        for (uint32_t i = tid; i < n_local; i += THREADS) {
            const uint32_t k = __ldcg(&src[i]);
            keys[i] = k;
            my_max = max(my_max, k);
        }
    }
    for (uint32_t pp0 = 0; !p.keys_in && 2 * pp0 < n_local; pp0 += PB * THREADS) {
        uint32_t idx[2 * PB];
        bool ok[2 * PB];
#pragma unroll
        for (int b = 0; b < PB; ++b) {
            const uint32_t pp = pp0 + b * THREADS + tid;
            const uint64_t j = (uint64_t)j0 + 2ull * pp;             // even sample of the pair
            ok[2 * b] = j < j1;
            ok[2 * b + 1] = j + 1 < j1;
            idx[2 * b] = idx[2 * b + 1] = 0;
            if (ok[2 * b]) {
                const Philox4 r = philox4x32_10((uint32_t)(j >> 1), (uint32_t)row, (uint32_t)(row >> 32), 0u,
                                                (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
                const uint64_t b0 = stratum_start(j, p.q, p.rem, p.S, p.inv_s);
                const uint64_t b1 = stratum_start(j + 1, p.q, p.rem, p.S, p.inv_s);
                idx[2 * b] = (uint32_t)(b0 + __umul64hi(((uint64_t)r.y << 32) | r.x, b1 - b0));
                if (ok[2 * b + 1]) {
                    const uint64_t b2 = stratum_start(j + 2, p.q, p.rem, p.S, p.inv_s);
                    idx[2 * b + 1] = (uint32_t)(b1 + __umul64hi(((uint64_t)r.w << 32) | r.z, b2 - b1));
                }
            }
        }
        // The sample positions do not depend on the data: only now does the kernel need the work queued
        // before it on the stream (whatever produced the input, or the previous call on this workspace).
        // (Their cache lines and address translations are requested meanwhile: a prefetch has no effect
        // on memory, and L2 is where a later write by that work lands too.)
        if (pp0 == 0) {
#pragma unroll
            for (int s = 0; s < 2 * PB; ++s)
                if (ok[s]) asm volatile("prefetch.global.L2 [%0];" ::"l"(rowp + idx[s]));
            pdl_wait();
        }
        T val[2 * PB];
#pragma unroll
        for (int s = 0; s < 2 * PB; ++s)
            if (ok[s]) val[s] = rowp[idx[s]];
#pragma unroll
        for (int s = 0; s < 2 * PB; ++s) {
            if (ok[s]) {
                const uint32_t pp = pp0 + (s >> 1) * THREADS + tid;
                const uint32_t local = 2 * pp + (s & 1);
                const uint32_t k = Elem<T>::key(val[s]);
                keys[local] = k;
                if (p.keys_store) p.keys_store[row * p.S + j0 + local] = k;
                my_max = max(my_max, k);
                if (p.sample_idx) p.sample_idx[row * p.S + j0 + local] = idx[s];
            }
        }
    }
    pdl_wait();                  // CTAs without a share of the sample have not waited yet
    // The filter kernel may start its prologue now -- and not earlier.  It reads tiles of the input before its own
    // wait, which covers this kernel only; this kernel's wait has just returned, so whatever produced the input has
    // finished, even a producer that released its own dependents early.  The filter's prologue still overlaps the
    // whole selection below.
    pdl_launch_dependents();
    if (p.zero)
        for (uint32_t i = blockIdx.x * THREADS + tid; i < p.zero_vecs; i += gridDim.x * THREADS) p.zero[i] = make_uint4(0u, 0u, 0u, 0u);
    if (crank == 0 && tid == 0) {
        if (p.ctl) {
            RowCtl* c = p.ctl + row;
            c->count = 0; c->collect = 0; c->status = 0; c->n_final = 0; c->capacity = p.capacity; c->pad = 0;
            if (p.part_counts)
                for (int j = 0; j < (int)FILTER_PARTS; ++j) p.part_counts[(row * FILTER_PARTS + j) * FILTER_PART_STRIDE] = 0;
        }
        if (p.header && row == 0) {
            p.header->bar_count = 0; p.header->error = 0; p.header->done = 0; p.header->n_failed = 0; p.header->tile_counter = 0;
            for (int g = 0; g < WS_GROUPS; ++g) p.header->group_bar[g][0] = 0;
        }
    }

    bool done = false;

    // ---- stage 2, short cut for small ranks -------------------------------------------
    // Deeper ranks, up to GROUPS per CTA of the cluster: every CTA takes the ceil(t / csize)-th largest of its group
    // maxima -- it has that many keys at or above it -- and the smallest of these bounds over the cluster has
    // csize * ceil(t / csize) >= t keys at or above it: one more exchange through the first CTA's shared memory.
    // (A cluster uses the cluster-wide bound from rank SEL_WIDE_MIN on: with a bound of its own every CTA sends two to
    // three times t keys, and towards t = 128 sixteen CTAs overflow the room for candidates and fall into the radix select.)
    const bool bounded = p.t <= (uint32_t)GROUPS && (csize == 1 || p.t < SEL_WIDE_MIN);
    const uint32_t cta_rank = bounded ? p.t : (p.t + csize - 1) / csize;
    const bool wide = GENERAL && !bounded && csize > 1 && cta_rank <= (uint32_t)GROUPS;
    if (bounded || wide || !GENERAL) {
        if (bounded || wide) {
        // maxima of the groups of 8 consecutive lanes
        uint32_t g = my_max;
        g = max(g, __shfl_xor_sync(FULL_MASK, g, 1));
        g = max(g, __shfl_xor_sync(FULL_MASK, g, 2));
        g = max(g, __shfl_xor_sync(FULL_MASK, g, 4));
        if ((tid & 7u) == 0) gmax[tid >> 3] = g;
        __syncthreads();
        {   // rank of group tid/8 among the 128 maxima, the eight lanes of the group sharing the loop
            const unsigned grp = tid >> 3, part = tid & 7u;
            const uint32_t mine = gmax[grp];
            uint32_t rank = 0;
#pragma unroll
            for (int jj = 0; jj < GROUPS / 8; ++jj) {
                const unsigned j = part * (GROUPS / 8) + jj;
                const uint32_t o = gmax[j];
                rank += (o > mine) || (o == mine && j < grp);
            }
            rank += __shfl_xor_sync(FULL_MASK, rank, 1);
            rank += __shfl_xor_sync(FULL_MASK, rank, 2);
            rank += __shfl_xor_sync(FULL_MASK, rank, 4);
            if (part == 0 && rank == cta_rank - 1) s_lower = mine;     // at least cta_rank keys of this CTA are >= mine
        }
        }                                   // (not bounded: the bound stays 0 and every key is a candidate)
        __syncthreads();
        uint32_t lower = s_lower;
        // every CTA sends its keys >= lower to the first CTA: one remote atomic per warp that has any
        uint64_t* cand0 = cluster.map_shared_rank(cand, 0);
        uint32_t* ncand0 = cluster.map_shared_rank(&s_ncand, 0);
        cluster.barrier_wait(std::move(zeroed));
        if (wide) {
            uint32_t* lmin0 = cluster.map_shared_rank(&s_lmin, 0);
            if (tid == 0) atomicMin(lmin0, lower);
            cluster.sync();
            lower = *lmin0;
        }
        for (uint32_t i = tid; i < n_round; i += THREADS) {
            const uint32_t k = i < n_local ? keys[i] : 0;
            const bool take = i < n_local && k >= lower;
            const unsigned bal = __ballot_sync(FULL_MASK, take);
            if (bal) {
                uint32_t base = 0;
                if (lane == 0) base = atomicAdd(ncand0, (uint32_t)__popc(bal));
                base = __shfl_sync(FULL_MASK, base, 0);
                const uint32_t slot = base + __popc(bal & ((1u << lane) - 1u));
                if (take && slot < SEL_CAND_CAP) cand0[slot] = ((uint64_t)k << 32) | (uint64_t)(0xFFFFFFFFu - (j0 + i));
            }
        }
        cluster.sync();                               // all candidates have arrived
        const uint32_t ncand = *ncand0;
        if (ncand <= SEL_CAND_CAP) {
            // Every CTA takes a copy of the candidates and looks at its share of them (candidate c goes to
            // CTA c mod csize): the t-th largest record is the one candidate with exactly t - 1 candidates
            // above it.  Eight lanes share one candidate's comparisons.
            // A handful of candidates (small ranks) is not worth the copies: the first CTA looks at all.
            const bool spread = ncand > SEL_SPREAD_MIN;
            if (spread && crank != 0)
                for (uint32_t i = tid; i < ncand; i += THREADS) cand[i] = cand0[i];
            auto seen = cluster.barrier_arrive();     // "I have read the first CTA's memory": it may leave after its peers did
            if (spread) __syncthreads();
            const unsigned part = tid & 7u;
            const uint32_t c_first = spread ? (tid >> 3) * csize + crank : crank == 0 ? (tid >> 3) : ncand;
            const uint32_t c_step = (THREADS / 8) * (spread ? csize : 1u);
            for (uint32_t c = c_first; c < ncand; c += c_step) {      // whole groups of eight lanes together
                const uint64_t mine = cand[c];
                uint32_t above = 0;
                for (uint32_t j = part; j < ncand; j += 8) above += cand[j] > mine;
                const unsigned group = 0xFFu << (lane & 24u);
                above += __shfl_xor_sync(group, above, 1);
                above += __shfl_xor_sync(group, above, 2);
                above += __shfl_xor_sync(group, above, 4);
                if (part == 0 && above == p.t - 1)                                                      // tau
                    publish_threshold(p, row, (uint32_t)(mine >> 32), 0xFFFFFFFFu - (uint32_t)mine);
            }
            done = true;
            cluster.barrier_wait(std::move(seen));
        } else {
            auto seen = cluster.barrier_arrive();
            cluster.barrier_wait(std::move(seen));
        }
    } else {
        cluster.barrier_wait(std::move(zeroed));
    }

    // ---- stage 2, general case: radix select over the cluster --------------------------
    if constexpr (GENERAL) {
    if (!done) {
        static_assert(sizeof(cand) >= 2 * SEL_BINS * sizeof(uint32_t), "the histograms fit in the candidates' space");
        uint32_t (*hist)[SEL_BINS] = reinterpret_cast<uint32_t (*)[SEL_BINS]>(cand);   // this CTA's histogram, double-buffered
        constexpr int NPASS = sizeof(T) == 4 ? 3 : 2;
        constexpr int KB = Elem<T>::KEY_BITS;
        const int shifts[3] = {KB - 11, sizeof(T) == 4 ? 10 : 0, 0};
        const int widths[3] = {11, sizeof(T) == 4 ? 11 : 5, 10};
        uint32_t prefix = 0;        // selected high bits so far (right-aligned)
        uint32_t need = p.t;        // rank among the keys that match the prefix, from the top
        int consumed = 0;           // number of high bits fixed
#pragma unroll
        for (int pass = 0; pass < NPASS; ++pass) {
            const int shift = shifts[pass], width = widths[pass];
            const uint32_t nbins = 1u << width;
            uint32_t* h = hist[pass & 1];
            for (uint32_t b = tid; b < nbins; b += THREADS) h[b] = 0;
            __syncthreads();
            for (uint32_t i = tid; i < n_round; i += THREADS) {
                const uint32_t k = i < n_local ? keys[i] : 0;
                const bool in_class = i < n_local && (consumed == 0 || (k >> (KB - consumed)) == prefix);
                const uint32_t digit = in_class ? (k >> shift) & (nbins - 1) : 0xFFFFFFFFu;
                const unsigned peers = __match_any_sync(FULL_MASK, digit);
                if (in_class && lane == (unsigned)(__ffs(peers) - 1)) atomicAdd(&h[digit], __popc(peers));
            }
            cluster.sync();   // every CTA's histogram of this pass is complete

            // Sum the histograms of all CTAs; thread t owns the two bins 2t, 2t+1 counted from the top.
            uint32_t c0 = 0, c1 = 0;
            const uint32_t rb0 = 2 * tid, rb1 = 2 * tid + 1;            // reversed bin numbers
            if (rb0 < nbins) {
#pragma unroll 4
                for (unsigned c = 0; c < csize; ++c) {
                    const uint32_t* ph = cluster.map_shared_rank(h, c);
                    c0 += ph[nbins - 1 - rb0];
                    c1 += ph[nbins - 1 - rb1];
                }
            }
            const uint32_t incl = block_inclusive_scan(c0 + c1, warp_sums);   // keys in reversed bins <= rb1
            const uint32_t before0 = incl - c0 - c1, before1 = incl - c1;
            if (before0 < need && need <= before0 + c0) { s_digit = nbins - 1 - rb0; s_before = before0; }
            else if (before1 < need && need <= before1 + c1) { s_digit = nbins - 1 - rb1; s_before = before1; }
            __syncthreads();
            prefix = (prefix << width) | s_digit;
            need -= s_before;
            consumed += width;
            __syncthreads();   // s_digit / s_before are rewritten in the next pass
        }
        const uint32_t tau_key = prefix << (KB - consumed);
        // Of the samples with exactly this key the threshold record is the need-th in sample order.  CTAs hold
        // consecutive runs of the sample: count the equal keys per CTA, find the CTA that holds the need-th,
        // and there the position by scans over runs of THREADS keys.
        uint32_t eq = 0;
        for (uint32_t i = tid; i < n_local; i += THREADS) eq += keys[i] == tau_key;
        eq = block_inclusive_scan(eq, warp_sums);
        if (tid == THREADS - 1) s_ncand = eq;           // (the candidates' counter is free by now)
        cluster.sync();
        uint32_t before = 0;
        for (unsigned c = 0; c < crank; ++c) before += *cluster.map_shared_rank(&s_ncand, c);
        const uint32_t mine_eq = s_ncand;
        if (before < need && need <= before + mine_eq) {             // uniform over the CTA
            uint32_t left = need - before;                           // 1-based among this CTA's equal keys
            for (uint32_t c0 = 0; c0 < n_local; c0 += THREADS) {
                const uint32_t i = c0 + tid;
                const uint32_t flag = i < n_local && keys[i] == tau_key;
                __syncthreads();                                     // warp_sums of the scan before
                const uint32_t incl = block_inclusive_scan(flag, warp_sums);
                if (flag && incl == left) publish_threshold(p, row, tau_key, j0 + i);
                __syncthreads();
                const uint32_t in_run = warp_sums[31];
                if (in_run >= left) break;
                left -= in_run;
            }
        }
        cluster.sync();   // no CTA leaves while a peer may still read its histogram or its count
    }
    }
}

}  // namespace profk
