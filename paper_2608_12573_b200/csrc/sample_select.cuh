// Stages 1 and 2 (Section 3, "Sampling" and "Threshold estimation"): gather S stratified
// Philox samples of a row and select the t-th largest as the threshold tau.
//
// One thread-block cluster handles one row.  Each CTA of the cluster gathers its share of
// the samples into shared memory as order keys; the t-th largest key is found by a radix
// select whose per-digit histograms are summed across the cluster through distributed
// shared memory (hardware cluster barriers only -- no spinning on global memory).
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace profk {

namespace cg = cooperative_groups;

constexpr int SEL_THREADS = 1024;
constexpr int SEL_BINS = 2048;       // 11-bit digits

// Per-row control block in the workspace.
struct RowCtl {
    uint32_t tau_bits;   // threshold (element bit pattern)
    uint32_t count;      // survivors appended by the filter (R, or something > capacity)
    uint32_t collect;    // records appended by the exact-selection path
    uint32_t status;     // PROFK_ROW_* (| 0x80000000 on a timeout)
    uint32_t n_final;    // records the refine step has to order
    uint32_t capacity;
    uint32_t pad[2];
};
static_assert(sizeof(RowCtl) == 32, "RowCtl is 32 bytes");

// Header of the workspace: state of the grid barrier used by the exact-selection kernel.
struct WsHeader {
    uint32_t bar_count;
    uint32_t bar_gen;
    uint32_t error;      // non-zero = a bounded wait gave up
    uint32_t pad[61];
};
static_assert(sizeof(WsHeader) == 256, "WsHeader is 256 bytes");

template <typename T> struct SelectParams {
    const T* in;
    uint64_t N;
    uint32_t S;            // sample size
    uint32_t t;            // rank, 1-based, t-th largest
    uint64_t seed;
    uint32_t per_cta;      // samples per CTA of the cluster = ceil(S / cluster size)
    T* tau;                // rows thresholds out
    RowCtl* ctl;           // may be null (stand-alone use)
    WsHeader* header;      // may be null
    uint32_t capacity;
    uint32_t* sample_idx;  // may be null; rows x S
};

// Block-wide inclusive scan of one value per thread (blockDim.x == SEL_THREADS).
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

template <typename T>
__global__ void __launch_bounds__(SEL_THREADS, 1) sample_select_kernel(const SelectParams<T> p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw);          // per_cta keys
    __shared__ uint32_t hist[2][SEL_BINS];                           // this CTA's histogram, double-buffered
    __shared__ uint32_t warp_sums[32];
    __shared__ uint32_t s_digit, s_before;

    cg::cluster_group cluster = cg::this_cluster();
    const unsigned csize = cluster.num_blocks();
    const unsigned crank = cluster.block_rank();
    const uint64_t row = blockIdx.x / csize;
    const unsigned tid = threadIdx.x;

    pdl_launch_dependents();   // the filter kernel may start its prologue now

    // ---- stage 1: gather this CTA's share of the sample -------------------------------
    const uint32_t j0 = crank * p.per_cta;
    const uint32_t j1 = min(p.S, j0 + p.per_cta);
    const uint32_t n_local = j1 > j0 ? j1 - j0 : 0;
    const T* rowp = p.in + row * p.N;
    for (uint32_t i = tid; i < n_local; i += SEL_THREADS) {
        const uint32_t idx = sample_index(p.N, p.S, j0 + i, row, p.seed);
        keys[i] = Elem<T>::key(rowp[idx]);
        if (p.sample_idx) p.sample_idx[row * p.S + j0 + i] = idx;
    }
    if (crank == 0 && tid == 0) {
        if (p.ctl) {
            RowCtl* c = p.ctl + row;
            c->count = 0; c->collect = 0; c->status = 0; c->n_final = 0; c->capacity = p.capacity;
        }
        if (p.header && row == 0) { p.header->bar_count = 0; p.header->error = 0; }
    }

    // ---- stage 2: radix select of the t-th largest key over the cluster ----------------
    constexpr int NPASS = sizeof(T) == 4 ? 3 : 2;
    const int shifts[3] = {21, sizeof(T) == 4 ? 10 : 16, 0};
    const int widths[3] = {11, sizeof(T) == 4 ? 11 : 5, 10};

    uint32_t prefix = 0;        // selected high bits so far (right-aligned)
    uint32_t need = p.t;        // rank among the keys that match the prefix, from the top
    int consumed = 0;           // number of high bits fixed
#pragma unroll
    for (int pass = 0; pass < NPASS; ++pass) {
        const int shift = shifts[pass], width = widths[pass];
        const uint32_t nbins = 1u << width;
        uint32_t* h = hist[pass & 1];
        for (uint32_t b = tid; b < nbins; b += SEL_THREADS) h[b] = 0;
        __syncthreads();
        for (uint32_t i = tid; i < n_local; i += SEL_THREADS) {
            const uint32_t k = keys[i];
            if (consumed == 0 || (k >> (32 - consumed)) == prefix) atomicAdd(&h[(k >> shift) & (nbins - 1)], 1u);
        }
        cluster.sync();   // every CTA's histogram of this pass is complete

        // Sum the histograms of all CTAs; thread t owns the two bins 2t, 2t+1 counted from the top.
        uint32_t c0 = 0, c1 = 0;
        const uint32_t rb0 = 2 * tid, rb1 = 2 * tid + 1;            // reversed bin numbers
        if (rb0 < nbins) {
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
    const uint32_t tau_key = prefix << (32 - consumed);

    if (crank == 0 && tid == 0) {
        const T tau = Elem<T>::from_key(tau_key);
        p.tau[row] = tau;
        if (p.ctl) p.ctl[row].tau_bits = Elem<T>::bits(tau);
    }
    cluster.sync();   // no CTA leaves while a peer may still read its histogram
}

}  // namespace profk
