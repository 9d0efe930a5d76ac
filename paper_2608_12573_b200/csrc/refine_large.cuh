// Stage 4 for large selections (k beyond what one CTA orders in shared memory; the flattened
// BatchTopK case of Section 5, "Application", selects K = B k = 131,072 values): the count
// check, then a full ascending sort of the row's candidate records -- which is "value
// descending, index ascending" -- by one thread-block cluster, and the first k are the answer.
//
// The sort is a bitonic network over P = 2^j records in the row's buffer (padded with all-ones
// records).  Exchanges at distance below one tile (16384 records = 128 KB) run in shared
// memory, tile by tile; the few longer ones run on the buffer in global memory, separated by
// hardware cluster barriers.  A bitonic network does the same work whatever the data, so
// heavy ties (bf16 inputs hold thousands of copies of each value near the threshold) cost
// nothing extra.
#pragma once

#include <cooperative_groups.h>

#include "refine.cuh"

namespace profk {

constexpr uint32_t BT_TILE = 16384;          // records per shared-memory tile
constexpr int BT_THREADS = 1024;

template <typename T> struct LargeParams {
    RowCtl* ctl;
    WsHeader* header;
    uint64_t* buf;           // rows x row_stride records; row_stride is a power of two >= capacity, >= BT_TILE
    uint64_t row_stride;
    uint32_t capacity;
    uint32_t k;
    uint32_t k_accept;
    int phase;               // 0 = count check, then sort the rows that pass; 1 = sort the rows the exact selection repaired
    T* out_vals;             // rows x k
    int64_t* out_idx;        // rows x k
    int use_pdl;
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

template <typename T>
__global__ void __launch_bounds__(BT_THREADS, 1) refine_large_kernel(const LargeParams<T> p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* tile = reinterpret_cast<uint64_t*>(smem_raw);          // BT_TILE records

    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned csize = cluster.num_blocks();
    const unsigned crank = cluster.block_rank();
    const uint64_t row = blockIdx.x / csize;
    const unsigned tid = threadIdx.x;
    const uint64_t gid = (uint64_t)crank * BT_THREADS + tid;         // thread index inside the cluster
    const uint64_t gthreads = (uint64_t)csize * BT_THREADS;

    pdl_launch_dependents();
    if (p.use_pdl) pdl_wait();

    // ---- which rows this launch handles (the decision is the same in every CTA of the cluster) ----
    const RowCtl ctl = p.ctl[row];
    uint32_t n;
    if (p.phase == 0) {
        const uint32_t R = ctl.count;
        const uint32_t status = R > p.capacity ? ROW_OVERFLOW : R < p.k_accept ? ROW_RECALL : ROW_OK;
        if (crank == 0 && tid == 0) {
            p.ctl[row].status = status;
            p.ctl[row].n_final = status ? p.k : R;
            if (status) atomicAdd(&p.header->n_failed, 1u);
        }
        if (status != ROW_OK) return;        // the exact-selection kernel and the second phase take this row
        n = R;
    } else {
        if (ctl.status == ROW_OK) return;    // already written by the first phase
        n = p.k;                             // the exact selection left exactly k records
    }
    const uint32_t kk = n < p.k ? n : p.k;
    uint64_t* G = p.buf + row * p.row_stride;
    uint64_t P = BT_TILE;
    while (P < n) P <<= 1;

    for (uint64_t j = kk + gid; j < p.k; j += gthreads) {            // relaxed mode: padding after a short buffer
        p.out_vals[row * (uint64_t)p.k + j] = Elem<T>::from_bits(Elem<T>::NEG_INF_BITS);
        p.out_idx[row * (uint64_t)p.k + j] = -1;
    }

    // ---- sort every tile (sizes 2 .. BT_TILE); positions beyond n hold all-ones padding ----
    const uint64_t tiles = P / BT_TILE;
    for (uint64_t t = crank; t < tiles; t += csize) {
        const uint64_t base = t * BT_TILE;
        for (uint32_t i = tid; i < BT_TILE; i += BT_THREADS) tile[i] = base + i < n ? __ldcg(&G[base + i]) : ~0ull;
        __syncthreads();
        bitonic_tile_steps(tile, base, 2, BT_TILE);
        for (uint32_t i = tid; i < BT_TILE; i += BT_THREADS) G[base + i] = tile[i];
        __syncthreads();
    }
    cluster.sync();

    // ---- merge: exchanges at distance >= BT_TILE on the buffer, the rest tile by tile ----
    for (uint64_t size = 2ull * BT_TILE; size <= P; size <<= 1) {
        for (uint64_t stride = size / 2; stride >= BT_TILE; stride >>= 1) {
            for (uint64_t q = gid; q < P / 2; q += gthreads) {
                const uint64_t lo = 2 * q - (q & (stride - 1));
                const uint64_t hi = lo + stride;
                const bool ascending = (lo & size) == 0;
                const uint64_t x = __ldcg(&G[lo]), y = __ldcg(&G[hi]);
                if ((x > y) == ascending) { G[lo] = y; G[hi] = x; }
            }
            cluster.sync();
        }
        for (uint64_t t = crank; t < tiles; t += csize) {
            const uint64_t base = t * BT_TILE;
            for (uint32_t i = tid; i < BT_TILE; i += BT_THREADS) tile[i] = __ldcg(&G[base + i]);
            __syncthreads();
            bitonic_tile_steps(tile, base, size, size);
            for (uint32_t i = tid; i < BT_TILE; i += BT_THREADS) G[base + i] = tile[i];
            __syncthreads();
        }
        cluster.sync();
    }

    for (uint64_t j = gid; j < kk; j += gthreads) write_output(p.out_vals, p.out_idx, p.k, row, (uint32_t)j, __ldcg(&G[j]));
}

}  // namespace profk
