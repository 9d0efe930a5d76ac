// One row split over several GPUs (the paper's "Limitations" leave distributed settings to future work; the four
// stages of Section 3 split at two exchange points): every GPU holds a contiguous shard of the row that is made of
// whole sampling strata, so
//   1. it gathers the keys of its own strata (gather_kernel with a pair offset) -- exchange: all-gather of the S keys;
//   2. every GPU selects the same threshold record from the S keys (sample_select_kernel on given keys);
//   3. it filters its shard with that threshold, indices local to the shard (filter_kernel; the threshold record is
//      first rewritten in the shard's coordinates, below) -- exchange: all-gather of (count, records);
//   4. the gathered records get their global indices and go through the ordinary count check and refinement.
// The two small kernels here do the rewriting (3) and the merge (4).  Remote memory is never an operand: the exchanges
// are made by the caller into local buffers.
#pragma once

#include "sample_select.cuh"

namespace profk {

constexpr int SHARD_MAX = 16;              // most shards of one row
constexpr int SHARD_STATE_WORDS = 8;       // per shard: [0] survivor count, [4..7] the threshold record in shard coordinates

struct ShardBases { long long base[SHARD_MAX]; };

// The row's threshold record {bits of tau, bits of the next value up, index of the threshold record or 0xFFFFFFFF, 0}
// in the coordinates of the shard [base, base + len): copies of tau are kept up to the record's index, so a shard that
// lies wholly before it keeps all of its copies, a shard wholly behind it none -- which is "everything from the next
// value up" (when tau is the largest bit pattern there is no such value and the shard keeps its copies: a superset,
// harmless to the result).  Also zeroes the shard's survivor count.
__global__ void localize_threshold_kernel(const uint4* thr_global, unsigned long long base, unsigned long long len, uint32_t* state) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const uint4 t = *thr_global;
    uint4 loc = t;
    if (t.z != 0xFFFFFFFFu) {
        if ((unsigned long long)t.z < base) { loc.x = t.y; loc.y = t.y; loc.z = 0xFFFFFFFFu; }
        else if ((unsigned long long)t.z >= base + len) loc.z = 0xFFFFFFFFu;
        else loc.z = (uint32_t)((unsigned long long)t.z - base);
    }
    state[0] = 0; state[1] = 0; state[2] = 0; state[3] = 0;
    *reinterpret_cast<uint4*>(state + 4) = loc;
}

// Merges the shards' candidate records into the row's buffer (global indices = local index + the shard's base), sets
// up the row's control block for the refine kernel that follows, and reports the count check: status_out[0] =
// ROW_OK / ROW_RECALL / ROW_OVERFLOW, status_out[1] = R (the sum of the shards' counts).  A shard whose own buffer
// overflowed makes the row overflow.
__global__ void merge_shards_kernel(const uint64_t* records, const uint32_t* states, ShardBases bases, uint32_t shards, uint32_t shard_cap,
                                    uint32_t capacity, uint32_t k, uint32_t k_accept, const uint4* thr_global, uint64_t* buf, RowCtl* ctl,
                                    WsHeader* header, uint32_t* status_out) {
    uint32_t first[SHARD_MAX + 1];
    bool shard_full = false;
    uint64_t total = 0;
    for (uint32_t g = 0; g < shards; ++g) {
        const uint32_t c = states[g * SHARD_STATE_WORDS];
        shard_full |= c > shard_cap;
        first[g] = (uint32_t)total;
        total += c < shard_cap ? c : shard_cap;
    }
    first[shards] = (uint32_t)total;
    const bool overflow = shard_full || total > capacity;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const uint4 t = *thr_global;
        RowCtl* c = ctl;
        c->tau_bits = t.x; c->count = overflow ? capacity + 1 : (uint32_t)total; c->collect = 0; c->status = 0; c->n_final = 0;
        c->capacity = capacity; c->tau_idx = t.z; c->pad = 0;
        header->bar_count = 0; header->error = 0; header->done = 0; header->n_failed = 0; header->tile_counter = 0;
        for (int g = 0; g < WS_GROUPS; ++g) header->group_bar[g][0] = 0;
        status_out[0] = overflow ? 2u : total < k_accept ? 1u : 0u;
        status_out[1] = total > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)total;
    }
    if (overflow) return;
    const uint64_t gthreads = (uint64_t)gridDim.x * blockDim.x;
    for (uint32_t g = 0; g < shards; ++g) {
        const uint32_t n = first[g + 1] - first[g];
        const uint64_t* src = records + (uint64_t)g * shard_cap;
        for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gthreads)
            buf[first[g] + i] = src[i] + (uint64_t)bases.base[g];
    }
}

}  // namespace profk
