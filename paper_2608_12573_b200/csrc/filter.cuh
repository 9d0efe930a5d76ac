// Stage 3, the filtering scan (Section 3, "Filtering"): stream every row once and append
// each element with x_i >= tau to the row's candidate buffer.
//
// The kernel is bound by HBM bandwidth: one 128-bit load per VEC elements, one compare
// per element, and nothing else on the common path.  Survivors are rare (1e-3 .. 1e-5 of
// the elements), so the append is a warp-cooperative slow path taken only when some lane
// of the warp saw a survivor: one atomic on the row's counter per warp and tile, records
// written straight to the row's buffer (eight counters and eight parts of the buffer for
// large selections from long rows).  Where survivors are dense -- one or more per
// warp-tile -- the DEFER build only notes its candidates while it streams and decides them
// afterwards, with every lane busy; its HIST form also counts the records it appends in
// the bins that the kernel behind it selects from.
#pragma once

#include "bins.cuh"
#include "rowscan.cuh"

// Launch shape of the filter kernel (tuned on B200; overridable at build time for experiments).
#ifndef PROFK_FILTER_THREADS
#define PROFK_FILTER_THREADS 512
#endif
#ifndef PROFK_FILTER_UNROLL
#define PROFK_FILTER_UNROLL 4
#endif
#ifndef PROFK_FILTER_MINBLOCKS_F32
#define PROFK_FILTER_MINBLOCKS_F32 3
#endif
#ifndef PROFK_FILTER_MINBLOCKS_BF16
#define PROFK_FILTER_MINBLOCKS_BF16 3            // the direct-append variant fits 40 registers without spills
#endif

namespace profk {

template <typename T> struct FilterParams {
    const T* in;
    uint64_t N;
    uint64_t rows;
    const T* tau;            // rows thresholds
    uint32_t capacity;       // records per row buffer
    uint64_t* buf;           // row r's records start at buf + r * buf_stride
    uint64_t buf_stride;
    uint32_t* counts;        // per-row survivor counter (stride in 32-bit words)
    uint32_t count_stride;
    uint64_t tiles_per_row;
    uint64_t total_tiles;
    int use_pdl;             // 1 = launched as a programmatic dependent of the threshold kernel
    uint32_t* tile_counter;  // zeroed counter that hands out the tiles from dyn_start on (null = fixed stride throughout)
    uint32_t dyn_start;      // first tile handed out dynamically (a multiple of the grid size)
    uint32_t dyn_chunk;      // consecutive tiles a CTA takes from the counter at a time (>= 1)
    // Partitioned append (the PARTS build of the kernel only).  With very many survivors the single counter of a
    // row becomes the bottleneck -- atomics on one address retire about 2 ns apart, 164 K of them are a quarter of
    // a 2^30-element scan -- so the row's buffer is cut into FILTER_PARTS equal parts, each with a counter in a
    // cache line of its own, and the survivors of a tile go to part (tile index in the row) mod FILTER_PARTS.
    uint32_t part_cap;       // records per part
    uint32_t* part_counts;   // row r, part j: part_counts[(r * FILTER_PARTS + j) * FILTER_PART_STRIDE] (zeroed)
    // Threshold records written by the threshold kernel (null = take `tau`, a value alone): row r's is {bits of tau,
    // bits of the value that follows tau in the total order, tau_idx, 0}.  Of the elements with exactly tau's bit
    // pattern only those with an index <= tau_idx are kept (0xFFFFFFFF: all of them), so that a flood of copies of tau
    // does not fill the buffer.
    const uint4* thr;
    // Tiles (0 or FILTER_PREFETCH) a CTA copies into its shared memory while it waits for the threshold kernel, beyond
    // the one it holds in registers: the input does not depend on the threshold, and HBM is idle meanwhile.
    uint32_t prefetch_tiles;
    // Polls of the mbarrier that counts those copies before the CTA gives up on them and reads the tiles with plain
    // loads (PREFETCH_SPIN_LIMIT; a test sets 0 to take that branch).  The wait before the CTA leaves always has the
    // full limit: shared memory must not be handed on while a copy into it is in flight.
    uint32_t prefetch_spin_limit;
    // The HIST build (one row, large selections): every record appended is also counted in the bins of bins.cuh -- the
    // fine bins at hist[0 .. BIN_COUNT) with one global atomic, the coarse ones through the CTA's shared memory -- so that
    // the kernel behind this one finds its histogram made (unless the flag word BIN_FLAG_UNCOUNTED says that some records
    // went uncounted).  All BIN_ROW_WORDS words are zero when the scan starts.
    uint32_t* hist;
    int idx_bits;            // bits an index of the row occupies
};

// What the appending code of the HIST build needs to count a record (an empty shell otherwise).
struct HistCtx {
    uint32_t* fine;          // global
    uint32_t* coarse;        // shared memory of the CTA
    uint32_t top_hi;         // high word of the largest record the filter keeps: tau's key, inverted
    int idx_bits;
    __device__ __forceinline__ void count(uint64_t rec) const {
        const uint32_t b = record_bin(rec, top_hi, idx_bits);
        atomicAdd(&fine[b], 1u);
        atomicAdd(&coarse[b / BIN_PER_COARSE], 1u);
    }
};

constexpr uint32_t FILTER_PREFETCH = 2;
constexpr uint32_t PREFETCH_SPIN_LIMIT = 1u << 22;

// Bit l set = element l of the vector is not below tau (the same test as vec_any_pass, per element).
__device__ __forceinline__ unsigned vec_pass_mask(const float4& v, float tau) {
    return (unsigned)!(v.x < tau) | ((unsigned)!(v.y < tau) << 1) | ((unsigned)!(v.z < tau) << 2) | ((unsigned)!(v.w < tau) << 3);
}
__device__ __forceinline__ unsigned vec_pass_mask(const uint4& v, __nv_bfloat16 tau) {
    const __nv_bfloat162 t2 = __halves2bfloat162(tau, tau);
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
    unsigned m = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const unsigned below = __hlt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&w[j]), t2);   // 0xFFFF per half that is < tau
        m |= ((~below & 1u) | ((~below >> 15) & 2u)) << (2 * j);
    }
    return m;
}

// Does the vector hold an element that floating point calls equal to tau, or unordered with it (a NaN on either
// side)?  Those are the elements on which the float test and the total order of the keys can differ: a copy of tau,
// a zero of the other sign, a NaN.  One "equal or unordered" comparison per element.
__device__ __forceinline__ bool vec_any_equal_or_unordered(const float4& v, float tau) {
    unsigned r;
    asm("{\n\t.reg .pred a, b, c, d;\n\t"
        "setp.equ.f32 a, %1, %5;\n\tsetp.equ.f32 b, %2, %5;\n\tsetp.equ.f32 c, %3, %5;\n\tsetp.equ.f32 d, %4, %5;\n\t"
        "or.pred a, a, b;\n\tor.pred c, c, d;\n\tor.pred a, a, c;\n\tselp.u32 %0, 1, 0, a;\n\t}"
        : "=r"(r) : "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "f"(tau));
    return r != 0;
}
__device__ __forceinline__ bool vec_any_equal_or_unordered(const uint4& v, __nv_bfloat16 tau) {
    const __nv_bfloat162 t2 = __halves2bfloat162(tau, tau);
    return (__hequ2_mask(*reinterpret_cast<const __nv_bfloat162*>(&v.x), t2) | __hequ2_mask(*reinterpret_cast<const __nv_bfloat162*>(&v.y), t2) |
            __hequ2_mask(*reinterpret_cast<const __nv_bfloat162*>(&v.z), t2) | __hequ2_mask(*reinterpret_cast<const __nv_bfloat162*>(&v.w), t2)) != 0;
}

// Index up to which copies of tau are kept in `row` (read on the slow paths only).
template <typename T>
__device__ __forceinline__ uint32_t tie_limit(const FilterParams<T>& p, uint32_t row) {
    return p.thr ? reinterpret_cast<const uint32_t*>(p.thr + row)[2] : 0xFFFFFFFFu;
}

// The exact test, in the total order of the keys, for the elements of a vector that passed the float test
// "not (x < tau)" (mask m; element l has index i0 + l): kept are the elements above tau and the copies of tau at
// or before the threshold record.  The float test lets through a few more: -0.0 for tau = +0.0, NaNs with the sign
// bit set (they rank lowest), copies of tau beyond the record.  An element that floating point puts strictly above
// tau is above it in the total order too, so only vectors with an element equal to tau or unordered with it -- rare
// -- are looked at, and the record's index is read only when a copy of tau turns up.
template <typename T>
__device__ __noinline__ unsigned confirm_each(const FilterParams<T>& p, uint32_t row, typename Elem<T>::vec_t v, unsigned m, int64_t i0, T tau) {
    unsigned keep = m;
    const uint32_t tau_key = Elem<T>::key(tau);
    while (m) {
        const int l = __ffs(m) - 1;
        m &= m - 1;
        const uint32_t key = Elem<T>::key(vec_elem(v, l));
        if (key < tau_key || (key == tau_key && i0 + l > (int64_t)tie_limit(p, row))) keep &= ~(1u << l);
    }
    return keep;
}
template <typename T>
__device__ __forceinline__ unsigned confirm_survivors(const FilterParams<T>& p, uint32_t row, const typename Elem<T>::vec_t& v,
                                                      unsigned m, int64_t i0, T tau) {
    return vec_any_equal_or_unordered(v, tau) ? confirm_each<T>(p, row, v, m, i0, tau) : m;
}


// not (x < tau) for every lane of a vector, OR-ed: does the vector hold any survivor?
__device__ __forceinline__ bool vec_any_pass(const float4& v, float tau) {
    return !(v.x < tau) | !(v.y < tau) | !(v.z < tau) | !(v.w < tau);
}
__device__ __forceinline__ bool vec_any_pass(const uint4& v, __nv_bfloat16 tau) {
    const __nv_bfloat162 t2 = __halves2bfloat162(tau, tau);
    const unsigned a = __hlt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&v.x), t2);
    const unsigned b = __hlt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&v.y), t2);
    const unsigned c = __hlt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&v.z), t2);
    const unsigned d = __hlt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&v.w), t2);
    return (a & b & c & d) != 0xFFFFFFFFu;    // some lane is not below tau
}

// Survivors of one thread's vectors of a tile: bit u * VEC + l set = element l of vector u is inside the row
// and kept.  Vectors without an element that is not below tau (nearly all) cost one packed test.
template <typename T, int THREADS, int UNROLL>
__device__ __forceinline__ uint32_t survivor_mask(const typename Elem<T>::vec_t (&v)[UNROLL], uint32_t inside_mask, uint64_t N,
                                                  uint64_t qbase, uint32_t mis, T tau, const FilterParams<T>& p, uint32_t row) {
    constexpr int VEC = Elem<T>::VEC;
    static_assert(VEC * UNROLL <= 32, "one bit per element of the thread's share of a tile");
    uint32_t mine = 0;
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
        if (((inside_mask >> u) & 1u) && vec_any_pass(v[u], tau)) {
            const uint64_t q = qbase + (uint64_t)u * THREADS + threadIdx.x;
            const int64_t i0 = (int64_t)(q * VEC) - (int64_t)mis;
            unsigned m = vec_pass_mask(v[u], tau);
            if (i0 < 0 || i0 + VEC > (int64_t)N) {          // a vector across an end of the row: drop the lanes outside
#pragma unroll
                for (int l = 0; l < VEC; ++l)
                    if (i0 + l < 0 || i0 + l >= (int64_t)N) m &= ~(1u << l);
            }
            mine |= confirm_survivors<T>(p, row, v[u], m, i0, tau) << (u * VEC);
        }
    }
    return mine;
}

// Exclusive prefix of cnt over the lanes of the warp, and the warp's total.  Survivors are rare: usually no
// lane has more than one, and a vote does it; otherwise a shuffle scan.
__device__ __forceinline__ unsigned warp_exclusive_count(unsigned cnt, unsigned lane, unsigned* total) {
    const unsigned has = __ballot_sync(FULL_MASK, cnt != 0);
    if (!__any_sync(FULL_MASK, cnt > 1)) {
        *total = __popc(has);
        return __popc(has & ((1u << lane) - 1u));
    }
    unsigned incl = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned nb = __shfl_up_sync(FULL_MASK, incl, d);
        if (lane >= (unsigned)d) incl += nb;
    }
    *total = __shfl_sync(FULL_MASK, incl, 31);
    return incl - cnt;
}

// Writes one thread's survivors as records to out[pos], out[pos + 1], ... (positions >= limit are dropped).
// Survivors are few: a loop over the set bits, each picking its element out of the registers.
template <typename T, int THREADS, int UNROLL, bool HIST = false>
__device__ __forceinline__ void emit_survivors(const typename Elem<T>::vec_t (&v)[UNROLL], uint32_t mine, uint64_t qbase,
                                               uint32_t mis, uint64_t* out, unsigned pos, unsigned limit, const HistCtx& hc = HistCtx{}) {
    constexpr int VEC = Elem<T>::VEC;
    static_assert(UNROLL == 4, "four vectors per thread and tile");
    while (mine) {
        const int b = __ffs(mine) - 1;
        mine &= mine - 1;
        const int u = b / VEC, l = b % VEC;
        const T x = u == 0 ? vec_elem(v[0], l) : u == 1 ? vec_elem(v[1], l) : u == 2 ? vec_elem(v[2], l) : vec_elem(v[3], l);
        const uint64_t q = qbase + (uint64_t)u * THREADS + threadIdx.x;
        const uint32_t i = (uint32_t)((int64_t)(q * VEC) - (int64_t)mis) + (uint32_t)l;
        if (pos < limit) {
            const uint64_t rec = make_record(Elem<T>::key(x), i);
            out[pos] = rec;
            if (HIST) hc.count(rec);
        }
        ++pos;
    }
}

// The slow path: one global atomic per warp and tile, records written straight to the row buffer.  Returns the row if its buffer has overflowed, else ~0.
template <typename T, int THREADS, int UNROLL, bool PARTS, bool HIST = false>
__device__ __forceinline__ uint32_t filter_slow_path_direct(const FilterParams<T>& p, const typename Elem<T>::vec_t (&v)[UNROLL],
                                                            uint32_t inside_mask, uint32_t row, uint64_t qbase, uint32_t mis, T tau,
                                                            uint32_t* hist_coarse = nullptr) {
    const unsigned lane = lane_id();
    const uint32_t mine = survivor_mask<T, THREADS, UNROLL>(v, inside_mask, p.N, qbase, mis, tau, p, row);
    const unsigned cnt = __popc(mine);
    unsigned total;
    const unsigned before = warp_exclusive_count(cnt, lane, &total);
    if (total == 0) return 0xFFFFFFFFu;
    uint32_t* counter = p.counts + (uint64_t)row * p.count_stride;
    uint64_t* dst = p.buf + (uint64_t)row * p.buf_stride;
    uint32_t cap = p.capacity;
    if (PARTS) {
        // (the part follows the tile, not the CTA: every part gets an eighth of the row's tiles whoever scans them --
        // with the tiles dealt from the counter, a few CTAs take most of a late row and their parts overflowed)
        const uint32_t part = (uint32_t)(qbase / ((uint64_t)THREADS * UNROLL)) % FILTER_PARTS;
        counter = p.part_counts + ((uint64_t)row * FILTER_PARTS + part) * FILTER_PART_STRIDE;
        dst += (uint64_t)part * p.part_cap;
        cap = p.part_cap;
    }
    unsigned base = 0;
    if (lane == 0) base = atomicAdd(counter, total);
    base = __shfl_sync(FULL_MASK, base, 0);
    if (cnt) {
        if (HIST) emit_survivors<T, THREADS, UNROLL, true>(v, mine, qbase, mis, dst, base + before, cap, HistCtx{p.hist, hist_coarse, ~Elem<T>::key(tau), p.idx_bits});
        else emit_survivors<T, THREADS, UNROLL>(v, mine, qbase, mis, dst, base + before, cap);
    }
    return (uint64_t)base + total > cap ? row : 0xFFFFFFFFu;
}

// DEFER build (many survivors: batches of short rows, dense selections).  With one or two survivors per warp-tile most
// tiles would take the slow path above, whose few hundred warp instructions -- executed for the sake of one or two lanes
// -- make the scan instruction-bound (359 warp instructions per bf16 warp-tile on 2^20-element rows with k = 32, against
// 164 with no survivor at all).  Here a warp whose tile holds a candidate only NOTES it: the lanes that hold an element
// not below the threshold -- one or two of the 32 as a rule -- reserve room with a shared-memory atomic and write the
// numbers of their candidate vectors into a list in the CTA's shared memory; the other lanes do nothing, and no global
// memory is touched.  When the CTA has streamed all its tiles it works the list off with every lane busy: thread i reads
// candidate vector i again (the candidates are a few percent of the input at most), decides its elements exactly and
// appends the survivors.  A warp that finds the list full takes the slow path above instead.
#ifndef PROFK_DEFER_CAP
#define PROFK_DEFER_CAP 6144
#endif
constexpr uint32_t DEFER_CAP = PROFK_DEFER_CAP;      // candidate vectors per CTA: 24 KB of shared memory
constexpr uint32_t DEFER_NONE = 0xFFFFFFFFu;          // a reserved slot that was not used

// One batch of 32 list entries worked off: lane by lane a candidate vector (number `vid` among the vectors of the launch,
// tiles in order; DEFER_NONE = none) is read again and decided in the total order of the keys; the survivors are
// appended with one atomic per row that has survivors among them.  All 32 lanes call it.
// A list entry decided: candidate vector number `vid` among the vectors of the launch (tiles in order; DEFER_NONE = none)
// is read again and its elements are tested in the total order of the keys.
template <typename T> struct DeferDecided {
    typename Elem<T>::vec_t v;
    int64_t i0;        // index of the vector's first element in its row
    uint32_t row;
    unsigned m;        // bit j: element j is kept
    uint32_t top_hi;   // (HIST) what HistCtx needs of the row's threshold
};
template <typename T, int THREADS, int UNROLL>
__device__ __forceinline__ DeferDecided<T> defer_decide(const FilterParams<T>& p, uint32_t vid) {
    constexpr int VEC = Elem<T>::VEC;
    constexpr uint32_t TILE_VECTORS = THREADS * UNROLL;
    DeferDecided<T> d = {};
    if (vid != DEFER_NONE) {
        const uint32_t tile = vid / TILE_VECTORS, within = vid % TILE_VECTORS;
        const uint32_t tiles_per_row = (uint32_t)p.tiles_per_row;
        uint32_t tin = tile;
        if (tiles_per_row != (uint32_t)p.total_tiles) { d.row = tile / tiles_per_row; tin = tile - d.row * tiles_per_row; }
        const RowView<T> rv = row_view(p.in, p.N, d.row);
        const T tau = p.thr ? Elem<T>::from_bits(reinterpret_cast<const uint32_t*>(p.thr + d.row)[0]) : p.tau[d.row];
        const uint64_t q = (uint64_t)tin * TILE_VECTORS + within;
        bool in;
        d.v = load_row_vector(rv, p.N, q, &in);
        if (in) {
            d.i0 = (int64_t)(q * VEC) - (int64_t)rv.mis;
            d.m = vec_pass_mask(d.v, tau);
            if (d.i0 < 0 || d.i0 + VEC > (int64_t)p.N) {
#pragma unroll
                for (int j = 0; j < VEC; ++j)
                    if (d.i0 + j < 0 || d.i0 + j >= (int64_t)p.N) d.m &= ~(1u << j);
            }
            d.m = confirm_survivors<T>(p, d.row, d.v, d.m, d.i0, tau);
            d.top_hi = ~Elem<T>::key(tau);
        }
    }
    return d;
}

// One batch of 32 list entries worked off, lane by lane one entry; the survivors are appended with one atomic per row
// that has survivors among them.  All 32 lanes call it.
template <typename T, int THREADS, int UNROLL, bool PARTS, bool HIST = false>
__device__ __forceinline__ void defer_process_batch(const FilterParams<T>& p, uint32_t vid, uint32_t* hist_coarse = nullptr) {
    const unsigned lane = lane_id();
    const DeferDecided<T> d = defer_decide<T, THREADS, UNROLL>(p, vid);
    const uint32_t row = d.row;
    const unsigned m = d.m;
    const typename Elem<T>::vec_t v = d.v;
    const int64_t i0 = d.i0;
    const HistCtx hc = {p.hist, hist_coarse, d.top_hi, p.idx_bits};
    // Append, one atomic per row that has survivors in this batch (32 consecutive entries of the list span a tile or two,
    // so one or two rows): the lanes of the first row with survivors form a group, scan their counts, their first lane
    // reserves the room; then the next row's lanes, until none is left.
    const unsigned cnt = __popc(m);
    unsigned left = __ballot_sync(FULL_MASK, cnt != 0);
    while (left) {
        const uint32_t row0 = __shfl_sync(FULL_MASK, row, __ffs(left) - 1);
        const bool mine = cnt != 0 && row == row0;
        const unsigned group = __ballot_sync(FULL_MASK, mine);
        unsigned incl = mine ? cnt : 0u;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned nb = __shfl_up_sync(FULL_MASK, incl, d);
            if (lane >= (unsigned)d) incl += nb;
        }
        const unsigned total = __shfl_sync(FULL_MASK, incl, 31);
        uint32_t* counter = p.counts + (uint64_t)row0 * p.count_stride;
        uint64_t* dst = p.buf + (uint64_t)row0 * p.buf_stride;
        uint32_t cap = p.capacity;
        if (PARTS) {
            const uint32_t part = blockIdx.x % FILTER_PARTS;
            counter = p.part_counts + ((uint64_t)row0 * FILTER_PARTS + part) * FILTER_PART_STRIDE;
            dst += (uint64_t)part * p.part_cap;
            cap = p.part_cap;
        }
        unsigned base = 0;
        if (lane == (unsigned)(__ffs(group) - 1)) base = atomicAdd(counter, total);
        base = __shfl_sync(FULL_MASK, base, __ffs(group) - 1);
        if (mine) {
            unsigned pos = base + incl - cnt;
            unsigned mm = m;
            while (mm) {
                const int b = __ffs(mm) - 1;
                mm &= mm - 1;
                if (pos < cap) {
                    const uint64_t rec = make_record(Elem<T>::key(vec_elem(v, b)), (uint32_t)(i0 + b));
                    dst[pos] = rec;
                    if (HIST) hc.count(rec);
                }
                ++pos;
            }
        }
        left &= ~group;
    }
}

// The same for a launch over ONE row, by the whole CTA: THREADS entries, one atomic.  When the scan ends every CTA of
// the grid works its list off at the same moment, and an atomic per warp -- seven thousand on the row's one counter --
// took longer than the rest of that work.  `scratch` holds THREADS / 32 + 1 words of shared memory; all threads call.
template <typename T, int THREADS, int UNROLL, bool HIST>
__device__ __noinline__ void defer_process_block(const FilterParams<T>& p, uint32_t vid, uint32_t* hist_coarse, uint32_t* scratch) {
    static_assert(THREADS / 32 <= 32, "one lane of the first warp per warp of the CTA");
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    const DeferDecided<T> d = defer_decide<T, THREADS, UNROLL>(p, vid);
    const unsigned cnt = __popc(d.m);
    unsigned incl = cnt;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const unsigned nb = __shfl_up_sync(FULL_MASK, incl, s);
        if (lane >= (unsigned)s) incl += nb;
    }
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const unsigned w = lane < THREADS / 32 ? scratch[lane] : 0u;
        unsigned wi = w;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            const unsigned nb = __shfl_up_sync(FULL_MASK, wi, s);
            if (lane >= (unsigned)s) wi += nb;
        }
        unsigned base = 0;
        if (lane == 31 && wi) base = atomicAdd(p.counts, wi);           // (row 0's counter)
        base = __shfl_sync(FULL_MASK, base, 31);
        if (lane < THREADS / 32) scratch[lane] = base + wi - w;         // first position of the warp's records
    }
    __syncthreads();
    if (cnt) {
        const HistCtx hc = {p.hist, hist_coarse, d.top_hi, p.idx_bits};
        unsigned pos = scratch[warp] + incl - cnt;
        unsigned mm = d.m;
        while (mm) {
            const int b = __ffs(mm) - 1;
            mm &= mm - 1;
            if (pos < p.capacity) {
                const uint64_t rec = make_record(Elem<T>::key(vec_elem(d.v, b)), (uint32_t)(d.i0 + b));
                p.buf[pos] = rec;
                if (HIST) hc.count(rec);
            }
            ++pos;
        }
    }
    __syncthreads();                   // scratch is rewritten by the next batch
}

// The HIST build's: out of line, so that the counting costs the streaming loop no registers.
template <typename T, int THREADS, int UNROLL, bool PARTS>
__device__ __noinline__ void defer_process_batch_counting(const FilterParams<T>& p, uint32_t vid, uint32_t* hist_coarse) {
    defer_process_batch<T, THREADS, UNROLL, PARTS, true>(p, vid, hist_coarse);
}

// Work distribution: a tile is TILE_VECTORS consecutive vectors of one row (32 KB), loaded by the
// whole CTA at once (every warp-level load is one contiguous 512-byte run, the CTA's loads one 32 KB
// run).  A CTA takes tiles blockIdx.x, + gridDim.x, ... with its warps running freely; the last few
// tiles of the launch (from dyn_start on) come from a global counter instead, so that SMs that saw
// less bandwidth take fewer of them and all CTAs finish together.  The counter is read one tile
// ahead, so its round trip hides behind the loads; only this tail needs a CTA barrier per tile
// (per chunk of dyn_chunk consecutive tiles: batches take four at a time).
template <typename T, int THREADS, int UNROLL, bool PARTS = false, bool DEFER = false, bool HIST = false>
__global__ void __launch_bounds__(THREADS, sizeof(T) == 4 ? PROFK_FILTER_MINBLOCKS_F32 : PROFK_FILTER_MINBLOCKS_BF16) filter_kernel(const __grid_constant__ FilterParams<T> p) {
    static_assert(!HIST || (DEFER && !PARTS), "only the deferring build counts its records");
    using V = typename Elem<T>::vec_t;
    constexpr uint32_t TILE_VECTORS = THREADS * UNROLL;
    __shared__ uint32_t hits[DEFER ? DEFER_CAP : 1];
    __shared__ uint32_t s_nhits;
    __shared__ uint32_t s_scan[DEFER ? THREADS / 32 + 1 : 1];
    __shared__ uint32_t s_hcoarse[HIST ? BIN_COARSE : 1];       // (HIST) this CTA's share of the coarse histogram
    if (DEFER || HIST) {
        if (threadIdx.x == 0) s_nhits = 0;
        if (HIST)
            for (uint32_t c = threadIdx.x; c < BIN_COARSE; c += THREADS) s_hcoarse[c] = 0;
        __syncthreads();
    }
    __shared__ uint32_t s_next[2];
    __shared__ __align__(8) uint64_t pf_bar;                         // counts the bytes of the prefetched tiles
    extern __shared__ __align__(128) unsigned char pf_smem[];        // p.prefetch_tiles tiles of 32 KB (or nothing)

    const unsigned lane = lane_id();

    constexpr int VEC = Elem<T>::VEC;
    constexpr uint32_t ALL_INSIDE = (1u << UNROLL) - 1u;
    const uint32_t total_tiles = (uint32_t)p.total_tiles, tiles_per_row = (uint32_t)p.tiles_per_row;
    const bool one_row = tiles_per_row == total_tiles;
    uint32_t tile = blockIdx.x;                  // the grid never exceeds the number of tiles (< 2^32)

    uint32_t row = 0;
    uint64_t qbase;                              // first vector of the tile inside its row
    RowView<T> rv;
    V v[UNROLL];
    uint32_t inside_mask;                        // bit u: vector u holds at least one element of the row
    // Row and position of `tile`, and its loads.  A tile that lies wholly inside its row -- all but the first
    // and the last of a row -- is four plain 128-bit loads off one pointer; the others take the checked path.
    uint32_t pf_left = 0;                        // tiles still waiting in shared memory (single rows only)
    auto decode_and_load = [&](bool first_time) {
        uint32_t nrow = 0, tin = tile;
        if (!one_row) { nrow = tile / tiles_per_row; tin = tile - nrow * tiles_per_row; }
        qbase = (uint64_t)tin * TILE_VECTORS;
        if (first_time || nrow != row) { row = nrow; rv = row_view(p.in, p.N, row); }
        if (pf_left) {
            // one of the tiles copied into shared memory before the wait for the threshold kernel
            const V* src = reinterpret_cast<const V*>(pf_smem) + (size_t)(p.prefetch_tiles - pf_left) * TILE_VECTORS + threadIdx.x;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) v[u] = src[u * THREADS];
            inside_mask = ALL_INSIDE;
            --pf_left;
        } else if (qbase * VEC >= rv.mis && (qbase + TILE_VECTORS) * VEC <= p.N + rv.mis) {
            const V* ptr = reinterpret_cast<const V*>(rv.aligned_base) + qbase + threadIdx.x;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) v[u] = ld_stream(ptr + u * THREADS);
            inside_mask = ALL_INSIDE;
        } else {
            inside_mask = 0;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                bool in;
                v[u] = load_row_vector(rv, p.N, qbase + (uint64_t)u * THREADS + threadIdx.x, &in);
                inside_mask |= in ? 1u << u : 0u;
            }
        }
    };

    // The first tile's loads are issued before waiting on the threshold kernel: the input does not depend on it.
    decode_and_load(true);

    // So are bulk copies of the CTA's next tiles into shared memory, when the launch asked for them (a single row,
    // tiles that lie wholly inside it and are dealt by the fixed stride): one thread issues them, an mbarrier counts
    // their bytes, and everybody waits on it -- with a limit -- when the first of them is due.
    bool pf_ok = false;
    if (p.prefetch_tiles) {
        const uint64_t last = (uint64_t)tile + (uint64_t)p.prefetch_tiles * gridDim.x;          // last tile to copy
        pf_ok = one_row && last < p.dyn_start && (uint64_t)tile * TILE_VECTORS * VEC >= rv.mis &&
                (last + 1) * TILE_VECTORS * VEC <= p.N + rv.mis;
        if (pf_ok) {
            const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&pf_bar);
            if (threadIdx.x == 0) {
                asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(p.prefetch_tiles * TILE_VECTORS * 16u) : "memory");
                for (uint32_t j = 0; j < p.prefetch_tiles; ++j) {
                    const V* src = reinterpret_cast<const V*>(rv.aligned_base) + ((uint64_t)tile + (uint64_t)(j + 1) * gridDim.x) * TILE_VECTORS;
                    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(pf_smem + (size_t)j * TILE_VECTORS * 16u);
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(dst), "l"(src), "r"(TILE_VECTORS * 16u), "r"(bar) : "memory");
                }
            }
            __syncthreads();            // the barrier is initialised before anyone may wait on it
        }
    }
    if (p.use_pdl) pdl_wait();
    pdl_launch_dependents();            // the refine kernel may be staged behind this one
    // The copies were issued microseconds ago; should they not have landed within the limit, the tiles are read with
    // plain loads instead and the copies are waited for once more before the CTA leaves.
    auto prefetch_landed = [&](uint32_t limit) {
        const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&pf_bar);
        for (uint32_t spin = 0; spin < limit; ++spin) {
            uint32_t done;
            asm volatile("{\n\t.reg .pred q;\n\tmbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                         : "=r"(done) : "r"(bar) : "memory");
            if (done) return true;
        }
        return false;
    };
    bool pf_pending = false;
    if (pf_ok) {
        if (prefetch_landed(p.prefetch_spin_limit)) pf_left = p.prefetch_tiles; else pf_pending = true;
    }

    uint32_t skip_row = 0xFFFFFFFFu;    // row whose buffer this warp has seen overflow: nothing more to append
    uint32_t parity = 0;
    uint32_t tau_row = row;
    // The row's threshold, and what the streaming test compares with: tau itself up to the tile that holds the
    // threshold record, the next value in the total order in the tiles after it -- there no copy of tau is
    // kept, and a row that is one flood of copies of tau stays on the fast path.  (Single rows only: in a batch a
    // CTA changes row at almost every tile, and the extra work at each change cost 2 % on rows without ties.)
    T tau_lo, tau_hi;
    uint32_t tie_tile;
    auto load_threshold = [&]() {
        if (p.thr && one_row) {
            const uint4 t = p.thr[row];
            tau_lo = Elem<T>::from_bits(t.x);
            tau_hi = Elem<T>::from_bits(t.y);
            tie_tile = t.z == 0xFFFFFFFFu ? 0xFFFFFFFFu : (uint32_t)(((uint64_t)t.z + rv.mis) / ((uint64_t)TILE_VECTORS * VEC));
        } else if (p.thr) {
            tau_lo = tau_hi = Elem<T>::from_bits(reinterpret_cast<const uint32_t*>(p.thr + row)[0]);
            tie_tile = 0xFFFFFFFFu;
        } else {
            tau_lo = tau_hi = p.tau[row];
            tie_tile = 0xFFFFFFFFu;
        }
    };
    load_threshold();
    while (true) {
        const T tau = (uint32_t)(qbase / TILE_VECTORS) > tie_tile ? tau_hi : tau_lo;
        // Tiles below dyn_start follow the fixed stride and the warps run freely; the last few tiles of
        // the launch are handed out by the counter.  Thread 0 asks for the next one now; the answer is
        // needed only after this tile.
        const bool dynamic = p.tile_counter != nullptr && tile + gridDim.x >= p.dyn_start;
        const bool claim = dynamic && (parity >> 1) == 0;        // (parity: bit 0 = which word of s_next, the rest = tiles left of the chunk)
        uint32_t upcoming = 0;
        if (claim && threadIdx.x == 0) {
            const uint32_t t = p.dyn_start + atomicAdd(p.tile_counter, p.dyn_chunk);
            upcoming = t < total_tiles ? t : total_tiles;
        }

        bool hit = false;
        bool h[UNROLL];                          // (DEFER) vector u holds an element that is not below tau
        if (DEFER) {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                h[u] = (inside_mask == ALL_INSIDE || ((inside_mask >> u) & 1u)) && vec_any_pass(v[u], tau);
                hit |= h[u];
            }
        } else if (inside_mask == ALL_INSIDE) {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) hit |= vec_any_pass(v[u], tau);
        } else {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) hit |= (((inside_mask >> u) & 1u) && vec_any_pass(v[u], tau));
        }

        if (__any_sync(FULL_MASK, hit) && row != skip_row) {
            uint32_t o = 0xFFFFFFFFu;
            bool noted = false;
            if (DEFER) {
                // Note the candidate vectors.  Only the lanes that hold one do anything: each reserves room for its own
                // (one shared-memory atomic; a tile rarely has more than two such lanes) and writes their numbers.
                uint32_t slot = 0, cnt = 0;
                if (hit) {
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) cnt += h[u] ? 1u : 0u;
                    slot = atomicAdd(&s_nhits, cnt);
                }
                noted = !__any_sync(FULL_MASK, hit && slot + cnt > DEFER_CAP);      // (a warp that does not fit leaves its slots unused)
                if (hit) {
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        if (h[u]) {
                            if (slot < DEFER_CAP) hits[slot] = noted ? tile * TILE_VECTORS + (uint32_t)u * THREADS + threadIdx.x : DEFER_NONE;
                            ++slot;
                        }
                    }
                }
            }
            if (!noted) {
                o = filter_slow_path_direct<T, THREADS, UNROLL, PARTS>(p, v, inside_mask, row, qbase, rv.mis, tau_lo);
                // (HIST) records appended on this way out of a full list are not counted: the kernel behind is told so
                if (HIST && lane == 0) p.hist[BIN_COUNT + BIN_FLAG_UNCOUNTED] = 1u;
            }
            if (o != 0xFFFFFFFFu) skip_row = o;
        }

        if (claim) {
            if (threadIdx.x == 0) s_next[parity & 1u] = upcoming;
            __syncthreads();
            tile = s_next[parity & 1u];
            parity = ((parity & 1u) ^ 1u) | ((p.dyn_chunk - 1u) << 1);
        } else if (dynamic) {
            tile = tile + 1u;                    // the next tile of the chunk this CTA holds
            parity -= 2u;
        } else {
            tile = total_tiles - tile <= gridDim.x ? total_tiles : tile + gridDim.x;
        }
        if (tile >= total_tiles) break;
        if (skip_row != 0xFFFFFFFFu && (one_row ? 0u : tile / tiles_per_row) == skip_row) {
            inside_mask = 0;            // this warp knows the row has overflowed: nothing to load (it stays in the
            continue;                   // loop: the hand-out of the last tiles is a matter for the whole CTA)
        }
        decode_and_load(false);
        if (row != tau_row) { tau_row = row; load_threshold(); }
    }
    if (DEFER) {
        // every tile of this CTA has been streamed: work the list off, one entry per thread
        __syncthreads();
        const uint32_t n = s_nhits < DEFER_CAP ? s_nhits : DEFER_CAP;
        for (uint32_t e0 = 0; e0 < n; e0 += THREADS) {          // whole warps take part in every batch
            const uint32_t e = e0 + threadIdx.x;
            if (one_row && !PARTS) {
                defer_process_block<T, THREADS, UNROLL, HIST>(p, e < n ? hits[e] : DEFER_NONE, s_hcoarse, s_scan);
            } else if (e0 + (threadIdx.x & ~31u) < n) {
                if (HIST) defer_process_batch_counting<T, THREADS, UNROLL, PARTS>(p, e < n ? hits[e] : DEFER_NONE, s_hcoarse);
                else defer_process_batch<T, THREADS, UNROLL, PARTS>(p, e < n ? hits[e] : DEFER_NONE);
            }
        }
    }
    if (HIST) {
        // this CTA's coarse counts join the row's (the fine bins were counted record by record)
        __syncthreads();
        uint32_t* coarse = p.hist + BIN_COUNT + BIN_FLAGS;
        for (uint32_t c = threadIdx.x; c < BIN_COARSE; c += THREADS) {
            const uint32_t n = s_hcoarse[c];
            if (n) atomicAdd(&coarse[c], n);
        }
    }
    if (pf_pending) prefetch_landed(PREFETCH_SPIN_LIMIT);
}

}  // namespace profk
