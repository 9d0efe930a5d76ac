// C ABI of the library (see profk.h): argument checks, workspace layout and the launch
// sequence  threshold -> filter -> count check + refine -> exact replacement of failed rows.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "batchtopk.cuh"
#include "fallback.cuh"
#include "filter.cuh"
#include "profk.h"
#include "refine.cuh"
#include "refine_large.cuh"
#include "sample_select.cuh"
#include "shard.cuh"

using namespace profk;

namespace {

#ifndef PROFK_DYNAMIC_ROUNDS
#define PROFK_DYNAMIC_ROUNDS 2      // fewest tiles per CTA (on average) that the filter hands out dynamically at the end
#endif
constexpr int FILTER_THREADS = PROFK_FILTER_THREADS;
constexpr int FILTER_UNROLL = PROFK_FILTER_UNROLL;
constexpr uint32_t SORT_CAP_MAX = 16384;         // largest k the single-CTA refine orders in shared memory
// Selections the whole grid refines (refine_large_kernel) instead of one CTA per row: beyond the single-CTA limit, and
// below it where that measured faster.  One CTA takes 100-280 us over 12000-16384 records (bf16, whose equal keys send
// the selection through the index digits, worst), the CTAs of several rows side by side; the grid takes 10-40 us per
// row, in up to 18 groups side by side, and its launch costs 7-9 us more.
//   one row: from k = 8193 on; bf16 from 3073 on, since the grid-wide path then starts from the filter's histogram
//     (2^28 bf16: k = 4096 137 -> 118 us, k = 8192 245 -> 114; 2^26: 58 -> 56, 106 -> 57; k = 2048 still 103 against
//     118; fp32 k = 8192: 186 against 193).
//   2 to 18 rows: from the k of large_switch_k on, read off sweeps over rows x k x N (2^20 .. 2^26) of both paths.  fp32:
//     the longer the rows and the more of them, the earlier (8 rows of 2^24, k = 6000: 203 us through one CTA each, 178
//     through the grid; of 2^22: 74 against 103).  bf16: near k = 6000 whatever the length (8 rows of 2^22: k = 5000 69
//     against 74, k = 6000 78 against 75, k = 8192 102 against 77, k = 16384 246 against 87).
//   more rows: the CTAs work side by side and win.
constexpr int64_t LARGE_FEW_ROWS = 4;
constexpr int64_t LARGE_SOME_ROWS = 18;
constexpr int64_t LARGE_FEW_K = 8192;
constexpr int64_t LARGE_FEW_K_HALF = 3072;
constexpr int64_t LARGE_SOME_K_MIN = 4096;       // no call of 2 to 18 rows switches at or below this k
// 2 to 18 rows: the largest k one CTA per row still orders.
inline int64_t large_switch_k(int64_t rows, size_t elem_size, int64_t N) {
    const int64_t never = (int64_t)SORT_CAP_MAX;
    if (elem_size == 2) return rows <= 8 ? 5632 : 6656;        // (at every row length from 2^20 to 2^26)
    if (N >= (1LL << 26)) return 6144;
    if (N >= (1LL << 25)) return rows <= 3 ? 8192 : 6144;
    if (N >= (1LL << 24)) return rows <= 4 ? 10240 : 6144;
    if (N >= (1LL << 23)) return 13312;
    return never;
}
inline bool large_selection(int64_t rows, int64_t k, size_t elem_size, int64_t N) {
    if (k > (int64_t)SORT_CAP_MAX) return true;
    if (rows == 1) return k > (elem_size == 2 ? LARGE_FEW_K_HALF : LARGE_FEW_K);
    if (rows > LARGE_SOME_ROWS) return false;
    return k > large_switch_k(rows, elem_size, N);
}
// The rule without the row length, as the allocation-free entry point applies it (its scratch holds the grid-wide
// layout of at most LARGE_FEW_ROWS rows).
inline bool large_selection_few(int64_t rows, int64_t k, size_t elem_size) {
    return k > (int64_t)SORT_CAP_MAX || (rows <= LARGE_FEW_ROWS && k > LARGE_FEW_K) || (rows == 1 && elem_size == 2 && k > LARGE_FEW_K_HALF);
}
// Whether some element type and row length send (rows, k) through the grid-wide layout.
inline bool large_possible(int64_t rows, int64_t k) {
    return k > (int64_t)SORT_CAP_MAX || (rows == 1 && k > LARGE_FEW_K_HALF) || (rows <= LARGE_SOME_ROWS && k > LARGE_SOME_K_MIN);
}
constexpr unsigned FB_MAX_CTAS = 256;             // most CTAs of the grid-wide exact selection (its per-CTA scratch is sized for them)
// Samples above this size are gathered by a kernel over all SMs (65536: 2^26, k = 16, S = 40529 took 49.7 us, not 47.0).
constexpr int64_t GATHER_MIN_SAMPLE = 32768;
constexpr int64_t GATHER_MAX_ROWS = PROFK_ALL_SM_GATHER_ROWS;   // most rows for which the sample may be gathered by a kernel of its own
constexpr int LARGE_MAX_CTAS = 1024;             // CTAs of the large refine (its per-CTA slots live in the 48 KB histogram area)
constexpr int64_t XS_MAX_ROWS = 18;              // most rows for which the refine kernel itself replaces failed rows
constexpr unsigned XS_MAX_SEGMENTS = 32;         // most (row, segment) pairs of that exact selection
constexpr unsigned REFINE_CLUSTER_THREADS = 512;   // fewest threads of a refine CTA that may have to read whole rows
constexpr size_t REFINE_SMEM_MAX = 160 * 1024;   // dynamic shared memory the refine kernel may ask for (it has ~41 KB static)
constexpr int64_t N_MAX = 4278190080LL;          // 2^32 - 2^24
constexpr int64_t M_MAX = 262144;                // largest sample the cluster select holds (8 CTAs x 32768 keys)
constexpr int64_t KEPT_SAMPLE_MAX = 131072;      // largest sample whose keys are kept for a second filtering pass when there are more than GATHER_MAX_ROWS rows
constexpr int64_t KEPT_SAMPLE_NOALLOC_MAX = 32768;   // ... in the scratch of the allocation-free entry point
constexpr int64_t KEPT_SAMPLE_BATCH_MAX = 4096;  // the same for batches of more than XS_MAX_ROWS rows

thread_local int g_launches = 0;
thread_local void* g_ws_override_ptr = nullptr;   // set by the allocation-free entry point for the duration of its call
thread_local size_t g_ws_override_bytes = 0;
std::atomic<uint32_t> g_prefetch_spin_limit{PREFETCH_SPIN_LIMIT};   // see profk_debug_set_prefetch_wait_polls
std::atomic<int> g_coop_pdl{-1};                 // -1 untried, 1 accepted, 0 refused by the runtime

struct DeviceInfo {
    int sm_count = 0;
    int filter_blocks_per_sm[2] = {0, 0};     // by dtype
    int filter_defer_blocks_per_sm[2] = {0, 0};
    int max_cluster[2] = {8, 8};              // 16 when the device can co-schedule 16 CTAs of the threshold kernel
    int refine_cluster[2] = {8, 8};           // same for the refine kernel at its largest footprint
    bool ready = false;
};

struct Workspace { void* ptr = nullptr; size_t bytes = 0; };

std::mutex g_mutex;
std::map<int, DeviceInfo> g_devinfo;
std::map<int, Workspace> g_workspace;
std::map<std::tuple<int64_t, int64_t, int64_t, double, double>, profk_plan_t> g_plan_cache;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct WsLayout {
    size_t off_header, off_ghist, off_ctl, off_tau, off_tau2, off_bins, off_xs_counters, off_xs_records, off_keys, off_fb_counters, off_fb_records, off_parts, off_buf, total;
};

// Records reserved per row: the capacity itself, or -- when k is too large for the single-CTA
// refine -- twice the power of two the cluster sort pads the row to (records, then scratch).
uint64_t row_stride_for(int64_t capacity, bool large) {
    if (!large) return (uint64_t)capacity;
    uint64_t p = BT_TILE;
    while (p < (uint64_t)capacity) p <<= 1;
    return 2 * p;
}

// `large` = the layout of large selections (bins, partitioned append counters, doubled row pitch): whenever
// large_selection(rows, k) says so, and always for the flattened BatchTopK calls, whose select works on the bins.
WsLayout ws_layout(int64_t rows, int64_t capacity, int64_t k, bool large, int64_t kept_sample_max = KEPT_SAMPLE_MAX) {
    WsLayout l;
    l.off_header = 0;
    l.off_ghist = sizeof(WsHeader);
    l.off_ctl = align_up(l.off_ghist + (size_t)FB_PASSES * FB_BINS * sizeof(uint32_t), 256);
    l.off_tau = align_up(l.off_ctl + (size_t)rows * sizeof(RowCtl), 256);
    l.off_tau2 = align_up(l.off_tau + (size_t)rows * sizeof(uint4), 256);       // threshold records of a second filtering pass
    l.off_bins = align_up(l.off_tau2 + (size_t)rows * sizeof(uint4), 256);
    const size_t bins_bytes = large ? (size_t)rows * BIN_ROW_WORDS * sizeof(uint32_t) : 0;
    // scratch of the in-refine exact selection (few rows, k within the single-CTA refine): up to
    // XS_MAX_SEGMENTS segments in all, each with a counter and k + XS_EDGE records
    const bool xs = rows <= XS_MAX_ROWS && !large;
    l.off_xs_counters = align_up(l.off_bins + bins_bytes, 256);
    l.off_xs_records = align_up(l.off_xs_counters + (xs ? XS_MAX_SEGMENTS * sizeof(uint32_t) : 0), 256);
    // keys of the sample when a kernel of its own gathers them (few rows only)
    l.off_keys = align_up(l.off_xs_records + (xs ? (size_t)XS_MAX_SEGMENTS * (size_t)(k + XS_EDGE) * sizeof(uint64_t) : 0), 256);
    // scratch of the grid-wide exact selection when it deals failed rows out one per CTA (many rows only)
    const bool fbp = rows > XS_MAX_ROWS && !large;
    // (up to GATHER_MAX_ROWS rows: room for the largest sample; up to XS_MAX_ROWS rows: for samples up to KEPT_SAMPLE_MAX,
    // larger batches: up to KEPT_SAMPLE_BATCH_MAX -- kept for the second filtering pass of a row that fails the count check)
    const size_t keys_per_row = rows <= GATHER_MAX_ROWS ? (size_t)M_MAX : rows <= XS_MAX_ROWS ? (size_t)kept_sample_max : !large ? (size_t)KEPT_SAMPLE_BATCH_MAX : 0;
    l.off_fb_counters = align_up(l.off_keys + (size_t)rows * keys_per_row * sizeof(uint32_t), 256);
    l.off_fb_records = align_up(l.off_fb_counters + (fbp ? FB_MAX_CTAS * sizeof(uint32_t) : 0), 256);
    // counters of the partitioned append (large selections only), each in a 256-byte line of its own
    l.off_parts = align_up(l.off_fb_records + (fbp ? (size_t)FB_MAX_CTAS * (size_t)(k + XS_EDGE) * sizeof(uint64_t) : 0), 256);
    l.off_buf = align_up(l.off_parts + (large ? (size_t)rows * FILTER_PARTS * FILTER_PART_STRIDE * sizeof(uint32_t) : 0), 256);
    l.total = align_up(l.off_buf + (size_t)rows * (size_t)row_stride_for(capacity, large) * sizeof(uint64_t), 256);
    return l;
}

#define CUDA_TRY(expr)                                   \
    do {                                                 \
        cudaError_t _e = (expr);                         \
        if (_e != cudaSuccess) { (void)cudaGetLastError(); return PROFK_ECUDA; } \
    } while (0)

template <typename T> constexpr int dtype_index() { return sizeof(T) == 4 ? 0 : 1; }

template <typename T> int ensure_device_info(int dev, DeviceInfo* out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo& di = g_devinfo[dev];
    if (!di.ready) {
        CUDA_TRY(cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev));
        di.ready = true;
    }
    const int d = dtype_index<T>();
    if (di.filter_blocks_per_sm[d] == 0) {
        int nb = 0;
        CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, filter_kernel<T, FILTER_THREADS, FILTER_UNROLL>,
                                                                 FILTER_THREADS, 0));
        di.filter_blocks_per_sm[d] = std::max(nb, 1);
        CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, filter_kernel<T, FILTER_THREADS, FILTER_UNROLL, false, true>,
                                                                 FILTER_THREADS, 0));
        di.filter_defer_blocks_per_sm[d] = std::max(nb, 1);
        CUDA_TRY(cudaFuncSetAttribute(sample_select_kernel<T, SEL_THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
        const int prefetch_bytes = (int)(FILTER_PREFETCH * FILTER_THREADS * FILTER_UNROLL * 16u);
        CUDA_TRY(cudaFuncSetAttribute(filter_kernel<T, FILTER_THREADS, FILTER_UNROLL>, cudaFuncAttributeMaxDynamicSharedMemorySize, prefetch_bytes));
        CUDA_TRY(cudaFuncSetAttribute(filter_kernel<T, FILTER_THREADS, FILTER_UNROLL, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, prefetch_bytes));
        // (the small build holds 33 KB of static shared memory: with 4096 keys it passes the 48 KB that need no opt-in)
        CUDA_TRY(cudaFuncSetAttribute(sample_select_kernel<T, SEL_SMALL_THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 16 * 1024));
        CUDA_TRY(cudaFuncSetAttribute(refine_kernel<T, 48>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)REFINE_SMEM_MAX));
        CUDA_TRY(cudaFuncSetAttribute(refine_kernel<T, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)REFINE_SMEM_MAX));
        CUDA_TRY(cudaFuncSetAttribute(fallback_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(SORT_CAP_MAX * 8)));
        // Clusters of 16 are beyond the portable size: allowed only where one actually fits.
        if (cudaFuncSetAttribute(sample_select_kernel<T, SEL_THREADS>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(16); cfg.blockDim = dim3(SEL_THREADS); cfg.dynamicSmemBytes = 16384 * sizeof(uint32_t);
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 16; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int nclusters = 0;
            if (cudaOccupancyMaxActiveClusters(&nclusters, sample_select_kernel<T, SEL_THREADS>, &cfg) == cudaSuccess && nclusters >= 1)
                di.max_cluster[d] = 16;
        }
        (void)cudaGetLastError();
        if (cudaFuncSetAttribute(refine_kernel<T, 48>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
            cudaFuncSetAttribute(refine_kernel<T, 64>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(16); cfg.blockDim = dim3(1024); cfg.dynamicSmemBytes = REFINE_SMEM_MAX;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 16; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int nclusters = 0;
            if (cudaOccupancyMaxActiveClusters(&nclusters, refine_kernel<T, 64>, &cfg) == cudaSuccess && nclusters >= 1)
                di.refine_cluster[d] = 16;
        }
        (void)cudaGetLastError();
        CUDA_TRY(cudaFuncSetAttribute(refine_large_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(BT_TILE * 8)));
        (void)cudaGetLastError();
    }
    *out = di;
    return PROFK_OK;
}

// Direct mode has no threshold / filter kernels: mark every row for exact selection.
__global__ void init_ctl_kernel(RowCtl* ctl, uint64_t rows, WsHeader* header, uint32_t capacity, uint32_t k) {
    const uint64_t r = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < rows) {
        RowCtl* c = ctl + r;
        c->tau_bits = 0; c->count = 0; c->collect = 0; c->status = ROW_DIRECT; c->n_final = k; c->capacity = capacity;
    }
    if (r == 0) {
        header->bar_count = 0; header->error = 0; header->done = 0; header->n_failed = (uint32_t)rows;
        for (int g = 0; g < WS_GROUPS; ++g) header->group_bar[g][0] = 0;
    }
}

// Cluster size for the threshold kernel: spread one row's gather over several SMs when
// there are few rows; never more keys per CTA than its shared memory holds.
int pick_cluster(int64_t rows, int64_t m, int max_cluster) {
    int c = rows <= 9 ? 16 : rows <= 18 ? 8 : rows <= 37 ? 4 : rows <= 74 ? 2 : 1;
    if (c > max_cluster) c = max_cluster;
    while (c < 8 && (m + c - 1) / c > 32766) c *= 2;
    return c;
}

template <typename T>
int launch_sample_select(const DeviceInfo& di, const T* in, int64_t rows, int64_t N, int64_t m, int64_t r, uint64_t seed, T* tau, RowCtl* ctl,
                         WsHeader* header, uint32_t capacity, uint32_t* sample_idx, uint32_t* keys_scratch, uint32_t* part_counts,
                         bool by_record, uint4* thr, cudaStream_t st, const uint32_t* keys_given = nullptr, uint32_t* keys_store = nullptr,
                         uint32_t* zero = nullptr, uint32_t zero_words = 0) {
    const int csize = pick_cluster(rows, m, di.max_cluster[dtype_index<T>()]);
    // A large sample, or a sample of a very long row (every element on a page of its own), is gathered by a
    // kernel over all SMs first; the cluster then only selects.  (keys_given: the caller already holds the sample's keys.)
    const bool spread_gather = !keys_given && keys_scratch != nullptr && rows <= GATHER_MAX_ROWS &&
                               (m > GATHER_MIN_SAMPLE || (int64_t)N * (int64_t)sizeof(T) >= (512LL << 20));
    if (spread_gather) {
        GatherParams<T> gp;
        gp.in = in; gp.N = (uint64_t)N; gp.rows = (uint64_t)rows; gp.S = (uint32_t)m; gp.seed = seed;
        gp.q = (uint64_t)(N / m); gp.rem = (uint32_t)(N % m); gp.inv_s = 1.0f / (float)m; gp.keys_out = keys_scratch;
        gp.pair_lo = 0; gp.pairs = (uint64_t)((m + 1) / 2); gp.base = 0;
        gp.zero = reinterpret_cast<uint4*>(zero); gp.zero_vecs = zero_words / 4;      // cleared by the wider of the two kernels
        const int64_t pairs = rows * ((m + 1) / 2);
        cudaLaunchConfig_t gcfg = {};
        gcfg.gridDim = dim3((unsigned)((pairs + GATHER_THREADS - 1) / GATHER_THREADS));
        gcfg.blockDim = dim3(GATHER_THREADS);
        gcfg.stream = st;
        cudaLaunchAttribute gattr[1];
        gattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        gattr[0].val.programmaticStreamSerializationAllowed = 1;
        gcfg.attrs = gattr; gcfg.numAttrs = 1;
        CUDA_TRY(cudaLaunchKernelEx(&gcfg, gather_kernel<T>, gp));
        ++g_launches;
    }
    SelectParams<T> sp;
    sp.keys_in = keys_given ? keys_given : spread_gather ? keys_scratch : nullptr;
    sp.keys_store = sp.keys_in ? nullptr : keys_store;       // (keys gathered by the kernel before are in memory already)
    sp.part_counts = part_counts;
    sp.by_record = by_record ? 1 : 0;
    sp.zero = spread_gather ? nullptr : reinterpret_cast<uint4*>(zero); sp.zero_vecs = zero_words / 4;
    sp.thr = thr;
    sp.in = in; sp.N = (uint64_t)N; sp.S = (uint32_t)m; sp.t = (uint32_t)r; sp.seed = seed;
    sp.per_cta = (uint32_t)(((m + csize - 1) / csize + 1) & ~1LL);      // even: samples are drawn in pairs
    sp.q = (uint64_t)(N / m); sp.rem = (uint32_t)(N % m); sp.inv_s = 1.0f / (float)m;
    sp.tau = tau; sp.ctl = ctl; sp.header = header; sp.capacity = capacity; sp.sample_idx = sample_idx;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(rows * csize));
    cfg.blockDim = dim3(SEL_THREADS);
    cfg.dynamicSmemBytes = (size_t)sp.per_cta * sizeof(uint32_t);
    cfg.stream = st;
    // The kernel may be staged behind whatever runs before it on the stream (it waits for that work
    // before it touches the input or the workspace): its launch and the computation of the sample
    // positions then overlap that work's tail.  Without a cluster dimension a kernel runs as implicit
    // clusters of one CTA, which is what a one-CTA cluster is.
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)csize; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = csize > 1 ? 2 : 1;
    // Batches of rows with small samples: one small CTA per row, four to an SM.
    if (csize == 1 && m <= (int64_t)SEL_CAND_CAP && r <= SEL_SMALL_THREADS / 8 && !sp.keys_in) {
        cfg.blockDim = dim3(SEL_SMALL_THREADS);
        CUDA_TRY(cudaLaunchKernelEx(&cfg, sample_select_kernel<T, SEL_SMALL_THREADS>, sp));
    } else {
        CUDA_TRY(cudaLaunchKernelEx(&cfg, sample_select_kernel<T, SEL_THREADS>, sp));
    }
    ++g_launches;
    return PROFK_OK;
}

template <typename T>
int launch_filter(const DeviceInfo& di, const T* in, int64_t rows, int64_t N, const T* tau, int64_t capacity, uint64_t* buf,
                  uint64_t buf_stride, uint32_t* counts, uint32_t count_stride, bool pdl, uint32_t* tile_counter, bool parts,
                  uint32_t part_cap, uint32_t* part_counts, const uint4* thr, cudaStream_t st, bool deferred = false, uint32_t* hist = nullptr) {
    FilterParams<T> fp;
    fp.hist = hist; fp.idx_bits = index_bits((uint64_t)N);
    fp.thr = thr;
    fp.in = in; fp.N = (uint64_t)N; fp.rows = (uint64_t)rows; fp.tau = tau; fp.capacity = (uint32_t)capacity;
    fp.buf = buf; fp.buf_stride = buf_stride; fp.counts = counts; fp.count_stride = count_stride;
    fp.tiles_per_row = tiles_per_row<T>((uint64_t)N, FILTER_THREADS * FILTER_UNROLL);
    fp.total_tiles = fp.tiles_per_row * (uint64_t)rows;
    if (fp.total_tiles >= (1ull << 32)) return PROFK_EINVAL;      // rows * N beyond 2^45 elements
    fp.use_pdl = pdl ? 1 : 0;
    fp.tile_counter = tile_counter;
    fp.part_cap = part_cap; fp.part_counts = part_counts;
    if (parts || fp.total_tiles * (uint64_t)(FILTER_THREADS * FILTER_UNROLL) >= (1ull << 32)) deferred = false;   // vectors are numbered in 32 bits
    const uint64_t max_grid = (uint64_t)di.sm_count *
        (deferred ? di.filter_defer_blocks_per_sm[dtype_index<T>()] : di.filter_blocks_per_sm[dtype_index<T>()]);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)std::min<uint64_t>(fp.total_tiles, max_grid));
    // All but the last few tiles per CTA follow the fixed stride; the rest come from a counter, so that all CTAs finish
    // together.  The longer the launch, the more of them: the three CTAs of an SM do not advance at the same rate (the
    // one that arrived first is a few per cent ahead: after 148 tiles its neighbours were 10-20 us behind), and two
    // rounds cannot level that.  An eighth of a single row's rounds, at most 32, one tile at a time; a quarter of a
    // batch's, at most 32, and there a CTA takes four consecutive tiles from the counter at a time (a dynamic tile costs a
    // batch a CTA barrier and a division): 2^30 fp32 605 -> 595 us, 2^29 bf16 K = 131072 207 -> 196, 512 rows of 2^20
    // 400 -> 386 (bf16 253 -> 242); 2^26 (18 rounds) keeps its two.
    const uint64_t rounds = fp.total_tiles / cfg.gridDim.x;
    const uint64_t dyn_rounds = rows > 1 ? std::min<uint64_t>(std::max<uint64_t>(rounds / 4, PROFK_DYNAMIC_ROUNDS), 32)
                                         : std::min<uint64_t>(std::max<uint64_t>(rounds / 8, PROFK_DYNAMIC_ROUNDS), 32);
    fp.dyn_chunk = rows > 1 ? (dyn_rounds >= 16 ? 4u : dyn_rounds >= 8 ? 2u : 1u) : 1u;
    fp.dyn_start = (uint32_t)((rounds > dyn_rounds ? rounds - dyn_rounds : 0) * cfg.gridDim.x);
    if (rounds <= dyn_rounds) fp.tile_counter = nullptr;
    cfg.blockDim = dim3(FILTER_THREADS);
    // A single row scanned behind the threshold kernel: each CTA copies its next tiles into shared memory while it waits.
    // (Not the build that defers its candidates: their list takes the shared memory.)
    const bool prefetch = pdl && !deferred && rows == 1 && fp.dyn_start >= (FILTER_PREFETCH + 1) * cfg.gridDim.x;
    fp.prefetch_tiles = prefetch ? FILTER_PREFETCH : 0u;
    fp.prefetch_spin_limit = g_prefetch_spin_limit.load();
    cfg.dynamicSmemBytes = prefetch ? FILTER_PREFETCH * FILTER_THREADS * FILTER_UNROLL * 16u : 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
    if (hist && (rows != 1 || !deferred)) return PROFK_EINVAL;      // (no caller asks for that)
    if (hist) CUDA_TRY(cudaLaunchKernelEx(&cfg, filter_kernel<T, FILTER_THREADS, FILTER_UNROLL, false, true, true>, fp));
    else if (deferred) CUDA_TRY(cudaLaunchKernelEx(&cfg, filter_kernel<T, FILTER_THREADS, FILTER_UNROLL, false, true>, fp));
    else if (parts) CUDA_TRY(cudaLaunchKernelEx(&cfg, filter_kernel<T, FILTER_THREADS, FILTER_UNROLL, true>, fp));
    else CUDA_TRY(cudaLaunchKernelEx(&cfg, filter_kernel<T, FILTER_THREADS, FILTER_UNROLL>, fp));
    ++g_launches;
    return PROFK_OK;
}

// Cooperative launch (all CTAs co-resident: the kernel uses grid barriers), staged behind the kernel before it
// when the runtime accepts a cooperative launch that is also a programmatic dependent.  `set_pdl` tells the
// kernel's parameters which way it went.
template <typename Kernel, typename Params, typename SetPdl>
int launch_cooperative(cudaLaunchConfig_t cfg, Kernel kernel, Params params, bool after_kernel, SetPdl set_pdl) {
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    if (after_kernel && g_coop_pdl.load() != 0) {
        cfg.numAttrs = 2;
        set_pdl(params, 1);
        if (cudaLaunchKernelEx(&cfg, kernel, params) == cudaSuccess) {
            g_coop_pdl.store(1);
            ++g_launches;
            return PROFK_OK;
        }
        (void)cudaGetLastError();
        g_coop_pdl.store(0);
    }
    cfg.numAttrs = 1;
    set_pdl(params, 0);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, params));
    ++g_launches;
    return PROFK_OK;
}

// Count check + ordering for large selections: the whole grid, one CTA per SM, one row after the other.
template <typename T>
int launch_refine_large(const DeviceInfo& di, RowCtl* ctl, WsHeader* header, uint64_t* buf, uint64_t row_pitch, uint32_t* bins,
                        unsigned long long* slots, bool parts, uint32_t part_cap, const uint32_t* part_counts, int64_t rows,
                        int64_t capacity, int64_t k, int64_t k_accept, int phase, T* out_vals, int64_t* out_idx, cudaStream_t st,
                        const FallbackParams<T>* fused_fb = nullptr, bool after_kernel = true, int64_t N = 0, bool hist_ready = false) {
    LargeParams<T> lp;
    lp.hist_ready = hist_ready ? 1 : 0;
    lp.idx_bits = 32;                            // (N unknown: every bit of the index word may be used)
    if (N > 1) { lp.idx_bits = 1; while (((int64_t)1 << lp.idx_bits) < N) ++lp.idx_bits; }
    lp.fused = fused_fb ? (rows == 1 ? 1 : 2) : 0;
    if (fused_fb) lp.fb = *fused_fb; else lp.fb = FallbackParams<T>{};
    lp.ctl = ctl; lp.header = header; lp.buf = buf; lp.row_stride = row_pitch / 2; lp.bins = bins; lp.slots = slots;
    lp.parts = (phase == 0 && parts) ? FILTER_PARTS : 1u; lp.part_cap = part_cap; lp.part_counts = part_counts;
    lp.rows = (uint64_t)rows; lp.capacity = (uint32_t)capacity;
    lp.k = (uint32_t)k; lp.k_accept = (uint32_t)k_accept; lp.phase = phase; lp.out_vals = out_vals; lp.out_idx = out_idx;
    lp.use_pdl = 0;
    cudaLaunchConfig_t cfg = {};
    // Several rows: the grid splits into groups of CTAs that take rows side by side (a row alone keeps all SMs).
    const unsigned groups = (unsigned)std::min<int64_t>(rows, WS_GROUPS);
    const unsigned ctas = (unsigned)std::min(di.sm_count, LARGE_MAX_CTAS);
    lp.groups = groups;
    cfg.gridDim = dim3(ctas / groups * groups);
    cfg.blockDim = dim3(BT_THREADS);
    cfg.dynamicSmemBytes = (size_t)BT_TILE * 8;
    cfg.stream = st;
    return launch_cooperative(cfg, refine_large_kernel<T>, lp, after_kernel, [](LargeParams<T>& q, int v) { q.use_pdl = v; });
}

// Who replaces a row that fails the count check.  With few rows each row gets a cluster of CTAs in
// the refine kernel, large enough to read a whole row at a good rate, and the call ends with that
// kernel.  With many rows a cluster per row would be mostly idle CTAs, and a single CTA is too slow a
// reader when failures are not rare (many rows, loose eps): the rows are left to a grid-wide
// cooperative kernel that follows, whose launch is a few microseconds in a call that is long anyway.
template <typename T> int refine_cluster_size(const DeviceInfo& di, int64_t rows, int64_t N) {
    int csize = rows <= 9 ? 16 : rows <= XS_MAX_ROWS ? 8 : 1;
    csize = std::min(csize, di.refine_cluster[dtype_index<T>()]);
    const int64_t tile_elems = (int64_t)1024 * XS_UNROLL * Elem<T>::VEC;      // the largest tile a CTA may have
    while (csize > 1 && (int64_t)csize * tile_elems > N) csize /= 2;       // no more CTAs than tiles of the row
    return csize;
}

// Count check + refine, one cluster of `csize` CTAs per row (see refine_cluster_size).
template <typename T>
int launch_refine(const DeviceInfo& di, const T* in, int64_t rows, int64_t N, RowCtl* ctl, WsHeader* header, uint64_t* buf,
                  uint64_t row_stride, int64_t capacity, int64_t k, int64_t k_accept, bool direct, int csize, uint64_t* xs_records,
                  uint32_t* xs_counters, T* out_vals, int64_t* out_idx, cudaStream_t st, const SampleInfo* sample = nullptr,
                  uint4* thr2 = nullptr) {
    uint32_t sort_cap = 32;
    while (sort_cap < (uint32_t)k && sort_cap < SORT_CAP_MAX) sort_cap <<= 1;
    RefineParams<T> rp;
    rp.in = in; rp.N = (uint64_t)N;
    rp.ctl = ctl; rp.header = header; rp.buf = buf; rp.buf_stride = row_stride; rp.capacity = (uint32_t)capacity; rp.k = (uint32_t)k;
    rp.k_accept = (uint32_t)k_accept;
    rp.sort_cap = sort_cap;
    rp.stage_cap = 0;            // the general select (crowded bins only) reads the buffer in place
    rp.out_vals = out_vals; rp.out_idx = out_idx;
    rp.use_pdl = direct ? 0 : 1;
    rp.direct = direct ? 1 : 0;
    rp.cluster_size = (uint32_t)csize;
    unsigned threads = csize > 1 ? REFINE_CLUSTER_THREADS : 128;      // a cluster may have to read whole rows
    while (threads < 1024 && threads * 8 < (unsigned)capacity) threads <<= 1;
    // More rows than SMs, one CTA per row: CTAs of 1024 threads run one to an SM, wave after wave (512 rows: 3.4 us a
    // row, the last done 17 us after the filter); CTAs of 256 threads all start at once.  A buffer is a third full as a
    // rule, so 256 threads hold a row's records in one batch of eight when the capacity is within 6144.
    if (csize == 1 && !direct && rows > di.sm_count && capacity <= 6144) threads = 256;
    // A failed row is cut into segments, one cluster each, so that all SMs read it: as many clusters per
    // row as the SMs hold at once, but no more than the row has tiles for.
    int64_t nseg = 1;
    if (csize > 1) {
        const int64_t tiles = (int64_t)tiles_per_row<T>((uint64_t)N, threads * XS_UNROLL);
        nseg = std::max<int64_t>(1, std::min<int64_t>({di.sm_count / (rows * csize), tiles / csize, (int64_t)XS_MAX_SEGMENTS / rows}));
    }
    rp.clusters_per_row = (uint32_t)nseg;
    rp.xs_records = xs_records; rp.xs_counters = xs_counters;
    rp.sample = sample ? *sample : SampleInfo{};
    rp.thr2 = thr2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(rows * nseg * csize));
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = ((size_t)sort_cap + RF_EDGE_CAP + rp.stage_cap) * 8;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    unsigned na = 0;
    if (csize > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)csize; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (!direct) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr; cfg.numAttrs = na;
    if (threads <= 512) CUDA_TRY(cudaLaunchKernelEx(&cfg, refine_kernel<T, 48>, rp));
    else CUDA_TRY(cudaLaunchKernelEx(&cfg, refine_kernel<T, 64>, rp));
    ++g_launches;
    return PROFK_OK;
}

// Which build of the filter takes a launch with this many survivors expected per warp-tile.  From about one survivor per
// warp-tile on, most tiles would run the slow path and the scan becomes instruction-bound; the build that only notes its
// candidates in shared memory and decides them after streaming (DEFER, filter.cuh) then wins for bf16 (twice the
// elements per warp-tile): 512 rows of 2^20, k = 32 (1.46 per warp-tile) 298 -> 260 us; the paper's SAE shape (3.2)
// 112 -> 97.  fp32: the SAE shape (1.6) 93.4 -> 89.3; batches of fp32 rows (0.73) lose 6 % (397 -> 422 us) and stay on
// the direct build.  (An earlier build that staged survivors per warp in shared memory has gone: this one beat it
// wherever it was chosen.)
// A large selection from a single row (and the BatchTopK entry points) gains more: the deferring build also hands the
// kernel behind it a finished histogram (HIST, filter.cuh) and needs no partitioned append; from 0.1 survivors per
// warp-tile on it wins (2^29 bf16, K = 131072 at 0.41: 218 -> 212 us; 2^26 fp32, k = 32768 at 0.36: 89 -> 81; 2^28 bf16,
// k = 20000 at 0.18: 127 -> 120; at 0.05 it loses half a percent to the direct build with its prefetched tiles).
template <typename T> bool defer_candidates(int64_t rows, double per_warp_tile, bool large_one_row = false) {
    if (large_one_row) return per_warp_tile > 0.1;
    if (sizeof(T) == 2) return per_warp_tile > 0.8;
    return rows == 1 && per_warp_tile > 1.0;
}

template <typename T>
int topk_planned(const T* in, int64_t rows, int64_t N, int64_t k, const profk_plan_t* plan, uint64_t seed, void* stream,
                 T* out_vals, int64_t* out_idx) {
    g_launches = 0;
    if (!in || !out_vals || !out_idx || !plan) return PROFK_EINVAL;
    if (rows < 1 || N < 1 || N > N_MAX || k < 1 || k > N) return PROFK_EINVAL;
    if (((uintptr_t)in % sizeof(T)) || ((uintptr_t)out_vals % sizeof(T)) || ((uintptr_t)out_idx % 8)) return PROFK_EINVAL;
    const int64_t capacity = plan->capacity;
    if (capacity < k || capacity > N || rows * capacity >= (1LL << 40)) return PROFK_EINVAL;
    if (plan->mode != 0 && plan->mode != 1) return PROFK_EINVAL;
    if (plan->tie_rule != PROFK_TIES_KEEP_ALL && plan->tie_rule != PROFK_TIES_BY_INDEX) return PROFK_EINVAL;
    if (plan->mode == 0) {
        if (plan->m < 1 || plan->m > std::min<int64_t>(N, M_MAX) || plan->r < 1 || plan->r > plan->m) return PROFK_EINVAL;
        if (plan->k_accept < 1 || plan->k_accept > k) return PROFK_EINVAL;
        if (plan->r_tight < 0 || plan->r_tight > plan->m || plan->r_loose < 0 || plan->r_loose > plan->m) return PROFK_EINVAL;
    }

    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    DeviceInfo di;
    int rc = ensure_device_info<T>(dev, &di);
    if (rc != PROFK_OK) return rc;

    Workspace ws;
    if (g_ws_override_ptr) {
        ws = Workspace{g_ws_override_ptr, g_ws_override_bytes};
    } else {
        std::lock_guard<std::mutex> lock(g_mutex);
        ws = g_workspace[dev];
    }
    const bool large = g_ws_override_ptr ? large_selection_few(rows, k, sizeof(T)) : large_selection(rows, k, sizeof(T), N);
    const int64_t kept_sample_max = g_ws_override_ptr ? KEPT_SAMPLE_NOALLOC_MAX : KEPT_SAMPLE_MAX;
    const WsLayout lay = ws_layout(rows, capacity, k, large, kept_sample_max);
    if (!ws.ptr || ws.bytes < lay.total) return PROFK_EWORKSPACE;
    const uint64_t row_stride = row_stride_for(capacity, large);
    unsigned char* base = static_cast<unsigned char*>(ws.ptr);
    WsHeader* header = reinterpret_cast<WsHeader*>(base + lay.off_header);
    uint32_t* ghist = reinterpret_cast<uint32_t*>(base + lay.off_ghist);
    RowCtl* ctl = reinterpret_cast<RowCtl*>(base + lay.off_ctl);
    uint4* thr = reinterpret_cast<uint4*>(base + lay.off_tau);
    uint64_t* buf = reinterpret_cast<uint64_t*>(base + lay.off_buf);
    uint32_t* bins = reinterpret_cast<uint32_t*>(base + lay.off_bins);
    uint32_t* xs_counters = reinterpret_cast<uint32_t*>(base + lay.off_xs_counters);
    uint64_t* xs_records = reinterpret_cast<uint64_t*>(base + lay.off_xs_records);
    uint32_t* keys_scratch = reinterpret_cast<uint32_t*>(base + lay.off_keys);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // Survivors expected per warp-tile (expected survivors per element ~ r / m) decide the build of the filter: sparse
    // survivors are appended directly, dense ones noted and decided after streaming.
    const double per_warp_tile = (double)plan->r / (double)std::max<int64_t>(plan->m, 1) * 32.0 * FILTER_UNROLL * Elem<T>::VEC;
    const bool deferred = plan->mode == 0 && defer_candidates<T>(rows, per_warp_tile, large && rows == 1);

    // Large selections keep so many survivors that a row's single append counter would hold the scan up:
    // the direct variant then appends to FILTER_PARTS parts of the buffer, each with a counter of its own.
    // (The deferring build appends once per 32 candidates, after streaming: one counter is enough for it.)
    const bool parts = large && !deferred && plan->mode == 0;
    const uint32_t part_cap = (uint32_t)(row_stride / 2 / FILTER_PARTS);
    uint32_t* part_counts = reinterpret_cast<uint32_t*>(base + lay.off_parts);

    const int csize = (large || rows > XS_MAX_ROWS) ? 1 : refine_cluster_size<T>(di, rows, N);
    const bool exact_in_refine = csize > 1;
    uint32_t fb_sort_cap = 32;
    while (fb_sort_cap < (uint32_t)k && fb_sort_cap < SORT_CAP_MAX) fb_sort_cap <<= 1;

    // A second filtering pass for rows that fail the count check (plan->r_tight / r_loose) needs the sample's keys: they
    // are kept when the workspace has room for them and a kernel that takes that pass does the repair: the refine
    // kernel's clusters, the grid-wide repair kernel (large selections: up to XS_MAX_ROWS rows), or the fused kernel of a
    // large selection from a single row.
    const bool keep_keys = (!large || rows <= XS_MAX_ROWS) && plan->mode == 0 && (plan->r_tight > 0 || plan->r_loose > 0) &&
                           (rows <= GATHER_MAX_ROWS || plan->m <= (rows <= XS_MAX_ROWS ? kept_sample_max : KEPT_SAMPLE_BATCH_MAX));
    SampleInfo sample = {};
    if (keep_keys) {
        sample.keys = keys_scratch; sample.S = (uint32_t)plan->m; sample.seed = seed;
        sample.q = (uint64_t)(N / plan->m); sample.rem = (uint32_t)(N % plan->m); sample.inv_s = 1.0f / (float)plan->m;
        sample.by_record = plan->tie_rule == PROFK_TIES_BY_INDEX ? 1 : 0;
        sample.r_tight = (uint32_t)plan->r_tight; sample.r_loose = (uint32_t)plan->r_loose;
    }
    uint4* thr2 = reinterpret_cast<uint4*>(base + lay.off_tau2);

    // What the grid-wide exact selection needs (the kernel of its own, or the large refine when it does that itself).
    FallbackParams<T> fb;
    fb.in = in; fb.N = (uint64_t)N; fb.rows = (uint64_t)rows; fb.k = (uint32_t)k;
    fb.capacity = (uint32_t)capacity; fb.ctl = ctl; fb.header = header; fb.ghist = ghist; fb.buf = buf;
    fb.buf_stride = row_stride; fb.sort_rows = large ? 0 : 1;
    fb.tiles_per_row = tiles_per_row<T>((uint64_t)N, FB_THREADS * FB_UNROLL);
    fb.use_pdl = 0;
    fb.out_vals = out_vals; fb.out_idx = out_idx;
    const bool fbp = rows > XS_MAX_ROWS && !large;
    fb.cta_records = fbp ? reinterpret_cast<uint64_t*>(base + lay.off_fb_records) : nullptr;
    fb.cta_counters = fbp ? reinterpret_cast<uint32_t*>(base + lay.off_fb_counters) : nullptr;
    fb.sort_cap = fb_sort_cap;
    fb.parallel = (fbp || large) ? 1 : 0;      // large selections write into the rows' own buffers
    fb.sample = keep_keys ? sample : SampleInfo{};
    fb.thr2 = thr2;
    // A large selection from a single row: the count check, the exact replacement of a row that fails it and the
    // ordering are one cooperative kernel (three launches otherwise, two of which do nothing when no row failed).
    const bool fused_large = large && rows == 1;
    // ... and from a few rows (not in direct mode): the groups of the grid order the rows that passed, then the whole
    // grid repairs and orders the rest -- the two cooperative launches saved cost 7-9 us each behind their predecessors.
    const bool fused_some = large && rows > 1 && rows <= XS_MAX_ROWS && plan->mode == 0;

    // ... and when its filter is the deferring build, that counts the records it appends in the bins the ordering starts
    // from (cleared by the threshold kernels).
    const bool hist = fused_large && deferred;

    if (plan->mode == 0) {
        rc = launch_sample_select<T>(di, in, rows, N, plan->m, plan->r, seed, nullptr, ctl, header, (uint32_t)capacity, nullptr,
                                     rows <= GATHER_MAX_ROWS ? keys_scratch : nullptr, parts ? part_counts : nullptr, plan->tie_rule == PROFK_TIES_BY_INDEX, thr, st,
                                     nullptr, keep_keys ? keys_scratch : nullptr, hist ? bins : nullptr, BIN_ROW_WORDS);
        if (rc != PROFK_OK) return rc;
        rc = launch_filter<T>(di, in, rows, N, nullptr, capacity, buf, row_stride, &ctl[0].count, sizeof(RowCtl) / 4, true, &header->tile_counter,
                              parts, part_cap, part_counts, thr, st, deferred, hist ? bins : nullptr);
        if (rc != PROFK_OK) return rc;

        if (large) {
            rc = launch_refine_large<T>(di, ctl, header, buf, row_stride, bins, reinterpret_cast<unsigned long long*>(ghist), parts, part_cap, part_counts, rows,
                                        capacity, k, plan->k_accept, 0, out_vals, out_idx, st, fused_large || fused_some ? &fb : nullptr, true, N, hist);
            if (fused_large || fused_some) return rc;
        } else {
            // count check and refine; with clusters, also the exact selection of the rows that fail the check
            rc = launch_refine<T>(di, in, rows, N, ctl, header, buf, row_stride, capacity, k, plan->k_accept, false, csize, xs_records, xs_counters, out_vals, out_idx, st,
                                  keep_keys ? &sample : nullptr, thr2);
        }
        if (rc != PROFK_OK) return rc;
    } else {
        init_ctl_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(ctl, (uint64_t)rows, header, (uint32_t)capacity, (uint32_t)k);
        CUDA_TRY(cudaGetLastError());
        ++g_launches;
        if (exact_in_refine)
            return launch_refine<T>(di, in, rows, N, ctl, header, buf, row_stride, capacity, k, k, true, csize, xs_records, xs_counters, out_vals, out_idx, st);
        if (fused_large)
            return launch_refine_large<T>(di, ctl, header, buf, row_stride, bins, reinterpret_cast<unsigned long long*>(ghist), false, part_cap, part_counts, rows,
                                          capacity, k, k, 0, out_vals, out_idx, st, &fb, false, N);
    }

    if (!exact_in_refine) {
        // Exact selection of the rows that failed the check (or, in direct mode, of all rows) by a grid-wide
        // cooperative kernel: all CTAs co-resident.  For large selections it runs between the two phases
        // of the large refine.
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(std::min<unsigned>((unsigned)di.sm_count, FB_MAX_CTAS));
        cfg.blockDim = dim3(FB_THREADS);
        cfg.dynamicSmemBytes = large ? 0 : (size_t)fb_sort_cap * 8;
        cfg.stream = st;
        rc = launch_cooperative(cfg, fallback_kernel<T>, fb, plan->mode == 0, [](FallbackParams<T>& q, int v) { q.use_pdl = v; });
        if (rc != PROFK_OK) return rc;
    }
    if (large) {   // the rows the exact selection repaired still have to be ordered and written
        rc = launch_refine_large<T>(di, ctl, header, buf, row_stride, bins, reinterpret_cast<unsigned long long*>(ghist), false, part_cap, part_counts, rows,
                                    capacity, k, k, 1, out_vals,
                                    out_idx, st, nullptr, true, N);
        if (rc != PROFK_OK) return rc;
    }
    return PROFK_OK;
}

// The library's plan for a shape, kept for the shapes seen (the plan costs some host time: tail sums, bisections).
int cached_plan(int64_t rows, int64_t N, int64_t k, double eps, double recall, profk_plan_t* plan) {
    std::lock_guard<std::mutex> lock(g_mutex);
    const int64_t plan_rows = rows <= GATHER_MAX_ROWS ? 1 : GATHER_MAX_ROWS + 1;     // the two classes the tuning knows
    const auto key = std::make_tuple(plan_rows, N, k, eps, recall);
    auto it = g_plan_cache.find(key);
    if (it == g_plan_cache.end()) {
        const int rc = profk_plan_batch(plan_rows, N, k, eps, recall, plan);
        if (rc != PROFK_OK) return rc;
        if (g_plan_cache.size() > 4096) g_plan_cache.clear();
        g_plan_cache[key] = *plan;
    } else {
        *plan = it->second;
    }
    return PROFK_OK;
}

template <typename T>
int topk_auto(const T* in, int64_t rows, int64_t N, int64_t k, double eps, double recall, uint64_t seed, void* stream,
              T* out_vals, int64_t* out_idx) {
    g_launches = 0;
    profk_plan_t plan;
    const int rc = cached_plan(rows, N, k, eps, recall, &plan);
    if (rc != PROFK_OK) return rc;
    return topk_planned<T>(in, rows, N, k, &plan, seed, stream, out_vals, out_idx);
}

// Flattened BatchTopK: stages 1-3 as in topk_planned (one row), then the kept set without ordering (batchtopk.cuh).
template <typename T>
int batchtopk_planned(const T* in, int64_t N, int64_t K, const profk_plan_t* plan, uint64_t seed, void* stream, T* sel_vals,
                      int64_t* sel_idx, uint32_t* mask, T* dense) {
    g_launches = 0;
    if (!in || !plan) return PROFK_EINVAL;
    if ((sel_vals == nullptr) != (sel_idx == nullptr)) return PROFK_EINVAL;
    if (!sel_vals && !mask && !dense) return PROFK_EINVAL;
    if (N < 1 || N > N_MAX || K < 1 || K > N) return PROFK_EINVAL;
    if (((uintptr_t)in % sizeof(T)) || ((uintptr_t)sel_vals % sizeof(T)) || ((uintptr_t)sel_idx % 8) || ((uintptr_t)mask % 4) ||
        ((uintptr_t)dense % sizeof(T)))
        return PROFK_EINVAL;
    const int64_t capacity = plan->capacity;
    if (capacity < K || capacity > N) return PROFK_EINVAL;
    if (plan->mode != 0 && plan->mode != 1) return PROFK_EINVAL;
    if (plan->tie_rule != PROFK_TIES_KEEP_ALL && plan->tie_rule != PROFK_TIES_BY_INDEX) return PROFK_EINVAL;
    if (plan->mode == 0) {
        if (plan->m < 1 || plan->m > std::min<int64_t>(N, M_MAX) || plan->r < 1 || plan->r > plan->m) return PROFK_EINVAL;
        if (plan->k_accept != K) return PROFK_EINVAL;          // the kept set has exactly K members: no relaxed mode
        if (plan->r_tight < 0 || plan->r_tight > plan->m || plan->r_loose < 0 || plan->r_loose > plan->m) return PROFK_EINVAL;
    }
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    DeviceInfo di;
    int rc = ensure_device_info<T>(dev, &di);
    if (rc != PROFK_OK) return rc;
    Workspace ws;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        ws = g_workspace[dev];
    }
    const WsLayout lay = ws_layout(1, capacity, K, true);
    if (!ws.ptr || ws.bytes < lay.total) return PROFK_EWORKSPACE;
    const uint64_t row_stride = row_stride_for(capacity, true);
    unsigned char* base = static_cast<unsigned char*>(ws.ptr);
    WsHeader* header = reinterpret_cast<WsHeader*>(base + lay.off_header);
    uint32_t* ghist = reinterpret_cast<uint32_t*>(base + lay.off_ghist);
    RowCtl* ctl = reinterpret_cast<RowCtl*>(base + lay.off_ctl);
    uint4* thr = reinterpret_cast<uint4*>(base + lay.off_tau);
    uint64_t* buf = reinterpret_cast<uint64_t*>(base + lay.off_buf);
    uint32_t* bins = reinterpret_cast<uint32_t*>(base + lay.off_bins);
    uint32_t* keys_scratch = reinterpret_cast<uint32_t*>(base + lay.off_keys);
    uint32_t* part_counts = reinterpret_cast<uint32_t*>(base + lay.off_parts);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    const double per_warp_tile = (double)plan->r / (double)std::max<int64_t>(plan->m, 1) * 32.0 * FILTER_UNROLL * Elem<T>::VEC;
    const bool deferred = plan->mode == 0 && defer_candidates<T>(1, per_warp_tile, true);       // as in topk_planned for a large selection
    const bool parts = !deferred && plan->mode == 0;
    const uint32_t part_cap = (uint32_t)(row_stride / 2 / FILTER_PARTS);
    const bool hist = deferred;

    if (plan->mode == 0) {
        // The filter counts the records it appends in the bins the emit kernel selects from (cleared by the threshold kernels).
        rc = launch_sample_select<T>(di, in, 1, N, plan->m, plan->r, seed, nullptr, ctl, header, (uint32_t)capacity, nullptr, keys_scratch,
                                     parts ? part_counts : nullptr, plan->tie_rule == PROFK_TIES_BY_INDEX, thr, st, nullptr,
                                     (plan->r_tight > 0 || plan->r_loose > 0) ? keys_scratch : nullptr, hist ? bins : nullptr, BIN_ROW_WORDS);
        if (rc != PROFK_OK) return rc;
        rc = launch_filter<T>(di, in, 1, N, nullptr, capacity, buf, row_stride, &ctl[0].count, sizeof(RowCtl) / 4, true, &header->tile_counter,
                              parts, part_cap, part_counts, thr, st, deferred, hist ? bins : nullptr);
        if (rc != PROFK_OK) return rc;
    } else {
        init_ctl_kernel<<<1, 256, 0, st>>>(ctl, 1, header, (uint32_t)capacity, (uint32_t)K);
        CUDA_TRY(cudaGetLastError());
        ++g_launches;
    }
    BatchTopkParams<T> bp;
    bp.fb.in = in; bp.fb.N = (uint64_t)N; bp.fb.rows = 1; bp.fb.k = (uint32_t)K; bp.fb.capacity = (uint32_t)capacity;
    bp.fb.ctl = ctl; bp.fb.header = header; bp.fb.ghist = ghist; bp.fb.buf = buf; bp.fb.buf_stride = row_stride; bp.fb.sort_rows = 0;
    bp.fb.tiles_per_row = tiles_per_row<T>((uint64_t)N, FB_THREADS * FB_UNROLL);
    bp.fb.use_pdl = 0; bp.fb.out_vals = nullptr; bp.fb.out_idx = nullptr; bp.fb.cta_records = nullptr; bp.fb.cta_counters = nullptr;
    bp.fb.sort_cap = 0; bp.fb.parallel = 0;
    // the sample's keys stay in the workspace for a second filtering pass of a row that fails the count check
    const bool keep_keys = plan->mode == 0 && (plan->r_tight > 0 || plan->r_loose > 0);
    bp.fb.sample = SampleInfo{};
    if (keep_keys) {
        SampleInfo& sm = bp.fb.sample;
        sm.keys = keys_scratch; sm.S = (uint32_t)plan->m; sm.seed = seed;
        sm.q = (uint64_t)(N / plan->m); sm.rem = (uint32_t)(N % plan->m); sm.inv_s = 1.0f / (float)plan->m;
        sm.by_record = plan->tie_rule == PROFK_TIES_BY_INDEX ? 1 : 0;
        sm.r_tight = (uint32_t)plan->r_tight; sm.r_loose = (uint32_t)plan->r_loose;
    }
    bp.fb.thr2 = reinterpret_cast<uint4*>(base + lay.off_tau2);
    bp.bins = bins;
    bp.hist_ready = hist ? 1 : 0;
    bp.edge = buf + row_stride / 2;                               // the scratch half of the row's buffer
    bp.parts = parts ? FILTER_PARTS : 1u; bp.part_cap = part_cap; bp.part_counts = part_counts;
    bp.sel_vals = sel_vals; bp.sel_idx = sel_idx; bp.mask = mask; bp.dense = dense;
    bp.use_pdl = 0; bp.direct = plan->mode == 1 ? 1 : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(std::min<unsigned>((unsigned)di.sm_count, FB_MAX_CTAS));
    cfg.blockDim = dim3(BK_THREADS);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    return launch_cooperative(cfg, batchtopk_emit_kernel<T>, bp, plan->mode == 0, [](BatchTopkParams<T>& q, int v) { q.use_pdl = v; });
}

template <typename T>
int batchtopk_auto(const T* in, int64_t N, int64_t K, double eps, uint64_t seed, void* stream, T* sel_vals, int64_t* sel_idx,
                   uint32_t* mask, T* dense) {
    g_launches = 0;
    profk_plan_t plan;
    const int rc = cached_plan(1, N, K, eps, 1.0, &plan);
    if (rc != PROFK_OK) return rc;
    return batchtopk_planned<T>(in, N, K, &plan, seed, stream, sel_vals, sel_idx, mask, dense);
}

template <typename T>
int filter_only(const T* in, int64_t rows, int64_t N, const T* tau, int64_t capacity, uint64_t* buf_keys, uint32_t* counts,
                void* stream) {
    if (!in || !tau || !buf_keys || !counts) return PROFK_EINVAL;
    if (rows < 1 || N < 1 || N > N_MAX || capacity < 1 || capacity > N_MAX) return PROFK_EINVAL;
    if ((uintptr_t)in % sizeof(T) || (uintptr_t)tau % sizeof(T) || (uintptr_t)buf_keys % 8 || (uintptr_t)counts % 32)
        return PROFK_EINVAL;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    DeviceInfo di;
    const int rc = ensure_device_info<T>(dev, &di);
    if (rc != PROFK_OK) return rc;
    // The same build of the kernel a whole call would pick for this density of survivors, estimated from the capacity
    // (a plan's capacity is about twice the survivors it expects).
    // (a single row whose capacity is beyond what one CTA refines: a whole call would treat it as a large selection)
    const double per_warp_tile = 0.5 * (double)capacity / (double)N * 32.0 * FILTER_UNROLL * Elem<T>::VEC;
    return launch_filter<T>(di, in, rows, N, tau, capacity, buf_keys, (uint64_t)capacity, counts, PROFK_FILTER_COUNT_STRIDE, false, nullptr, false,
                            0u, nullptr, nullptr, static_cast<cudaStream_t>(stream), defer_candidates<T>(rows, per_warp_tile, rows == 1 && capacity > 32768));
}

template <typename T>
int sample_threshold(const T* in, int64_t rows, int64_t N, int64_t m, int64_t r, uint64_t seed, T* tau, uint32_t* sample_idx,
                     void* stream) {
    if (!in || !tau) return PROFK_EINVAL;
    if (rows < 1 || N < 1 || N > N_MAX || m < 1 || m > std::min<int64_t>(N, M_MAX) || r < 1 || r > m) return PROFK_EINVAL;
    if ((uintptr_t)in % sizeof(T) || (uintptr_t)tau % sizeof(T) || (uintptr_t)sample_idx % 4) return PROFK_EINVAL;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    DeviceInfo di;
    const int rc = ensure_device_info<T>(dev, &di);
    if (rc != PROFK_OK) return rc;
    return launch_sample_select<T>(di, in, rows, N, m, r, seed, tau, nullptr, nullptr, 0, sample_idx, nullptr, nullptr, false, nullptr,
                                   static_cast<cudaStream_t>(stream));
}

// ---- one row over several GPUs: the stage calls (shard.cuh) ----

// floor(j * N / m) on the host, as the kernels compute it.
int64_t stratum_start_host(int64_t j, int64_t N, int64_t m) { return (int64_t)(((unsigned __int128)j * (unsigned __int128)N) / (unsigned __int128)m); }

template <typename T>
int shard_sample_keys(const T* shard, int64_t shard_base, int64_t shard_len, int64_t N, int64_t m, int64_t j_lo, int64_t j_hi, uint64_t seed,
                      uint32_t* keys_out, void* stream) {
    if (!shard || !keys_out) return PROFK_EINVAL;
    if (N < 1 || N > N_MAX || m < 1 || m > std::min<int64_t>(N, M_MAX) || shard_len < 1 || shard_base < 0 || shard_base + shard_len > N) return PROFK_EINVAL;
    if (j_lo < 0 || j_hi <= j_lo || j_hi > m || (j_lo & 1) || ((j_hi & 1) && j_hi != m)) return PROFK_EINVAL;      // whole pairs of strata
    if (stratum_start_host(j_lo, N, m) < shard_base || stratum_start_host(j_hi, N, m) > shard_base + shard_len) return PROFK_EINVAL;
    if ((uintptr_t)shard % sizeof(T) || (uintptr_t)keys_out % 4) return PROFK_EINVAL;
    GatherParams<T> gp;
    gp.in = shard; gp.N = (uint64_t)N; gp.rows = 1; gp.S = (uint32_t)m; gp.seed = seed;
    gp.q = (uint64_t)(N / m); gp.rem = (uint32_t)(N % m); gp.inv_s = 1.0f / (float)m; gp.keys_out = keys_out;
    gp.pair_lo = (uint64_t)(j_lo / 2); gp.pairs = (uint64_t)((j_hi - j_lo + 1) / 2); gp.base = (uint64_t)shard_base;
    gp.zero = nullptr; gp.zero_vecs = 0;
    gather_kernel<T><<<(unsigned)((gp.pairs + GATHER_THREADS - 1) / GATHER_THREADS), GATHER_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(gp);
    CUDA_TRY(cudaGetLastError());
    return PROFK_OK;
}

template <typename T>
int threshold_from_keys(const uint32_t* keys, int64_t N, int64_t m, int64_t r, uint64_t seed, int tie_rule, uint32_t* thr_record, void* stream) {
    if (!keys || !thr_record) return PROFK_EINVAL;
    if (N < 1 || N > N_MAX || m < 1 || m > std::min<int64_t>(N, M_MAX) || r < 1 || r > m) return PROFK_EINVAL;
    if (tie_rule != PROFK_TIES_KEEP_ALL && tie_rule != PROFK_TIES_BY_INDEX) return PROFK_EINVAL;
    if ((uintptr_t)keys % 4 || (uintptr_t)thr_record % 16) return PROFK_EINVAL;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    DeviceInfo di;
    const int rc = ensure_device_info<T>(dev, &di);
    if (rc != PROFK_OK) return rc;
    return launch_sample_select<T>(di, nullptr, 1, N, m, r, seed, nullptr, nullptr, nullptr, 0, nullptr, nullptr, nullptr,
                                   tie_rule == PROFK_TIES_BY_INDEX, reinterpret_cast<uint4*>(thr_record), static_cast<cudaStream_t>(stream), keys);
}

template <typename T>
int filter_shard(const T* shard, int64_t shard_base, int64_t shard_len, const uint32_t* thr_record, int64_t capacity, uint64_t* records,
                 uint32_t* state, void* stream) {
    if (!shard || !thr_record || !records || !state) return PROFK_EINVAL;
    if (shard_len < 1 || shard_base < 0 || shard_base + shard_len > N_MAX || capacity < 1 || capacity > N_MAX) return PROFK_EINVAL;
    if ((uintptr_t)shard % sizeof(T) || (uintptr_t)thr_record % 16 || (uintptr_t)records % 8 || (uintptr_t)state % 16) return PROFK_EINVAL;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    DeviceInfo di;
    const int rc = ensure_device_info<T>(dev, &di);
    if (rc != PROFK_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    localize_threshold_kernel<<<1, 32, 0, st>>>(reinterpret_cast<const uint4*>(thr_record), (unsigned long long)shard_base,
                                                (unsigned long long)shard_len, state);
    CUDA_TRY(cudaGetLastError());
    return launch_filter<T>(di, shard, 1, shard_len, nullptr, capacity, records, (uint64_t)capacity, state, 1, false, nullptr, false, 0u,
                            nullptr, reinterpret_cast<const uint4*>(state + 4), st);
}

template <typename T>
int refine_gathered(const uint64_t* records, const uint32_t* states, const int64_t* bases, int64_t shards, int64_t shard_capacity,
                    const uint32_t* thr_record, int64_t capacity, int64_t k, int64_t k_accept, T* out_vals, int64_t* out_idx,
                    uint32_t* status_out, void* stream) {
    g_launches = 0;
    if (!records || !states || !bases || !thr_record || !out_vals || !out_idx || !status_out) return PROFK_EINVAL;
    if (shards < 1 || shards > SHARD_MAX || shard_capacity < 1 || capacity < k || k < 1 || k_accept < 1 || k_accept > k || capacity > N_MAX) return PROFK_EINVAL;
    if ((uintptr_t)records % 8 || (uintptr_t)states % 16 || (uintptr_t)thr_record % 16 || (uintptr_t)out_vals % sizeof(T) || (uintptr_t)out_idx % 8 ||
        (uintptr_t)status_out % 4)
        return PROFK_EINVAL;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    DeviceInfo di;
    int rc = ensure_device_info<T>(dev, &di);
    if (rc != PROFK_OK) return rc;
    Workspace ws;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        ws = g_workspace[dev];
    }
    const bool large = large_selection(1, k, sizeof(T), 0);
    const WsLayout lay = ws_layout(1, capacity, k, large);
    if (!ws.ptr || ws.bytes < lay.total) return PROFK_EWORKSPACE;
    const uint64_t row_stride = row_stride_for(capacity, large);
    unsigned char* base = static_cast<unsigned char*>(ws.ptr);
    WsHeader* header = reinterpret_cast<WsHeader*>(base + lay.off_header);
    uint32_t* ghist = reinterpret_cast<uint32_t*>(base + lay.off_ghist);
    RowCtl* ctl = reinterpret_cast<RowCtl*>(base + lay.off_ctl);
    uint64_t* buf = reinterpret_cast<uint64_t*>(base + lay.off_buf);
    uint32_t* bins = reinterpret_cast<uint32_t*>(base + lay.off_bins);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ShardBases sb = {};
    for (int64_t g = 0; g < shards; ++g) {
        if (bases[g] < 0 || bases[g] > N_MAX) return PROFK_EINVAL;
        sb.base[g] = bases[g];
    }
    merge_shards_kernel<<<di.sm_count, 256, 0, st>>>(records, states, sb, (uint32_t)shards, (uint32_t)std::min<int64_t>(shard_capacity, 0xFFFFFFFFll),
                                                     (uint32_t)capacity, (uint32_t)k, (uint32_t)k_accept, reinterpret_cast<const uint4*>(thr_record),
                                                     buf, ctl, header, status_out);
    CUDA_TRY(cudaGetLastError());
    ++g_launches;
    // The ordinary count check and refinement of one row.  A row that fails the check is left alone here (its exact
    // replacement needs the whole row, which no single GPU holds): the caller reads status_out and repairs it.
    if (large)
        return launch_refine_large<T>(di, ctl, header, buf, row_stride, bins, reinterpret_cast<unsigned long long*>(ghist), false, 0u, nullptr, 1,
                                      capacity, k, k_accept, 0, out_vals, out_idx, st);
    return launch_refine<T>(di, static_cast<const T*>(nullptr), 1, 1, ctl, header, buf, row_stride, capacity, k, k_accept, false, 1, nullptr, nullptr,
                            out_vals, out_idx, st);
}

}  // namespace

// --------------------------------------------------------------------------------------- C ABI
extern "C" {

int profk_workspace_bytes(int64_t rows, int64_t capacity, int64_t k, size_t* bytes) {
    if (!bytes || rows < 1 || capacity < 1 || k < 1 || capacity < k || capacity > N_MAX || rows * capacity >= (1LL << 40))
        return PROFK_EINVAL;
    // (enough for either element type and any row length: they take the grid-wide layout from different k on)
    size_t need = 0;
    if (k <= (int64_t)SORT_CAP_MAX) need = ws_layout(rows, capacity, k, false).total;
    if (large_possible(rows, k)) need = std::max(need, ws_layout(rows, capacity, k, true).total);
    *bytes = need;
    return PROFK_OK;
}

int profk_set_workspace(void* dev_ptr, size_t bytes) {
    if ((dev_ptr == nullptr) != (bytes == 0)) return PROFK_EINVAL;
    if ((uintptr_t)dev_ptr % 256) return PROFK_EINVAL;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(g_mutex);
    g_workspace[dev] = Workspace{dev_ptr, bytes};
    return PROFK_OK;
}

int profk_topk_f32(const float* in, int64_t rows, int64_t N, int64_t k, double eps, double recall, uint64_t seed,
                   void* stream, float* out_vals, int64_t* out_idx) {
    return topk_auto<float>(in, rows, N, k, eps, recall, seed, stream, out_vals, out_idx);
}

int profk_batchtopk_workspace_bytes(int64_t capacity, int64_t K, size_t* bytes) {
    if (!bytes || capacity < 1 || K < 1 || capacity < K || capacity > N_MAX) return PROFK_EINVAL;
    *bytes = ws_layout(1, capacity, K, true).total;
    return PROFK_OK;
}

int profk_batchtopk_f32(const float* in, int64_t N, int64_t K, double eps, uint64_t seed, void* stream, float* sel_vals,
                        int64_t* sel_idx, uint32_t* mask, float* dense) {
    return batchtopk_auto<float>(in, N, K, eps, seed, stream, sel_vals, sel_idx, mask, dense);
}

int profk_batchtopk_bf16(const void* in, int64_t N, int64_t K, double eps, uint64_t seed, void* stream, void* sel_vals,
                         int64_t* sel_idx, uint32_t* mask, void* dense) {
    return batchtopk_auto<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(in), N, K, eps, seed, stream,
                                         static_cast<__nv_bfloat16*>(sel_vals), sel_idx, mask, static_cast<__nv_bfloat16*>(dense));
}

int profk_batchtopk_planned_f32(const float* in, int64_t N, int64_t K, const profk_plan_t* plan, uint64_t seed, void* stream,
                                float* sel_vals, int64_t* sel_idx, uint32_t* mask, float* dense) {
    return batchtopk_planned<float>(in, N, K, plan, seed, stream, sel_vals, sel_idx, mask, dense);
}

int profk_batchtopk_planned_bf16(const void* in, int64_t N, int64_t K, const profk_plan_t* plan, uint64_t seed, void* stream,
                                 void* sel_vals, int64_t* sel_idx, uint32_t* mask, void* dense) {
    return batchtopk_planned<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(in), N, K, plan, seed, stream,
                                            static_cast<__nv_bfloat16*>(sel_vals), sel_idx, mask, static_cast<__nv_bfloat16*>(dense));
}

int profk_topk_bf16(const void* in, int64_t rows, int64_t N, int64_t k, double eps, double recall, uint64_t seed,
                    void* stream, void* out_vals, int64_t* out_idx) {
    return topk_auto<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(in), rows, N, k, eps, recall, seed, stream,
                                    static_cast<__nv_bfloat16*>(out_vals), out_idx);
}

int profk_topk_planned_f32(const float* in, int64_t rows, int64_t N, int64_t k, const profk_plan_t* plan, uint64_t seed,
                           void* stream, float* out_vals, int64_t* out_idx) {
    return topk_planned<float>(in, rows, N, k, plan, seed, stream, out_vals, out_idx);
}

int profk_topk_planned_bf16(const void* in, int64_t rows, int64_t N, int64_t k, const profk_plan_t* plan, uint64_t seed,
                            void* stream, void* out_vals, int64_t* out_idx) {
    return topk_planned<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(in), rows, N, k, plan, seed, stream,
                                       static_cast<__nv_bfloat16*>(out_vals), out_idx);
}

int profk_filter_f32(const float* in, int64_t rows, int64_t N, const float* tau, int64_t capacity, uint64_t* buf_keys,
                     uint32_t* counts, void* stream) {
    return filter_only<float>(in, rows, N, tau, capacity, buf_keys, counts, stream);
}

int profk_filter_bf16(const void* in, int64_t rows, int64_t N, const void* tau, int64_t capacity, uint64_t* buf_keys,
                      uint32_t* counts, void* stream) {
    return filter_only<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(in), rows, N, static_cast<const __nv_bfloat16*>(tau),
                                      capacity, buf_keys, counts, stream);
}

int profk_sample_threshold_f32(const float* in, int64_t rows, int64_t N, int64_t m, int64_t r, uint64_t seed, float* tau,
                               uint32_t* sample_idx, void* stream) {
    return sample_threshold<float>(in, rows, N, m, r, seed, tau, sample_idx, stream);
}

int profk_sample_threshold_bf16(const void* in, int64_t rows, int64_t N, int64_t m, int64_t r, uint64_t seed, void* tau,
                                uint32_t* sample_idx, void* stream) {
    return sample_threshold<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(in), rows, N, m, r, seed,
                                           static_cast<__nv_bfloat16*>(tau), sample_idx, stream);
}

// ---- allocation-free entry point -------------------------------------------------------------
// Scratch for profk_topk_noalloc_f32: part of the library image, so every GPU that loads the
// library holds these 16 MiB until the process exits, whether or not the entry point is used.
constexpr size_t NOALLOC_SCRATCH_BYTES = (size_t)16 << 20;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

int profk_topk_noalloc_f32(const float* in, int64_t rows, int64_t N, int64_t k, double eps, double recall, uint64_t seed,
                           void* stream, float* out_vals, int64_t* out_idx) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    // In host code `g_noalloc_scratch` is only a handle of the symbol, not a device address: the
    // address on the current device comes from the runtime, once per device, and is kept.  Both
    // tables below have a fixed size, so that nothing here allocates on the host either.
    constexpr int MAX_DEVICES = 64;
    constexpr int PLAN_SLOTS = 16;
    struct PlanSlot { int64_t rows_class, N, k; double eps, recall; profk_plan_t plan; bool used; };
    static std::mutex table_mutex;
    static void* ptr_by_device[MAX_DEVICES] = {};
    static PlanSlot plans[PLAN_SLOTS] = {};
    static int next_slot = 0;
    if (dev < 0 || dev >= MAX_DEVICES) return PROFK_EINVAL;
    if (rows < 1) return PROFK_EINVAL;
    void* scratch = nullptr;
    profk_plan_t plan;
    {
        std::lock_guard<std::mutex> lock(table_mutex);
        if (!ptr_by_device[dev]) {
            void* p = nullptr;
            CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
            if (!p) return PROFK_ECUDA;
            ptr_by_device[dev] = p;
        }
        scratch = ptr_by_device[dev];
        // the plan costs some host time (tail sums, bisections): kept for the last few shapes
        const int64_t rows_class = rows <= GATHER_MAX_ROWS ? 1 : GATHER_MAX_ROWS + 1;     // the two classes the tuning knows
        const PlanSlot* hit = nullptr;
        for (const PlanSlot& ps : plans)
            if (ps.used && ps.rows_class == rows_class && ps.N == N && ps.k == k && ps.eps == eps && ps.recall == recall) hit = &ps;
        if (hit) {
            plan = hit->plan;
        } else {
            const int prc = profk_plan_batch(rows_class, N, k, eps, recall, &plan);
            if (prc != PROFK_OK) return prc;
            plans[next_slot] = PlanSlot{rows_class, N, k, eps, recall, plan, true};
            next_slot = (next_slot + 1) % PLAN_SLOTS;
        }
    }
    if (rows * plan.capacity >= (1LL << 40)) return PROFK_EINVAL;
    if (ws_layout(rows, plan.capacity, k, large_selection_few(rows, k, sizeof(float)), KEPT_SAMPLE_NOALLOC_MAX).total > NOALLOC_SCRATCH_BYTES) return PROFK_ETOOLARGE;
    g_ws_override_ptr = scratch;
    g_ws_override_bytes = NOALLOC_SCRATCH_BYTES;
    const int rc = topk_planned<float>(in, rows, N, k, &plan, seed, stream, out_vals, out_idx);
    g_ws_override_ptr = nullptr;
    g_ws_override_bytes = 0;
    return rc;
}

int profk_shard_bounds(int64_t N, int64_t m, int64_t shards, int64_t shard, int64_t* j_lo, int64_t* j_hi, int64_t* elem_lo, int64_t* elem_hi) {
    if (!j_lo || !j_hi || !elem_lo || !elem_hi) return PROFK_EINVAL;
    if (N < 1 || N > N_MAX || m < 1 || m > std::min<int64_t>(N, M_MAX) || shards < 1 || shards > SHARD_MAX || shard < 0 || shard >= shards) return PROFK_EINVAL;
    const int64_t pairs = (m + 1) / 2;                    // strata travel in pairs (one Philox block serves two)
    if (pairs < shards) return PROFK_EINVAL;
    const int64_t lo = 2 * (pairs * shard / shards), hi = shard + 1 == shards ? m : 2 * (pairs * (shard + 1) / shards);
    *j_lo = lo; *j_hi = hi;
    *elem_lo = stratum_start_host(lo, N, m);
    *elem_hi = stratum_start_host(hi, N, m);
    return PROFK_OK;
}

int profk_shard_sample_keys_f32(const float* shard, int64_t shard_base, int64_t shard_len, int64_t N, int64_t m, int64_t j_lo, int64_t j_hi,
                                uint64_t seed, uint32_t* keys_out, void* stream) {
    return shard_sample_keys<float>(shard, shard_base, shard_len, N, m, j_lo, j_hi, seed, keys_out, stream);
}
int profk_shard_sample_keys_bf16(const void* shard, int64_t shard_base, int64_t shard_len, int64_t N, int64_t m, int64_t j_lo, int64_t j_hi,
                                 uint64_t seed, uint32_t* keys_out, void* stream) {
    return shard_sample_keys<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(shard), shard_base, shard_len, N, m, j_lo, j_hi, seed, keys_out, stream);
}
int profk_threshold_from_keys_f32(const uint32_t* keys, int64_t N, int64_t m, int64_t r, uint64_t seed, int tie_rule, uint32_t* thr_record, void* stream) {
    return threshold_from_keys<float>(keys, N, m, r, seed, tie_rule, thr_record, stream);
}
int profk_threshold_from_keys_bf16(const uint32_t* keys, int64_t N, int64_t m, int64_t r, uint64_t seed, int tie_rule, uint32_t* thr_record, void* stream) {
    return threshold_from_keys<__nv_bfloat16>(keys, N, m, r, seed, tie_rule, thr_record, stream);
}
int profk_filter_shard_f32(const float* shard, int64_t shard_base, int64_t shard_len, const uint32_t* thr_record, int64_t capacity,
                           uint64_t* records, uint32_t* state, void* stream) {
    return filter_shard<float>(shard, shard_base, shard_len, thr_record, capacity, records, state, stream);
}
int profk_filter_shard_bf16(const void* shard, int64_t shard_base, int64_t shard_len, const uint32_t* thr_record, int64_t capacity,
                            uint64_t* records, uint32_t* state, void* stream) {
    return filter_shard<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(shard), shard_base, shard_len, thr_record, capacity, records, state, stream);
}
int profk_refine_gathered_f32(const uint64_t* records, const uint32_t* states, const int64_t* bases, int64_t shards, int64_t shard_capacity,
                              const uint32_t* thr_record, int64_t capacity, int64_t k, int64_t k_accept, float* out_vals, int64_t* out_idx,
                              uint32_t* status_out, void* stream) {
    return refine_gathered<float>(records, states, bases, shards, shard_capacity, thr_record, capacity, k, k_accept, out_vals, out_idx, status_out, stream);
}
int profk_refine_gathered_bf16(const uint64_t* records, const uint32_t* states, const int64_t* bases, int64_t shards, int64_t shard_capacity,
                               const uint32_t* thr_record, int64_t capacity, int64_t k, int64_t k_accept, void* out_vals, int64_t* out_idx,
                               uint32_t* status_out, void* stream) {
    return refine_gathered<__nv_bfloat16>(records, states, bases, shards, shard_capacity, thr_record, capacity, k, k_accept,
                                          static_cast<__nv_bfloat16*>(out_vals), out_idx, status_out, stream);
}

int profk_read_stats(void* stream, int64_t rows, profk_row_stats_t* out) {
    if (!out || rows < 1) return PROFK_EINVAL;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    Workspace ws;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        ws = g_workspace[dev];
    }
    const WsLayout lay = ws_layout(rows, 1, 1, false);
    if (!ws.ptr || ws.bytes < lay.off_ctl + (size_t)rows * sizeof(RowCtl)) return PROFK_EWORKSPACE;
    std::vector<RowCtl> host((size_t)rows);
    WsHeader hdr;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* base = static_cast<unsigned char*>(ws.ptr);
    CUDA_TRY(cudaMemcpyAsync(host.data(), base + lay.off_ctl, (size_t)rows * sizeof(RowCtl), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaMemcpyAsync(&hdr, base + lay.off_header, sizeof(WsHeader), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    for (int64_t r = 0; r < rows; ++r) {
        out[r].tau_bits = host[r].tau_bits;
        out[r].survivors = host[r].count;
        out[r].capacity = host[r].capacity;
        out[r].status = host[r].status | (hdr.error ? 0x80000000u : 0u);
    }
    return hdr.error ? PROFK_ETIMEOUT : PROFK_OK;
}

int profk_last_launch_count(void) { return g_launches; }

int profk_debug_set_prefetch_wait_polls(int64_t polls) {
    g_prefetch_spin_limit.store(polls < 0 ? PREFETCH_SPIN_LIMIT : (uint32_t)std::min<int64_t>(polls, PREFETCH_SPIN_LIMIT));
    return PROFK_OK;
}

const char* profk_strerror(int code) {
    switch (code) {
        case PROFK_OK: return "ok";
        case PROFK_EINVAL: return "invalid argument";
        case PROFK_EWORKSPACE: return "workspace missing or too small";
        case PROFK_ECUDA: return "CUDA runtime error";
        case PROFK_ETIMEOUT: return "device-side wait timed out";
        case PROFK_ETOOLARGE: return "problem too large for the built-in scratch of the allocation-free entry point";
        default: return "unknown status";
    }
}

}  // extern "C"
