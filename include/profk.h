/*
 * profk.h -- C ABI of the Prof-K top-k library for NVIDIA B200 (sm_100a).
 *
 * Prof-K (Section 3 of the paper, "The Prof-K algorithm") returns the k largest
 * entries of each row of a rows x N matrix together with their indices by
 *   1. drawing a small sample of S positions,
 *   2. taking the t-th largest sampled value as threshold tau,
 *   3. streaming the row once and appending every element x_i >= tau to a
 *      candidate buffer of capacity M,
 *   4. running an exact top-k on that buffer; when fewer than k candidates were
 *      kept or the buffer overflowed, an exact top-k of the whole row replaces it.
 * In this library every stage, the check of step 4 and the exact replacement
 * run on the GPU; no call copies anything to the host or waits for the device.
 *
 * Conventions for every entry point
 *   - Pointers marked [device] are device addresses valid on the current CUDA
 *     device; [host] are ordinary host addresses.  The library never allocates,
 *     frees or keeps device memory: inputs, outputs and the workspace belong to
 *     the caller.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Work is only enqueued; results are valid once the caller has
 *     synchronised the stream.
 *   - Return value: PROFK_OK (0) or a negative profk_status_t.  No exception
 *     crosses the boundary.  A repaired failure of the probabilistic filter is
 *     not an error: it shows only in the per-row statistics.
 *   - Layout: `in` is row-major, contiguous, rows x N; element (row, i) is at
 *     in[row * N + i].  Outputs are rows x k.  Indices are 0-based positions
 *     inside the row.  Each output row is ordered by value descending, equal
 *     values by index ascending; values are ordered through the total order
 *     -NaN < -inf < ... < -0 < +0 < ... < +inf < +NaN of their bit patterns.
 *   - Limits: 1 <= k <= N <= 2^32 - 2^24 per row, rows >= 1, rows * capacity < 2^40.
 *   - Two calls that use the same workspace must not overlap on the device.
 *   - Ordinary stream order is all a caller relies on.  The kernels of a call
 *     are enqueued as programmatic dependents of one another and of whatever
 *     precedes the call on the stream.  The call's first kernel computes its
 *     sample positions early but waits for the work before it
 *     (griddepcontrol.wait) before it reads the input or touches the workspace,
 *     and only after that wait does it release the kernels behind it.  The
 *     filtering scan does read tiles of the input before its own wait -- by then
 *     the first kernel's wait has returned, so whatever wrote the input has
 *     finished and its writes are visible, also when that producer itself
 *     released its dependents early (a GEMM epilogue with programmatic launch,
 *     or this library's own last kernel when one call's output feeds the next).
 *     A call can be captured into a CUDA graph once its shape has been used
 *     outside a capture (the first use sets kernel attributes).
 */
#ifndef PROFK_H
#define PROFK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum profk_status {
    PROFK_OK = 0,
    PROFK_EINVAL = -1,     /* bad argument (range, null pointer, alignment) */
    PROFK_EWORKSPACE = -2, /* no workspace registered on this device, or it is too small */
    PROFK_ECUDA = -3,      /* a CUDA runtime call or launch reported an error */
    PROFK_ETIMEOUT = -4,   /* profk_read_stats: a bounded device-side wait gave up during the call (result invalid) */
    PROFK_ETOOLARGE = -5   /* profk_topk_noalloc_f32 only: the shape needs more than the built-in scratch */
} profk_status_t;

typedef enum profk_dtype { PROFK_F32 = 0, PROFK_BF16 = 1 } profk_dtype_t;

/* Per-row outcome of the count check of stage 4. */
enum {
    PROFK_ROW_OK = 0,       /* k_accept <= R <= capacity: answer refined from the buffer   */
    PROFK_ROW_RECALL = 1,   /* R < k_accept: too few candidates, exact selection ran       */
    PROFK_ROW_OVERFLOW = 2, /* R > capacity: buffer overflowed, exact selection ran        */
    PROFK_ROW_DIRECT = 3,   /* plan mode 1: exact selection without sampling or filtering  */
    PROFK_ROW_RECALL_REFILTERED = 4,   /* R < k_accept, then k <= R' <= capacity with the looser rank r_loose:
                                          answer refined from the second filtering pass (tau, R report that pass) */
    PROFK_ROW_OVERFLOW_REFILTERED = 5  /* R > capacity, then k <= R' <= capacity with the tighter rank r_tight */
};

/* How the filter of stage 3 treats copies of the threshold value (profk_plan_t.tie_rule).
 *   PROFK_TIES_KEEP_ALL  Section 3 as printed: tau is the t-th largest sampled value and every x_i >= tau
 *                        is kept.  The analysis of Section 4 assumes distinct values; on a row with very
 *                        many copies of tau all of them survive and the buffer overflows.
 *   PROFK_TIES_BY_INDEX  tau is the t-th sampled element under (value descending, index ascending), a value
 *                        and an index, and of the elements whose bit pattern equals tau's only those with an
 *                        index <= tau's are kept.  Elements then have distinct ranks, the rank law of Lemma 1
 *                        holds for any input, and R is the rank of the threshold element.  On a row with no
 *                        second copy of tau both rules keep the same elements.  profk_plan's choice. */
enum {
    PROFK_TIES_KEEP_ALL = 0,
    PROFK_TIES_BY_INDEX = 1
};

/*
 * The parameters (S, t, M) of Section 4 / Algorithm 1, as this library chooses them.
 *   m         sample size S: Algorithm 1 steps 1-4 (Eq. optimal_S with log2 k,
 *             rounded, clamped to [s_min, s_max]) and never more than N.
 *   r         sample rank t (1-based): the smallest rank whose recall-failure
 *             bound Pr(R < k_accept) is <= eps/2.  Algorithm 1's last step
 *             (t <- 1 in the sparse regime) is NOT applied: it breaks the eps
 *             budget of Theorem 1 that this plan keeps.
 *   capacity  buffer capacity M: max(ceil(Eq. M), smallest M whose overflow
 *             bound Pr(R > M) is <= eps/2), never more than N.
 *   k_accept  k in exact mode (recall == 1), ceil(recall * k) in relaxed mode.
 *   mode      0 = sample / filter / refine; 1 = direct exact selection, chosen
 *             when 2 * capacity >= N or N <= 2 * m (the filter would not pay).
 *   tie_rule  PROFK_TIES_*; profk_plan and profk_plan_ex set PROFK_TIES_BY_INDEX.
 *   z, alpha  Algorithm 1's z = 2 Phi^{-1}(1 - eps/2) and alpha = k / N.
 *   p_recall_fail, p_overflow   the two bounds for the returned (m, r, capacity).
 *   r_tight, r_loose   second-chance ranks (0 = none).  Section 3, "Refinement", sends a row that fails the count
 *             check to an exact top-k of the full input; the appendix ("Fallback as a Safety Mechanism") argues
 *             that this is rare enough not to matter.  It is also avoidable most of the time: the sample is still
 *             there, so after an overflow the row is filtered once more with the threshold of the TIGHTER rank
 *             r_tight < r, after a recall failure with that of the LOOSER rank r_loose > r, into the same buffer
 *             with the same check k <= R <= M -- one more read of the row at streaming speed -- and only a row
 *             that fails again is selected exactly.  The ranks aim midway between k and M:
 *             r_tight = floor(r (k + M) / (2 M)), r_loose = r + ceil((M - k) m / (2 N)).  Used when the sample's keys
 *             are kept: any sample for up to four rows, m <= 131072 for up to 18 rows; for larger batches m <= 4096,
 *             when one CTA orders each row's selection (k <= 16384; there the grid-wide repair kernel takes the
 *             pass, as long as fewer than eight rows of the call failed).  Which kernel takes the pass follows from
 *             who orders the selection: the refine kernel's clusters where one CTA orders a row (k <= 16384; from
 *             one to 18 rows the library hands selections above 4096 -- one row: above 8192, bf16 above 3072 --
 *             to the whole grid where that measured faster, by element type, row count and row length), the one
 *             kernel after the filter for a grid-ordered selection from 1 to 18 rows and for the BatchTopK entry
 *             points.  Grid-ordered selections from more rows and anything else go straight to the exact
 *             selection.
 * Both bounds are binomial tail bounds valid for the stratified sampler the
 * library uses (one uniform draw from each of m equal strata of the row).
 */
typedef struct profk_plan {
    int64_t m;
    int64_t r;
    int64_t capacity;
    int64_t k_accept;
    int32_t mode;
    int32_t tie_rule;
    double z;
    double alpha;
    double p_recall_fail;
    double p_overflow;
    int64_t r_tight;
    int64_t r_loose;
} profk_plan_t;

/* Tuning inputs of Algorithm 1.  The paper's values (Section 4) are
 * s_min = 32768, s_max = 131072, cost_ratio (tau_B / tau_A) = 1; profk_plan_ex
 * takes them when `tuning` is NULL.  profk_plan_batch and the profk_topk_*
 * entry points use profk_default_tuning_batch(rows, N), tuned on B200:
 *   - the floor on the sample size follows the row length for short rows,
 *         s_min = min(32768, max(1024, N / 512)),
 *     because on this GPU a sample of 32768 elements touches every 128-byte
 *     line of a row of 2^20 elements (the sample pass would read the whole
 *     row) and rows of 2^16 elements would not be filtered at all;
 *   - the cost ratio grows with the row length, N / 2^22 clamped to [1, 16]
 *     for up to PROFK_ALL_SM_GATHER_ROWS rows (their sample is gathered by a
 *     kernel over all SMs, cheap at any size, while every survivor costs a
 *     trip through the filter's slow path and a record in the refine step),
 *     clamped to [1, 4] for larger batches.
 * profk_default_tuning(N) and profk_plan(N, ...) are the one-row forms.  Any
 * choice keeps the failure budget: rank and capacity are derived from the
 * bounds for the S in use. */
#define PROFK_ALL_SM_GATHER_ROWS 4

typedef struct profk_tuning {
    int64_t s_min;
    int64_t s_max;
    double cost_ratio;
} profk_tuning_t;

/* What happened to one row (read back with profk_read_stats). */
typedef struct profk_row_stats {
    uint32_t tau_bits;   /* threshold tau: fp32 bit pattern, or bf16 pattern in the low 16 bits */
    uint32_t survivors;  /* R, the elements the filter kept (|{i : x_i >= tau}| less the dropped copies of tau);
                            exact when <= capacity, otherwise only "> capacity" */
    uint32_t capacity;   /* M used for the row */
    uint32_t status;     /* PROFK_ROW_*; bit 31 set = a device-side wait timed out (result invalid) */
} profk_row_stats_t;

/*
 * Host, pure: Algorithm 1 with the guard described at profk_plan_t.
 *   N, k      row length and selection size, 1 <= k <= N <= 2^32 - 2^24
 *   eps       total failure budget, 0 < eps < 1 (the paper's default is 1e-3)
 *   recall    1.0 = exact mode; rho in (0,1) = relaxed mode (accept ceil(rho k) survivors)
 *   out       [host] receives the plan
 * Returns PROFK_EINVAL on a bad argument.  profk_plan_ex takes the tuning
 * inputs explicitly (NULL = the paper's constants); profk_default_tuning
 * writes the ones profk_plan uses for a row of length N.
 */
int profk_default_tuning(int64_t N, profk_tuning_t* tuning /* [host] out */);
int profk_default_tuning_batch(int64_t rows, int64_t N, profk_tuning_t* tuning /* [host] out */);
int profk_plan(int64_t N, int64_t k, double eps, double recall, profk_plan_t* out);
int profk_plan_batch(int64_t rows, int64_t N, int64_t k, double eps, double recall, profk_plan_t* out);
int profk_plan_ex(int64_t N, int64_t k, double eps, double recall, const profk_tuning_t* tuning,
                  profk_plan_t* out);

/*
 * Workspace.  profk_workspace_bytes gives the size the calls below need for
 * `rows` rows with buffer capacity `capacity` and selection size k (take
 * capacity from profk_plan; it does not depend on the element type: the size
 * is enough for either).
 * profk_set_workspace registers a caller-owned device allocation (256-byte
 * aligned) for the current device; it stays registered until replaced or
 * cleared with (NULL, 0).  Its contents need no initialisation and are
 * overwritten by every call.
 */
int profk_workspace_bytes(int64_t rows, int64_t capacity, int64_t k, size_t* bytes /* [host] */);
int profk_set_workspace(void* dev_ptr /* [device] */, size_t bytes);

/*
 * Top-k of every row (the problem statement of Section 3), all four stages on
 * the GPU.  Equivalent to profk_plan followed by profk_topk_planned_*.
 *   in        [device] rows x N elements, fp32 / bf16, aligned to the element size
 *   seed      keys the Philox4x32-10 sample; in exact mode the result does not
 *             depend on it, only tau, the buffer and the repair decision do
 *   out_vals  [device] rows x k, same element type as `in`
 *   out_idx   [device] rows x k int64
 * Relaxed mode (recall < 1): a row whose buffer holds R < k (but >= k_accept)
 * candidates returns its R best in order followed by padding (value -inf,
 * index -1); the result is always a prefix of the exact answer.
 * Errors: PROFK_EINVAL, PROFK_EWORKSPACE, PROFK_ECUDA.
 */
int profk_topk_f32(const float* in, int64_t rows, int64_t N, int64_t k, double eps, double recall,
                   uint64_t seed, void* stream, float* out_vals, int64_t* out_idx);
int profk_topk_bf16(const void* in, int64_t rows, int64_t N, int64_t k, double eps, double recall,
                    uint64_t seed, void* stream, void* out_vals, int64_t* out_idx);

/*
 * Same with the plan given explicitly (stages 1-4 of Section 3 with the
 * caller's S = m, t = r, M = capacity).  Any plan returns the exact answer,
 * because the count check repairs a bad one: capacity == k forces overflows,
 * r == 1 with a large m forces recall failures, mode == 1 skips the filter.
 * Requires 1 <= r <= m <= min(N, 262144), k <= capacity <= N,
 * 1 <= k_accept <= k (mode 0).
 */
int profk_topk_planned_f32(const float* in, int64_t rows, int64_t N, int64_t k, const profk_plan_t* plan,
                           uint64_t seed, void* stream, float* out_vals, int64_t* out_idx);
int profk_topk_planned_bf16(const void* in, int64_t rows, int64_t N, int64_t k, const profk_plan_t* plan,
                            uint64_t seed, void* stream, void* out_vals, int64_t* out_idx);

/*
 * Flattened BatchTopK (Section 5, "Application: BatchTopK sparse autoencoders"): the B x d_dict matrix of
 * pre-activations is read as ONE row of N = B * d_dict elements, its K = B * k largest entries are kept and every
 * other entry becomes zero.  Stages 1-3 and the count check of Section 3 run as in profk_topk_*; stage 4 only finds
 * the K-th best candidate and emits the kept set -- nothing is sorted, because the consumer of a BatchTopK does not
 * need an order.  The kept set is exactly the set profk_topk_* would return for (1 row, N, K): ties at the K-th value
 * go to the lowest indices, also when the count check fails and the exact selection of the whole row replaces the
 * buffer.  Exact mode only.  The set comes in up to three forms; pass NULL for a form that is not wanted (at least one
 * is; sel_vals and sel_idx go together):
 *   sel_vals, sel_idx  [device] K values and K int64 indices of the kept entries, in no particular order (the order
 *                      may differ from call to call; compare as a set)
 *   mask               [device] ceil(N / 32) uint32 words; bit (i % 32) of word i / 32 is set iff entry i is kept
 *   dense              [device] N elements: entry i holds in[i] (bit for bit) if it is kept, else +0.0.  May be `in`
 *                      itself (in place): the input is then overwritten once the kernels have finished reading it.
 * All outputs are written entirely by the call (mask and dense are zeroed first); none is read.
 *   in     [device] N elements;  eps, seed, stream as for profk_topk_*
 * The workspace must hold profk_batchtopk_workspace_bytes(capacity, K) bytes, capacity from profk_plan(N, K, eps, 1)
 * (a little more than profk_workspace_bytes(1, capacity, K) when K <= 8192).  profk_read_stats(stream, 1, ..) reports
 * the row as after profk_topk_*.  The _planned forms take (S, t, M) explicitly (k_accept must equal K): the test hook
 * that forces overflow, recall failure and direct mode.
 * Errors: PROFK_EINVAL, PROFK_EWORKSPACE, PROFK_ECUDA.
 */
int profk_batchtopk_workspace_bytes(int64_t capacity, int64_t K, size_t* bytes /* [host] */);
int profk_batchtopk_f32(const float* in, int64_t N, int64_t K, double eps, uint64_t seed, void* stream,
                        float* sel_vals, int64_t* sel_idx, uint32_t* mask, float* dense);
int profk_batchtopk_bf16(const void* in, int64_t N, int64_t K, double eps, uint64_t seed, void* stream,
                         void* sel_vals, int64_t* sel_idx, uint32_t* mask, void* dense);
int profk_batchtopk_planned_f32(const float* in, int64_t N, int64_t K, const profk_plan_t* plan, uint64_t seed, void* stream,
                                float* sel_vals, int64_t* sel_idx, uint32_t* mask, float* dense);
int profk_batchtopk_planned_bf16(const void* in, int64_t N, int64_t K, const profk_plan_t* plan, uint64_t seed, void* stream,
                                 void* sel_vals, int64_t* sel_idx, uint32_t* mask, void* dense);

/*
 * Stage 3 alone (the filtering scan of Section 3): for every row append the
 * elements with x_i >= tau[row] to the row's buffer and count them.  The
 * comparison is taken in the total order of the values (-NaN < -inf < ... <
 * -0 < +0 < ... < +inf < +NaN, by bit pattern), the order the sample is
 * sorted in; the threshold is a value alone (tie rule PROFK_TIES_KEEP_ALL).
 *   tau        [device] rows thresholds of the element type
 *   buf_keys   [device] rows x capacity uint64 candidate records (see below)
 *   counts     [device] rows x PROFK_FILTER_COUNT_STRIDE uint32 words, 32-byte aligned, zero on entry; on return word
 *              row * PROFK_FILTER_COUNT_STRIDE holds the row's number of survivors (exact if <= capacity, else some
 *              value > capacity).  One counter per 32 bytes: the rows' append atomics then do not share a memory sector
 *              (with adjacent counters a batch of 512 fp32 rows took 439 us instead of 345)
 * A candidate record packs the complemented order key of the value in the high
 * 32 bits (bf16: the 16-bit key in bits 47..32, bits 63..48 all ones) and the
 * index in the low 32 bits, so that ascending records are "value descending,
 * index ascending".  Records are
 * appended in no particular order.  Needs no workspace.  The launch takes the build of the kernel a whole call would
 * take for the density of survivors that `capacity` suggests (a plan's capacity is about twice the survivors it
 * expects): from about one survivor per warp-tile on (a tenth of one for a single row with a capacity beyond 32768
 * records, as for a large selection), the build that notes candidates in shared memory while streaming and decides
 * them afterwards.
 */
#define PROFK_FILTER_COUNT_STRIDE 8
int profk_filter_f32(const float* in, int64_t rows, int64_t N, const float* tau, int64_t capacity,
                     uint64_t* buf_keys, uint32_t* counts, void* stream);
int profk_filter_bf16(const void* in, int64_t rows, int64_t N, const void* tau, int64_t capacity,
                      uint64_t* buf_keys, uint32_t* counts, void* stream);

/*
 * Stages 1-2 alone (sampling and threshold estimation of Section 3): tau[row]
 * = the r-th largest of m stratified Philox samples of the row.  Also writes
 * the sampled indices when sample_idx != NULL ([device] rows x m uint32).
 */
int profk_sample_threshold_f32(const float* in, int64_t rows, int64_t N, int64_t m, int64_t r, uint64_t seed,
                               float* tau, uint32_t* sample_idx, void* stream);
int profk_sample_threshold_bf16(const void* in, int64_t rows, int64_t N, int64_t m, int64_t r, uint64_t seed,
                                void* tau, uint32_t* sample_idx, void* stream);

/*
 * ONE ROW SPLIT OVER SEVERAL GPUS.  The paper runs on a single GPU and leaves distributed settings to future work
 * (Section "Limitations"); the four stages of Section 3 split at two exchange points, and these stage calls are the
 * pieces between them.  Every GPU holds a contiguous shard of the row made of whole sampling strata
 * (profk_shard_bounds), so the sample -- and with it the threshold -- is the one the unsharded call draws for the same
 * seed.  The caller makes the two exchanges (an all-gather each) into LOCAL buffers; no call here touches another
 * GPU's memory.  Per row:
 *   1. profk_shard_sample_keys_*      stage 1 on the shard: the order keys of the samples of its strata
 *      -> all-gather the m keys (in stratum order)
 *   2. profk_threshold_from_keys_*    stage 2: the r-th largest sampled record, as a 16-byte threshold record
 *                                     {bits of tau, bits of the next value up, index of the record or 0xFFFFFFFF, 0}
 *   3. profk_filter_shard_*           stage 3 on the shard, indices local to the shard; state = 8 uint32 words,
 *                                     [0] = the shard's survivor count on return (the call zeroes it first)
 *      -> all-gather (state, records), `capacity` records per shard
 *   4. profk_refine_gathered_*        the count check on the summed counts and stage 4 on the merged records (global
 *                                     index = local index + bases[g]); status_out[0] = PROFK_ROW_OK / _RECALL /
 *                                     _OVERFLOW, status_out[1] = R.  Needs the registered workspace of
 *                                     profk_workspace_bytes(1, capacity, k).  On a status other than OK the outputs
 *                                     are not written: the exact replacement needs the whole row, which no single GPU
 *                                     holds -- the caller repairs the row (e.g. the exact top-k of every shard with
 *                                     profk_topk_*, gathered and selected from once more).
 * Arguments: shard [device] the shard's elements, shard_base / shard_len its position in the row of length N;
 * j_lo, j_hi the shard's strata [j_lo, j_hi) of m (j_lo even; j_hi even or m); keys_out / keys [device] uint32;
 * thr_record [device] 4 uint32, 16-byte aligned; records [device] uint64; state / states [device] 16-byte aligned;
 * bases [host] `shards` int64; shards <= 16.  m, r, capacity, k_accept, tie_rule come from profk_plan(N, k, ...).
 * Errors: PROFK_EINVAL, PROFK_EWORKSPACE, PROFK_ECUDA.
 */
int profk_shard_bounds(int64_t N, int64_t m, int64_t shards, int64_t shard,
                       int64_t* j_lo, int64_t* j_hi, int64_t* elem_lo, int64_t* elem_hi /* [host] out */);
int profk_shard_sample_keys_f32(const float* shard, int64_t shard_base, int64_t shard_len, int64_t N, int64_t m,
                                int64_t j_lo, int64_t j_hi, uint64_t seed, uint32_t* keys_out, void* stream);
int profk_shard_sample_keys_bf16(const void* shard, int64_t shard_base, int64_t shard_len, int64_t N, int64_t m,
                                 int64_t j_lo, int64_t j_hi, uint64_t seed, uint32_t* keys_out, void* stream);
int profk_threshold_from_keys_f32(const uint32_t* keys, int64_t N, int64_t m, int64_t r, uint64_t seed, int tie_rule,
                                  uint32_t* thr_record, void* stream);
int profk_threshold_from_keys_bf16(const uint32_t* keys, int64_t N, int64_t m, int64_t r, uint64_t seed, int tie_rule,
                                   uint32_t* thr_record, void* stream);
int profk_filter_shard_f32(const float* shard, int64_t shard_base, int64_t shard_len, const uint32_t* thr_record,
                           int64_t capacity, uint64_t* records, uint32_t* state, void* stream);
int profk_filter_shard_bf16(const void* shard, int64_t shard_base, int64_t shard_len, const uint32_t* thr_record,
                            int64_t capacity, uint64_t* records, uint32_t* state, void* stream);
int profk_refine_gathered_f32(const uint64_t* records, const uint32_t* states, const int64_t* bases, int64_t shards,
                              int64_t shard_capacity, const uint32_t* thr_record, int64_t capacity, int64_t k,
                              int64_t k_accept, float* out_vals, int64_t* out_idx, uint32_t* status_out, void* stream);
int profk_refine_gathered_bf16(const uint64_t* records, const uint32_t* states, const int64_t* bases, int64_t shards,
                               int64_t shard_capacity, const uint32_t* thr_record, int64_t capacity, int64_t k,
                               int64_t k_accept, void* out_vals, int64_t* out_idx, uint32_t* status_out, void* stream);

/*
 * (This entry point has no counterpart in the paper; it exists for callers that must not
 * allocate.)  Same result as profk_topk_f32, but no workspace has to be registered and the
 * entry point calls no allocator, neither cudaMalloc / cudaFree nor an allocating library
 * routine: the scratch is a 16 MiB array that is part of the library itself.  It is meant for code
 * that runs where an allocation is forbidden or would deadlock -- a callback of a memory
 * pool that is itself inside an allocation, a real-time or plug-in context that was handed
 * its buffers up front, a host that has already given all device memory to another
 * allocator -- and still needs a top-k of buffers it already owns.
 *   - Limit: the workspace the call lays out in the array (never more than profk_workspace_bytes
 *     for rows, the plan's capacity and k; this entry point keeps samples of 5 to 18 rows for the
 *     second filtering pass up to 32768 keys only, and hands selections from 2 to 4 rows to the
 *     whole grid from k = 8193 on whatever the rows' length) must fit 16 MiB; roughly
 *     rows * capacity <= 2,000,000 records, e.g.
 *     one row of any length up to the library limit with small k, or 512 rows of 2^20
 *     elements with k = 32.  Anything larger returns PROFK_ETOOLARGE and does nothing.
 *   - Every GPU that loads the library holds the 16 MiB until the process exits.
 *   - The first call on each device is a set-up call: it looks up the array's device address
 *     (and keeps it), and like any first use of this library on a device it may make the driver
 *     load the library's code and the array onto the device, sets kernel attributes and fills a
 *     small host-side table.  Make that first call before the region in which nothing may be
 *     allocated, and outside any stream capture; in a process whose device memory is already
 *     exhausted it can fail with PROFK_ECUDA.  Calls after it allocate nothing, on the host side
 *     of CUDA or on the device; the plan of the last 16 shapes is kept in a fixed table.
 *   - All calls share the one array, and it keeps whatever the last call left in it.  Each
 *     call re-initialises the parts that must start at zero, so calls issued one after the
 *     other on a stream are fine; two calls that overlap on the GPU (different streams,
 *     different threads) race on it and give wrong answers.
 *   - profk_read_stats does not see this call (it reads the registered workspace).
 * Arguments, layout and the other errors are those of profk_topk_f32.
 */
int profk_topk_noalloc_f32(const float* in, int64_t rows, int64_t N, int64_t k, double eps, double recall,
                           uint64_t seed, void* stream, float* out_vals, int64_t* out_idx);

/*
 * Copies the statistics of the last call that used the registered workspace to
 * the host and waits for `stream`.  out: [host] rows entries.  Every wait inside
 * the kernels is bounded (the grid barriers of the exact-selection and large-k
 * kernels); when one gave up, the kernels returned early, the call's outputs are
 * invalid, every status word has bit 31 set and the return value is
 * PROFK_ETIMEOUT (the entries are filled in all the same).  The next call on the
 * workspace clears the flag.
 */
int profk_read_stats(void* stream, int64_t rows, profk_row_stats_t* out);

/* Number of kernels the last profk_topk* call on this thread enqueued. */
int profk_last_launch_count(void);

/*
 * Diagnostic: how many polls a CTA of the filtering scan spends on the tiles it copied into shared memory while
 * the threshold was being computed before it reads them with plain loads instead (negative = the default, 2^22;
 * 0 = never use the copies).  Results do not depend on it.  Process-wide.
 */
int profk_debug_set_prefetch_wait_polls(int64_t polls);

/* Static text for a status code. */
const char* profk_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* PROFK_H */
