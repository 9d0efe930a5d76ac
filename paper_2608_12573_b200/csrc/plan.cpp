// Parameter selection (S, t, M) on the host: Algorithm 1 of the paper with the
// exact-tail guard that keeps Theorem 1's failure budget.  Pure double-precision
// arithmetic, no CUDA.  See profk_plan_t in profk.h for what each field means.
#include <cmath>
#include <cstdint>
#include <cstring>

#include "profk.h"

namespace {

// x with Pr(Z > x) = q for a standard normal Z, by bisection on erfc (monotone, so
// the bracket closes to the last bit in ~110 halvings of [-40, 40]).
double normal_upper_quantile(double q) {
    double lo = -40.0, hi = 40.0;
    for (int it = 0; it < 200; ++it) {
        double mid = 0.5 * (lo + hi);
        if (mid == lo || mid == hi) break;
        if (0.5 * std::erfc(mid * M_SQRT1_2) > q) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

double log_binom_pmf(int64_t n, int64_t x, double p) {
    return std::lgamma((double)n + 1.0) - std::lgamma((double)x + 1.0) - std::lgamma((double)(n - x) + 1.0) +
           (double)x * std::log(p) + (double)(n - x) * std::log1p(-p);
}

// Pr(Bin(n, p) >= t), summed upward from t (terms fall off geometrically past the mean).
double binom_upper_tail(int64_t n, double p, int64_t t) {
    if (t <= 0) return 1.0;
    if (t > n || p <= 0.0) return 0.0;
    if (p >= 1.0) return 1.0;
    double term = std::exp(log_binom_pmf(n, t, p));
    double sum = 0.0;
    const double odds = p / (1.0 - p);
    for (int64_t x = t; x <= n; ++x) {
        sum += term;
        if (term < 1e-18 * sum && (double)x > (double)n * p) break;
        term *= (double)(n - x) / (double)(x + 1) * odds;
    }
    return sum < 1.0 ? sum : 1.0;
}

// Pr(Bin(n, p) <= c), summed downward from c (terms fall off below the mean).
double binom_lower_tail(int64_t n, double p, int64_t c) {
    if (c < 0) return 0.0;
    if (c >= n || p <= 0.0) return 1.0;
    if (p >= 1.0) return 0.0;
    double term = std::exp(log_binom_pmf(n, c, p));
    double sum = 0.0;
    const double inv_odds = (1.0 - p) / p;
    for (int64_t x = c; x >= 0; --x) {
        sum += term;
        if (term < 1e-18 * sum && (double)x < (double)n * p) break;
        term *= (double)x / (double)(n - x + 1) * inv_odds;
    }
    return sum < 1.0 ? sum : 1.0;
}

// Bound on Pr(R < k_accept): the number of sample draws among the top k_accept-1 ranks
// is a sum of S independent Bernoullis (one per stratum) with mean at most
// mu = (k_accept-1) / floor(N/S); beyond the mean its upper tail is bounded by the
// binomial's (Hoeffding 1956), below it by Markov's inequality.
double recall_fail_bound(int64_t N, int64_t S, int64_t t, int64_t k_accept) {
    if (k_accept <= 1) return 0.0;
    double pa = (double)(k_accept - 1) / ((double)S * (double)(N / S));
    if (pa > 1.0) pa = 1.0;
    const double mu = (double)S * pa;
    if ((double)(t - 1) >= mu) return binom_upper_tail(S, pa, t);
    const double markov = mu / (double)t;
    return markov < 1.0 ? markov : 1.0;
}

// Bound on Pr(R > M): the number of draws among the top M ranks has mean at least
// mu = M / ceil(N/S); below the mean its lower tail is bounded by the binomial's.
double overflow_bound(int64_t N, int64_t S, int64_t t, int64_t M) {
    if (M >= N) return 0.0;
    double pb = (double)M / ((double)S * (double)((N + S - 1) / S));
    if (pb > 1.0) pb = 1.0;
    if ((double)t <= (double)S * pb) return binom_lower_tail(S, pb, t - 1);
    return 1.0;
}

}  // namespace

extern "C" int profk_plan_ex(int64_t N, int64_t k, double eps, double recall, const profk_tuning_t* tuning,
                             profk_plan_t* out) {
    if (!out) return PROFK_EINVAL;
    if (N < 1 || N > 4278190080LL || k < 1 || k > N) return PROFK_EINVAL;
    if (!(eps > 0.0 && eps < 1.0) || !(recall > 0.0 && recall <= 1.0)) return PROFK_EINVAL;
    int64_t s_min = 32768, s_max = 131072;
    double cost_ratio = 1.0;
    if (tuning) {
        s_min = tuning->s_min;
        s_max = tuning->s_max;
        cost_ratio = tuning->cost_ratio;
        if (s_min < 1 || s_max < s_min || s_max > 262144 || !(cost_ratio > 0.0)) return PROFK_EINVAL;
    }
    std::memset(out, 0, sizeof(*out));

    // Algorithm 1, steps 1-4.
    const double z = 2.0 * normal_upper_quantile(eps / 2.0);
    const double alpha = (double)k / (double)N;
    const double s_star = std::pow(z * cost_ratio * std::log2((double)k) / 2.0, 2.0 / 3.0) *
                          std::pow((double)k * (double)(N - k), 1.0 / 3.0);
    int64_t S = (int64_t)std::floor(s_star + 0.5);
    if (S < s_min) S = s_min;
    if (S > s_max) S = s_max;
    if (S > N) S = N;

    // Relaxed recall: accept ceil(recall * k) survivors.
    int64_t k_acc = (int64_t)std::ceil(recall * (double)k - 1e-9);
    if (k_acc < 1) k_acc = 1;
    if (k_acc > k) k_acc = k;

    // Smallest rank whose recall-failure bound fits eps/2 (the bound falls with t).
    const double eps_half = eps / 2.0;
    int64_t t = S;
    if (recall_fail_bound(N, S, S, k_acc) <= eps_half) {
        int64_t lo = 1, hi = S;
        while (lo < hi) {
            int64_t mid = (lo + hi) / 2;
            if (recall_fail_bound(N, S, mid, k_acc) <= eps_half) hi = mid; else lo = mid + 1;
        }
        t = lo;
    }

    // Smallest capacity whose overflow bound fits eps/2 (the bound falls with M, 0 at M = N).
    int64_t lo = k, hi = N;
    while (lo < hi) {
        int64_t mid = lo + (hi - lo) / 2;
        if (overflow_bound(N, S, t, mid) <= eps_half) hi = mid; else lo = mid + 1;
    }
    const int64_t m_exact = lo;

    // Eq. (M) / Algorithm 1 step 7.
    const double f = 1.0 - (double)S / (double)N;
    const int64_t m_paper = (int64_t)std::ceil((double)k + z * std::sqrt((double)k * (double)(N - k) / (double)S * f));

    int64_t capacity = m_exact > m_paper ? m_exact : m_paper;
    if (capacity > N) capacity = N;

    out->m = S;
    out->r = t;
    out->capacity = capacity;
    out->k_accept = k_acc;
    out->mode = (2 * capacity >= N || N <= 2 * S) ? 1 : 0;
    out->tie_rule = PROFK_TIES_BY_INDEX;
    out->z = z;
    out->alpha = alpha;
    out->p_recall_fail = recall_fail_bound(N, S, t, k_acc);
    out->p_overflow = overflow_bound(N, S, t, capacity);
    // Second-chance ranks (see profk_plan_t): the sample ranks whose expected survivor count lies midway between k and
    // the capacity, seen from a threshold that kept just too many (tight) or just too few (loose).
    const int64_t tight = (int64_t)(((__int128)t * (__int128)(k + capacity)) / ((__int128)2 * capacity));
    out->r_tight = (tight >= 1 && tight < t) ? tight : 0;
    const int64_t loose = t + (int64_t)((((__int128)(capacity - k) * (__int128)S) + (__int128)2 * N - 1) / ((__int128)2 * N));
    out->r_loose = (loose > t && loose <= S) ? loose : 0;
    return PROFK_OK;
}

// The library's own choice of the tuning inputs.  Section 4's floor S_min = 32768 is kept for long rows.
// For a short row it is lowered to N / 512 (not below 1024): on this GPU DRAM delivers 128 bytes per sampled
// element, so 32768 samples of a 2^20-element row read the whole row once before the filtering scan reads
// it again, and 2^16-element rows would not be filtered at all (N <= 2 S).  The guarded rank and capacity
// keep the failure budget for any S.
//
// The cost ratio tau_B / tau_A of Eq. (cost_model) -- what a unit of buffer work costs against a sampled
// element -- is 1 in the paper and grows here with the row length, N / 2^22 clamped to [1, 16] for up to
// PROFK_ALL_SM_GATHER_ROWS rows and to [1, 4] for larger batches: the sample of a long row is gathered by a
// kernel over all SMs in a few microseconds whatever its size, while every survivor costs a trip through the
// filter's slow path and a record in the refine step.  Measured on B200: 2^26, k = 256, eps = 1e-4: 51.3 -> 49.0 us;
// k = 4096: 63.6 -> 60.0; 2^30 Cauchy, k = 64: 631 -> 610; four rows of 2^26, k = 256: 187 -> 167; rows of 2^22 and
// shorter are planned as before.  S_max stays Section 4's 131072: with 262144 the selection of a deep rank among
// so many keys cost the flattened BatchTopK shape (2^29, K = 131072) 16 us and gained the others 1-2.
extern "C" int profk_default_tuning_batch(int64_t rows, int64_t N, profk_tuning_t* tuning) {
    if (!tuning || N < 1 || rows < 1) return PROFK_EINVAL;
    int64_t s_min = N / 512;
    if (s_min < 1024) s_min = 1024;
    if (s_min > 32768) s_min = 32768;
    const bool all_sm_gather = rows <= PROFK_ALL_SM_GATHER_ROWS;
    double ratio = (double)N / 4194304.0;
    const double ratio_max = all_sm_gather ? 16.0 : 4.0;
    if (ratio < 1.0) ratio = 1.0;
    if (ratio > ratio_max) ratio = ratio_max;
    tuning->s_min = s_min;
    tuning->s_max = 131072;
    tuning->cost_ratio = ratio;
    return PROFK_OK;
}

extern "C" int profk_default_tuning(int64_t N, profk_tuning_t* tuning) { return profk_default_tuning_batch(1, N, tuning); }

extern "C" int profk_plan_batch(int64_t rows, int64_t N, int64_t k, double eps, double recall, profk_plan_t* out) {
    profk_tuning_t tuning;
    if (profk_default_tuning_batch(rows, N, &tuning) != PROFK_OK) return PROFK_EINVAL;
    return profk_plan_ex(N, k, eps, recall, &tuning, out);
}

extern "C" int profk_plan(int64_t N, int64_t k, double eps, double recall, profk_plan_t* out) {
    return profk_plan_batch(1, N, k, eps, recall, out);
}
