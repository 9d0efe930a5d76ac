// The bins of the large selections (k beyond what one CTA orders; the flattened BatchTopK case of Section 5,
// "Application"): the kernels that order or select among some 10^5 candidate records of a row first count them in
// 2^18 bins by how far they lie from the threshold record, and the filtering scan can do that counting itself while it
// appends the records (stage 3 of Section 3 then hands stage 4 a histogram along with the buffer).
//
// A record r (value key above a 32-bit index, smaller = better) is measured from `top`, the largest record the filter
// can have kept: tau's key with the last index.  D = top - r with the index word's unused bits squeezed out (a row of N
// elements uses ceil(log2 N) of the 32), so that the bits right below the key difference are real index bits and
// thousands of copies of one bf16 value spread over many bins instead of crowding one.  D >= 0 for every kept record,
// larger D = better record.  D is binned on a logarithmic scale -- 6 bits of exponent, 12 of mantissa: fine where the
// records are dense, right above the threshold, and never stretched by an outlier -- and the bins are numbered from
// the best record's end, so that a prefix sum over the bins walks the records from the best down.
#pragma once

#include "common.cuh"

namespace profk {

constexpr int BIN_BITS = 18;
constexpr uint32_t BIN_COUNT = 1u << BIN_BITS;
constexpr uint32_t BIN_FLAGS = 8;                 // words after the bins, for the kernel that uses them
constexpr uint32_t BIN_FLAG_UNCOUNTED = 7;        // flag word set by a filter kernel that appended records without counting them
constexpr uint32_t BIN_COARSE = 512;              // coarse bins after the flags, each the sum of BIN_PER_COARSE fine ones
constexpr uint32_t BIN_PER_COARSE = BIN_COUNT / BIN_COARSE;
constexpr uint32_t BIN_ROW_WORDS = BIN_COUNT + BIN_FLAGS + BIN_COARSE;     // words of one row's bins in the workspace

// Bits an index of a row of N elements occupies (1 .. 32).
__host__ __device__ __forceinline__ int index_bits(uint64_t N) {
    int b = 1;
    while (b < 32 && (1ull << b) < N) ++b;
    return b;
}

// D of a record below the record (top_hi, last index); top_hi = the high word (inverted key) of the largest record kept.
__device__ __forceinline__ uint64_t record_dist(uint64_t rec, uint32_t top_hi, int idx_bits) {
    const uint64_t idx_top = (1ull << idx_bits) - 1ull;
    return ((uint64_t)(top_hi - (uint32_t)(rec >> 32)) << idx_bits) | (idx_top - (rec & 0xFFFFFFFFull));
}

// Bin of the logarithmic scale: exponent e = floor(log2 D) in the top 6 bits, the 12 bits after the leading one below.
// Monotone in D.  D = 0 shares bin 0 with D = 1.
__device__ __forceinline__ uint32_t log_bin(uint64_t D) {
    if (D < 2) return 0;
    const int e = 63 - __clzll((long long)D);
    const uint64_t frac = D ^ (1ull << e);
    const uint32_t m = e >= 12 ? (uint32_t)(frac >> (e - 12)) : (uint32_t)(frac << (12 - e));
    return ((uint32_t)e << 12) | m;
}
// The D range of a bin of the logarithmic scale: [lo, lo + 2^w).
__device__ __forceinline__ void log_bin_range(uint32_t bin, uint64_t* lo, int* w) {
    if (bin == 0) { *lo = 0; *w = 1; return; }
    const int e = (int)(bin >> 12);
    const uint64_t m = bin & 4095u;
    if (e >= 12) { *lo = (1ull << e) | (m << (e - 12)); *w = e - 12; }
    else { *lo = (1ull << e) + (m >> (12 - e)); *w = 0; }
}

// Number of the bin that counts `rec`, best records first.
__device__ __forceinline__ uint32_t record_bin(uint64_t rec, uint32_t top_hi, int idx_bits) {
    return BIN_COUNT - 1 - log_bin(record_dist(rec, top_hi, idx_bits));
}

}  // namespace profk
