// Tiled, vectorised, alignment-safe traversal of the rows x N input.
//
// A row r starts at element address in + r*N, which need not be 16-byte aligned (N odd,
// or a caller-offset base pointer).  Each row is therefore addressed in "virtual"
// coordinates v = i + mis_r, where mis_r is the number of elements between the previous
// 16-byte boundary and the row start: vector q of the row covers v in [q*VEC, (q+1)*VEC)
// and is always a naturally aligned 128-bit load.  Vectors that straddle the row's ends
// are read element by element, so nothing outside [row start, row end) is ever touched.
//
// A tile is THREADS * UNROLL consecutive vectors of one row; thread t of the CTA owns
// vectors t, t + THREADS, ... of the tile, so every load instruction of a warp is one
// contiguous 512-byte run.
#pragma once

#include "common.cuh"

namespace profk {

template <typename T> struct RowView {
    const T* aligned_base;  // row start rounded down to 16 bytes
    uint32_t mis;           // elements between aligned_base and the row start
};

template <typename T>
__device__ __forceinline__ RowView<T> row_view(const T* in, uint64_t N, uint64_t row) {
    const T* start = in + row * N;
    const uint32_t mis = (uint32_t)(((uintptr_t)start & 15u) / sizeof(T));
    return RowView<T>{start - mis, mis};
}

// Number of tiles that cover any row of length N (uniform over rows: mis < VEC).
template <typename T>
__host__ __device__ inline uint64_t tiles_per_row(uint64_t N, uint32_t tile_vectors) {
    const uint64_t vec = Elem<T>::VEC;
    const uint64_t vectors = (N + vec - 1 + vec - 1) / vec;   // ceil((N + VEC-1) / VEC)
    return (vectors + tile_vectors - 1) / tile_vectors;
}

// Loads vector q of the row.  Lanes outside the row get the bit pattern of -inf.
// *inside_any says whether at least one lane lies inside the row.
template <typename T>
__device__ __forceinline__ typename Elem<T>::vec_t load_row_vector(const RowView<T>& rv, uint64_t N, uint64_t q,
                                                                    bool* inside_any) {
    using V = typename Elem<T>::vec_t;
    constexpr int VEC = Elem<T>::VEC;
    const int64_t i0 = (int64_t)(q * VEC) - (int64_t)rv.mis;   // row index of lane 0
    const T* p = rv.aligned_base + q * VEC;
    if (i0 >= 0 && (uint64_t)i0 + VEC <= N) {
        *inside_any = true;
        return ld_stream(reinterpret_cast<const V*>(p));
    }
    union { V v; T e[VEC]; } u;
#pragma unroll
    for (int l = 0; l < VEC; ++l) u.e[l] = Elem<T>::from_bits(Elem<T>::NEG_INF_BITS);
    bool any = false;
    if (i0 + VEC > 0 && i0 < (int64_t)N) {
#pragma unroll
        for (int l = 0; l < VEC; ++l) {
            const int64_t i = i0 + l;
            if (i >= 0 && i < (int64_t)N) { u.e[l] = p[l]; any = true; }
        }
    }
    *inside_any = any;
    return u.v;
}

// Element l of a vector.
__device__ __forceinline__ float vec_elem(const float4& v, int l) {
    return l == 0 ? v.x : l == 1 ? v.y : l == 2 ? v.z : v.w;
}
__device__ __forceinline__ __nv_bfloat16 vec_elem(const uint4& v, int l) {
    const uint32_t w = (l >> 1) == 0 ? v.x : (l >> 1) == 1 ? v.y : (l >> 1) == 2 ? v.z : v.w;
    return __ushort_as_bfloat16((unsigned short)((l & 1) ? (w >> 16) : (w & 0xFFFFu)));
}

}  // namespace profk
