// Shared device helpers: order-preserving keys, candidate records, Philox4x32-10,
// element-type traits and small warp / block utilities.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace profk {

constexpr unsigned FULL_MASK = 0xFFFFFFFFu;

// Partitioned append of the filter (large selections): parts of a row's buffer, each with a counter of its own.
#ifndef PROFK_FILTER_PARTS
#define PROFK_FILTER_PARTS 8
#endif
constexpr uint32_t FILTER_PARTS = PROFK_FILTER_PARTS;
constexpr uint32_t FILTER_PART_STRIDE = 64;     // words between two counters: 256 bytes

// ---------------------------------------------------------------------------------------
// Order keys.  key(x) is an unsigned integer whose order is the total order
// -NaN < -inf < ... < -0 < +0 < ... < +inf < +NaN of the bit patterns.  Keys travel in 32-bit
// words; a bf16 key is the 16-bit key of its pattern in the lower half (KEY_BITS = 16), so that
// in a candidate record it sits directly above the index.
__device__ __forceinline__ uint32_t key_from_bits32(uint32_t b) {
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ uint32_t bits32_from_key(uint32_t k) {
    return (k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k;
}

// Bit pattern of a float through an opaque move: the compiler must not rewrite the integer
// key arithmetic below as floating-point sign / abs operations, which would replace a NaN's
// payload by the canonical NaN and so change its key.
__device__ __forceinline__ uint32_t float_bits_exact(float v) {
    uint32_t b;
    asm("mov.b32 %0, %1;" : "=r"(b) : "f"(v));
    return b;
}

template <typename T> struct Elem;

template <> struct Elem<float> {
    using vec_t = float4;                       // 128-bit vector
    static constexpr int VEC = 4;               // elements per vector
    static constexpr int KEY_BITS = 32;
    static constexpr uint32_t NEG_INF_BITS = 0xFF800000u;
    static __device__ __forceinline__ uint32_t bits(float v) { return float_bits_exact(v); }
    static __device__ __forceinline__ uint32_t key(float v) { return key_from_bits32(float_bits_exact(v)); }
    static __device__ __forceinline__ float from_key(uint32_t k) { return __uint_as_float(bits32_from_key(k)); }
    static __device__ __forceinline__ float from_bits(uint32_t b) { return __uint_as_float(b); }
    static __device__ __forceinline__ float as_float(float v) { return v; }
};

template <> struct Elem<__nv_bfloat16> {
    using vec_t = uint4;                        // 8 bf16 in 128 bits
    static constexpr int VEC = 8;
    static constexpr int KEY_BITS = 16;
    static constexpr uint32_t NEG_INF_BITS = 0xFF80u;
    static __device__ __forceinline__ uint32_t bits(__nv_bfloat16 v) { return (uint32_t)__bfloat16_as_ushort(v); }
    static __device__ __forceinline__ uint32_t key(__nv_bfloat16 v) {
        return key_from_bits32((uint32_t)__bfloat16_as_ushort(v) << 16) >> 16;
    }
    static __device__ __forceinline__ __nv_bfloat16 from_key(uint32_t k) {
        const uint32_t k16 = k & 0xFFFFu;
        const uint32_t b = (k16 & 0x8000u) ? (k16 & 0x7FFFu) : (~k16 & 0xFFFFu);
        return __ushort_as_bfloat16((unsigned short)b);
    }
    static __device__ __forceinline__ __nv_bfloat16 from_bits(uint32_t b) { return __ushort_as_bfloat16((unsigned short)b); }
    static __device__ __forceinline__ float as_float(__nv_bfloat16 v) {
        return __uint_as_float((uint32_t)__bfloat16_as_ushort(v) << 16);
    }
};

// Candidate record: ascending record order == (value descending, index ascending).
__device__ __forceinline__ uint64_t make_record(uint32_t key, uint32_t idx) {
    return ((uint64_t)(~key) << 32) | (uint64_t)idx;
}
__device__ __forceinline__ uint32_t record_key(uint64_t rec) { return ~(uint32_t)(rec >> 32); }
__device__ __forceinline__ uint32_t record_idx(uint64_t rec) { return (uint32_t)rec; }

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds, key bumped by the Weyl constants between rounds.
struct Philox4 { uint32_t x, y, z, w; };

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t k0, uint32_t k1) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k0 += W0; k1 += W1; }
        const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    }
    return Philox4{c0, c1, c2, c3};
}

// ---------------------------------------------------------------------------------------
// Streaming loads: the input is read exactly once, so keep it out of L1.

__device__ __forceinline__ float4 ld_stream(const float4* p) {
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ unsigned lane_id() { return threadIdx.x & 31u; }

// Programmatic dependent launch: wait for the preceding kernel's memory to be visible /
// allow the following kernel to start its prologue.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace profk
