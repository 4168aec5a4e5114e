// Lane-group primitives shared by the decode kernels: a group of LPH lanes of a warp owns one (batch, head).
#pragma once

#include "internal.cuh"

namespace sketchssm {

__device__ __forceinline__ void ld4(const float* p, float* d) {
    const float4 t = *reinterpret_cast<const float4*>(p);
    d[0] = t.x; d[1] = t.y; d[2] = t.z; d[3] = t.w;
}
__device__ __forceinline__ void ld4(const __nv_bfloat16* p, float* d) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    d[0] = __uint_as_float(t.x << 16); d[1] = __uint_as_float(t.x & 0xffff0000u);
    d[2] = __uint_as_float(t.y << 16); d[3] = __uint_as_float(t.y & 0xffff0000u);
}
__device__ __forceinline__ void st4(float* p, const float* s) {
    *reinterpret_cast<float4*>(p) = make_float4(s[0], s[1], s[2], s[3]);
}
__device__ __forceinline__ void st4(__nv_bfloat16* p, const float* s) {
    __nv_bfloat162 a = __floats2bfloat162_rn(s[0], s[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(s[2], s[3]);
    uint2 t;
    t.x = *reinterpret_cast<uint32_t*>(&a);
    t.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = t;
}

// A lane j of a group owns the element chunks {4 (j + LPH m) .. +3 : m = 0 .. E/4-1} of a row.
template <int E, int LPH, typename T>
__device__ __forceinline__ void load_row(const T* row, int j, float (&d)[E]) {
#pragma unroll
    for (int m = 0; m < E / 4; ++m) ld4(row + 4 * (j + LPH * m), &d[4 * m]);
}
template <int E, int LPH, typename T>
__device__ __forceinline__ void store_row(T* row, int j, const float (&s)[E]) {
#pragma unroll
    for (int m = 0; m < E / 4; ++m) st4(row + 4 * (j + LPH * m), &s[4 * m]);
}

// Ask L2 to fetch a byte range (16-byte aligned, size a multiple of 16) without occupying shared memory.
__device__ __forceinline__ void prefetch_l2(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

template <int LPH>
__device__ __forceinline__ float group_sum(float x) {
#pragma unroll
    for (int o = LPH / 2; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Transposing butterfly over the LPH lanes of a group: on entry every lane holds M partial sums v[0..M);
// on exit lane j holds the complete sums of indices (M/LPH) j .. (M/LPH) j + M/LPH - 1 in v[0..M/LPH)
// (if M < LPH: v[0] holds the sum of index j / (LPH/M)).  Each value crosses lanes once per level.
template <int LPH, int M>
__device__ __forceinline__ void group_reduce_transpose(float (&v)[M], int j) {
    int m = M;
#pragma unroll
    for (int o = LPH / 2; o > 0; o >>= 1) {
        if (m > 1) {
            const int half = m / 2;
            const bool upper = (j & o) != 0;
#pragma unroll
            for (int i = 0; i < M / 2; ++i) {
                if (i < half) {
                    const float send = upper ? v[i] : v[i + half];
                    const float keep = upper ? v[i + half] : v[i];
                    v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                }
            }
            m = half;
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
        }
    }
}


}  // namespace sketchssm
