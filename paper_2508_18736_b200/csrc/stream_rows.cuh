// Pieces shared by the kernels that stream centroid rows through registers (lookup_stream.cu, lookup_noalloc.cu):
// 128-bit row loads that bypass L1, and the transposing warp reduction of many partial dot products at once.
#pragma once

#include "common.cuh"

namespace siso {

// 8 consecutive elements of a row as fp32
template <typename T> struct Chunk8;
template <> struct Chunk8<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&f)[8]) {
        uint4 u;
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w) : "l"(p));
        f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xFFFF0000u);
        f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xFFFF0000u);
        f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xFFFF0000u);
        f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xFFFF0000u);
    }
    static __device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
};
template <> struct Chunk8<float> {
    static __device__ __forceinline__ void load(const float *p, float (&f)[8]) {
        uint4 u, w;
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w) : "l"(p));
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "l"(p + 4));
        f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
        f[4] = __uint_as_float(w.x); f[5] = __uint_as_float(w.y); f[6] = __uint_as_float(w.z); f[7] = __uint_as_float(w.w);
    }
    static __device__ __forceinline__ float to_f32(float v) { return v; }
};

// Sum V per-lane values across the 32 lanes.  Afterwards v[0] of lane L holds the complete sum
// of value number L >> (5 - log2 V); lanes that share that number hold the same sum.
template <int N, int STRIDE, int V> __device__ __forceinline__ void transpose_reduce_step(float (&v)[V], int lane) {
    if constexpr (STRIDE >= 1) {
        if constexpr (N > 1) {
            constexpr int HALF = N / 2;
            const bool upper = (lane & STRIDE) != 0;
#pragma unroll
            for (int i = 0; i < HALF; ++i) {
                const float send = upper ? v[i] : v[i + HALF];
                const float keep = upper ? v[i + HALF] : v[i];
                v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, STRIDE);
            }
            transpose_reduce_step<HALF, STRIDE / 2, V>(v, lane);
        } else {
            v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], STRIDE);
            transpose_reduce_step<1, STRIDE / 2, V>(v, lane);
        }
    }
}
template <int V> __device__ __forceinline__ void warp_transpose_reduce(float (&v)[V], int lane) {
    transpose_reduce_step<V, 16, V>(v, lane);
}

}  // namespace siso
