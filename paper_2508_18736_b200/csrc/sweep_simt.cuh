// CUDA-core similarity sweep: one 128x128 tile of S = A * B^T (rows of A against rows of B,
// both row-major [rows, D]) accumulated in fp32 with FFMA.  Products of bf16 inputs are exact
// in fp32; fp32 inputs are multiplied in full precision (tensor-core TF32 would not meet the
// 1e-5 tolerance of the fp32 configurations).  The tile is left in shared memory for the
// caller's epilogue: S is never written to global memory.
#pragma once

#include "common.cuh"

namespace siso {
namespace sweep {

constexpr int BM = 128, BN = 128, BK = 16;
constexpr int THREADS = 256;
constexpr int S_STRIDE = 130;                                  // floats per row of the result tile in smem
constexpr int OPER_FLOATS = 2 * BK * BM;                       // one operand, double-buffered
constexpr int SMEM_FLOATS_MAINLOOP = 2 * OPER_FLOATS;          // A and B
constexpr int SMEM_FLOATS_RESULT = BM * S_STRIDE;
constexpr int SMEM_BYTES = (SMEM_FLOATS_RESULT > SMEM_FLOATS_MAINLOOP ? SMEM_FLOATS_RESULT : SMEM_FLOATS_MAINLOOP) * 4;

// Four consecutive K elements of one row as fp32 (zero beyond the row count or beyond D).
template <typename T> struct Frag;
template <> struct Frag<float> {
    static __device__ __forceinline__ float4 load(const float *base, int64_t row, int64_t rows, int k, int D) {
        if (row < rows && k < D) return __ldg(reinterpret_cast<const float4 *>(base + row * D + k));
        return make_float4(0.f, 0.f, 0.f, 0.f);
    }
};
template <> struct Frag<__nv_bfloat16> {
    static __device__ __forceinline__ float4 load(const __nv_bfloat16 *base, int64_t row, int64_t rows, int k, int D) {
        if (row < rows && k < D) {
            uint2 u = __ldg(reinterpret_cast<const uint2 *>(base + row * D + k));
            return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u),
                               __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xFFFF0000u));
        }
        return make_float4(0.f, 0.f, 0.f, 0.f);
    }
};

// Computes the tile (rows a0..a0+127 of A) x (rows b0..b0+127 of B) and leaves it in smem as
// S[r * S_STRIDE + c].  All 256 threads must call it; it ends with __syncthreads().
template <typename T>
__device__ __forceinline__ void tile_to_smem(const T *__restrict__ A, int64_t a_rows, int64_t a0,
                                             const T *__restrict__ Bm, int64_t b_rows, int64_t b0, int D,
                                             float *smem) {
    float *As = smem;                 // [2][BK][BM]
    float *Bs = smem + OPER_FLOATS;   // [2][BK][BN]
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    // loader mapping: element idx = tid + 256*j covers (row = idx % 128, kq = idx / 128), kq in 0..3
    const int lrow = tid & 127, lkq = tid >> 7;

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    float4 ra[2], rb[2];
    const int ktiles = (D + BK - 1) / BK;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        ra[j] = Frag<T>::load(A, a0 + lrow, a_rows, (lkq + 2 * j) * 4, D);
        rb[j] = Frag<T>::load(Bm, b0 + lrow, b_rows, (lkq + 2 * j) * 4, D);
    }
    __syncthreads();   // previous users of smem (the caller's epilogue) are done
    for (int kt = 0; kt < ktiles; ++kt) {
        const int buf = kt & 1;
        float *as = As + buf * BK * BM, *bs = Bs + buf * BK * BN;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int kk = (lkq + 2 * j) * 4;
            as[(kk + 0) * BM + lrow] = ra[j].x; as[(kk + 1) * BM + lrow] = ra[j].y;
            as[(kk + 2) * BM + lrow] = ra[j].z; as[(kk + 3) * BM + lrow] = ra[j].w;
            bs[(kk + 0) * BN + lrow] = rb[j].x; bs[(kk + 1) * BN + lrow] = rb[j].y;
            bs[(kk + 2) * BN + lrow] = rb[j].z; bs[(kk + 3) * BN + lrow] = rb[j].w;
        }
        __syncthreads();
        if (kt + 1 < ktiles) {
            const int kbase = (kt + 1) * BK;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                ra[j] = Frag<T>::load(A, a0 + lrow, a_rows, kbase + (lkq + 2 * j) * 4, D);
                rb[j] = Frag<T>::load(Bm, b0 + lrow, b_rows, kbase + (lkq + 2 * j) * 4, D);
            }
        }
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a0v = *reinterpret_cast<const float4 *>(as + k * BM + ty * 4);
            const float4 a1v = *reinterpret_cast<const float4 *>(as + k * BM + 64 + ty * 4);
            const float4 b0v = *reinterpret_cast<const float4 *>(bs + k * BN + tx * 4);
            const float4 b1v = *reinterpret_cast<const float4 *>(bs + k * BN + 64 + tx * 4);
            const float a[8] = {a0v.x, a0v.y, a0v.z, a0v.w, a1v.x, a1v.y, a1v.z, a1v.w};
            const float b[8] = {b0v.x, b0v.y, b0v.z, b0v.w, b1v.x, b1v.y, b1v.z, b1v.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        // the other buffer is written next iteration; it was last read one iteration ago, and every
        // thread has passed this iteration's barrier since, so no second barrier is needed
    }
    __syncthreads();   // all reads of As/Bs done before the result tile overwrites them
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = (i < 4) ? ty * 4 + i : 64 + ty * 4 + (i - 4);
        float *row = smem + r * S_STRIDE;
        *reinterpret_cast<float2 *>(row + tx * 4) = make_float2(acc[i][0], acc[i][1]);
        *reinterpret_cast<float2 *>(row + tx * 4 + 2) = make_float2(acc[i][2], acc[i][3]);
        *reinterpret_cast<float2 *>(row + 64 + tx * 4) = make_float2(acc[i][4], acc[i][5]);
        *reinterpret_cast<float2 *>(row + 64 + tx * 4 + 2) = make_float2(acc[i][6], acc[i][7]);
    }
    __syncthreads();
}

}  // namespace sweep
}  // namespace siso
