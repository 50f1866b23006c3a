// Small-batch lookup: one pass over the centroid matrix at HBM speed.  Queries (at most BQ = 8
// per pass) sit in shared memory as fp32; each warp streams centroid rows with 128-bit
// loads, four rows in flight, multiplies them against every query with FFMA, reduces the
// partial dot products across the warp with shuffles (a transposing reduction: 31 shuffles
// for 32 values) and keeps a running top-k per query in registers.  Exact: bf16 products
// are exact in fp32 and the sum is fp32.
#include "common.cuh"
#include "stream_rows.cuh"

namespace siso {

constexpr int ST_THREADS = 256;
constexpr int ST_WARPS = ST_THREADS / 32;
constexpr int ST_ROWS = 4;            // centroid rows in flight per warp

// grid.x CTAs split the rows [0, rows_alloc) into contiguous chunks (multiples of ST_ROWS*ST_WARPS).
template <typename T, int BQ, int KMAX>
__global__ void __launch_bounds__(ST_THREADS)
lookup_stream_kernel(const T *__restrict__ Q, int nq, const T *__restrict__ C, const uint8_t *__restrict__ valid,
                     int64_t N, int D, int64_t rows_per_cta, unsigned long long *__restrict__ partial, int splits) {
    extern __shared__ __align__(16) float qs[];     // [BQ][D], zero rows beyond nq
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < BQ * D; i += ST_THREADS) {
        const int b = i / D;
        qs[i] = b < nq ? Chunk8<T>::to_f32(Q[static_cast<int64_t>(b) * D + (i - b * D)]) : 0.f;
    }
    __syncthreads();

    constexpr int V = ST_ROWS * BQ;                 // values reduced per step; value index = r * BQ + b
    constexpr int SHARE = 32 / V;                   // lanes that end up holding the same value
    const int my_val = lane / SHARE;
    const int my_r = my_val / BQ, my_b = my_val % BQ;
    TopK<KMAX> top;
    top.clear();

    const int64_t row_begin = static_cast<int64_t>(blockIdx.x) * rows_per_cta;
    const int64_t row_end = min(N, row_begin + rows_per_cta);
    const int chunks = D / 8;
    for (int64_t n0 = row_begin + warp * ST_ROWS; n0 < row_end; n0 += ST_WARPS * ST_ROWS) {
        // valid flags of the four rows (the arrays are padded to a multiple of 256 rows)
        const uint32_t vmask = *reinterpret_cast<const uint32_t *>(valid + n0);
        float acc[V];
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = 0.f;
        if (vmask != 0u) {
            for (int ch = lane; ch < chunks; ch += 32) {
                float cf[ST_ROWS][8];
#pragma unroll
                for (int r = 0; r < ST_ROWS; ++r) Chunk8<T>::load(C + (n0 + r) * D + ch * 8, cf[r]);
#pragma unroll
                for (int b = 0; b < BQ; ++b) {
                    const float4 q0 = *reinterpret_cast<const float4 *>(qs + b * D + ch * 8);
                    const float4 q1 = *reinterpret_cast<const float4 *>(qs + b * D + ch * 8 + 4);
#pragma unroll
                    for (int r = 0; r < ST_ROWS; ++r) {
                        float a = acc[r * BQ + b];
                        a = fmaf(cf[r][0], q0.x, a); a = fmaf(cf[r][1], q0.y, a);
                        a = fmaf(cf[r][2], q0.z, a); a = fmaf(cf[r][3], q0.w, a);
                        a = fmaf(cf[r][4], q1.x, a); a = fmaf(cf[r][5], q1.y, a);
                        a = fmaf(cf[r][6], q1.z, a); a = fmaf(cf[r][7], q1.w, a);
                        acc[r * BQ + b] = a;
                    }
                }
            }
            warp_transpose_reduce<V>(acc, lane);
            const int64_t n = n0 + my_r;
            if ((lane % SHARE) == 0 && ((vmask >> (8 * my_r)) & 0xFFu) && n < N) top.push(acc[0], static_cast<int32_t>(n));
        }
    }
    // combine: every owner lane publishes its list; one thread per query merges them
    __syncthreads();
    unsigned long long *lists = reinterpret_cast<unsigned long long *>(qs);     // [ST_THREADS][KMAX], reuses qs
#pragma unroll
    for (int j = 0; j < KMAX; ++j) lists[tid * KMAX + j] = ((lane % SHARE) == 0) ? top.key(j) : 0ull;
    __syncthreads();
    if (tid < nq) {
        KeyList<KMAX> out;
        out.clear();
        for (int t = 0; t < ST_THREADS; ++t) {
            const int l = t & 31;
            if ((l % SHARE) != 0 || ((l / SHARE) % BQ) != tid) continue;
#pragma unroll
            for (int j = 0; j < KMAX; ++j) out.insert(lists[t * KMAX + j]);
        }
        unsigned long long *dst = partial + (static_cast<int64_t>(tid) * splits + blockIdx.x) * KMAX;
#pragma unroll
        for (int j = 0; j < KMAX; ++j) dst[j] = out.k[j];
    }
}

template <typename T, int BQ, int KMAX>
static siso_status_t run_stream(Cache *c, const void *q, int nq, int64_t rows_per_cta, int splits,
                                unsigned long long *partial, cudaStream_t s) {
    auto kern = lookup_stream_kernel<T, BQ, KMAX>;
    const size_t smem = max(sizeof(float) * BQ * c->dim, sizeof(unsigned long long) * ST_THREADS * KMAX);
    if (smem > 48 * 1024) SISO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<splits, ST_THREADS, smem, s>>>(static_cast<const T *>(q), nq, static_cast<const T *>(c->vecs), c->valid,
                                          c->capacity, c->dim, rows_per_cta, partial, splits);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

template <typename T, int KMAX>
static siso_status_t run_stream_bq(Cache *c, const void *q, int nq, int64_t rows_per_cta, int splits,
                                   unsigned long long *partial, cudaStream_t s) {
    if (nq <= 1) return run_stream<T, 1, KMAX>(c, q, nq, rows_per_cta, splits, partial, s);
    if (nq <= 2) return run_stream<T, 2, KMAX>(c, q, nq, rows_per_cta, splits, partial, s);
    if (nq <= 4) return run_stream<T, 4, KMAX>(c, q, nq, rows_per_cta, splits, partial, s);
    return run_stream<T, 8, KMAX>(c, q, nq, rows_per_cta, splits, partial, s);
}

siso_status_t launch_lookup_stream(Cache *c, const void *q, int64_t B, const float *theta, float theta_s, int k,
                                   int32_t *idx, float *sim, uint8_t *hit, cudaStream_t s) {
    const int kmax = k == 1 ? 1 : (k <= 4 ? 4 : 8);
    // about 4 CTAs per SM, chunks in multiples of the rows one CTA sweeps per iteration
    const int64_t gran = ST_ROWS * ST_WARPS;
    int64_t rows_per_cta = (c->rows_alloc + 4 * c->sm_count - 1) / (4 * c->sm_count);
    rows_per_cta = ((rows_per_cta + gran - 1) / gran) * gran;
    const int splits = static_cast<int>((c->capacity + rows_per_cta - 1) / rows_per_cta);
    const int bq_max = (static_cast<size_t>(c->dim) * 8 * sizeof(float) <= 96 * 1024) ? 8 : 4;
    Scratch scr;
    SISO_TRY(scratch_reserve(c, pad256(sizeof(unsigned long long) * bq_max * splits * kmax), s, &scr));
    unsigned long long *partial = scr.take<unsigned long long>(static_cast<size_t>(bq_max) * splits * kmax);
    const size_t esz = c->dtype == SISO_F32 ? 4 : 2;
    for (int64_t b0 = 0; b0 < B; b0 += bq_max) {
        const int nq = static_cast<int>(std::min<int64_t>(bq_max, B - b0));
        const void *qp = static_cast<const char *>(q) + b0 * c->dim * esz;
        siso_status_t st;
        if (c->dtype == SISO_F32) {
            st = kmax == 1 ? run_stream_bq<float, 1>(c, qp, nq, rows_per_cta, splits, partial, s)
               : kmax == 4 ? run_stream_bq<float, 4>(c, qp, nq, rows_per_cta, splits, partial, s)
                           : run_stream_bq<float, 8>(c, qp, nq, rows_per_cta, splits, partial, s);
        } else {
            st = kmax == 1 ? run_stream_bq<__nv_bfloat16, 1>(c, qp, nq, rows_per_cta, splits, partial, s)
               : kmax == 4 ? run_stream_bq<__nv_bfloat16, 4>(c, qp, nq, rows_per_cta, splits, partial, s)
                           : run_stream_bq<__nv_bfloat16, 8>(c, qp, nq, rows_per_cta, splits, partial, s);
        }
        SISO_TRY(st);
        SISO_TRY(launch_topk_finalize(c, partial, nq, splits, kmax, k, theta ? theta + b0 : nullptr, theta_s,
                                      idx + b0 * k, sim + b0 * k, hit + b0, s));
    }
    return SISO_OK;
}

}  // namespace siso
