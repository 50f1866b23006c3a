// Lookup on CUDA cores: tiled similarity sweep with a fused per-query top-k epilogue, and the
// small kernel that merges per-split partial results and applies the hit threshold.
// FindClosestCentroid / CosineSimilarity of Algorithm 1 evaluated exactly for a batch.
#include "sweep_simt.cuh"

namespace siso {

using namespace sweep;

// grid = (splits, m_tiles).  Each CTA owns 128 queries and a contiguous range of centroid tiles;
// thread t scans row t/2 of every result tile, columns of parity t%2, in ascending slot order.
template <typename T, int KMAX>
__global__ void __launch_bounds__(THREADS, 2)
lookup_simt_kernel(const T *__restrict__ Q, int64_t B, const T *__restrict__ C, const uint8_t *__restrict__ valid,
                   int64_t N, int D, int tiles_per_split, int n_tiles, unsigned long long *__restrict__ partial,
                   int splits) {
    extern __shared__ __align__(16) float smem[];
    __shared__ uint8_t valid_s[BN];
    const int split = blockIdx.x;
    const int64_t q0 = static_cast<int64_t>(blockIdx.y) * BM;
    const int tid = threadIdx.x;
    const int row = tid >> 1, par = tid & 1;

    TopK<KMAX> top;
    top.clear();
    const int t_begin = split * tiles_per_split;
    const int t_end = min(n_tiles, t_begin + tiles_per_split);
    for (int t = t_begin; t < t_end; ++t) {
        const int64_t n0 = static_cast<int64_t>(t) * BN;
        tile_to_smem<T>(Q, B, q0, C, N, n0, D, smem);
        if (tid < BN) valid_s[tid] = (n0 + tid < N) ? valid[n0 + tid] : 0;
        __syncthreads();
        const float *srow = smem + row * S_STRIDE;
#pragma unroll 8
        for (int i = 0; i < BN / 2; ++i) {
            const int cidx = par + 2 * i;
            const float v = srow[cidx];
            if (valid_s[cidx]) top.push(v, static_cast<int32_t>(n0 + cidx));
        }
        // the next tile_to_smem starts with a barrier before it touches smem
    }
    __syncthreads();
    // merge the two parity lists of each row through shared memory (packed keys: exact order)
    unsigned long long *lists = reinterpret_cast<unsigned long long *>(smem);   // [256][KMAX]
#pragma unroll
    for (int j = 0; j < KMAX; ++j) lists[tid * KMAX + j] = top.key(j);
    __syncthreads();
    if (par == 0 && q0 + row < B) {
        KeyList<KMAX> out;
        out.clear();
#pragma unroll
        for (int j = 0; j < KMAX; ++j) {
            out.insert(lists[tid * KMAX + j]);
            out.insert(lists[(tid + 1) * KMAX + j]);
        }
        unsigned long long *dst = partial + ((q0 + row) * splits + split) * KMAX;
#pragma unroll
        for (int j = 0; j < KMAX; ++j) dst[j] = out.k[j];
    }
}

// One warp per query: the lanes split the splits*kmax packed keys, merge their lists with shuffles, and lane 0
// writes the k best and applies the strict threshold test.
template <int KMAX>
__global__ void __launch_bounds__(1024)
topk_finalize_kernel(const unsigned long long *__restrict__ partial, int64_t B, int splits, int k,
                     const float *__restrict__ theta, float theta_s, int32_t *__restrict__ idx,
                     float *__restrict__ sim, uint8_t *__restrict__ hit, long long *counters) {
    __shared__ int hits_s;
    if (threadIdx.x == 0) hits_s = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t b = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (b < B) {
        KeyList<KMAX> out;
        out.clear();
        const unsigned long long *src = partial + b * splits * KMAX;
        for (int s = lane; s < splits * KMAX; s += 32) out.insert(src[s]);
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            unsigned long long other[KMAX];
#pragma unroll
            for (int j = 0; j < KMAX; ++j) other[j] = __shfl_xor_sync(0xFFFFFFFFu, out.k[j], o);
#pragma unroll
            for (int j = 0; j < KMAX; ++j) out.insert(other[j]);
        }
        if (lane == 0) {
#pragma unroll
            for (int j = 0; j < KMAX; ++j) {
                if (j < k) {
                    const unsigned long long key = out.k[j];
                    idx[b * k + j] = key ? key_slot(key) : -1;
                    sim[b * k + j] = key ? key_sim(key) : -INFINITY;
                }
            }
            const float th = theta ? theta[b] : theta_s;
            const int is_hit = (out.k[0] != 0ull && key_sim(out.k[0]) > th) ? 1 : 0;
            hit[b] = static_cast<uint8_t>(is_hit);
            if (is_hit) atomicAdd(&hits_s, 1);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (hits_s) atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_HITS), static_cast<unsigned long long>(hits_s));
        if (blockIdx.x == 0) atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_LOOKUPS), static_cast<unsigned long long>(B));
    }
}

siso_status_t launch_topk_finalize(Cache *c, const unsigned long long *partial, int64_t B, int splits, int kmax, int k,
                                   const float *theta, float theta_s, int32_t *idx, float *sim, uint8_t *hit,
                                   cudaStream_t s) {
    const int threads = B >= 4096 ? 1024 : 256;              // one warp per query
    const int per_block = threads / 32;
    const unsigned blocks = static_cast<unsigned>((B + per_block - 1) / per_block);
    if (kmax == 1) topk_finalize_kernel<1><<<blocks, threads, 0, s>>>(partial, B, splits, k, theta, theta_s, idx, sim, hit, c->counters);
    else if (kmax == 4) topk_finalize_kernel<4><<<blocks, threads, 0, s>>>(partial, B, splits, k, theta, theta_s, idx, sim, hit, c->counters);
    else topk_finalize_kernel<8><<<blocks, threads, 0, s>>>(partial, B, splits, k, theta, theta_s, idx, sim, hit, c->counters);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

template <typename T, int KMAX>
static siso_status_t run_simt(Cache *c, const void *q, int64_t B, int tiles_per_split, int n_tiles, int splits,
                              int m_tiles, unsigned long long *partial, cudaStream_t s) {
    auto kern = lookup_simt_kernel<T, KMAX>;
    bool &attr_set = c->simt_attr_set[sizeof(T) == 2 ? 1 : 0][KMAX == 1 ? 0 : (KMAX == 4 ? 1 : 2)];
    if (!attr_set) {
        SISO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        attr_set = true;
    }
    dim3 grid(splits, m_tiles);
    kern<<<grid, THREADS, SMEM_BYTES, s>>>(static_cast<const T *>(q), B, static_cast<const T *>(c->vecs), c->valid,
                                           c->capacity, c->dim, tiles_per_split, n_tiles, partial, splits);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

siso_status_t launch_lookup_simt(Cache *c, const void *q, int64_t B, const float *theta, float theta_s, int k,
                                 int32_t *idx, float *sim, uint8_t *hit, cudaStream_t s) {
    const int kmax = k == 1 ? 1 : (k <= 4 ? 4 : 8);
    const int n_tiles = static_cast<int>((c->capacity + BN - 1) / BN);
    const int64_t m_tiles64 = (B + BM - 1) / BM;
    if (m_tiles64 > 65535) return SISO_ERR_UNSUPPORTED;
    const int m_tiles = static_cast<int>(m_tiles64);
    // enough CTAs for about four waves of two CTAs per SM, but never fewer than one tile per split
    int want = (8 * c->sm_count + m_tiles - 1) / m_tiles;
    int splits = max(1, min(n_tiles, want));
    const int tiles_per_split = (n_tiles + splits - 1) / splits;
    splits = (n_tiles + tiles_per_split - 1) / tiles_per_split;
    Scratch scr;
    SISO_TRY(scratch_reserve(c, pad256(sizeof(unsigned long long) * B * splits * kmax), s, &scr));
    unsigned long long *partial = scr.take<unsigned long long>(static_cast<size_t>(B) * splits * kmax);
    siso_status_t st;
    if (c->dtype == SISO_F32) {
        st = kmax == 1 ? run_simt<float, 1>(c, q, B, tiles_per_split, n_tiles, splits, m_tiles, partial, s)
           : kmax == 4 ? run_simt<float, 4>(c, q, B, tiles_per_split, n_tiles, splits, m_tiles, partial, s)
                       : run_simt<float, 8>(c, q, B, tiles_per_split, n_tiles, splits, m_tiles, partial, s);
    } else {
        st = kmax == 1 ? run_simt<__nv_bfloat16, 1>(c, q, B, tiles_per_split, n_tiles, splits, m_tiles, partial, s)
           : kmax == 4 ? run_simt<__nv_bfloat16, 4>(c, q, B, tiles_per_split, n_tiles, splits, m_tiles, partial, s)
                       : run_simt<__nv_bfloat16, 8>(c, q, B, tiles_per_split, n_tiles, splits, m_tiles, partial, s);
    }
    SISO_TRY(st);
    return launch_topk_finalize(c, partial, B, splits, kmax, k, theta, theta_s, idx, sim, hit, s);
}

}  // namespace siso
