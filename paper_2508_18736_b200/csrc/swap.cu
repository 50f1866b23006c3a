// Algorithm 1 around MergeCentroids and FilteringCentroids: "C_new <- C_cur" (its first line) and the update step
// (Sec. 4.2): C_cur takes the contents of C_new a small group of slots at a time, so that the cache keeps serving
// lookups between the groups.  On the GPU every step is a kernel in stream order: a lookup issued between two groups
// sees each slot either wholly old or wholly new.
//   cache_copy        every slot of src into the same slot of dst (dst may be larger; its other slots become empty)
//   update plan       the live entries of C_new, in ascending slot order, numbered 0, 1, ...: one CTA-wide scan of the
//                     valid flags writes source_of[d] = slot of entry number d (made when the first group is copied)
//   update group      destination slots [first, first + n): slot d receives entry number d (vector, master, cluster_size,
//                     access_count, last_access) or becomes empty; one CTA per slot
#include "common.cuh"

namespace siso {

namespace {

__global__ void __launch_bounds__(1024)
swap_plan_kernel(const uint8_t *__restrict__ valid, int64_t n_src, int64_t dst_capacity, int32_t *__restrict__ source_of,
                 long long *n_live_out, int *status) {
    __shared__ int warp_sum[32];
    __shared__ long long run_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) run_s = 0;
    __syncthreads();
    for (int64_t base = 0; base < n_src; base += 1024) {
        const int64_t i = base + tid;
        const int live = (i < n_src && valid[i]) ? 1 : 0;
        int x = live;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) warp_sum[warp] = x;
        __syncthreads();
        int before = 0, all = 0;
        for (int w = 0; w < 32; ++w) { if (w < warp) before += warp_sum[w]; all += warp_sum[w]; }
        const long long pos = run_s + before + x - live;
        if (live && pos < dst_capacity) source_of[pos] = static_cast<int32_t>(i);
        __syncthreads();
        if (tid == 0) run_s += all;
        __syncthreads();
    }
    if (tid == 0) {
        *n_live_out = run_s;
        if (run_s > dst_capacity) set_status(status, SISO_ERR_CAPACITY);
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
swap_group_kernel(const int32_t *__restrict__ source_of, const long long *__restrict__ n_live_p, int64_t first, int64_t n,
                  int64_t dst_capacity, int D, const T *__restrict__ s_vecs, const float *__restrict__ s_master,
                  const double *__restrict__ s_size, const uint32_t *__restrict__ s_access,
                  const unsigned long long *__restrict__ s_last, T *__restrict__ d_vecs, float *__restrict__ d_master,
                  double *__restrict__ d_size, uint32_t *__restrict__ d_access, unsigned long long *__restrict__ d_last,
                  uint8_t *__restrict__ d_valid, long long *d_counters) {
    const long long n_live = *n_live_p;
    if (n_live > dst_capacity) return;                 // C_new does not fit: nothing is copied (status already set)
    const int64_t d = first + blockIdx.x;
    if (d >= first + n || d >= dst_capacity) return;
    const int was = d_valid[d] ? 1 : 0;
    int now = 0;
    if (d < n_live) {
        const int64_t src = source_of[d];
        const T *sv = s_vecs + src * D;
        T *dv = d_vecs + d * D;
        for (int k = threadIdx.x; k < D; k += 256) dv[k] = sv[k];
        if (sizeof(T) == 2) {                          // bf16 caches: the fp32 master too
            const float *sm = s_master + src * D;
            float *dm = d_master + d * D;
            for (int k = threadIdx.x; k < D; k += 256) dm[k] = sm[k];
        }
        if (threadIdx.x == 0) {
            d_size[d] = s_size[src];
            d_access[d] = s_access[src];
            d_last[d] = s_last[src];
            d_valid[d] = 1;
        }
        now = 1;
    } else if (threadIdx.x == 0) {
        d_valid[d] = 0;
    }
    if (threadIdx.x == 0 && now != was)
        atomicAdd(reinterpret_cast<unsigned long long *>(d_counters + CNT_OCCUPANCY),
                  static_cast<unsigned long long>(static_cast<long long>(now - was)));
}

__global__ void swap_clear_tail_kernel(uint8_t *valid, int64_t from, int64_t to) {
    const int64_t i = from + static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < to) valid[i] = 0;
}

__global__ void swap_copy_counters_kernel(const long long *__restrict__ src, long long *__restrict__ dst) {
    if (threadIdx.x < CNT_SPARE) dst[threadIdx.x] = src[threadIdx.x];
}

}  // namespace

siso_status_t launch_cache_copy(Cache *dst, const Cache *src, cudaStream_t s) {
    dst->vec_epoch += 1;          // the vectors may change: derived copies (the split-bf16 parts) are stale
    const size_t n = static_cast<size_t>(src->capacity), D = static_cast<size_t>(src->dim);
    const size_t esz = src->dtype == SISO_F32 ? 4 : 2;
    SISO_CUDA(cudaMemcpyAsync(dst->master, src->master, n * D * 4, cudaMemcpyDeviceToDevice, s));
    if (src->dtype != SISO_F32) SISO_CUDA(cudaMemcpyAsync(dst->vecs, src->vecs, n * D * esz, cudaMemcpyDeviceToDevice, s));
    SISO_CUDA(cudaMemcpyAsync(dst->size, src->size, n * 8, cudaMemcpyDeviceToDevice, s));
    SISO_CUDA(cudaMemcpyAsync(dst->access, src->access, n * 4, cudaMemcpyDeviceToDevice, s));
    SISO_CUDA(cudaMemcpyAsync(dst->last, src->last, n * 8, cudaMemcpyDeviceToDevice, s));
    SISO_CUDA(cudaMemcpyAsync(dst->valid, src->valid, n, cudaMemcpyDeviceToDevice, s));
    if (dst->capacity > src->capacity) {
        const int64_t extra = dst->capacity - src->capacity;
        swap_clear_tail_kernel<<<static_cast<unsigned>((extra + 255) / 256), 256, 0, s>>>(dst->valid, src->capacity, dst->capacity);
        SISO_LAUNCHED(dst);
    }
    swap_copy_counters_kernel<<<1, 32, 0, s>>>(src->counters, dst->counters);
    SISO_LAUNCHED(dst);
    return SISO_OK;
}

siso_status_t launch_update_centroids(Cache *cur, Cache *c_new, int64_t first, int64_t n, cudaStream_t s) {
    cur->vec_epoch += 1;          // the vectors may change: derived copies (the split-bf16 parts) are stale
    if (!c_new->swap_plan) {
        // source_of[capacity of C_new] and the live count behind it; lives as long as C_new
        c_new->swap_plan = cache_alloc_zeroed(c_new, pad256(sizeof(int32_t) * c_new->capacity) + 256);
        if (!c_new->swap_plan) return SISO_ERR_OOM;
    }
    int32_t *source_of = static_cast<int32_t *>(c_new->swap_plan);
    long long *n_live = reinterpret_cast<long long *>(static_cast<char *>(c_new->swap_plan) + pad256(sizeof(int32_t) * c_new->capacity));
    if (first == 0) {
        swap_plan_kernel<<<1, 1024, 0, s>>>(c_new->valid, c_new->capacity, std::min(cur->capacity, c_new->capacity), source_of,
                                            n_live, cur->status);
        SISO_LAUNCHED(cur);
    }
    const int64_t count = std::min(n, cur->capacity - first);
    if (count <= 0) return SISO_OK;
    if (cur->dtype == SISO_F32)
        swap_group_kernel<float><<<static_cast<unsigned>(count), 256, 0, s>>>(
            source_of, n_live, first, count, cur->capacity, cur->dim, static_cast<const float *>(c_new->vecs), c_new->master,
            c_new->size, c_new->access, c_new->last, static_cast<float *>(cur->vecs), cur->master, cur->size, cur->access,
            cur->last, cur->valid, cur->counters);
    else
        swap_group_kernel<__nv_bfloat16><<<static_cast<unsigned>(count), 256, 0, s>>>(
            source_of, n_live, first, count, cur->capacity, cur->dim, static_cast<const __nv_bfloat16 *>(c_new->vecs),
            c_new->master, c_new->size, c_new->access, c_new->last, static_cast<__nv_bfloat16 *>(cur->vecs), cur->master,
            cur->size, cur->access, cur->last, cur->valid, cur->counters);
    SISO_LAUNCHED(cur);
    return SISO_OK;
}

}  // namespace siso
