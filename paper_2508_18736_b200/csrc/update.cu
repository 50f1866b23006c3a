// Hit update: running mean of every centroid that was hit in this batch, then renormalisation.
//     c_j <- normalise(cluster_size_j * c_j + sum_{b in H_j} q_b)      (H_j in ascending query order)
// The hits are grouped by slot with a stable sort, so each sum runs in one fixed order; sums and
// the norm are accumulated in fp64, the result is rounded once to the fp32 master and, for bf16
// caches, once more to the bf16 lookup copy.
#include "common.cuh"

namespace siso {

constexpr int UP_THREADS = 256;

// keys: slot of each hit row, `capacity` (sorts last) for rows that are not hits; vals: row number
__global__ void update_keys_kernel(const int32_t *__restrict__ idx, int idx_stride, const uint8_t *__restrict__ hit,
                                   const uint8_t *__restrict__ valid, int64_t B, int64_t capacity,
                                   uint32_t *__restrict__ keys, uint32_t *__restrict__ vals, long long *counters,
                                   int *status) {
    const int64_t b = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (b == 0) counters[CNT_CLOCK] += 1;      // the cache clock advances once per update call
    if (b >= B) return;
    uint32_t key = static_cast<uint32_t>(capacity);
    if (hit[b]) {
        const int64_t j = idx[b * idx_stride];
        if (j >= 0 && j < capacity && valid[j]) key = static_cast<uint32_t>(j);
        else set_status(status, SISO_ERR_INVALID_ARG);   // a hit must name a live slot; the row is skipped
    }
    keys[b] = key;
    vals[b] = static_cast<uint32_t>(b);
}

// four consecutive elements of a row as fp32 (one 8- or 16-byte load)
template <typename T> __device__ __forceinline__ float4 load4(const T *p);
template <> __device__ __forceinline__ float4 load4<float>(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
template <> __device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16 *p) {
    const uint2 u = __ldg(reinterpret_cast<const uint2 *>(p));
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xFFFF0000u));
}

__device__ __forceinline__ double block_sum_f64(double v, double *red) {
    // fixed-shape tree: the same order of additions on every run
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < UP_THREADS / 32; ++w) t += red[w];
    return t;
}

// One CTA per position of the sorted hit list.  A group (the hits of one slot, ascending query order) is cut into
// chunks of `chunk` rows; the CTA at the first row of a chunk sums that chunk in fp64.  A group of one chunk is
// finished on the spot.  Otherwise the chunk sums go to scratch and the CTA that arrives last (a counter per
// group) adds them up in chunk order and finishes, so a centroid that takes hundreds of hits is not one CTA's
// serial work and the result is still the same on every run.
template <typename T>
__global__ void __launch_bounds__(UP_THREADS)
update_apply_kernel(const uint32_t *__restrict__ keys, const uint32_t *__restrict__ rows, int64_t B, int64_t capacity,
                    int D, int chunk, const T *__restrict__ Q, float *__restrict__ master, T *__restrict__ vecs,
                    double *__restrict__ size, uint32_t *__restrict__ access, unsigned long long *__restrict__ last,
                    const long long *__restrict__ counters, double *__restrict__ partial,
                    unsigned int *__restrict__ arrived) {
    extern __shared__ double acc[];          // [D]
    __shared__ double red[UP_THREADS / 32];
    __shared__ int last_s;
    const int64_t p = blockIdx.x;
    // this position, its left neighbour and the position one chunk to the left, requested together: most CTAs
    // learn from them alone whether they start a chunk
    const uint32_t slot = keys[p];
    const uint32_t left = p > 0 ? keys[p - 1] : 0xFFFFFFFFu;
    const uint32_t far_left = p >= chunk ? keys[p - chunk] : 0xFFFFFFFFu;
    if (slot >= capacity) return;
    int64_t head = p;                        // first position of this slot in the sorted list
    if (left == slot) {
        // not the first row of the group.  If the row one chunk to the left belongs to another slot, the group began
        // less than a chunk ago and this row starts no chunk; only long groups need their first position
        if (far_left != slot) return;
        int64_t lo = 0, hi = p;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if (keys[mid] < slot) lo = mid + 1; else hi = mid;
        }
        head = lo;
        if ((p - head) % chunk != 0) return;
    }
    const bool is_head = p == head;
    // everything the CTA needs of the slot and the first rows of the chunk, requested before the chunk's end is known
    const double n_old = size[slot];
    const uint32_t access_old = access[slot];
    float *m = master + static_cast<int64_t>(slot) * D;
    constexpr int MR = 4;                    // master elements per thread fetched ahead (covers D <= 1024)
    float mreg[MR];
#pragma unroll
    for (int j = 0; j < MR; ++j) { const int d = threadIdx.x + j * UP_THREADS; mreg[j] = (is_head && d < D) ? m[d] : 0.0f; }
    uint32_t row4[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) row4[r] = p + r < B ? rows[p + r] : 0u;
    // the end of this chunk, eight positions at a time; one position beyond the chunk tells whether the group goes on
    int64_t e = p + 1;
    const int64_t limit = min(B, p + static_cast<int64_t>(chunk) + 1);
    while (e < limit) {
        uint32_t k8[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) k8[u] = e + u < limit ? keys[e + u] : 0xFFFFFFFFu;
        int same = 0;
#pragma unroll
        for (int u = 0; u < 8; ++u) same += (same == u && k8[u] == slot) ? 1 : 0;
        e += same;
        if (same < 8) break;
    }
    const bool more = e > p + chunk;
    if (more) e = p + chunk;
#pragma unroll
    for (int j = 0; j < MR; ++j) { const int d = threadIdx.x + j * UP_THREADS; if (d < D) acc[d] = is_head ? n_old * static_cast<double>(mreg[j]) : 0.0; }
    for (int d = threadIdx.x + MR * UP_THREADS; d < D; d += UP_THREADS) acc[d] = is_head ? n_old * static_cast<double>(m[d]) : 0.0;
    __syncthreads();      // the accumulation below uses a different thread-to-element mapping
    // the rows four at a time: the loads of a quartet are in flight together, additions stay in ascending order
    const int quads = D / 4;
    for (int64_t t = p; t < e; t += 4) {
        const int nrow = static_cast<int>(e - t < 4 ? e - t : 4);
        const T *q[4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
            q[r] = Q + static_cast<int64_t>(t == p ? row4[r < nrow ? r : 0] : rows[t + (r < nrow ? r : 0)]) * D;
        for (int g = threadIdx.x; g < quads; g += UP_THREADS) {
            float4 v[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) v[r] = load4<T>(q[r] + 4 * g);
            double a0 = acc[4 * g], a1 = acc[4 * g + 1], a2 = acc[4 * g + 2], a3 = acc[4 * g + 3];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                if (r < nrow) { a0 += v[r].x; a1 += v[r].y; a2 += v[r].z; a3 += v[r].w; }
            }
            acc[4 * g] = a0; acc[4 * g + 1] = a1; acc[4 * g + 2] = a2; acc[4 * g + 3] = a3;   // each thread owns its g
        }
    }
    __syncthreads();
    long long count = e - p;
    if (!(is_head && !more)) {
        // several chunks: publish this chunk's sum, the last arriver combines.  A chunk's scratch row is
        // 2 * (start / chunk) + (1 if it is the group's first chunk): unique, because chunks of one group start
        // `chunk` rows apart and a first chunk of a several-chunk group is at least `chunk` rows from the next group.
        const int64_t my_id = 2 * (p / chunk) + (is_head ? 1 : 0);
        for (int d = threadIdx.x; d < D; d += UP_THREADS) partial[my_id * D + d] = acc[d];
        int64_t glo = e, ghi = B;            // first position past the group
        while (glo < ghi) {
            const int64_t mid = (glo + ghi) >> 1;
            if (keys[mid] <= slot) glo = mid + 1; else ghi = mid;
        }
        const int64_t gend = glo;
        const int64_t n_chunks = (gend - head + chunk - 1) / chunk;
        const int64_t head_id = 2 * (head / chunk) + 1;
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) last_s = (atomicAdd(&arrived[head_id], 1u) == static_cast<unsigned int>(n_chunks - 1)) ? 1 : 0;
        __syncthreads();
        if (!last_s) return;
        __threadfence();
        for (int d = threadIdx.x; d < D; d += UP_THREADS) {
            double v = __ldcg(&partial[head_id * D + d]);
            for (int64_t cidx = 1; cidx < n_chunks; ++cidx)
                v += __ldcg(&partial[(2 * ((head + cidx * chunk) / chunk)) * D + d]);
            acc[d] = v;
        }
        __syncthreads();
        count = gend - head;
    }
    double ss = 0.0;
    for (int d = threadIdx.x; d < D; d += UP_THREADS) ss += acc[d] * acc[d];
    const double norm = sqrt(block_sum_f64(ss, red));
    T *v = vecs + static_cast<int64_t>(slot) * D;
    for (int d = threadIdx.x; d < D; d += UP_THREADS) {
        const float f = static_cast<float>(acc[d] / norm);
        m[d] = f;
        if constexpr (sizeof(T) == 2) v[d] = __float2bfloat16_rn(f);
    }
    if (threadIdx.x == 0) {
        size[slot] = n_old + static_cast<double>(count);
        const unsigned long long a = static_cast<unsigned long long>(access_old) + static_cast<unsigned long long>(count);
        access[slot] = (access_old == SISO_ACCESS_INF || a >= SISO_ACCESS_INF) ? SISO_ACCESS_INF : static_cast<uint32_t>(a);
        last[slot] = static_cast<unsigned long long>(counters[CNT_CLOCK]);
    }
}

// Small batches (at most UPS_MAX_B rows): one launch.  CTA b looks at row b; it works only if row b is the first
// hit of its slot in the batch, then collects the later hits of that slot in ascending order (an ordered
// compaction in shared memory) and applies them exactly like update_apply_kernel.  Every CTA reads the clock
// before it signs off on a completion counter; the last CTA to sign off advances the clock, so no CTA can
// see the new value.
constexpr int UPS_MAX_B = 1024;

template <typename T>
__global__ void __launch_bounds__(UP_THREADS)
update_small_kernel(const int32_t *__restrict__ idx, int idx_stride, const uint8_t *__restrict__ hit, int B,
                    int64_t capacity, int D, const T *__restrict__ Q, float *__restrict__ master, T *__restrict__ vecs,
                    double *__restrict__ size, uint32_t *__restrict__ access, unsigned long long *__restrict__ last,
                    const uint8_t *__restrict__ valid, long long *counters, int *status) {
    extern __shared__ double acc[];          // [D]
    __shared__ double red[UP_THREADS / 32];
    __shared__ uint16_t members[UPS_MAX_B];
    __shared__ int warp_cnt[UP_THREADS / 32];
    __shared__ long long clock_s;
    __shared__ int n_members_s;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) clock_s = counters[CNT_CLOCK];
    bool work = false;
    int64_t slot = -1;
    if (hit[b]) {
        slot = idx[static_cast<int64_t>(b) * idx_stride];
        if (slot >= 0 && slot < capacity && valid[slot]) work = true;
        else if (tid == 0) set_status(status, SISO_ERR_INVALID_ARG);     // a hit must name a live slot; the row is skipped
    }
    if (work) {
        // is an earlier row a hit on the same slot?  then that row's CTA owns the group
        int earlier = 0;
        for (int r = tid; r < b; r += UP_THREADS) earlier |= (hit[r] && idx[static_cast<int64_t>(r) * idx_stride] == slot) ? 1 : 0;
        work = __syncthreads_or(earlier) == 0;
    }
    if (work) {
        // members of the group in ascending row order: rows b.. in chunks of 256, ballot-ordered
        int base_count = 0;
        for (int r0 = b; r0 < B; r0 += UP_THREADS) {
            const int r = r0 + tid;
            const bool mine = r < B && hit[r] && idx[static_cast<int64_t>(r) * idx_stride] == slot;
            const unsigned ballot = __ballot_sync(0xFFFFFFFFu, mine);
            if (lane == 0) warp_cnt[warp] = __popc(ballot);
            __syncthreads();
            int before = base_count, total = 0;
            for (int w = 0; w < UP_THREADS / 32; ++w) { if (w < warp) before += warp_cnt[w]; total += warp_cnt[w]; }
            if (mine) members[before + __popc(ballot & ((1u << lane) - 1u))] = static_cast<uint16_t>(r);
            base_count += total;
            __syncthreads();
        }
        if (tid == 0) n_members_s = base_count;
        const double n_old = size[slot];
        float *m = master + slot * D;
        for (int d = tid; d < D; d += UP_THREADS) acc[d] = n_old * static_cast<double>(m[d]);
        __syncthreads();
        const int count = n_members_s;
        const int quads = D / 4;
        constexpr int R = 8;                 // rows in flight per trip; additions stay in ascending row order
        for (int t = 0; t < count; t += R) {
            const int nrow = count - t < R ? count - t : R;
            const T *q[R];
#pragma unroll
            for (int r = 0; r < R; ++r) q[r] = Q + static_cast<int64_t>(members[t + (r < nrow ? r : 0)]) * D;
            for (int g = tid; g < quads; g += UP_THREADS) {
                float4 v[R];
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = load4<T>(q[r] + 4 * g);
                double a0 = acc[4 * g], a1 = acc[4 * g + 1], a2 = acc[4 * g + 2], a3 = acc[4 * g + 3];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    if (r < nrow) { a0 += v[r].x; a1 += v[r].y; a2 += v[r].z; a3 += v[r].w; }
                }
                acc[4 * g] = a0; acc[4 * g + 1] = a1; acc[4 * g + 2] = a2; acc[4 * g + 3] = a3;
            }
        }
        __syncthreads();
        double ss = 0.0;
        for (int d = tid; d < D; d += UP_THREADS) ss += acc[d] * acc[d];
        const double norm = sqrt(block_sum_f64(ss, red));
        T *v = vecs + slot * D;
        for (int d = tid; d < D; d += UP_THREADS) {
            const float f = static_cast<float>(acc[d] / norm);
            m[d] = f;
            if constexpr (sizeof(T) == 2) v[d] = __float2bfloat16_rn(f);
        }
        if (tid == 0) {
            size[slot] = n_old + static_cast<double>(count);
            const unsigned long long a = static_cast<unsigned long long>(access[slot]) + static_cast<unsigned long long>(count);
            access[slot] = (access[slot] == SISO_ACCESS_INF || a >= SISO_ACCESS_INF) ? SISO_ACCESS_INF : static_cast<uint32_t>(a);
            last[slot] = static_cast<unsigned long long>(clock_s + 1);
        }
    }
    // sign off; the last CTA advances the clock (every CTA has read it by then) and re-arms the counter
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned long long done = atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_SYNC), 1ull);
        if (done == gridDim.x - 1) {
            counters[CNT_CLOCK] = clock_s + 1;
            counters[CNT_SYNC] = 0;
        }
    }
}

siso_status_t launch_update(Cache *c, const void *q, int64_t B, const int32_t *idx, int idx_stride, const uint8_t *hit,
                            cudaStream_t s) {
    c->vec_epoch += 1;          // the vectors may change: derived copies (the split-bf16 parts) are stale
    if (B >= (1ll << 31)) return SISO_ERR_UNSUPPORTED;
    if (B >= 1 && B <= UPS_MAX_B) {
        const size_t smem_small = sizeof(double) * c->dim;
        if (c->dtype == SISO_F32)
            update_small_kernel<float><<<static_cast<unsigned>(B), UP_THREADS, smem_small, s>>>(
                idx, idx_stride, hit, static_cast<int>(B), c->capacity, c->dim, static_cast<const float *>(q), c->master,
                static_cast<float *>(c->vecs), c->size, c->access, c->last, c->valid, c->counters, c->status);
        else
            update_small_kernel<__nv_bfloat16><<<static_cast<unsigned>(B), UP_THREADS, smem_small, s>>>(
                idx, idx_stride, hit, static_cast<int>(B), c->capacity, c->dim, static_cast<const __nv_bfloat16 *>(q),
                c->master, static_cast<__nv_bfloat16 *>(c->vecs), c->size, c->access, c->last, c->valid, c->counters,
                c->status);
        SISO_LAUNCHED(c);
        return SISO_OK;
    }
    Scratch scr;
    const int chunk = static_cast<int>(std::max<int64_t>(32, (B + 4095) / 4096));
    const size_t n_ids = 2 * static_cast<size_t>(B / chunk + 1);
    const size_t need = 4 * pad256(sizeof(uint32_t) * B) + sort_pairs_scratch_bytes(B) +
                        pad256(sizeof(double) * n_ids * c->dim) + pad256(sizeof(unsigned int) * n_ids);
    SISO_TRY(scratch_reserve(c, need, s, &scr));
    uint32_t *keys = scr.take<uint32_t>(B), *vals = scr.take<uint32_t>(B);
    uint32_t *keys2 = scr.take<uint32_t>(B), *vals2 = scr.take<uint32_t>(B);
    const int threads = 256;
    // B == 0 still advances the clock
    const unsigned blocks = static_cast<unsigned>((std::max<int64_t>(B, 1) + threads - 1) / threads);
    update_keys_kernel<<<blocks, threads, 0, s>>>(idx, idx_stride, hit, c->valid, B, c->capacity, keys, vals,
                                                  c->counters, c->status);
    SISO_LAUNCHED(c);
    if (B == 0) return SISO_OK;
    int key_bits = 1;
    while ((1ll << key_bits) <= c->capacity) ++key_bits;      // keys go up to `capacity` inclusive
    uint32_t *ks, *vs;
    SISO_TRY(launch_sort_pairs(c, &scr, keys, vals, keys2, vals2, B, key_bits, &ks, &vs, s));
    const size_t smem = sizeof(double) * c->dim;
    double *partial = scr.take<double>(n_ids * c->dim);
    unsigned int *arrived = scr.take<unsigned int>(n_ids);
    SISO_CUDA(cudaMemsetAsync(arrived, 0, sizeof(unsigned int) * n_ids, s));
    if (c->dtype == SISO_F32) {
        update_apply_kernel<float><<<static_cast<unsigned>(B), UP_THREADS, smem, s>>>(
            ks, vs, B, c->capacity, c->dim, chunk, static_cast<const float *>(q), c->master, static_cast<float *>(c->vecs),
            c->size, c->access, c->last, c->counters, partial, arrived);
    } else {
        update_apply_kernel<__nv_bfloat16><<<static_cast<unsigned>(B), UP_THREADS, smem, s>>>(
            ks, vs, B, c->capacity, c->dim, chunk, static_cast<const __nv_bfloat16 *>(q), c->master,
            static_cast<__nv_bfloat16 *>(c->vecs), c->size, c->access, c->last, c->counters, partial, arrived);
    }
    SISO_LAUNCHED(c);
    return SISO_OK;
}

}  // namespace siso
