// Eviction (FilteringCentroids of Algorithm 1) and insertion of new entries.
//
// Eviction removes the m entries that come first in ascending (cluster_size, access_count,
// last_access, slot) order.  Sorting the whole cache for a few victims would cost far more
// than the metadata scan, so the kernels select instead:
//   plan    one CTA ranks a strided sample of live entries and picks a pivot key that, with
//           overwhelming probability, has at least m entries at or below it but not many more;
//   filter  every live entry with key <= pivot is appended to a candidate list;
//   rank    each candidate counts the candidates below it; rank < m means victim number `rank`.
// If the pivot turned out too low (fewer than m candidates), a second filter/rank pair with an
// infinite pivot redoes the selection exactly; both pairs are always launched and the second is a
// no-op when the first succeeded.  The result never depends on the sample: it is the exact order.
#include "common.cuh"

namespace siso {

struct EvictKey {
    double size;
    unsigned long long last;
    uint32_t access;
    int32_t slot;
};
__device__ __forceinline__ bool key_less(const EvictKey &a, const EvictKey &b) {
    if (a.size != b.size) return a.size < b.size;
    if (a.access != b.access) return a.access < b.access;
    if (a.last != b.last) return a.last < b.last;
    return a.slot < b.slot;
}

struct EvictPlan {
    EvictKey pivot;
    long long m;            // victims to produce (clamped to the occupancy)
    int pivot_all;          // 1: pivot is +infinity
    unsigned int ncand[2];  // candidates found by attempt 0 / 1
};

constexpr int EV_SAMPLE = 1024;

__device__ __forceinline__ int block_exclusive_scan_1024(int v, int *total, int *warp_sum) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xFFFFFFFFu, x, o);
        if (lane >= o) x += y;
    }
    __syncthreads();
    if (lane == 31) warp_sum[warp] = x;
    __syncthreads();
    if (warp == 0) {
        int s = warp_sum[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xFFFFFFFFu, s, o);
            if (lane >= o) s += y;
        }
        warp_sum[lane] = s;
    }
    __syncthreads();
    *total = warp_sum[31];
    return (warp ? warp_sum[warp - 1] : 0) + x - v;
}

__global__ void __launch_bounds__(1024)
evict_plan_kernel(long long m_req, const uint8_t *__restrict__ hit, long long n_hit, long long capacity,
                  const double *__restrict__ size, const uint32_t *__restrict__ access,
                  const unsigned long long *__restrict__ last, const uint8_t *__restrict__ valid,
                  const long long *__restrict__ counters, EvictPlan *plan, int32_t *victims, long long n_victims_out) {
    __shared__ EvictKey sample[EV_SAMPLE];
    __shared__ int warp_sum[32];
    __shared__ long long m_s;
    const int tid = threadIdx.x;
    const long long occupancy = counters[CNT_OCCUPANCY];
    // how many to evict: given, or what the misses of this batch lack in free slots
    if (m_req < 0) {
        int miss = 0;
        for (long long b = tid; b < n_hit; b += 1024) miss += hit[b] ? 0 : 1;
        int total;
        block_exclusive_scan_1024(miss, &total, warp_sum);
        if (tid == 0) {
            const long long lack = static_cast<long long>(total) - (capacity - occupancy);
            m_s = lack > 0 ? lack : 0;
        }
    } else if (tid == 0) {
        m_s = m_req;
    }
    __syncthreads();
    const long long m = m_s < occupancy ? m_s : occupancy;
    for (long long r = m + tid; r < n_victims_out; r += 1024) victims[r] = -1;
    if (tid == 0) { plan->m = m; plan->ncand[0] = 0; plan->ncand[1] = 0; plan->pivot_all = 0; }
    if (m == 0) return;
    // strided sample: thread t looks at slots [t*stride, (t+1)*stride) and takes the first live one
    const long long stride = (capacity + EV_SAMPLE - 1) / EV_SAMPLE;
    int have = 0;
    EvictKey mine;
    mine.size = 0.0; mine.last = 0; mine.access = 0; mine.slot = -1;
    const long long lo = tid * stride, hi = min(capacity, lo + stride);
    for (long long sl = lo; sl < hi && sl < lo + 64; ++sl) {
        if (valid[sl]) {
            mine.size = size[sl]; mine.access = access[sl]; mine.last = last[sl]; mine.slot = static_cast<int32_t>(sl);
            have = 1;
            break;
        }
    }
    sample[tid] = mine;
    int n_sample;
    block_exclusive_scan_1024(have, &n_sample, warp_sum);
    __syncthreads();
    // which rank of the sample becomes the pivot
    long long r;
    if (stride == 1) {
        r = m;                                     // the sample is the whole cache: exact
    } else {
        const double mu = static_cast<double>(m) * n_sample / static_cast<double>(occupancy);
        r = static_cast<long long>(ceil(mu + 12.0 + 8.0 * sqrt(mu)));
    }
    if (r > n_sample || n_sample == 0) {
        if (tid == 0) plan->pivot_all = 1;
        return;
    }
    if (have) {
        int rank = 0;
        for (int j = 0; j < EV_SAMPLE; ++j) {
            const EvictKey o = sample[j];
            rank += (o.slot >= 0 && key_less(o, mine)) ? 1 : 0;
        }
        if (rank == r - 1) plan->pivot = mine;
    }
}

__global__ void __launch_bounds__(256)
evict_filter_kernel(int attempt, long long capacity, const double *__restrict__ size,
                    const uint32_t *__restrict__ access, const unsigned long long *__restrict__ last,
                    const uint8_t *__restrict__ valid, EvictPlan *plan, EvictKey *__restrict__ cand) {
    const long long m = plan->m;
    if (m == 0) return;
    if (attempt == 1 && plan->ncand[0] >= m) return;
    const bool all = attempt == 1 || plan->pivot_all;
    const EvictKey pivot = plan->pivot;
    const int lane = threadIdx.x & 31;
    for (long long base = static_cast<long long>(blockIdx.x) * blockDim.x; base < capacity;
         base += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long sl = base + threadIdx.x;
        bool take = false;
        EvictKey k;
        if (sl < capacity && valid[sl]) {
            k.size = size[sl]; k.access = access[sl]; k.last = last[sl]; k.slot = static_cast<int32_t>(sl);
            take = all || !key_less(pivot, k);
        }
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, take);
        if (ballot) {
            unsigned int warp_base = 0;
            if (lane == 0) warp_base = atomicAdd(&plan->ncand[attempt], static_cast<unsigned int>(__popc(ballot)));
            warp_base = __shfl_sync(0xFFFFFFFFu, warp_base, 0);
            if (take) cand[warp_base + __popc(ballot & ((1u << lane) - 1u))] = k;
        }
    }
}

__global__ void __launch_bounds__(256)
evict_rank_kernel(int attempt, EvictPlan *plan, const EvictKey *__restrict__ cand, uint8_t *__restrict__ valid,
                  int32_t *__restrict__ victims, long long *counters) {
    const long long m = plan->m;
    if (m == 0) return;
    if (attempt == 1 && plan->ncand[0] >= m) return;
    const unsigned int n = plan->ncand[attempt];
    if (n < m) return;                 // attempt 0 fell short: attempt 1 redoes it; attempt 1 never falls short
    __shared__ EvictKey tile[256];
    const unsigned int rounds = (n + gridDim.x * blockDim.x - 1) / (gridDim.x * blockDim.x);
    for (unsigned int rd = 0; rd < rounds; ++rd) {
        const unsigned int i = (rd * gridDim.x + blockIdx.x) * blockDim.x + threadIdx.x;
        EvictKey mine;
        if (i < n) mine = cand[i];
        unsigned int rank = 0;
        for (unsigned int t0 = 0; t0 < n; t0 += 256) {
            __syncthreads();
            if (t0 + threadIdx.x < n) tile[threadIdx.x] = cand[t0 + threadIdx.x];
            __syncthreads();
            const unsigned int lim = min(256u, n - t0);
            if (i < n)
                for (unsigned int j = 0; j < lim; ++j) rank += key_less(tile[j], mine) ? 1u : 0u;
        }
        if (i < n && rank < m) {
            if (victims) victims[rank] = mine.slot;
            valid[mine.slot] = 0;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        counters[CNT_OCCUPANCY] -= m;
        counters[CNT_EVICTIONS] += m;
    }
}

__global__ void decay_kernel(long long capacity, double decay, double *__restrict__ size, uint32_t *__restrict__ access,
                             const uint8_t *__restrict__ valid) {
    const long long sl = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (sl < capacity && valid[sl]) {
        size[sl] = __ddiv_rn(size[sl], decay);
        access[sl] = 0;
    }
}

// n_evict >= 0: evict that many; n_evict < 0: evict max(0, #rows with hit == 0 - #free slots).
siso_status_t launch_evict(Cache *c, int64_t n_evict, const uint8_t *hit, int64_t n_hit, uint32_t flags,
                           int32_t *victims, int64_t n_victims_out, cudaStream_t s) {
    Scratch scr;
    SISO_TRY(scratch_reserve(c, pad256(sizeof(EvictPlan)) + pad256(sizeof(EvictKey) * c->capacity), s, &scr));
    EvictPlan *plan = scr.take<EvictPlan>(1);
    EvictKey *cand = scr.take<EvictKey>(c->capacity);
    evict_plan_kernel<<<1, 1024, 0, s>>>(n_evict, hit, n_hit, c->capacity, c->size, c->access, c->last, c->valid,
                                         c->counters, plan, victims, victims ? n_victims_out : 0);
    SISO_LAUNCHED(c);
    const int grid = static_cast<int>(std::min<int64_t>((c->capacity + 255) / 256, 4ll * c->sm_count));
    for (int attempt = 0; attempt < 2; ++attempt) {
        evict_filter_kernel<<<grid, 256, 0, s>>>(attempt, c->capacity, c->size, c->access, c->last, c->valid, plan, cand);
        SISO_LAUNCHED(c);
        evict_rank_kernel<<<grid, 256, 0, s>>>(attempt, plan, cand, c->valid, victims, c->counters);
        SISO_LAUNCHED(c);
    }
    if (flags & SISO_EVICT_DECAY) {
        decay_kernel<<<static_cast<unsigned>((c->capacity + 255) / 256), 256, 0, s>>>(c->capacity, c->decay, c->size,
                                                                                      c->access, c->valid);
        SISO_LAUNCHED(c);
    }
    return SISO_OK;
}

// ---------------------------------------------------------------------------------------------
// insertion: rows with hit == 0 (all rows if hit == NULL), ascending, take the free slots, ascending
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
insert_plan_kernel(const uint8_t *__restrict__ hit, long long n, long long capacity, const uint8_t *__restrict__ valid,
                   long long *counters, int32_t *__restrict__ free_list, int32_t *__restrict__ slots, int *status) {
    __shared__ int warp_sum[32];
    __shared__ long long carry_s;
    const int tid = threadIdx.x;
    // how many rows want a slot
    int want = 0;
    for (long long b = tid; b < n; b += 1024) want += (!hit || !hit[b]) ? 1 : 0;
    int n_ins;
    block_exclusive_scan_1024(want, &n_ins, warp_sum);
    const long long n_free = capacity - counters[CNT_OCCUPANCY];
    if (n_ins > n_free) {
        for (long long b = tid; b < n; b += 1024) slots[b] = -1;
        if (tid == 0) set_status(status, SISO_ERR_CAPACITY);
        return;
    }
    // the first n_ins free slots, ascending: each thread inspects 16 consecutive slots per step
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (long long base = 0; base < capacity; base += 1024 * 16) {
        const long long lo = base + tid * 16;
        uint32_t free_mask = 0;
        if (lo + 16 <= capacity) {
            const uint4 v = *reinterpret_cast<const uint4 *>(valid + lo);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 16; ++i) free_mask |= (((w[i >> 2] >> (8 * (i & 3))) & 0xFFu) == 0u) ? (1u << i) : 0u;
        } else {
            for (int i = 0; i < 16; ++i)
                if (lo + i < capacity && !valid[lo + i]) free_mask |= 1u << i;
        }
        int total;
        const int before = block_exclusive_scan_1024(__popc(free_mask), &total, warp_sum);
        const long long carry = carry_s;
        long long rank = carry + before;
        for (int i = 0; i < 16 && free_mask; ++i) {
            if (free_mask & (1u << i)) {
                if (rank < n_ins) free_list[rank] = static_cast<int32_t>(lo + i);
                ++rank;
            }
        }
        __syncthreads();
        if (tid == 0) carry_s = carry + total;
        __syncthreads();
        if (carry + total >= n_ins) break;
    }
    // rows -> slots
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (long long base = 0; base < n; base += 1024) {
        const long long b = base + tid;
        const int w = (b < n && (!hit || !hit[b])) ? 1 : 0;
        int total;
        const int before = block_exclusive_scan_1024(w, &total, warp_sum);
        const long long carry = carry_s;
        if (b < n) slots[b] = w ? free_list[carry + before] : -1;
        __syncthreads();
        if (tid == 0) carry_s = carry + total;
        __syncthreads();
    }
    if (tid == 0) {
        counters[CNT_OCCUPANCY] += n_ins;
        counters[CNT_INSERTS] += n_ins;
    }
}

template <typename T>
__global__ void __launch_bounds__(128)
insert_copy_kernel(const T *__restrict__ rows, const double *__restrict__ sizes_in, const int32_t *__restrict__ slots,
                   int D, T *__restrict__ vecs, float *__restrict__ master, double *__restrict__ size,
                   uint32_t *__restrict__ access, unsigned long long *__restrict__ last, uint8_t *__restrict__ valid,
                   const long long *__restrict__ counters) {
    const long long b = blockIdx.x;
    const int32_t slot = slots[b];
    if (slot < 0) return;
    const T *src = rows + b * D;
    T *dv = vecs + static_cast<long long>(slot) * D;
    float *dm = master + static_cast<long long>(slot) * D;
    for (int d = threadIdx.x; d < D; d += 128) {
        const T x = src[d];
        dv[d] = x;
        if constexpr (sizeof(T) == 2) dm[d] = __bfloat162float(x);
    }
    if (threadIdx.x == 0) {
        size[slot] = sizes_in ? sizes_in[b] : 1.0;
        access[slot] = SISO_ACCESS_INF;
        last[slot] = static_cast<unsigned long long>(counters[CNT_CLOCK]);
        valid[slot] = 1;
    }
}

siso_status_t launch_insert(Cache *c, const void *vecs, const double *sizes, const uint8_t *hit, int64_t n,
                            int32_t *slots_out, cudaStream_t s) {
    if (n == 0) return SISO_OK;
    if (n >= (1ll << 31)) return SISO_ERR_UNSUPPORTED;
    Scratch scr;
    SISO_TRY(scratch_reserve(c, 2 * pad256(sizeof(int32_t) * n), s, &scr));
    int32_t *free_list = scr.take<int32_t>(n);
    int32_t *slots = slots_out ? slots_out : scr.take<int32_t>(n);
    insert_plan_kernel<<<1, 1024, 0, s>>>(hit, n, c->capacity, c->valid, c->counters, free_list, slots, c->status);
    SISO_LAUNCHED(c);
    if (c->dtype == SISO_F32) {
        insert_copy_kernel<float><<<static_cast<unsigned>(n), 128, 0, s>>>(
            static_cast<const float *>(vecs), sizes, slots, c->dim, static_cast<float *>(c->vecs), c->master, c->size,
            c->access, c->last, c->valid, c->counters);
    } else {
        insert_copy_kernel<__nv_bfloat16><<<static_cast<unsigned>(n), 128, 0, s>>>(
            static_cast<const __nv_bfloat16 *>(vecs), sizes, slots, c->dim, static_cast<__nv_bfloat16 *>(c->vecs),
            c->master, c->size, c->access, c->last, c->valid, c->counters);
    }
    SISO_LAUNCHED(c);
    return SISO_OK;
}

}  // namespace siso
