// Eviction (FilteringCentroids of Algorithm 1) and insertion of new entries.
//
// Eviction removes the m entries that come first in ascending (cluster_size, access_count,
// last_access, slot) order.  Sorting the whole cache for a few victims would cost far more than the
// metadata scan, so the kernels select, exactly, in the manner of a sample sort:
//   sample   one CTA gathers a strided sample of 256 live entries and sorts it (bitonic, in
//            shared memory): the sorted sample keys are splitters
//   bucket   every live entry finds its bucket (number of splitters below its key, binary search)
//            and the buckets are counted
//   collect  the smallest bucket index p whose cumulative count reaches m is found from the counts;
//            entries in buckets <= p (at least m of them, about m + capacity/256) become candidates
//   rank     one warp per candidate counts the candidates below it; rank < m means victim number rank
// Keys are compared as three 64-bit integers (order-preserving image of the fp64 cluster_size, then
// access_count | last_access | slot), so the order is the exact lexicographic order and total.
#include "evict_keys.cuh"

namespace siso {

constexpr int EV_SAMPLE = 256;

struct EvictPlan {
    long long m;             // victims to produce (clamped to the occupancy)
    int n_sample;            // live splitters
    unsigned int n_cand;
    unsigned int hist[EV_SAMPLE + 1];
};

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
evict_sample_kernel(long long m_req, const uint8_t *__restrict__ hit, long long n_hit, long long capacity,
                    const double *__restrict__ size, const uint32_t *__restrict__ access,
                    const unsigned long long *__restrict__ last, const uint8_t *__restrict__ valid,
                    const long long *__restrict__ counters, EvictPlan *plan, Key3 *__restrict__ splitters,
                    int32_t *victims, long long n_victims_out) {
    __shared__ unsigned long long k0[EV_SAMPLE], k1[EV_SAMPLE], k2[EV_SAMPLE];
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
    if (tid == 0) { plan->m = m; plan->n_cand = 0; }
    if (tid <= EV_SAMPLE) plan->hist[tid] = 0;
    if (m == 0) return;
    // strided sample: thread t < EV_SAMPLE takes the first live slot of window [t*stride, (t+1)*stride), starting
    // at an offset that changes from call to call (at most 64 probes)
    const long long stride = (capacity + EV_SAMPLE - 1) / EV_SAMPLE;
    const long long lo = tid * stride, hi = tid < EV_SAMPLE ? min(capacity, lo + stride) : lo;
    const long long span = hi - lo;
    int have = 0;
    Key3 mine;
    mine.w0 = mine.w1 = mine.w2 = ~0ull;                 // sentinel: sorts after every real key
    if (span > 0) {
        const long long start = static_cast<long long>((static_cast<unsigned long long>(counters[CNT_CLOCK]) * 2654435761ull) % static_cast<unsigned long long>(span));
        const long long probes = span < 64 ? span : 64;
        for (long long i = 0; i < probes; ++i) {
            long long sl = lo + start + i;
            if (sl >= hi) sl -= span;
            if (valid[sl]) { mine = make_key(size[sl], access[sl], last[sl], static_cast<uint32_t>(sl)); have = 1; break; }
        }
    }
    if (tid < EV_SAMPLE) { k0[tid] = mine.w0; k1[tid] = mine.w1; k2[tid] = mine.w2; }
    int n_sample;
    block_exclusive_scan_1024(have, &n_sample, warp_sum);
    __syncthreads();
    // bitonic sort, ascending
    for (int k = 2; k <= EV_SAMPLE; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            const int partner = tid ^ j;
            if (tid < EV_SAMPLE && partner > tid) {
                Key3 a, b;
                a.w0 = k0[tid]; a.w1 = k1[tid]; a.w2 = k2[tid];
                b.w0 = k0[partner]; b.w1 = k1[partner]; b.w2 = k2[partner];
                const bool up = (tid & k) == 0;
                if (key_less(b, a) == up) {
                    k0[tid] = b.w0; k1[tid] = b.w1; k2[tid] = b.w2;
                    k0[partner] = a.w0; k1[partner] = a.w1; k2[partner] = a.w2;
                }
            }
            __syncthreads();
        }
    }
    if (tid < EV_SAMPLE) {
        Key3 out;
        out.w0 = k0[tid]; out.w1 = k1[tid]; out.w2 = k2[tid];
        splitters[tid] = out;
    }
    if (tid == 0) plan->n_sample = n_sample;
}

// bucket(key) = number of live splitters strictly below the key, in [0, n_sample]
__global__ void __launch_bounds__(256)
evict_bucket_kernel(long long capacity, const double *__restrict__ size, const uint32_t *__restrict__ access,
                    const unsigned long long *__restrict__ last, const uint8_t *__restrict__ valid, EvictPlan *plan,
                    const Key3 *__restrict__ splitters, uint16_t *__restrict__ bucket) {
    if (plan->m == 0) return;
    __shared__ unsigned long long s0[EV_SAMPLE], s1[EV_SAMPLE], s2[EV_SAMPLE];
    __shared__ unsigned int hist[EV_SAMPLE + 1];
    const int n_sample = plan->n_sample;
    for (int i = threadIdx.x; i < EV_SAMPLE; i += 256) {
        const Key3 k = splitters[i];
        s0[i] = k.w0; s1[i] = k.w1; s2[i] = k.w2;
        hist[i] = 0;
    }
    if (threadIdx.x == 0) hist[EV_SAMPLE] = 0;
    __syncthreads();
    for (long long sl = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x; sl < capacity;
         sl += static_cast<long long>(gridDim.x) * 256) {
        if (!valid[sl]) continue;
        const Key3 k = make_key(size[sl], access[sl], last[sl], static_cast<uint32_t>(sl));
        int lo = 0, hi = n_sample;                       // first index whose splitter is >= k
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            Key3 sp;
            sp.w0 = s0[mid]; sp.w1 = s1[mid]; sp.w2 = s2[mid];
            if (key_less(sp, k)) lo = mid + 1; else hi = mid;
        }
        bucket[sl] = static_cast<uint16_t>(lo);
        atomicAdd(&hist[lo], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i <= EV_SAMPLE; i += 256)
        if (hist[i]) atomicAdd(&plan->hist[i], hist[i]);
}

__global__ void __launch_bounds__(256)
evict_collect_kernel(long long capacity, const double *__restrict__ size, const uint32_t *__restrict__ access,
                     const unsigned long long *__restrict__ last, const uint8_t *__restrict__ valid, EvictPlan *plan,
                     const uint16_t *__restrict__ bucket, Key3 *__restrict__ cand) {
    const long long m = plan->m;
    if (m == 0) return;
    __shared__ int p_s;
    if (threadIdx.x < 32) {
        // smallest p with hist[0] + ... + hist[p] >= m (exists: the live entries number at least m)
        long long run = 0;
        int found = EV_SAMPLE;
        for (int base = 0; base <= EV_SAMPLE && found == EV_SAMPLE; base += 32) {
            const int i = base + threadIdx.x;
            long long x = i <= EV_SAMPLE ? plan->hist[i] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const long long y = __shfl_up_sync(0xFFFFFFFFu, x, o);
                if (static_cast<int>(threadIdx.x) >= o) x += y;
            }
            const unsigned reach = __ballot_sync(0xFFFFFFFFu, run + x >= m);
            if (reach) found = base + __ffs(reach) - 1;
            run += __shfl_sync(0xFFFFFFFFu, x, 31);
        }
        if (threadIdx.x == 0) p_s = found;
    }
    __syncthreads();
    const int p = p_s;
    const int lane = threadIdx.x & 31;
    for (long long base = static_cast<long long>(blockIdx.x) * 256; base < capacity;
         base += static_cast<long long>(gridDim.x) * 256) {
        const long long sl = base + threadIdx.x;
        const bool take = sl < capacity && valid[sl] && bucket[sl] <= p;
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, take);
        if (ballot) {
            unsigned int warp_base = 0;
            if (lane == 0) warp_base = atomicAdd(&plan->n_cand, static_cast<unsigned int>(__popc(ballot)));
            warp_base = __shfl_sync(0xFFFFFFFFu, warp_base, 0);
            if (take) cand[warp_base + __popc(ballot & ((1u << lane) - 1u))] =
                          make_key(size[sl], access[sl], last[sl], static_cast<uint32_t>(sl));
        }
    }
}

// one warp per candidate
__global__ void __launch_bounds__(256)
evict_rank_kernel(EvictPlan *plan, const Key3 *__restrict__ cand, uint8_t *__restrict__ valid,
                  int32_t *__restrict__ victims, long long *counters, Key3 *__restrict__ keys_out, unsigned long long slot_offset,
                  int apply) {
    const long long m = plan->m;
    if (m == 0) return;
    const unsigned int n = plan->n_cand;
    const int lane = threadIdx.x & 31;
    const unsigned int warps = gridDim.x * (blockDim.x >> 5);
    for (unsigned int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); i < n; i += warps) {
        const Key3 mine = cand[i];
        unsigned int rank = 0;
        for (unsigned int j = lane; j < n; j += 32) rank += key_less(cand[j], mine) ? 1u : 0u;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, o);
        if (lane == 0 && rank < m) {
            const int32_t slot = static_cast<int32_t>(mine.w2 & 0xFFFFFFFFull);
            if (victims) victims[rank] = slot;
            if (keys_out) {                  // the key with the slot made global (slot + offset < 2^32: no carry into last_access)
                Key3 k = mine;
                k.w2 += slot_offset;
                keys_out[rank] = k;
            }
            if (apply) valid[slot] = 0;
        }
    }
    if (apply && blockIdx.x == 0 && threadIdx.x == 0) {
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
    SISO_TRY(scratch_reserve(c, pad256(sizeof(EvictPlan)) + pad256(sizeof(Key3) * EV_SAMPLE) +
                                    pad256(sizeof(uint16_t) * c->capacity) + pad256(sizeof(Key3) * c->capacity), s, &scr));
    EvictPlan *plan = scr.take<EvictPlan>(1);
    Key3 *splitters = scr.take<Key3>(EV_SAMPLE);
    uint16_t *bucket = scr.take<uint16_t>(c->capacity);
    Key3 *cand = scr.take<Key3>(c->capacity);
    evict_sample_kernel<<<1, 1024, 0, s>>>(n_evict, hit, n_hit, c->capacity, c->size, c->access, c->last, c->valid,
                                           c->counters, plan, splitters, victims, victims ? n_victims_out : 0);
    SISO_LAUNCHED(c);
    const int grid = static_cast<int>(std::min<int64_t>((c->capacity + 255) / 256, 4ll * c->sm_count));
    const int grid_bucket = static_cast<int>(std::min<int64_t>((c->capacity + 255) / 256, 8ll * c->sm_count));
    evict_bucket_kernel<<<grid_bucket, 256, 0, s>>>(c->capacity, c->size, c->access, c->last, c->valid, plan, splitters, bucket);
    SISO_LAUNCHED(c);
    evict_collect_kernel<<<grid, 256, 0, s>>>(c->capacity, c->size, c->access, c->last, c->valid, plan, bucket, cand);
    SISO_LAUNCHED(c);
    evict_rank_kernel<<<grid, 256, 0, s>>>(plan, cand, c->valid, victims, c->counters, nullptr, 0ull, 1);
    SISO_LAUNCHED(c);
    if (flags & SISO_EVICT_DECAY) {
        decay_kernel<<<static_cast<unsigned>((c->capacity + 255) / 256), 256, 0, s>>>(c->capacity, c->decay, c->size,
                                                                                      c->access, c->valid);
        SISO_LAUNCHED(c);
    }
    return SISO_OK;
}

// ---------------------------------------------------------------------------------------------
// eviction over a cache partitioned across GPUs: every shard reports its n lowest keys (global slots), the n_take lowest
// of all reported keys are the victims, every shard drops those it holds
// ---------------------------------------------------------------------------------------------
siso_status_t launch_evict_keys(Cache *c, int64_t n, int64_t slot_offset, unsigned long long *keys_out, cudaStream_t s) {
    Scratch scr;
    SISO_TRY(scratch_reserve(c, pad256(sizeof(EvictPlan)) + pad256(sizeof(Key3) * EV_SAMPLE) +
                                    pad256(sizeof(uint16_t) * c->capacity) + pad256(sizeof(Key3) * c->capacity), s, &scr));
    EvictPlan *plan = scr.take<EvictPlan>(1);
    Key3 *splitters = scr.take<Key3>(EV_SAMPLE);
    uint16_t *bucket = scr.take<uint16_t>(c->capacity);
    Key3 *cand = scr.take<Key3>(c->capacity);
    SISO_CUDA(cudaMemsetAsync(keys_out, 0xFF, sizeof(Key3) * n, s));           // padding: sorts after every real key
    evict_sample_kernel<<<1, 1024, 0, s>>>(n, nullptr, 0, c->capacity, c->size, c->access, c->last, c->valid, c->counters, plan,
                                           splitters, nullptr, 0);
    SISO_LAUNCHED(c);
    const int grid = static_cast<int>(std::min<int64_t>((c->capacity + 255) / 256, 4ll * c->sm_count));
    const int grid_bucket = static_cast<int>(std::min<int64_t>((c->capacity + 255) / 256, 8ll * c->sm_count));
    evict_bucket_kernel<<<grid_bucket, 256, 0, s>>>(c->capacity, c->size, c->access, c->last, c->valid, plan, splitters, bucket);
    SISO_LAUNCHED(c);
    evict_collect_kernel<<<grid, 256, 0, s>>>(c->capacity, c->size, c->access, c->last, c->valid, plan, bucket, cand);
    SISO_LAUNCHED(c);
    evict_rank_kernel<<<grid, 256, 0, s>>>(plan, cand, c->valid, nullptr, c->counters, reinterpret_cast<Key3 *>(keys_out),
                                           static_cast<unsigned long long>(slot_offset), 0);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

namespace {

// keys [n_lists, n] (Key3), every list ascending with all-ones padding; one thread per key: its rank among all keys is the
// sum over the lists of the number of smaller keys there (binary search); the n_take lowest give victims[rank] = global slot
__global__ void __launch_bounds__(256)
evict_select_kernel(const Key3 *__restrict__ keys, int n_lists, long long n, long long n_take, const long long *__restrict__ plan,
                    long long *__restrict__ victims) {
    const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= n * n_lists) return;
    if (plan) n_take = plan[1] < n ? plan[1] : n;               // decided on the device (siso_shard_plan)
    const Key3 mine = keys[t];
    if ((mine.w0 & mine.w1 & mine.w2) == ~0ull) return;
    long long rank = 0;
    for (int l = 0; l < n_lists; ++l) {
        const Key3 *list = keys + static_cast<long long>(l) * n;
        long long lo = 0, hi = n;                                  // first position whose key is not below mine
        while (lo < hi) {
            const long long mid = (lo + hi) >> 1;
            if (key_less(list[mid], mine)) lo = mid + 1; else hi = mid;
        }
        rank += lo;
    }
    if (rank < n_take) victims[rank] = static_cast<long long>(mine.w2 & 0xFFFFFFFFull);
}

// one CTA: drops the victims that fall into [slot_offset, slot_offset + capacity)
__global__ void __launch_bounds__(1024)
evict_slots_kernel(const long long *__restrict__ victims, long long n, long long slot_offset, long long capacity,
                   uint8_t *__restrict__ valid, long long *counters) {
    __shared__ int warp_sum[32];
    int dropped = 0;
    for (long long i = threadIdx.x; i < n; i += 1024) {
        const long long v = victims[i] - slot_offset;
        if (victims[i] >= 0 && v >= 0 && v < capacity && valid[v]) {
            valid[v] = 0;
            ++dropped;
        }
    }
    int total;
    block_exclusive_scan_1024(dropped, &total, warp_sum);
    if (threadIdx.x == 0) {
        counters[CNT_OCCUPANCY] -= total;
        counters[CNT_EVICTIONS] += total;
    }
}

}  // namespace

siso_status_t launch_evict_select(const unsigned long long *keys, int n_lists, int64_t n, int64_t n_take, long long *victims,
                                  cudaStream_t s, const long long *plan) {
    SISO_CUDA(cudaMemsetAsync(victims, 0xFF, sizeof(long long) * n_take, s));  // -1: fewer live entries than asked for
    if (n > 0)
        evict_select_kernel<<<static_cast<unsigned>((n * n_lists + 255) / 256), 256, 0, s>>>(
            reinterpret_cast<const Key3 *>(keys), n_lists, n, n_take, plan, victims);
    return check_cuda(cudaGetLastError(), "evict_select_kernel");
}

siso_status_t launch_evict_slots(Cache *c, const long long *victims, int64_t n, int64_t slot_offset, uint32_t flags, cudaStream_t s) {
    if (n > 0) {
        evict_slots_kernel<<<1, 1024, 0, s>>>(victims, n, slot_offset, c->capacity, c->valid, c->counters);
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
    c->vec_epoch += 1;          // the vectors may change: derived copies (the split-bf16 parts) are stale
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
