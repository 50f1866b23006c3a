// Centroid-sharded lookup: the cache's rows are partitioned over several GPUs, every GPU scores the whole query batch
// against its own rows (FindClosestCentroid of Algorithm 1 restricted to a shard), and the shards' results are
// combined after ONE exchange of a few bytes per query.  What crosses between GPUs are packed 64-bit keys,
// (order-preserving similarity bits << 32) | (2^32 - 1 - global slot), whose maximum is the best match with ties to the
// lower global slot, so that the combined result does not depend on the number of shards or on their order.
//   pack     a shard's (idx, sim) lists -> keys with the shard's slot offset added
//   combine  per query the k largest of n_lists * k keys -> global slot (int64), similarity, strict threshold test
//   route    the combined (global slot, hit) of a batch -> what THIS shard has to do: the hits on its own rows as local
//            slots (for the running-mean update), and the misses it stores: misses are numbered in ascending row order and
//            take the free slots of the whole cache in ascending global order, so a shard with `take` free slots after
//            `skip` free slots on the shards before it stores misses number skip .. skip + take - 1
#include "common.cuh"

namespace siso {

namespace {

__global__ void shard_pack_kernel(const int32_t *__restrict__ idx, const float *__restrict__ sim, long long n, long long slot_offset,
                                  unsigned long long *__restrict__ keys) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t s = idx[i];
    keys[i] = s < 0 ? 0ull : pack_key(sim[i], static_cast<uint32_t>(static_cast<long long>(s) + slot_offset));
}

// one warp per query; keys [n, n_lists, k]
template <int KMAX>
__global__ void __launch_bounds__(256)
shard_combine_kernel(const unsigned long long *__restrict__ keys, long long n, int n_lists, int k, const float *__restrict__ theta,
                     float theta_s, long long *__restrict__ idx, float *__restrict__ sim, uint8_t *__restrict__ hit) {
    const int lane = threadIdx.x & 31;
    const long long b = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (b >= n) return;
    KeyList<KMAX> out;
    out.clear();
    const unsigned long long *src = keys + b * n_lists * k;
    for (int s = lane; s < n_lists * k; s += 32) out.insert(src[s]);
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
                idx[b * k + j] = key ? static_cast<long long>(0xFFFFFFFFu - static_cast<uint32_t>(key)) : -1ll;
                sim[b * k + j] = key ? key_sim(key) : -INFINITY;
            }
        }
        const float th = theta ? theta[b] : theta_s;
        hit[b] = (out.k[0] != 0ull && key_sim(out.k[0]) > th) ? 1 : 0;
    }
}

// one CTA
__global__ void __launch_bounds__(1024)
shard_route_kernel(const long long *__restrict__ idx, long long idx_stride, const uint8_t *__restrict__ hit, long long n,
                   long long slot_lo, long long slot_hi, long long skip, long long take, const long long *__restrict__ plan,
                   int32_t *__restrict__ idx_local, uint8_t *__restrict__ upd_hit, uint8_t *__restrict__ ins_hit) {
    __shared__ int warp_cnt[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (plan) { skip = plan[2]; take = plan[3]; }              // decided on the device (siso_shard_plan)
    long long base = 0;                                          // misses in the rows already visited, the same in every thread
    for (long long b0 = 0; b0 < n; b0 += 1024) {
        const long long b = b0 + tid;
        const bool miss = b < n && hit[b] == 0;
        const unsigned int ballot = __ballot_sync(0xFFFFFFFFu, miss);
        if (lane == 0) warp_cnt[warp] = __popc(ballot);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < 32; ++w) {
            const int c = warp_cnt[w];
            before += w < warp ? c : 0;
            total += c;
        }
        if (b < n) {
            const long long g = idx[b * idx_stride];
            const bool mine = !miss && g >= slot_lo && g < slot_hi;
            idx_local[b] = mine ? static_cast<int32_t>(g - slot_lo) : -1;
            upd_hit[b] = mine ? 1 : 0;
            const long long number = base + before + __popc(ballot & ((1u << lane) - 1u));
            ins_hit[b] = (miss && number >= skip && number < skip + take) ? 0 : 1;      // 0 = store this row here
        }
        base += total;
        __syncthreads();
    }
}

// one CTA: what the batch's misses need, from the hit flags and the free slots of every shard
//   plan[0] misses   plan[1] entries to evict over the whole cache (misses - free slots, at least 0)
//   plan[2] free slots on the shards before this one   plan[3] free slots on this shard
__global__ void __launch_bounds__(1024)
shard_plan_kernel(const uint8_t *__restrict__ hit, long long n, const long long *__restrict__ free_all, int world, int rank,
                  long long *__restrict__ plan) {
    __shared__ int warp_cnt[32];
    int miss = 0;
    for (long long b = threadIdx.x; b < n; b += 1024) miss += hit[b] == 0 ? 1 : 0;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) miss += __shfl_xor_sync(0xFFFFFFFFu, miss, o);
    if ((threadIdx.x & 31) == 0) warp_cnt[threadIdx.x >> 5] = miss;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long n_miss = 0, total = 0, before = 0;
        for (int w = 0; w < 32; ++w) n_miss += warp_cnt[w];
        for (int r = 0; r < world; ++r) { total += free_all[r]; before += r < rank ? free_all[r] : 0; }
        plan[0] = n_miss;
        plan[1] = n_miss > total ? n_miss - total : 0;
        plan[2] = before;
        plan[3] = free_all[rank];
    }
}

__global__ void free_slots_kernel(const long long *__restrict__ counters, long long capacity, long long *__restrict__ out) {
    out[0] = capacity - counters[CNT_OCCUPANCY];
}

}  // namespace

siso_status_t launch_shard_plan(const uint8_t *hit, int64_t n, const long long *free_all, int world, int rank, long long *plan,
                                cudaStream_t s) {
    shard_plan_kernel<<<1, 1024, 0, s>>>(hit, n, free_all, world, rank, plan);
    return check_cuda(cudaGetLastError(), "shard_plan_kernel");
}

siso_status_t launch_free_slots(Cache *c, long long *out, cudaStream_t s) {
    free_slots_kernel<<<1, 1, 0, s>>>(c->counters, c->capacity, out);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

siso_status_t launch_shard_route(const long long *idx, long long idx_stride, const uint8_t *hit, int64_t n, int64_t slot_lo,
                                 int64_t slot_hi, int64_t skip, int64_t take, int32_t *idx_local, uint8_t *upd_hit,
                                 uint8_t *ins_hit, cudaStream_t s, const long long *plan) {
    shard_route_kernel<<<1, 1024, 0, s>>>(idx, idx_stride, hit, n, slot_lo, slot_hi, skip, take, plan, idx_local, upd_hit, ins_hit);
    return check_cuda(cudaGetLastError(), "shard_route_kernel");
}

siso_status_t launch_shard_pack(Cache *c, const int32_t *idx, const float *sim, int64_t n, int64_t slot_offset,
                                unsigned long long *keys, cudaStream_t s) {
    shard_pack_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, s>>>(idx, sim, n, slot_offset, keys);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

siso_status_t launch_shard_combine(const unsigned long long *keys, int64_t n, int n_lists, int k, const float *theta,
                                   float theta_s, long long *idx, float *sim, uint8_t *hit, cudaStream_t s) {
    const unsigned blocks = static_cast<unsigned>((n + 7) / 8);
    if (k == 1) shard_combine_kernel<1><<<blocks, 256, 0, s>>>(keys, n, n_lists, k, theta, theta_s, idx, sim, hit);
    else if (k <= 4) shard_combine_kernel<4><<<blocks, 256, 0, s>>>(keys, n, n_lists, k, theta, theta_s, idx, sim, hit);
    else shard_combine_kernel<8><<<blocks, 256, 0, s>>>(keys, n, n_lists, k, theta, theta_s, idx, sim, hit);
    return check_cuda(cudaGetLastError(), "shard_combine_kernel");
}

}  // namespace siso
