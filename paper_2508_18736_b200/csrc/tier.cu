// Locality-ordered exact search: the exact-search counterpart of the placement of Sec. 4.3 ("Searching for vectors in
// semantic cache"), where centroids with strong semantic locality sit in the upper levels of the index so that most
// queries end their search there.
//
// The cache is held as two tiers: a small HOT tier (the entries FilteringCentroids would evict last: largest
// cluster_size, then access count) and the COLD rest.  Every query is scored against the hot tier first.  If its best
// hot similarity s exceeds an exit similarity derived from how far apart hot and cold entries are, no cold entry can
// reach s, and the query is finished: with unit vectors, angle(q, c) >= angle(h, c) - angle(q, h), so when every
// hot/cold pair has cos <= sep and angle(q, h) < acos(sep) / 2, every cold c is farther from q than h is.  Only the
// remaining queries are gathered into a dense batch and scored against the cold tier.  The result equals the plain
// top-1 over the whole cache.
//   select   which queries go on (best hot similarity <= exit_sim, or no hot entry), as an ascending row list
//   gather   those query rows into a dense batch
//   finish   per query the better of its hot and cold keys -> cache slot, similarity, strict threshold test
#include <cmath>

#include "common.cuh"

namespace siso {

namespace {

// one CTA; rows [n] receives the ascending indexes of the queries that go on to the cold tier, count[0] their number
__global__ void __launch_bounds__(1024)
tier_select_kernel(const unsigned long long *__restrict__ hot_keys, long long n, float exit_sim, int32_t *__restrict__ rows,
                   long long *__restrict__ count) {
    __shared__ int warp_cnt[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    long long base = 0;                                          // the same in every thread
    for (long long b0 = 0; b0 < n; b0 += 1024) {
        const long long b = b0 + tid;
        bool go = false;
        if (b < n) {
            const unsigned long long key = hot_keys[b];
            go = key == 0ull || !(key_sim(key) > exit_sim);
        }
        const unsigned int ballot = __ballot_sync(0xFFFFFFFFu, go);
        if (lane == 0) warp_cnt[warp] = __popc(ballot);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < 32; ++w) {
            const int c = warp_cnt[w];
            before += w < warp ? c : 0;
            total += c;
        }
        if (go) rows[base + before + __popc(ballot & ((1u << lane) - 1u))] = static_cast<int32_t>(b);
        base += total;
        __syncthreads();
    }
    if (tid == 0) count[0] = base;
}

// one warp per gathered row, 16 bytes per lane and step; the number of rows is read on the device
__global__ void __launch_bounds__(256)
tier_gather_kernel(const uint4 *__restrict__ src, const int32_t *__restrict__ rows, const long long *__restrict__ count,
                   int row_vec16, uint4 *__restrict__ dst) {
    const long long n = count[0];
    const int lane = threadIdx.x & 31;
    const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    for (long long i = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); i < n; i += warps) {
        const uint4 *s = src + static_cast<long long>(rows[i]) * row_vec16;
        uint4 *d = dst + i * row_vec16;
        for (int v = lane; v < row_vec16; v += 32) d[v] = s[v];
    }
}

// one thread per query that went on to the cold tier: the better of its hot and cold keys, ties to the lower cache slot
__global__ void __launch_bounds__(256)
tier_finish_kernel(const unsigned long long *__restrict__ hot_keys, long long n, const unsigned long long *__restrict__ cold_keys,
                   const int32_t *__restrict__ rows, long long n_cold, const int32_t *__restrict__ hot_slot,
                   const int32_t *__restrict__ cold_slot, const float *__restrict__ theta, float theta_s,
                   int32_t *__restrict__ idx, float *__restrict__ sim, uint8_t *__restrict__ hit) {
    const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t < n_cold) {
        const long long b = rows[t];
        const unsigned long long hk = hot_keys[b], ck = cold_keys[t];
        int32_t best_slot = -1;
        float best_sim = -INFINITY;
        if (hk) {
            best_slot = hot_slot ? hot_slot[key_slot(hk)] : key_slot(hk);
            best_sim = key_sim(hk);
        }
        if (ck) {
            const int32_t cs = cold_slot ? cold_slot[key_slot(ck)] : key_slot(ck);
            const float s = key_sim(ck);
            if (best_slot < 0 || s > best_sim || (s == best_sim && cs < best_slot)) {
                best_slot = cs;
                best_sim = s;
            }
        }
        idx[b] = best_slot;
        sim[b] = best_sim;
        hit[b] = (best_slot >= 0 && best_sim > (theta ? theta[b] : theta_s)) ? 1 : 0;
    }
}

// one thread per query; writes those that ended in the hot tier (the same test as tier_select_kernel)
__global__ void __launch_bounds__(256)
tier_finish_settled_kernel(const unsigned long long *__restrict__ hot_keys, long long n, float exit_sim,
                           const int32_t *__restrict__ hot_slot, const float *__restrict__ theta, float theta_s,
                           int32_t *__restrict__ idx, float *__restrict__ sim, uint8_t *__restrict__ hit) {
    const long long b = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (b >= n) return;
    const unsigned long long hk = hot_keys[b];
    if (hk == 0ull || !(key_sim(hk) > exit_sim)) return;         // went on to the cold tier: written by tier_finish_kernel
    const float s = key_sim(hk);
    idx[b] = hot_slot ? hot_slot[key_slot(hk)] : key_slot(hk);
    sim[b] = s;
    hit[b] = s > (theta ? theta[b] : theta_s) ? 1 : 0;
}

// ---- building the tiers ------------------------------------------------------------------------------------------
// cold[slot] = 1 for the slots named by the eviction keys (low 32 bits of a key's third word)
__global__ void tier_mark_cold_kernel(const unsigned long long *__restrict__ keys, long long n, long long capacity,
                                      uint32_t *__restrict__ cold) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const unsigned long long w2 = keys[3 * i + 2];
    if (keys[3 * i] == ~0ull && w2 == ~0ull) return;              // padding: fewer live entries than asked for
    const long long slot = static_cast<long long>(w2 & 0xFFFFFFFFull);
    if (slot < capacity) cold[slot] = 1u;
}

// hot[slot] = live and not cold; both arrays have capacity + 1 places (the last one 0) for the scans that follow
__global__ void tier_flags_kernel(const uint8_t *__restrict__ valid, long long capacity, const uint32_t *__restrict__ cold,
                                  uint32_t *__restrict__ hot) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i > capacity) return;
    hot[i] = (i < capacity && valid[i] && !cold[i]) ? 1u : 0u;
}

// One CTA per slot of the source cache: the entry goes to place pos[slot] of its tier (ascending slot order), with its
// vectors (lookup copy and fp32 master) and its metadata; `list` receives the source slot of every place.
template <typename T>
__global__ void __launch_bounds__(128)
tier_copy_kernel(const uint32_t *__restrict__ flag_pos, const uint8_t *__restrict__ valid, const uint32_t *__restrict__ cold,
                 int want_cold, int D, const T *__restrict__ src_vecs, const float *__restrict__ src_master,
                 const double *__restrict__ src_size, const uint32_t *__restrict__ src_access,
                 const unsigned long long *__restrict__ src_last, T *__restrict__ dst_vecs, float *__restrict__ dst_master,
                 double *__restrict__ dst_size, uint32_t *__restrict__ dst_access, unsigned long long *__restrict__ dst_last,
                 uint8_t *__restrict__ dst_valid, int32_t *__restrict__ list) {
    const long long slot = blockIdx.x;
    const bool is_cold = cold[slot] != 0u;
    if (!valid[slot] || is_cold != (want_cold != 0)) return;
    const long long at = flag_pos[slot];
    const float4 *sm = reinterpret_cast<const float4 *>(src_master + slot * D);
    float4 *dm = reinterpret_cast<float4 *>(dst_master + at * D);
    for (int q = threadIdx.x; q < D / 4; q += blockDim.x) dm[q] = sm[q];
    if constexpr (sizeof(T) == 2) {
        const uint4 *sv = reinterpret_cast<const uint4 *>(src_vecs + slot * D);
        uint4 *dv = reinterpret_cast<uint4 *>(dst_vecs + at * D);
        for (int q = threadIdx.x; q < D / 8; q += blockDim.x) dv[q] = sv[q];
    }
    if (threadIdx.x == 0) {
        dst_size[at] = src_size[slot];
        dst_access[at] = src_access[slot];
        dst_last[at] = src_last[slot];
        dst_valid[at] = 1;
        list[at] = static_cast<int32_t>(slot);
    }
}

__global__ void tier_counters_kernel(const uint32_t *__restrict__ hot_pos, const uint32_t *__restrict__ cold_pos, long long capacity,
                                     const long long *__restrict__ src_counters, long long *hot_counters, long long *cold_counters,
                                     long long *out2) {
    const long long n_hot = hot_pos[capacity], n_cold = cold_pos[capacity];
    hot_counters[CNT_OCCUPANCY] = n_hot;
    cold_counters[CNT_OCCUPANCY] = n_cold;
    hot_counters[CNT_CLOCK] = cold_counters[CNT_CLOCK] = src_counters[CNT_CLOCK];
    out2[0] = n_hot;
    out2[1] = n_cold;
}

}  // namespace

}  // namespace siso

using namespace siso;

extern "C" {

siso_status_t siso_tier_build(siso_cache_t *cache_h, int64_t hot_rows, double sep_sim, siso_cache_t *hot_h, siso_cache_t *cold_h,
                              int32_t *d_hot_slot, int32_t *d_cold_slot, int64_t *h_counts, void *stream) {
    Cache *c = reinterpret_cast<Cache *>(cache_h), *hot = reinterpret_cast<Cache *>(hot_h), *cold = reinterpret_cast<Cache *>(cold_h);
    if (!c || !hot || !cold || hot == cold || hot == c || cold == c || hot_rows < 0 || !d_hot_slot || !d_cold_slot || !h_counts)
        return SISO_ERR_INVALID_ARG;
    if (hot->dim != c->dim || cold->dim != c->dim || hot->dtype != c->dtype || cold->dtype != c->dtype ||
        hot->device != c->device || cold->device != c->device)
        return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    long long occ = 0;
    SISO_CUDA(cudaMemcpyAsync(&occ, c->counters + CNT_OCCUPANCY, sizeof(occ), cudaMemcpyDeviceToHost, s));
    SISO_CUDA(cudaStreamSynchronize(s));
    const int64_t n_hot = std::min<int64_t>(hot_rows, occ), n_cold = occ - n_hot;
    if (n_hot > hot->capacity || n_cold > cold->capacity) return SISO_ERR_CAPACITY;
    const int64_t cap = c->capacity;
    // the lists and flags live in the HOT tier's scratch (the source cache's own scratch serves its eviction-order selection)
    Scratch scr;
    SISO_TRY(scratch_reserve(hot, 2 * pad256(sizeof(uint32_t) * (cap + 1)) + pad256(sizeof(unsigned long long) * 3 * std::max<int64_t>(n_cold, 1)) +
                                      pad256(2 * sizeof(long long)) + 256, s, &scr));
    uint32_t *cold_pos = scr.take<uint32_t>(cap + 1), *hot_pos = scr.take<uint32_t>(cap + 1);
    unsigned long long *keys = scr.take<unsigned long long>(3 * std::max<int64_t>(n_cold, 1));
    long long *d_out2 = scr.take<long long>(2);
    SISO_CUDA(cudaMemsetAsync(cold_pos, 0, sizeof(uint32_t) * (cap + 1), s));
    if (n_cold > 0) {
        // the cold tier = what FilteringCentroids would remove to leave n_hot entries (nothing is removed here)
        SISO_TRY(launch_evict_keys(c, n_cold, 0, keys, s));
        tier_mark_cold_kernel<<<static_cast<unsigned>((n_cold + 255) / 256), 256, 0, s>>>(keys, n_cold, cap, cold_pos);
        SISO_LAUNCHED(c);
    }
    const unsigned nblk = static_cast<unsigned>((cap + 1 + 255) / 256);
    tier_flags_kernel<<<nblk, 256, 0, s>>>(c->valid, cap, cold_pos, hot_pos);
    SISO_LAUNCHED(c);
    // cold flags are still needed as flags by the copy: scan a copy of them
    uint32_t *cold_flag = cold_pos;
    Scratch scr2;
    SISO_TRY(scratch_reserve(cold, pad256(sizeof(uint32_t) * (cap + 1)) + 256, s, &scr2));
    uint32_t *cold_scan = scr2.take<uint32_t>(cap + 1);
    SISO_CUDA(cudaMemcpyAsync(cold_scan, cold_flag, sizeof(uint32_t) * (cap + 1), cudaMemcpyDeviceToDevice, s));
    SISO_TRY(launch_exclusive_scan_u32(c, cold_scan, cap + 1, s));
    SISO_TRY(launch_exclusive_scan_u32(c, hot_pos, cap + 1, s));
    for (Cache *t : {hot, cold}) {
        SISO_CUDA(cudaMemsetAsync(t->valid, 0, static_cast<size_t>(t->rows_alloc), s));
        SISO_CUDA(cudaMemsetAsync(t->counters, 0, sizeof(long long) * CNT_N, s));
        t->vec_epoch += 1;
        t->low_dirty = true;
    }
    for (int want_cold = 0; want_cold < 2; ++want_cold) {
        Cache *t = want_cold ? cold : hot;
        const uint32_t *pos = want_cold ? cold_scan : hot_pos;
        int32_t *list = want_cold ? d_cold_slot : d_hot_slot;
        if (c->dtype == SISO_F32)
            tier_copy_kernel<float><<<static_cast<unsigned>(cap), 128, 0, s>>>(
                pos, c->valid, cold_flag, want_cold, c->dim, static_cast<const float *>(c->vecs), c->master, c->size, c->access, c->last,
                static_cast<float *>(t->vecs), t->master, t->size, t->access, t->last, t->valid, list);
        else
            tier_copy_kernel<__nv_bfloat16><<<static_cast<unsigned>(cap), 128, 0, s>>>(
                pos, c->valid, cold_flag, want_cold, c->dim, static_cast<const __nv_bfloat16 *>(c->vecs), c->master, c->size, c->access,
                c->last, static_cast<__nv_bfloat16 *>(t->vecs), t->master, t->size, t->access, t->last, t->valid, list);
        SISO_LAUNCHED(c);
    }
    tier_counters_kernel<<<1, 1, 0, s>>>(hot_pos, cold_scan, cap, c->counters, hot->counters, cold->counters, d_out2);
    SISO_LAUNCHED(c);
    long long out2[2] = {0, 0};
    SISO_CUDA(cudaMemcpyAsync(out2, d_out2, sizeof(out2), cudaMemcpyDeviceToHost, s));
    SISO_CUDA(cudaStreamSynchronize(s));
    h_counts[0] = out2[0];
    h_counts[1] = out2[1];
    h_counts[2] = -1;
    // the exit rule rests on every hot/cold pair being at most sep_sim similar: count the pairs above it (exact fp64
    // similarities of the vectors that lookups read) with the block sweep of the sharded MergeCentroids, hot tier as the peer block
    if (sep_sim == sep_sim && out2[0] > 0 && out2[1] > 0) {
        Scratch scr3;
        SISO_TRY(scratch_reserve(hot, pad256(12 * 64) + pad256(sizeof(long long)) + 256, s, &scr3));
        int32_t *cand = scr3.take<int32_t>(3 * 64);
        long long *n_cand = scr3.take<long long>(1);
        SISO_CUDA(cudaMemsetAsync(n_cand, 0, sizeof(long long), s));
        SISO_TRY(launch_pair_sweep_block(cold, 0, hot->vecs, hot->valid, out2[0], cold->capacity, static_cast<float>(sep_sim), cand, 64,
                                         reinterpret_cast<int64_t *>(n_cand), true, s));
        long long above = 0;
        SISO_CUDA(cudaMemcpyAsync(&above, n_cand, sizeof(above), cudaMemcpyDeviceToHost, s));
        SISO_CUDA(cudaStreamSynchronize(s));
        // more than 64 such pairs leave SISO_ERR_OVERFLOW in the cold tier's status word: the count is what matters here
        int discard = 0;
        SISO_CUDA(cudaMemcpyAsync(&discard, cold->status, sizeof(int), cudaMemcpyDeviceToHost, s));
        SISO_CUDA(cudaMemsetAsync(cold->status, 0, sizeof(int), s));
        SISO_CUDA(cudaStreamSynchronize(s));
        if (discard != 0 && discard != SISO_ERR_OVERFLOW) return static_cast<siso_status_t>(discard);
        h_counts[2] = discard == SISO_ERR_OVERFLOW ? std::max<long long>(above, 65) : above;
    }
    return SISO_OK;
}

int64_t siso_tier_work_bytes(int64_t n_queries, int32_t dim, int32_t dtype) {
    if (n_queries < 0 || dim < 1) return 0;
    const size_t row = static_cast<size_t>(dim) * (dtype == SISO_F32 ? 4 : 2);
    return static_cast<int64_t>(2 * pad256(sizeof(uint64_t) * n_queries) + pad256(sizeof(int32_t) * n_queries) +
                                pad256(row * n_queries) + 256);
}

siso_status_t siso_tier_lookup(siso_cache_t *hot, siso_cache_t *cold, const int32_t *d_hot_slot, const int32_t *d_cold_slot,
                               const void *d_queries, int64_t n_queries, float exit_sim, const float *d_theta, float theta_scalar,
                               void *d_work, int32_t *d_idx, float *d_sim, uint8_t *d_hit, int64_t *h_settled, void *stream) {
    if (!hot || !cold || n_queries < 0) return SISO_ERR_INVALID_ARG;
    if (n_queries == 0) { if (h_settled) *h_settled = 0; return SISO_OK; }
    if (!d_queries || !d_work || !d_idx || !d_sim || !d_hit || (reinterpret_cast<uintptr_t>(d_work) & 255u)) return SISO_ERR_INVALID_ARG;
    Cache *h = reinterpret_cast<Cache *>(hot), *c = reinterpret_cast<Cache *>(cold);
    if (h->dim != c->dim || h->dtype != c->dtype || h->device != c->device) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(h->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t row = static_cast<size_t>(h->dim) * (h->dtype == SISO_F32 ? 4 : 2);
    char *p = static_cast<char *>(d_work);
    uint64_t *hk = reinterpret_cast<uint64_t *>(p); p += pad256(sizeof(uint64_t) * n_queries);
    uint64_t *ck = reinterpret_cast<uint64_t *>(p); p += pad256(sizeof(uint64_t) * n_queries);
    int32_t *rows = reinterpret_cast<int32_t *>(p); p += pad256(sizeof(int32_t) * n_queries);
    void *packed = p; p += pad256(row * n_queries);
    int64_t *count = reinterpret_cast<int64_t *>(p);
    // the whole batch against the hot tier; the queries that may still find something better go on, packed
    SISO_TRY(siso_lookup_keys(hot, d_queries, n_queries, 1, 0, hk, stream));
    SISO_TRY(siso_tier_select(hk, n_queries, exit_sim, d_queries, static_cast<int64_t>(row), packed, rows, count, stream));
    long long n_go = 0;                              // one 8-byte read sizes the cold tier's sweep
    SISO_CUDA(cudaMemcpyAsync(&n_go, count, sizeof(n_go), cudaMemcpyDeviceToHost, s));
    SISO_CUDA(cudaStreamSynchronize(s));
    if (n_go > 0) SISO_TRY(siso_lookup_keys(cold, packed, n_go, 1, 0, ck, stream));
    if (h_settled) *h_settled = n_queries - n_go;
    return siso_tier_finish(hk, n_queries, exit_sim, ck, rows, n_go, d_hot_slot, d_cold_slot, d_theta, theta_scalar, d_idx, d_sim,
                            d_hit, stream);
}

double siso_tier_exit_sim(double sep_sim, double norm_slack) {
    // Vectors (queries and entries) have norms in [1 - d, 1 + d]; every hot/cold pair has dot product <= sep.
    // With s = <q, h>: cos(angle(q, h)) >= s / (1 + d)^2 and cos(angle(h, c)) <= sep / (1 - d)^2 =: g, so
    // <q, c> <= (1 + d)^2 cos(acos(g) - acos(s / (1 + d)^2)) while that difference of angles is positive.  The exit
    // similarity is the smallest s above which this bound stays below s (found by bisection; the bound falls and s
    // rises), plus 1e-5 for the rounding of the computed similarities themselves.
    if (!(norm_slack >= 0.0) || !(norm_slack < 0.25) || !(sep_sim == sep_sim)) return INFINITY;
    const double up = (1.0 + norm_slack) * (1.0 + norm_slack), dn = (1.0 - norm_slack) * (1.0 - norm_slack);
    const double g = (sep_sim > 0.0 ? sep_sim : 0.0) / dn;
    if (!(g < 1.0)) return INFINITY;
    const double beta = std::acos(g);
    auto safe = [&](double s) {
        const double ca = s / up;
        if (!(ca > 0.0)) return false;
        const double alpha = std::acos(ca < 1.0 ? ca : 1.0);
        const double gap = beta - alpha;
        if (!(gap > alpha)) return false;                         // needs angle(q, c) > angle(q, h) with room to spare
        return up * std::cos(gap) < s;
    };
    double lo = 0.0, hi = up;
    if (!safe(hi)) return INFINITY;
    for (int it = 0; it < 80; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (safe(mid)) hi = mid; else lo = mid;
    }
    return hi + 1e-5;
}

siso_status_t siso_tier_select(const uint64_t *d_hot_keys, int64_t n_queries, float exit_sim, const void *d_queries,
                               int64_t row_bytes, void *d_cold_queries, int32_t *d_rows, int64_t *d_count, void *stream) {
    if (n_queries < 0 || row_bytes <= 0 || row_bytes % 16 != 0 || n_queries > 0x7FFFFFFFll) return SISO_ERR_INVALID_ARG;
    if (!d_count) return SISO_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n_queries == 0) return check_cuda(cudaMemsetAsync(d_count, 0, sizeof(int64_t), s), "tier_select count");
    if (!d_hot_keys || !d_queries || !d_cold_queries || !d_rows) return SISO_ERR_INVALID_ARG;
    tier_select_kernel<<<1, 1024, 0, s>>>(reinterpret_cast<const unsigned long long *>(d_hot_keys), n_queries, exit_sim, d_rows,
                                          reinterpret_cast<long long *>(d_count));
    const unsigned blocks = static_cast<unsigned>(std::min<int64_t>((n_queries + 7) / 8, 148 * 8));
    tier_gather_kernel<<<blocks, 256, 0, s>>>(static_cast<const uint4 *>(d_queries), d_rows,
                                              reinterpret_cast<const long long *>(d_count), static_cast<int>(row_bytes / 16),
                                              static_cast<uint4 *>(d_cold_queries));
    return check_cuda(cudaGetLastError(), "tier_select");
}

siso_status_t siso_tier_finish(const uint64_t *d_hot_keys, int64_t n_queries, float exit_sim, const uint64_t *d_cold_keys,
                               const int32_t *d_rows, int64_t n_cold, const int32_t *d_hot_slot, const int32_t *d_cold_slot,
                               const float *d_theta, float theta_scalar, int32_t *d_idx, float *d_sim, uint8_t *d_hit,
                               void *stream) {
    if (n_queries < 0 || n_cold < 0 || n_cold > n_queries) return SISO_ERR_INVALID_ARG;
    if (n_queries == 0) return SISO_OK;
    if (!d_hot_keys || !d_idx || !d_sim || !d_hit || (n_cold > 0 && (!d_cold_keys || !d_rows))) return SISO_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const unsigned long long *hk = reinterpret_cast<const unsigned long long *>(d_hot_keys);
    tier_finish_settled_kernel<<<static_cast<unsigned>((n_queries + 255) / 256), 256, 0, s>>>(hk, n_queries, exit_sim, d_hot_slot,
                                                                                              d_theta, theta_scalar, d_idx, d_sim, d_hit);
    if (n_cold > 0)
        tier_finish_kernel<<<static_cast<unsigned>((n_cold + 255) / 256), 256, 0, s>>>(
            hk, n_queries, reinterpret_cast<const unsigned long long *>(d_cold_keys), d_rows, n_cold, d_hot_slot, d_cold_slot,
            d_theta, theta_scalar, d_idx, d_sim, d_hit);
    return check_cuda(cudaGetLastError(), "tier_finish");
}

}  // extern "C"
