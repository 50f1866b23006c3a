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

}  // namespace

}  // namespace siso

using namespace siso;

extern "C" {

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
