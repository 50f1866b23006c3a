// Threshold control of Sec. 4.3: the threshold-to-hit-ratio (T2H) table and the M/D/1 waiting-time model.
//
// The table is one batched lookup of a sample of queries (k = 1, exact) followed by a counting kernel: for every
// threshold of the grid, how many sampled queries have a best similarity strictly above it.  The model (Eq. 1 with
// E = L (1 - h), i.e. Eq. 2) and the choice of the highest threshold that meets the SLO are scalar host arithmetic.
#include <cmath>

#include "common.cuh"

namespace siso {

constexpr int T2H_MAX_THETAS = 1024;

// grid = thresholds; one CTA counts over all queries
__global__ void __launch_bounds__(256)
t2h_count_kernel(const float *__restrict__ best, long long n, const float *__restrict__ thetas,
                 long long *__restrict__ hits) {
    __shared__ long long warp_cnt[8];
    const float th = thetas[blockIdx.x];
    long long c = 0;
    for (long long i = threadIdx.x; i < n; i += 256) c += (best[i] > th) ? 1 : 0;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
    if ((threadIdx.x & 31) == 0) warp_cnt[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long t = 0;
        for (int w = 0; w < 8; ++w) t += warp_cnt[w];
        hits[blockIdx.x] = t;
    }
}

}  // namespace siso

using namespace siso;

extern "C" {

siso_status_t siso_t2h(siso_cache_t *c, const void *d_queries, int64_t n_queries, const float *d_thetas,
                       int32_t n_thetas, int64_t *d_hits, void *stream) {
    Cache *cc = reinterpret_cast<Cache *>(c);
    if (!cc || n_queries < 1 || !d_queries || !d_thetas || !d_hits || n_thetas < 1) return SISO_ERR_INVALID_ARG;
    if (n_thetas > T2H_MAX_THETAS) return SISO_ERR_UNSUPPORTED;
    SISO_CUDA(cudaSetDevice(cc->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // results of the test lookups live in the staging buffer (the lookup itself uses the scratch buffer)
    const size_t ib = pad256(sizeof(int32_t) * n_queries), sb = pad256(sizeof(float) * n_queries), hb = pad256(n_queries);
    SISO_TRY(stage_reserve(cc, ib + sb + hb, s));
    char *p = static_cast<char *>(cc->stage);
    int32_t *idx = reinterpret_cast<int32_t *>(p);
    float *best = reinterpret_cast<float *>(p + ib);
    uint8_t *hit = reinterpret_cast<uint8_t *>(p + ib + sb);
    // a threshold of +infinity: these test lookups never count as hits in the cache statistics
    SISO_TRY(siso_lookup(c, d_queries, n_queries, nullptr, INFINITY, 1, idx, best, hit, stream));
    t2h_count_kernel<<<n_thetas, 256, 0, s>>>(best, n_queries, d_thetas, reinterpret_cast<long long *>(d_hits));
    SISO_LAUNCHED(cc);
    return SISO_OK;
}

double siso_md1_wait(double llm_latency, double arrival_rate, double hit_ratio) {
    const double e = llm_latency * (1.0 - hit_ratio);
    const double rho = arrival_rate * e;
    if (!(rho < 1.0)) return INFINITY;
    return e + arrival_rate * e * e / (2.0 * (1.0 - rho));
}

int32_t siso_choose_theta(const float *h_thetas, const double *h_hit_ratio, int32_t n_thetas, double llm_latency,
                          double arrival_rate, double slo, double *h_wait_out) {
    int32_t best = -1;
    double best_w = INFINITY;
    if (h_thetas && h_hit_ratio) {
        for (int32_t t = 0; t < n_thetas; ++t) {
            const double w = siso_md1_wait(llm_latency, arrival_rate, h_hit_ratio[t]);
            if (w < slo && (best < 0 || h_thetas[t] > h_thetas[best])) { best = t; best_w = w; }
        }
    }
    if (h_wait_out) *h_wait_out = best_w;
    return best;
}

int32_t siso_correct_theta(const float *h_thetas, int32_t n_thetas, int32_t chosen, double wait_estimated,
                           double wait_measured) {
    if (!h_thetas || chosen < 0 || chosen >= n_thetas || !(wait_measured > 0.0)) return chosen;
    if (std::fabs(wait_estimated - wait_measured) / wait_measured <= 0.10) return chosen;
    const bool lower = wait_measured > wait_estimated;     // the LLM is slower than modelled: send it less traffic
    int32_t next = -1;
    for (int32_t t = 0; t < n_thetas; ++t) {
        if (lower ? (h_thetas[t] < h_thetas[chosen]) : (h_thetas[t] > h_thetas[chosen])) {
            if (next < 0 || (lower ? h_thetas[t] > h_thetas[next] : h_thetas[t] < h_thetas[next])) next = t;
        }
    }
    return next < 0 ? chosen : next;
}

}  // extern "C"
