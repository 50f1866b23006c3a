// Large-batch lookup of fp32 caches on the tensor cores (FindClosestCentroid of Algorithm 1 as a dense contraction).
//
// fp32 inputs cannot go through TF32 under a 1e-5 tolerance.  Queries and centroids are split as x = hi + lo + r with
// hi = bf16(x), lo = bf16(x - hi), and the sweep accumulates hi.hi + hi.lo + lo.hi in fp32 on tcgen05 (three MMAs per
// 16 K-elements); what is left out stays below 6e-5 for unit vectors.  The sweep therefore SELECTS, it does not
// decide: every (query, centroid split) keeps its 8 best approximate similarities, lookup_rescore_kernel recomputes
// all rows on a query's lists exactly (fp64 sums of the fp32 values) and returns the k <= 4 best; the answer is
// accepted only if the k-th exact similarity exceeds the last entry of every full list by more than 6e-5, which
// proves that no row outside the lists can belong to the top k.  A query that fails the test (one split holds more
// than 8 - k rows within the margin of the k-th best) is looked up again by a plain exact scan
// (lookup_rescan_kernel).  The results are those of an exact sweep.
//
// The sweep kernel is the CTA-pair kernel of the bf16 lookup with four operand tiles per stage (64 KiB, three
// stages) and three MMAs per K step; see lookup_tensor_pair.cu for the roles and barriers.
#include <cuda.h>

#include <cmath>
#include <cstring>

#include "umma_pair.cuh"

namespace siso {
namespace tc3 {

constexpr int TM = 128;             // queries per CTA
constexpr int TN = 256;             // centroids per tile (both CTAs together stage them, 128 rows each)
constexpr int TK = 64;
constexpr int STAGES = 3;
constexpr int ACC_STAGES = 2;
constexpr int THREADS = 192;
constexpr uint32_t OPER_BYTES = TM * TK * 2;         // 16 KiB: 128 rows x 64 bf16
constexpr uint32_t STAGE_BYTES = 4 * OPER_BYTES;     // q hi, q lo, this CTA's half of the centroid tile hi and lo
constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256;
constexpr uint32_t TMEM_COLS = ACC_STAGES * TN;

using namespace umma2;

// D fp32, A and B bf16, K-major, N = 256, M = 256 (128 rows per CTA of the pair)
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(TN >> 3) << 17) |
                           (static_cast<uint32_t>((2 * TM) >> 4) << 24);

struct Barriers {
    uint64_t full[STAGES], empty[STAGES], acc_full[ACC_STAGES], acc_empty[ACC_STAGES];
    uint32_t tmem_base;
    int abort_flag;
};

template <int KMAX>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
lookup_tensor_split_kernel(const __grid_constant__ CUtensorMap map_q_hi, const __grid_constant__ CUtensorMap map_q_lo,
                           const __grid_constant__ CUtensorMap map_c_hi, const __grid_constant__ CUtensorMap map_c_lo,
                           const uint8_t *__restrict__ valid, int64_t B, int D, int tiles_per_split, int n_tiles,
                           unsigned long long *__restrict__ partial, int splits, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    Barriers *bars = reinterpret_cast<Barriers *>(tiles + STAGES * STAGE_BYTES);
    volatile int *abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();              // 0 = leader
    const int split = blockIdx.y;
    const int q0 = blockIdx.x * TM;                    // this CTA's own 128 queries
    const int t_begin = split * tiles_per_split;
    const int t_end = min(n_tiles, t_begin + tiles_per_split);
    const int k_slabs = (D + TK - 1) / TK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        for (int a = 0; a < ACC_STAGES; ++a) { mbar_init(&bars->acc_full[a], 1); mbar_init(&bars->acc_empty[a], 8); }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // the same warp of both CTAs allocates the pair's tensor memory (512 columns in each)
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&bars->tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync();                                    // both CTAs' barriers are initialised before any remote use
    tcgen05_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int t = t_begin; t < t_end && ok; ++t) {
                const int n0 = t * TN + static_cast<int>(rank) * (TN / 2);     // this CTA's half of the centroid tile
                for (int ks = 0; ks < k_slabs; ++ks) {
                    if (!mbar_wait(&bars->empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t *dst = tiles + stage * STAGE_BYTES;
                    const uint32_t full_leader = cluster_addr(smem_u32(&bars->full[stage]), 0);
                    if (rank == 0) mbar_arrive_expect_tx(&bars->full[stage], 2 * STAGE_BYTES);   // both CTAs' bytes
                    tma_load_2d_pair(dst, &map_q_hi, ks * TK, q0, full_leader);
                    tma_load_2d_pair(dst + OPER_BYTES, &map_q_lo, ks * TK, q0, full_leader);
                    tma_load_2d_pair(dst + 2 * OPER_BYTES, &map_c_hi, ks * TK, n0, full_leader);
                    tma_load_2d_pair(dst + 3 * OPER_BYTES, &map_c_lo, ks * TK, n0, full_leader);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader only)
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int t = t_begin; t < t_end && ok; ++t) {
                if (!mbar_wait(&bars->acc_empty[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + acc * TN;
                for (int ks = 0; ks < k_slabs; ++ks) {
                    if (!mbar_wait(&bars->full[stage], phase, abort_flag)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t base = smem_u32(tiles + stage * STAGE_BYTES);
                    const uint64_t q_hi = smem_desc_sw128(base), q_lo = smem_desc_sw128(base + OPER_BYTES);
                    const uint64_t c_hi = smem_desc_sw128(base + 2 * OPER_BYTES), c_lo = smem_desc_sw128(base + 3 * OPER_BYTES);
#pragma unroll
                    for (int kk = 0; kk < TK / 16; ++kk) {
                        const uint64_t o = static_cast<uint64_t>(2 * kk);
                        umma_bf16_pair(d_tmem, q_hi + o, c_hi + o, IDESC, (ks | kk) ? 1u : 0u);
                        umma_bf16_pair(d_tmem, q_hi + o, c_lo + o, IDESC, 1u);
                        umma_bf16_pair(d_tmem, q_lo + o, c_hi + o, IDESC, 1u);
                    }
                    // stage reusable in BOTH CTAs once these MMAs have read it
                    umma_commit_both(&bars->empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit_both(&bars->acc_full[acc]);
                if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5 of both CTAs)
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        TopK<KMAX> top;
        top.clear();
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int t = t_begin; t < t_end && ok; ++t) {
            const int n0 = t * TN;
            // live flags of the tile's 256 slots (lane l holds slots l, l+32, ...): fetched before the wait
            unsigned long long vflags = 0ull;       // bit ch: slot n0 + 32*ch + lane is live
#pragma unroll
            for (int ch = 0; ch < TN / 32; ++ch)
                vflags |= static_cast<unsigned long long>(valid[static_cast<int64_t>(n0) + ch * 32 + lane] != 0) << ch;
            if (!mbar_wait(&bars->acc_full[acc], acc_phase, abort_flag)) { ok = false; break; }
            tcgen05_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * TN;
            drain_accumulator<KMAX, TN>(taddr, vflags, n0, top);
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(cluster_addr(smem_u32(&bars->acc_empty[acc]), 0));
            if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
        }
        if (ok && static_cast<int64_t>(q0) + row < B) {
            unsigned long long *dst = partial + ((static_cast<int64_t>(q0) + row) * splits + split) * KMAX;
#pragma unroll
            for (int j = 0; j < KMAX; ++j) dst[j] = top.key(j);
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        if (threadIdx.x == 0) set_status(status, SISO_ERR_TIMEOUT);
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync();          // neither CTA frees tensor memory or exits while the other may still use its memory
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

constexpr int CAND = 8;                   // approximate best matches kept per query and split
// bound on |approximate - exact| for norms up to 1.002: bf16 keeps 8 significant bits, u = 2^-8, so |x - hi| <= u |x| and
// |x - hi - lo| <= u^2 |x|; left out are lo.lo (<= u^2) and the two remainder terms (<= 2 u^2): 3 u^2 = 4.6e-5; the fp32
// accumulator is rounded once per 16 K-elements (dim / 16 roundings of 2^-23 of a sum below 1: 7.6e-6 at dim 1024)
constexpr double ACCEPT_MARGIN = 6e-5;

// exact similarity of query row q and centroid row c (fp64 sums of the fp32 values): this lane's share of a group of
// 8 lanes, then the sum over the group (to be called by all lanes of the warp together)
__device__ __forceinline__ double dot_share_of_8(const float4 *__restrict__ q, const float4 *__restrict__ c, int quads, int sub) {
    double acc = 0.0;
    for (int t = sub; t < quads; t += 8) {
        const float4 x = __ldg(q + t), y = __ldg(c + t);
        acc += static_cast<double>(x.x) * static_cast<double>(y.x) + static_cast<double>(x.y) * static_cast<double>(y.y) +
               static_cast<double>(x.z) * static_cast<double>(y.z) + static_cast<double>(x.w) * static_cast<double>(y.w);
    }
    return acc;
}
__device__ __forceinline__ double sum_over_8_lanes(double acc) {
#pragma unroll
    for (int o = 4; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    return acc;
}

// (v, sl) into a list of 4 ordered by similarity descending, slot ascending; empty places have slot -1
__device__ __forceinline__ void insert_best4(double (&best)[4], int32_t (&best_slot)[4], double v, int32_t sl) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const bool before = sl >= 0 && (best_slot[j] < 0 || v > best[j] || (v == best[j] && sl < best_slot[j]));
        if (before) {
            const double tv = best[j]; best[j] = v; v = tv;
            const int32_t ts = best_slot[j]; best_slot[j] = sl; sl = ts;
        }
    }
}

// One warp per query: the rows on the query's per-split lists (up to CAND per split) again, exactly; the k best of them
// are the answer if the k-th beats, by more than the margin, the last entry of every FULL list: a row that is on no
// list scored at most that entry approximately, so it cannot reach the top k.  Otherwise the query is passed on to
// the exact scan.  Rows whose approximate similarity lies more than two margins below the k-th approximate one cannot
// be among the k best and are not recomputed.  Four rows at a time, eight lanes each.
__global__ void __launch_bounds__(256)
lookup_rescore_kernel(const float *__restrict__ Q, const float *__restrict__ C, int64_t B, int D, int k, int splits,
                      const unsigned long long *__restrict__ partial, const float *__restrict__ theta, float theta_s,
                      int32_t *__restrict__ idx, float *__restrict__ sim, uint8_t *__restrict__ hit,
                      int32_t *__restrict__ flagged, unsigned int *__restrict__ n_flagged, long long *counters) {
    const int lane = threadIdx.x & 31, group = lane >> 3, sub = lane & 7;
    const int64_t b = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (blockIdx.x == 0 && threadIdx.x == 0)
        atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_LOOKUPS), static_cast<unsigned long long>(B));
    if (b >= B) return;
    const float4 *q = reinterpret_cast<const float4 *>(Q + b * D);
    const unsigned long long *lists = partial + b * splits * CAND;
    const int n_keys = splits * CAND;
    // the k-th largest approximate similarity over all lists, and the largest last entry of a full list
    KeyList<4> top;
    top.clear();
    float bound_f = -2.0f;
    for (int e = lane; e < n_keys; e += 32) {
        const unsigned long long key = lists[e];
        top.insert(key);
        if (key != 0ull && (e % CAND) == CAND - 1) bound_f = fmaxf(bound_f, key_sim(key));
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        unsigned long long other[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) other[j] = __shfl_xor_sync(0xFFFFFFFFu, top.k[j], o);
#pragma unroll
        for (int j = 0; j < 4; ++j) top.insert(other[j]);
        bound_f = fmaxf(bound_f, __shfl_xor_sync(0xFFFFFFFFu, bound_f, o));
    }
    unsigned long long kth_key = 0ull;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (j == k - 1) kth_key = top.k[j];
    const float cutoff = kth_key ? key_sim(kth_key) - static_cast<float>(2.0 * ACCEPT_MARGIN) - 1e-6f : -2.0f;
    double best[4];                        // the same in all lanes
    int32_t best_slot[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) { best[j] = 0.0; best_slot[j] = -1; }
    for (int e0 = 0; e0 < n_keys; e0 += 4) {
        const int e = e0 + group;
        const unsigned long long key = e < n_keys ? lists[e] : 0ull;
        const bool take = key != 0ull && key_sim(key) >= cutoff;
        if (!__any_sync(0xFFFFFFFFu, take)) continue;
        const int32_t slot = take ? key_slot(key) : -1;
        double v = 0.0;
        if (take) v = dot_share_of_8(q, reinterpret_cast<const float4 *>(C + static_cast<int64_t>(slot) * D), D / 4, sub);
        v = sum_over_8_lanes(v);
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const double vg = __shfl_sync(0xFFFFFFFFu, v, g * 8);
            const int32_t sg = __shfl_sync(0xFFFFFFFFu, slot, g * 8);
            insert_best4(best, best_slot, vg, sg);
        }
    }
    if (lane != 0) return;
    double kth = 0.0;
    int32_t kth_slot = -1;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (j == k - 1) { kth = best[j]; kth_slot = best_slot[j]; }
    // a full list exists only if its split has at least CAND live rows
    if (bound_f > -2.0f && !(kth_slot >= 0 && kth > static_cast<double>(bound_f) + ACCEPT_MARGIN)) {
        flagged[atomicAdd(n_flagged, 1u)] = static_cast<int32_t>(b);
        atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_RESCANS), 1ull);
        return;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (j < k) {
            idx[b * k + j] = best_slot[j];
            sim[b * k + j] = best_slot[j] >= 0 ? static_cast<float>(best[j]) : -INFINITY;
        }
    }
    const float th = theta ? theta[b] : theta_s;
    const int is_hit = (best_slot[0] >= 0 && best[0] > static_cast<double>(th)) ? 1 : 0;
    hit[b] = static_cast<uint8_t>(is_hit);
    if (is_hit) atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_HITS), 1ull);
}

// The queries the rescoring could not settle: an exact scan of all live rows.  CTA c scans its share of the rows for
// every such query (four rows at a time per warp, eight lanes each) and leaves its 4 best as packed keys;
// lookup_rescan_finish_kernel combines the CTAs' lists.
__global__ void __launch_bounds__(256)
lookup_rescan_kernel(const float *__restrict__ Q, const float *__restrict__ C, const uint8_t *__restrict__ valid, int64_t N, int D,
                     const int32_t *__restrict__ flagged, const unsigned int *__restrict__ n_flagged,
                     unsigned long long *__restrict__ rescan_keys /* [n_flagged, gridDim.x, 4] */) {
    __shared__ unsigned long long lists[8][4];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, group = lane >> 3, sub = lane & 7;
    const unsigned int n = *n_flagged;
    const int64_t per = (N + gridDim.x - 1) / gridDim.x;
    const int64_t r_lo = min(N, static_cast<int64_t>(blockIdx.x) * per), r_hi = min(N, r_lo + per);
    for (unsigned int f = 0; f < n; ++f) {
        const float4 *q = reinterpret_cast<const float4 *>(Q + static_cast<int64_t>(flagged[f]) * D);
        KeyList<4> best;
        best.clear();
        for (int64_t r0 = r_lo + warp * 4; r0 < r_hi; r0 += 32) {
            const int64_t r = r0 + group;
            const bool live = r < r_hi && valid[r] != 0;
            double v = 0.0;
            if (live) v = dot_share_of_8(q, reinterpret_cast<const float4 *>(C + r * D), D / 4, sub);
            v = sum_over_8_lanes(v);
            const unsigned long long key = live ? pack_key(static_cast<float>(v), static_cast<uint32_t>(r)) : 0ull;
#pragma unroll
            for (int g = 0; g < 4; ++g) best.insert(__shfl_sync(0xFFFFFFFFu, key, g * 8));
        }
        __syncthreads();
        if (lane == 0)
            for (int j = 0; j < 4; ++j) lists[warp][j] = best.k[j];
        __syncthreads();
        if (threadIdx.x == 0) {
            KeyList<4> all;
            all.clear();
            for (int w = 0; w < 8; ++w)
                for (int j = 0; j < 4; ++j) all.insert(lists[w][j]);
            unsigned long long *dst = rescan_keys + (static_cast<size_t>(f) * gridDim.x + blockIdx.x) * 4;
            for (int j = 0; j < 4; ++j) dst[j] = all.k[j];
        }
    }
}

// one warp per rescanned query
__global__ void __launch_bounds__(256)
lookup_rescan_finish_kernel(const unsigned long long *__restrict__ rescan_keys, int n_lists, int k,
                            const int32_t *__restrict__ flagged, const unsigned int *__restrict__ n_flagged,
                            const float *__restrict__ theta, float theta_s, int32_t *__restrict__ idx, float *__restrict__ sim,
                            uint8_t *__restrict__ hit, long long *counters) {
    const int lane = threadIdx.x & 31;
    const unsigned int n = *n_flagged;
    for (unsigned int f = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); f < n; f += gridDim.x * (blockDim.x >> 5)) {
        KeyList<4> all;
        all.clear();
        const unsigned long long *src = rescan_keys + static_cast<size_t>(f) * n_lists * 4;
        for (int e = lane; e < n_lists * 4; e += 32) all.insert(src[e]);
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            unsigned long long other[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) other[j] = __shfl_xor_sync(0xFFFFFFFFu, all.k[j], o);
#pragma unroll
            for (int j = 0; j < 4; ++j) all.insert(other[j]);
        }
        if (lane == 0) {
            const int64_t b = flagged[f];
            for (int j = 0; j < k; ++j) {
                idx[b * k + j] = all.k[j] ? key_slot(all.k[j]) : -1;
                sim[b * k + j] = all.k[j] ? key_sim(all.k[j]) : -INFINITY;
            }
            const float th = theta ? theta[b] : theta_s;
            const int is_hit = (all.k[0] != 0ull && key_sim(all.k[0]) > th) ? 1 : 0;
            hit[b] = static_cast<uint8_t>(is_hit);
            if (is_hit) atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_HITS), 1ull);
        }
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static siso_status_t encode_rows_map(EncodeTiledFn fn, CUtensorMap *map, const void *base, uint64_t rows, uint64_t dim) {
    cuuint64_t gdim[2] = {dim, rows};
    cuuint64_t gstride[1] = {dim * 2};
    cuuint32_t box[2] = {static_cast<cuuint32_t>(TK), static_cast<cuuint32_t>(TM)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return check_cuda(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return SISO_OK;
}

}  // namespace tc3

// fp32 caches, k <= 4.  Returns SISO_ERR_UNSUPPORTED otherwise (the caller then takes the CUDA-core sweep).
siso_status_t launch_lookup_tensor_f32(Cache *c, const void *q, int64_t B, const float *theta, float theta_s, int k,
                                       int32_t *idx, float *sim, uint8_t *hit, cudaStream_t s) {
    if (c->dtype != SISO_F32 || k > 4) return SISO_ERR_UNSUPPORTED;
    static tc3::EncodeTiledFn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        SISO_CUDA(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres));
        if (!fn || qres != cudaDriverEntryPointSuccess) return check_cuda(cudaErrorNotSupported, "cuTensorMapEncodeTiled lookup");
        encode = reinterpret_cast<tc3::EncodeTiledFn>(fn);
    }
    const int D = c->dim;
    const int64_t rows = c->rows_alloc;
    const int n_tiles = static_cast<int>((c->capacity + tc3::TN - 1) / tc3::TN);
    const int64_t m_tiles64 = (B + tc3::TM - 1) / tc3::TM;
    if (m_tiles64 > 0x7FFFFFFE) return SISO_ERR_UNSUPPORTED;
    const int m_ctas = static_cast<int>((m_tiles64 + 1) / 2 * 2);           // CTA pairs; an odd count is padded with an idle CTA
    // wave count by the same cost model as the bf16 kernel: rounds x (tiles per CTA + start-up cost in tiles)
    const int64_t units = static_cast<int64_t>(m_ctas) * n_tiles;
    const int wave_cap = static_cast<int>(std::min<int64_t>(16, std::max<int64_t>(1, units / (8ll * c->sm_count))));
    int splits = 1, tiles_per_split = n_tiles;
    int64_t best_cost = -1;
    const int candidates[] = {1, 2, 4, 6, 8, 12, 16};
    for (int ci = 0; ci < 7; ++ci) {
        const int w = std::min(candidates[ci], wave_cap);
        int sp = std::max(1, std::min(std::min(n_tiles, 65535), (c->sm_count * w) / m_ctas));
        const int tps = (n_tiles + sp - 1) / sp;
        sp = (n_tiles + tps - 1) / tps;
        const int64_t rounds = (static_cast<int64_t>(m_ctas) * sp + c->sm_count - 1) / c->sm_count;
        const int64_t cost = rounds * (tps + 6);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; splits = sp; tiles_per_split = tps; }
    }
    const size_t c_elems = static_cast<size_t>(rows) * D, q_elems = static_cast<size_t>(B) * D;
    Scratch scr;
    const size_t need = 2 * pad256(q_elems * 2) + pad256(sizeof(unsigned long long) * B * splits * tc3::CAND) +
                        pad256(4 * B) + pad256(sizeof(unsigned long long) * 4 * B * c->sm_count) + 512;
    SISO_TRY(scratch_reserve(c, need, s, &scr));
    // the centroids' parts are kept until the vectors change (every entry point that writes vectors raises vec_epoch)
    if (!c->split_hi) {
        c->split_hi = cache_alloc_zeroed(c, c_elems * 2);
        c->split_lo = cache_alloc_zeroed(c, c_elems * 2);
        if (!c->split_hi || !c->split_lo) return SISO_ERR_OOM;
        c->split_epoch = ~0ull;
    }
    __nv_bfloat16 *c_hi = static_cast<__nv_bfloat16 *>(c->split_hi), *c_lo = static_cast<__nv_bfloat16 *>(c->split_lo);
    __nv_bfloat16 *q_hi = scr.take<__nv_bfloat16>(q_elems), *q_lo = scr.take<__nv_bfloat16>(q_elems);
    unsigned long long *partial = scr.take<unsigned long long>(static_cast<size_t>(B) * splits * tc3::CAND);
    int32_t *flagged = scr.take<int32_t>(B);
    unsigned int *n_flagged = scr.take<unsigned int>(1);
    unsigned long long *rescan_keys = scr.take<unsigned long long>(static_cast<size_t>(4) * B * c->sm_count);
    SISO_CUDA(cudaMemsetAsync(n_flagged, 0, sizeof(unsigned int), s));
    if (c->split_epoch != c->vec_epoch) {
        SISO_TRY(launch_split_bf16(c, c->master, c_hi, c_lo, static_cast<long long>(c_elems / 4), s));
        c->split_epoch = c->vec_epoch;
    }
    SISO_TRY(launch_split_bf16(c, static_cast<const float *>(q), q_hi, q_lo, static_cast<long long>(q_elems / 4), s));
    CUtensorMap map_q_hi, map_q_lo, map_c_hi, map_c_lo;
    SISO_TRY(tc3::encode_rows_map(encode, &map_q_hi, q_hi, static_cast<uint64_t>(B), static_cast<uint64_t>(D)));
    SISO_TRY(tc3::encode_rows_map(encode, &map_q_lo, q_lo, static_cast<uint64_t>(B), static_cast<uint64_t>(D)));
    SISO_TRY(tc3::encode_rows_map(encode, &map_c_hi, c_hi, static_cast<uint64_t>(rows), static_cast<uint64_t>(D)));
    SISO_TRY(tc3::encode_rows_map(encode, &map_c_lo, c_lo, static_cast<uint64_t>(rows), static_cast<uint64_t>(D)));
    auto kern = tc3::lookup_tensor_split_kernel<tc3::CAND>;
    if (!c->split_attr_set) {
        SISO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc3::SMEM_BYTES));
        c->split_attr_set = true;
    }
    kern<<<dim3(m_ctas, splits), tc3::THREADS, tc3::SMEM_BYTES, s>>>(map_q_hi, map_q_lo, map_c_hi, map_c_lo, c->valid, B, D,
                                                                      tiles_per_split, n_tiles, partial, splits, c->status);
    SISO_LAUNCHED(c);
    tc3::lookup_rescore_kernel<<<static_cast<unsigned>((B + 7) / 8), 256, 0, s>>>(
        static_cast<const float *>(q), c->master, B, D, k, splits, partial, theta, theta_s, idx, sim, hit, flagged, n_flagged,
        c->counters);
    SISO_LAUNCHED(c);
    const int scan_ctas = c->sm_count;
    tc3::lookup_rescan_kernel<<<scan_ctas, 256, 0, s>>>(static_cast<const float *>(q), c->master, c->valid, c->capacity, D, flagged,
                                                       n_flagged, rescan_keys);
    SISO_LAUNCHED(c);
    tc3::lookup_rescan_finish_kernel<<<32, 256, 0, s>>>(rescan_keys, scan_ctas, k, flagged, n_flagged, theta, theta_s, idx, sim, hit,
                                                        c->counters);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

}  // namespace siso
