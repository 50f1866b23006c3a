// Large-batch lookup on tensor cores with CTA pairs (tcgen05 cta_group::2).
//
// Two CTAs of a cluster work on 256 queries x 256 centroids at a time.  Each CTA stages its own
// 128-query slab of Q and HALF of the centroid tile (128 rows of C), so for the same flops per SM
// a third less data crosses L2 -> shared memory than in the single-CTA kernel (which reloads the
// whole 256-row centroid tile for every 128 queries).  The leader CTA (cluster rank 0) issues one
// M=256 MMA per 16 K-elements; the result rows 0..127 land in the leader's TMEM, rows 128..255 in
// the peer's, and each CTA's epilogue warps scan their own rows exactly as in the single-CTA kernel.
//   full[s]       (leader's)  both CTAs' TMA loads of stage s report their bytes here
//   empty[s]      (each CTA)  one tcgen05.commit of the leader arrives on both when the MMAs have read stage s
//   acc_full[a]   (each CTA)  committed by the leader when a 256-column accumulator is complete
//   acc_empty[a]  (leader's)  the 8 epilogue warps of both CTAs arrive when they have drained it
// No load is multicast: every CTA fetches what it needs itself.  All waits are bounded (see
// lookup_tensor.cu); a CTA that gives up sets SISO_ERR_TIMEOUT and still reaches the final cluster barrier.
#include <cuda.h>

#include <cstring>

#include "umma_pair.cuh"

namespace siso {
namespace tc2 {

constexpr int TM = 128;             // queries per CTA
constexpr int TN = 256;             // centroids per tile (both CTAs together stage them, 128 rows each)
constexpr int TK = 64;
constexpr int STAGES = 6;
constexpr int ACC_STAGES = 2;
constexpr int THREADS = 192;
constexpr uint32_t A_BYTES = TM * TK * 2;            // 16 KiB
constexpr uint32_t B_BYTES = (TN / 2) * TK * 2;      // 16 KiB: this CTA's half of the centroid tile
constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
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
    int is_last;
};

// Top-1 lookups of at most two query tiles (a streaming micro-batch) are finished inside the sweep: every CTA folds
// the best key of each of its rows into a per-row word with an atomic maximum, and the CTA that is the last of its
// query tile to have done so (a ticket counter per query tile, no waiting) reads the words out and applies the threshold.  That saves a kernel launch, or a phase and
// a grid-wide barrier of the streaming maintenance kernel.  counter == NULL: the partial results are all there is.
struct TailFinal {
    unsigned int *counter;     // [query tiles], zero between launches
    unsigned long long *best;  // [256] best key of every row so far, zero between launches
    const float *theta;
    float theta_s;
    int32_t *idx;              // [B]
    float *sim;                // [B]
    uint8_t *hit;              // [B]
    long long *counters;       // lookups and hits are counted here unless NULL (the caller then counts them itself)
};

template <int KMAX>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
lookup_tensor_pair_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_c_half,
                          const uint8_t *__restrict__ valid, int64_t B, int D, int tiles_per_split, int n_tiles,
                          unsigned long long *__restrict__ partial, int splits, int stream_c, int *status,
                          const TailFinal tail) {
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
            const uint64_t policy = stream_c ? l2_evict_first_policy() : 0ull;
            for (int t = t_begin; t < t_end && ok; ++t) {
                const int n0 = t * TN + static_cast<int>(rank) * (TN / 2);     // this CTA's half of the centroid tile
                for (int ks = 0; ks < k_slabs; ++ks) {
                    if (!mbar_wait(&bars->empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t *a_dst = tiles + stage * STAGE_BYTES;
                    uint8_t *b_dst = a_dst + A_BYTES;
                    const uint32_t full_leader = cluster_addr(smem_u32(&bars->full[stage]), 0);
                    if (rank == 0) mbar_arrive_expect_tx(&bars->full[stage], 2 * STAGE_BYTES);   // both CTAs' bytes
                    tma_load_2d_pair(a_dst, &map_q, ks * TK, q0, full_leader);
                    if (stream_c) tma_load_2d_pair_hint(b_dst, &map_c_half, ks * TK, n0, full_leader, policy);
                    else tma_load_2d_pair(b_dst, &map_c_half, ks * TK, n0, full_leader);
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
                    const uint32_t a_addr = smem_u32(tiles + stage * STAGE_BYTES);
                    const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
                    for (int kk = 0; kk < TK / 16; ++kk)
                        umma_bf16_pair(d_tmem, da + static_cast<uint64_t>(2 * kk), db + static_cast<uint64_t>(2 * kk), IDESC,
                                       (ks | kk) ? 1u : 0u);
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
            if (KMAX == 1 && tail.counter) {
                atomicMax(tail.best + static_cast<int64_t>(q0) + row, top.key(0));
                __threadfence();                                  // folded in before this CTA takes its ticket
            }
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
    if constexpr (KMAX == 1) {
        if (tail.counter) {
            if (threadIdx.x == 0) {
                __threadfence();
                const unsigned int ticket = atomicAdd(&tail.counter[blockIdx.x], 1u);
                bars->is_last = ticket == static_cast<unsigned int>(splits) - 1u ? 1 : 0;
            }
            __syncthreads();
            if (bars->is_last) {
                __threadfence();
                // every CTA has folded its rows' best keys into tail.best with an atomic maximum: read them out,
                // one thread per row (little code: this runs once per launch, from a cold instruction cache)
                const int n_rows = static_cast<int>(min(static_cast<int64_t>(TM), B - q0));
                int is_hit = 0;
                if (static_cast<int>(threadIdx.x) < n_rows) {
                    const int64_t b = static_cast<int64_t>(q0) + threadIdx.x;
                    const unsigned long long key = __ldcg(tail.best + b);
                    tail.best[b] = 0ull;                                   // ready for the next launch
                    tail.idx[b] = key ? key_slot(key) : -1;
                    tail.sim[b] = key ? key_sim(key) : -INFINITY;
                    const float th = tail.theta ? tail.theta[b] : tail.theta_s;
                    is_hit = (key != 0ull && key_sim(key) > th) ? 1 : 0;
                    tail.hit[b] = static_cast<uint8_t>(is_hit);
                }
                if (tail.counters) {
                    const int n_hit = __syncthreads_count(is_hit);
                    if (threadIdx.x == 0 && n_rows > 0) {
                        if (n_hit) atomicAdd(reinterpret_cast<unsigned long long *>(tail.counters + CNT_HITS), static_cast<unsigned long long>(n_hit));
                        atomicAdd(reinterpret_cast<unsigned long long *>(tail.counters + CNT_LOOKUPS), static_cast<unsigned long long>(n_rows));
                    }
                }
                if (threadIdx.x == 0) tail.counter[blockIdx.x] = 0u;      // ready for the next launch
            }
        }
    }
}

}  // namespace tc2

template <int KMAX>
static siso_status_t run_pair(Cache *c, bool *attr_set, const CUtensorMap &map_q, const CUtensorMap &map_c_half, int64_t B,
                              int tiles_per_split, int n_tiles, int splits, int m_tiles_even, unsigned long long *partial,
                              const tc2::TailFinal &tail, cudaStream_t s) {
    auto kern = tc2::lookup_tensor_pair_kernel<KMAX>;
    if (!*attr_set) {
        SISO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc2::SMEM_BYTES));
        *attr_set = true;
    }
    dim3 grid(m_tiles_even, splits);
    // one pair covers the whole batch: every centroid tile is read by exactly one cluster, so it need not stay in L2
    kern<<<grid, tc2::THREADS, tc2::SMEM_BYTES, s>>>(map_q, map_c_half, c->valid, B, c->dim, tiles_per_split, n_tiles,
                                                     partial, splits, m_tiles_even == 2 ? 1 : 0, c->status, tail);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

// Called by launch_lookup_tensor when the batch spans at least two query tiles.  With `tail_counter` (k = 1 only) the
// kernel also writes idx / sim / hit itself (see TailFinal).
siso_status_t launch_lookup_tensor_pair(Cache *c, bool *attr_set3, const CUtensorMap &map_q, const CUtensorMap &map_c_half,
                                        int64_t B, int kmax, int tiles_per_split, int n_tiles, int splits, int m_tiles_even,
                                        unsigned long long *partial, unsigned int *tail_counter, const float *theta,
                                        float theta_s, int32_t *idx, float *sim, uint8_t *hit, long long *counters,
                                        cudaStream_t s) {
    tc2::TailFinal tail;
    tail.counter = kmax == 1 ? tail_counter : nullptr;
    tail.best = tail_counter ? reinterpret_cast<unsigned long long *>(tail_counter + 64) : nullptr;     // 256 bytes in
    tail.theta = theta; tail.theta_s = theta_s; tail.idx = idx; tail.sim = sim; tail.hit = hit; tail.counters = counters;
    return kmax == 1 ? run_pair<1>(c, attr_set3 + 0, map_q, map_c_half, B, tiles_per_split, n_tiles, splits, m_tiles_even, partial, tail, s)
         : kmax == 4 ? run_pair<4>(c, attr_set3 + 1, map_q, map_c_half, B, tiles_per_split, n_tiles, splits, m_tiles_even, partial, tail, s)
                     : run_pair<8>(c, attr_set3 + 2, map_q, map_c_half, B, tiles_per_split, n_tiles, splits, m_tiles_even, partial, tail, s);
}

}  // namespace siso
