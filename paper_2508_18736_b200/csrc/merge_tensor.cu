// Pairwise similarity sweep of MergeCentroids (Algorithm 1: every entry against the earlier entries of C_new) as a
// dense contraction on the tensor cores, for fp32 vectors.
//
// An fp32 value x is split as x = hi + lo + r with hi = bf16(x), lo = bf16(x - hi), |r| <= 2^-16 |x|.  The sweep
// accumulates hi_i.hi_j + hi_i.lo_j + lo_i.hi_j in fp32 on tcgen05 (three MMAs per 16 K-elements, one TMEM
// accumulator); what it leaves out (lo.lo, the r terms) and the fp32 accumulation stay below 6e-5 for unit
// vectors.  So the tensor cores only FILTER: every pair whose approximate similarity exceeds theta_C - 1e-4
// becomes a provisional candidate, and merge_verify_kernel recomputes exactly these pairs from the fp32 vectors
// in fp64 and keeps those whose exact similarity exceeds theta_C.  The decisions are therefore those of an exact
// fp64 sweep; the tensor cores do the 2 N^2 D flops, the exact arithmetic touches the few candidates only.
//
// By default even less is asked of the tensor cores: the rows rounded to bf16 are multiplied ONCE (one MMA per 16
// K-elements, half the operand bytes) and the filter margin is widened to the bound of that rounding (one_part_margin, 8.1e-3);
// a few more pairs reach the exact check, the decisions stay the same.
//
// Kernel layout (CTA pairs, cta_group::2, as in the large-batch lookup): a cluster works on 256 rows i x 256 rows j
// at a time; each CTA stages its own 128 rows i and half of the rows j: 32 KiB per stage and six stages with one
// part, 64 KiB (hi and lo of both) and three stages with three parts; warp 0 = TMA producer, warp 1 = MMA issuer
// (leader CTA), warps 2-9 = epilogue (thread = row i, two warps per 32 rows, 128 columns each) over two TMEM
// accumulators.  The tile pairs of the lower triangle (one set) or of the whole matrix (two sets) are
// listed block by block (9 x 9 tiles) and dealt to the clusters round robin, so the clusters that run at the same
// time work inside one block and share its rows through L2.  No load is multicast; every wait is bounded.
#include <cstring>
#include <vector>

#include "umma_pair.cuh"

namespace siso {

struct MergeCandidate {
    int32_t i, j;
    float sim;
};
struct MergeCtlView {                 // same layout as MergeCtl in merge.cu
    unsigned long long n_cand;
    int overflow;
    int n_merged;
};

namespace tcm {

using namespace umma2;

constexpr int TM = 128;             // rows i per CTA
constexpr int TN = 256;             // rows j per tile (128 staged by each CTA)
constexpr int TK = 64;
constexpr int MAX_STAGES = 6;
constexpr int ACC_STAGES = 2;
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;
constexpr uint32_t OPER_BYTES = TM * TK * 2;              // 16 KiB: 128 rows x 64 bf16
constexpr uint32_t RING_BYTES = 12 * OPER_BYTES;          // six stages of (hi_i, hi_j half) or three of (hi_i, lo_i, hi_j half, lo_j half)
constexpr uint32_t SMEM_BYTES = RING_BYTES + 1024 + 4096;
constexpr uint32_t TMEM_COLS = ACC_STAGES * TN;
constexpr float FILTER_MARGIN = 1e-4f;             // three-part products (or rows that are bf16 values): left-out terms and fp32 sums
// One-part filter on fp32 rows.  bf16 keeps 8 significant bits: with x^ = bf16(x), |x - x^| <= u |x| for u = 2^-8 (round
// to nearest), so |x.y - x^.y^| <= (2u + u^2) |x| |y| = 7.99e-3 for norms up to 1.01 (what checked mode accepts); the fp32 accumulator is rounded
// once per 16 K-elements (dim / 16 roundings of 2^-23 of a sum below 1).
__host__ inline float one_part_margin(int dim) { return 8.1e-3f + 1.0e-8f * static_cast<float>(dim); }

// D fp32, A and B bf16, K-major, N = 256, M = 256 (128 rows per CTA of the pair)
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(TN >> 3) << 17) |
                           (static_cast<uint32_t>((2 * TM) >> 4) << 24);

struct Shared {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], acc_full[ACC_STAGES], acc_empty[ACC_STAGES];
    uint32_t tmem_base;
    int abort_flag;
};

// tile pair number -> (row tile I, column tile t), from the list the host wrote
__device__ __forceinline__ void pair_to_tiles(const uint32_t *__restrict__ pair_list, long long p, int *I, int *t) {
    const uint32_t v = __ldg(pair_list + p);
    *I = static_cast<int>(v >> 16);
    *t = static_cast<int>(v & 0xFFFFu);
}

// SPLIT: three products of bf16 parts per pair and K step (false: one product of the rounded rows); a template
// parameter so that the MMA-issuing thread runs straight-line code
template <bool SPLIT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
merge_sweep_tensor_kernel(const __grid_constant__ CUtensorMap map_hi, const __grid_constant__ CUtensorMap map_lo,
                          const uint8_t *__restrict__ valid, const uint8_t *__restrict__ seed, int64_t N, int D,
                          const uint32_t *__restrict__ pair_list, long long n_pairs, float theta_filter, MergeCtlView *ctl,
                          MergeCandidate *__restrict__ cand, unsigned long long max_cand, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *stage_mem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    Shared *sh = reinterpret_cast<Shared *>(stage_mem + RING_BYTES);
    constexpr bool split = SPLIT;
    constexpr uint32_t STAGES = split ? 3u : 6u;
    constexpr uint32_t STAGE_BYTES = split ? 4 * OPER_BYTES : 2 * OPER_BYTES;
    constexpr uint32_t OFF_J = split ? 2 * OPER_BYTES : OPER_BYTES;       // where the rows j start inside a stage
    volatile int *abort_flag = &sh->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const bool two_sets = seed != nullptr;
    const long long p_begin = blockIdx.x >> 1;             // this cluster's tile pairs: p_begin, p_begin + clusters, ...
    const long long p_step = gridDim.x >> 1;
    const long long p_end = n_pairs;
    const int k_slabs = (D + TK - 1) / TK;
    const bool skip = ctl->overflow != 0;           // set before the launch (two sets: the insertion failed)

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        for (int a = 0; a < ACC_STAGES; ++a) { mbar_init(&sh->acc_full[a], 1); mbar_init(&sh->acc_empty[a], 2 * EPI_WARPS); }
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sh->tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync();
    tcgen05_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    if (skip) {
        // nothing to do; fall through to the common teardown
    } else if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (long long p = p_begin; p < p_end && ok; p += p_step) {
                int I, t;
                pair_to_tiles(pair_list, p, &I, &t);
                const int i0 = I * (2 * TM) + static_cast<int>(rank) * TM;        // this CTA's own rows i
                const int n0 = t * TN + static_cast<int>(rank) * (TN / 2);        // its half of the rows j
                for (int ks = 0; ks < k_slabs; ++ks) {
                    if (!mbar_wait(&sh->empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t *dst = stage_mem + stage * STAGE_BYTES;
                    const uint32_t full_leader = cluster_addr(smem_u32(&sh->full[stage]), 0);
                    // bf16 inputs have no second part: only the hi tiles are loaded and one MMA per K step is issued
                    if (rank == 0) mbar_arrive_expect_tx(&sh->full[stage], 2 * STAGE_BYTES);   // both CTAs' loads of the stage
                    tma_load_2d_pair(dst, &map_hi, ks * TK, i0, full_leader);
                    if (split) tma_load_2d_pair(dst + OPER_BYTES, &map_lo, ks * TK, i0, full_leader);
                    tma_load_2d_pair(dst + OFF_J, &map_hi, ks * TK, n0, full_leader);
                    if (split) tma_load_2d_pair(dst + OFF_J + OPER_BYTES, &map_lo, ks * TK, n0, full_leader);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader only)
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (long long p = p_begin; p < p_end && ok; p += p_step) {
                if (!mbar_wait(&sh->acc_empty[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + acc * TN;
                for (int ks = 0; ks < k_slabs; ++ks) {
                    if (!mbar_wait(&sh->full[stage], phase, abort_flag)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t base = smem_u32(stage_mem + stage * STAGE_BYTES);
                    const uint64_t a_hi = smem_desc_sw128(base), a_lo = smem_desc_sw128(base + OPER_BYTES);
                    const uint64_t b_hi = smem_desc_sw128(base + OFF_J), b_lo = smem_desc_sw128(base + OFF_J + OPER_BYTES);
#pragma unroll
                    for (int kk = 0; kk < TK / 16; ++kk) {
                        const uint64_t o = static_cast<uint64_t>(2 * kk);
                        umma_bf16_pair(d_tmem, a_hi + o, b_hi + o, IDESC, (ks | kk) ? 1u : 0u);
                        if constexpr (split) {
                            umma_bf16_pair(d_tmem, a_hi + o, b_lo + o, IDESC, 1u);
                            umma_bf16_pair(d_tmem, a_lo + o, b_hi + o, IDESC, 1u);
                        }
                    }
                    umma_commit_both(&sh->empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit_both(&sh->acc_full[acc]);
                if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9 of both CTAs)
        // a warp reads the 32 TMEM lanes of its quarter (warp % 4) and one half of the tile's 256 columns
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        constexpr int CHUNKS = TN / 64;          // chunks of 32 columns per warp
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        constexpr int RUN = 128;                 // places of the candidate list a warp reserves at a time
        unsigned long long run_base = 0;         // the warp's current run (the same in all lanes)
        int run_left = 0;
        int last_I = -1;
        bool row_ok = false;
        long long gi = 0;
        for (long long p = p_begin; p < p_end && ok; p += p_step) {
            int I, t;
            pair_to_tiles(pair_list, p, &I, &t);
            const long long n0 = static_cast<long long>(t) * TN + half * (TN / 2);
            if (I != last_I) {
                last_I = I;
                gi = static_cast<long long>(I) * (2 * TM) + static_cast<long long>(rank) * TM + quarter * 32 + lane;
                // a row takes part if it is live and not a member of C_cur (those are never merged into others)
                row_ok = gi < N && valid[gi] != 0 && !(two_sets && seed[gi] != 0);
            }
            // the warp's 128 rows j as bit masks per chunk of 32 (the same in all lanes): live, member of C_cur
            uint32_t live_mask[CHUNKS], seed_mask[CHUNKS];
#pragma unroll
            for (int h = 0; h < CHUNKS; ++h) {
                const long long gj = n0 + h * 32 + lane;
                const bool lv = gj < N && valid[gj] != 0;
                live_mask[h] = __ballot_sync(0xFFFFFFFFu, lv);
                seed_mask[h] = two_sets ? __ballot_sync(0xFFFFFFFFu, lv && seed[gj] != 0) : 0u;
            }
            if (!mbar_wait(&sh->acc_full[acc], acc_phase, abort_flag)) { ok = false; break; }
            tcgen05_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * TN + half * (TN / 2);
            uint32_t ra[32], rb[32];
            auto scan = [&](uint32_t (&r)[32], int ch) {
                // the largest of the row's 32 values, by four independent chains
                float m0 = __uint_as_float(r[0]), m1 = __uint_as_float(r[1]), m2 = __uint_as_float(r[2]), m3 = __uint_as_float(r[3]);
#pragma unroll
                for (int j = 4; j < 32; j += 4) {
                    m0 = fmaxf(m0, __uint_as_float(r[j]));
                    m1 = fmaxf(m1, __uint_as_float(r[j + 1]));
                    m2 = fmaxf(m2, __uint_as_float(r[j + 2]));
                    m3 = fmaxf(m3, __uint_as_float(r[j + 3]));
                }
                const bool look = row_ok && fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) > theta_filter;
                if (!__any_sync(0xFFFFFFFFu, look)) return;            // the common case: nothing above the filter
                // which values of this row are pairs of the sweep
                uint32_t take = 0;
                if (look) {
                    // columns that come before row gi in C_new: members of C_cur, or a lower slot
                    const long long below = gi - (n0 + ch * 32);             // columns 0..below-1 of the chunk are lower slots
                    const uint32_t lower = below <= 0 ? 0u : (below >= 32 ? 0xFFFFFFFFu : ((1u << below) - 1u));
                    uint32_t ok_mask = live_mask[ch] & (seed_mask[ch] | lower);
                    if (below >= 0 && below < 32) ok_mask &= ~(1u << below);   // never the row itself
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (__uint_as_float(r[j]) > theta_filter) take |= 1u << j;
                    take &= ok_mask;
                }
                // places in the warp's reserved run of the candidate list (one global atomic per RUN places: a single
                // counter that every row hits would serialise them).  Few rows of a chunk hold pairs, so their places
                // are dealt by walking the lanes that have some.
                uint32_t holders = __ballot_sync(0xFFFFFFFFu, take != 0u);
                if (holders == 0u) return;
                const int mine = __popc(take);
                int before = 0, total = 0;
                while (holders) {
                    const int src = __ffs(holders) - 1;
                    holders &= holders - 1u;
                    const int cnt = __shfl_sync(0xFFFFFFFFu, mine, src);
                    if (src < lane) before += cnt;
                    total += cnt;
                }
                if (total > run_left) {
                    // give the rest of the old run back as empty records and take a new one
                    for (int t = lane; t < run_left; t += 32)
                        if (run_base + t < max_cand) cand[run_base + t].i = -1;
                    const int want = total > RUN ? total : RUN;
                    unsigned long long nb = 0;
                    if (lane == 0) nb = atomicAdd(&ctl->n_cand, static_cast<unsigned long long>(want));
                    run_base = __shfl_sync(0xFFFFFFFFu, nb, 0);
                    run_left = want;
                    if (run_base + want > max_cand && lane == 0) ctl->overflow = 1;
                }
                // the exact check writes the similarity of the pairs it confirms; the filter's value is not kept
                unsigned long long pos = run_base + static_cast<unsigned long long>(before);
                while (take) {
                    const int j = __ffs(take) - 1;
                    take &= take - 1u;
                    if (pos < max_cand) {
                        MergeCandidate cd;
                        cd.i = static_cast<int32_t>(gi);
                        cd.j = static_cast<int32_t>(n0 + ch * 32 + j);
                        cd.sim = 0.0f;
                        cand[pos] = cd;
                    }
                    ++pos;
                }
                run_base += static_cast<unsigned long long>(total);
                run_left -= total;
            };
            tmem_ld_32x32(taddr, ra);
#pragma unroll 1
            for (int ch = 0; ch < CHUNKS; ch += 2) {
                tmem_ld_fence(ra);
                tmem_ld_32x32(taddr + (ch + 1) * 32, rb);
                scan(ra, ch);
                tmem_ld_fence(rb);
                if (ch + 2 < CHUNKS) tmem_ld_32x32(taddr + (ch + 2) * 32, ra);
                scan(rb, ch + 1);
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(cluster_addr(smem_u32(&sh->acc_empty[acc]), 0));
            if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
        }
        // what is left of the last run holds no pair
        for (int t = lane; t < run_left; t += 32)
            if (run_base + t < max_cand) cand[run_base + t].i = -1;
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        if (threadIdx.x == 0) set_status(status, SISO_ERR_TIMEOUT);
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// x -> (bf16(x), bf16(x - bf16(x))), four elements per thread
__global__ void split_bf16_kernel(const float *__restrict__ x, __nv_bfloat16 *__restrict__ hi, __nv_bfloat16 *__restrict__ lo,
                                  long long n4) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    const float4 v = __ldg(reinterpret_cast<const float4 *>(x) + i);
    const float f[4] = {v.x, v.y, v.z, v.w};
    __nv_bfloat16 h[4], l[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        h[k] = __float2bfloat16_rn(f[k]);
        l[k] = __float2bfloat16_rn(f[k] - __bfloat162float(h[k]));
    }
    *reinterpret_cast<uint2 *>(hi + 4 * i) = *reinterpret_cast<const uint2 *>(h);
    if (lo) *reinterpret_cast<uint2 *>(lo + 4 * i) = *reinterpret_cast<const uint2 *>(l);
}

// One warp per provisional candidate: exact similarity of the fp32 vectors (products and sums in fp64).  The pair
// stays a candidate if it exceeds theta_C (strict, as in Algorithm 1); otherwise its row index becomes -1.
__global__ void __launch_bounds__(256)
merge_verify_kernel(const MergeCtlView *ctl, const float *__restrict__ C, int D, float theta, MergeCandidate *__restrict__ cand,
                    unsigned long long max_cand, uint32_t *__restrict__ row_count) {
    if (ctl->overflow) return;
    const unsigned long long n = ctl->n_cand < max_cand ? ctl->n_cand : max_cand;
    const int lane = threadIdx.x & 31;
    const unsigned long long warps = static_cast<unsigned long long>(gridDim.x) * (blockDim.x >> 5);
    for (unsigned long long e = static_cast<unsigned long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); e < n; e += warps) {
        const MergeCandidate cd = cand[e];
        if (cd.i < 0) continue;                      // an unused place of a warp's reserved run
        const float4 *a = reinterpret_cast<const float4 *>(C + static_cast<long long>(cd.i) * D);
        const float4 *b = reinterpret_cast<const float4 *>(C + static_cast<long long>(cd.j) * D);
        double s = 0.0;
        for (int q = lane; q < D / 4; q += 32) {
            const float4 x = __ldg(a + q), y = __ldg(b + q);
            s += static_cast<double>(x.x) * static_cast<double>(y.x) + static_cast<double>(x.y) * static_cast<double>(y.y) +
                 static_cast<double>(x.z) * static_cast<double>(y.z) + static_cast<double>(x.w) * static_cast<double>(y.w);
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        if (lane == 0) {
            if (s > static_cast<double>(theta)) {
                cand[e].sim = static_cast<float>(s);
                if (row_count) atomicAdd(&row_count[cd.i], 1u);
            } else {
                cand[e].i = -1;
            }
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

}  // namespace tcm

siso_status_t launch_split_bf16(Cache *c, const float *x, __nv_bfloat16 *hi, __nv_bfloat16 *lo, long long n4, cudaStream_t s) {
    if (n4 <= 0) return SISO_OK;
    tcm::split_bf16_kernel<<<static_cast<unsigned>((n4 + 255) / 256), 256, 0, s>>>(x, hi, lo, n4);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

size_t pair_sweep_tensor_scratch_bytes(int64_t n, int64_t rows, int dim) {
    const size_t tiles = static_cast<size_t>((n + 2 * tcm::TM - 1) / (2 * tcm::TM));
    return 2 * pad256(static_cast<size_t>(rows) * dim * sizeof(__nv_bfloat16)) + pad256(sizeof(uint32_t) * tiles * tiles);
}
size_t merge_tensor_scratch_bytes(const Cache *c) { return pair_sweep_tensor_scratch_bytes(c->capacity, c->rows_alloc, c->dim); }

// Sweep + exact check over the rows of X ([rows, dim] fp32; if the values are in fact bf16 values, `rows_bf16` is the
// same matrix in bf16 and the sweep needs one MMA per K step instead of three; the first N rows take part, `valid` [N] saying which
// are live, `seed` [N] or NULL marking the members of C_cur).  `ctl` and `row_count` are zeroed (or carry the two-set
// insertion's failure flag); on return (in stream order) cand[0 .. min(n_cand, max_cand)) holds the provisional
// pairs, the confirmed ones with their exact similarity and i >= 0, and row_count[i] (if not NULL) counts the
// confirmed pairs of row i.
// `cross_rows` > 0 (a multiple of 256, with `seed` marking exactly the rows below it): only the pairs of a row at or
// beyond cross_rows with a row below it are swept, i.e. one block of rows against another block.
siso_status_t launch_pair_sweep_tensor(Cache *c, Scratch *scr, const float *X, int64_t N, int64_t rows, const uint8_t *valid,
                                       const uint8_t *seed, float theta_c, void *ctl, void *cand, size_t max_cand,
                                       uint32_t *row_count, cudaStream_t s, const void *rows_bf16, int64_t cross_rows) {
    static tcm::EncodeTiledFn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        SISO_CUDA(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres));
        if (!fn || qres != cudaDriverEntryPointSuccess) return check_cuda(cudaErrorNotSupported, "cuTensorMapEncodeTiled lookup");
        encode = reinterpret_cast<tcm::EncodeTiledFn>(fn);
    }
    const size_t elems = static_cast<size_t>(rows) * c->dim;
    // rows that ARE bf16 values need no second part.  fp32 rows: by default the sweep is a FILTER on the rounded rows
    // alone (one MMA per K step, half the operand bytes) with a margin that covers the rounding, and the exact check
    // below decides; with three parts the margin is the one of the fp32 sums and fewer pairs reach the check.
    const int split = (!rows_bf16 && c->merge_sweep_parts == 3) ? 1 : 0;
    const float margin = (rows_bf16 || split) ? tcm::FILTER_MARGIN : tcm::one_part_margin(c->dim);
    const __nv_bfloat16 *hi, *lo;
    if (!rows_bf16) {
        __nv_bfloat16 *h = scr->take<__nv_bfloat16>(elems), *l = split ? scr->take<__nv_bfloat16>(elems) : nullptr;
        const long long n4 = static_cast<long long>(elems / 4);
        tcm::split_bf16_kernel<<<static_cast<unsigned>((n4 + 255) / 256), 256, 0, s>>>(X, h, l, n4);
        SISO_LAUNCHED(c);
        hi = h;
        lo = split ? l : h;
    } else {
        hi = lo = static_cast<const __nv_bfloat16 *>(rows_bf16);
    }
    CUtensorMap map_hi, map_lo;
    SISO_TRY(tcm::encode_rows_map(encode, &map_hi, hi, static_cast<uint64_t>(rows), static_cast<uint64_t>(c->dim)));
    SISO_TRY(tcm::encode_rows_map(encode, &map_lo, lo, static_cast<uint64_t>(rows), static_cast<uint64_t>(c->dim)));
    const int tiles = static_cast<int>((N + 2 * tcm::TM - 1) / (2 * tcm::TM));       // 256 rows per tile
    if (tiles > 0xFFFF) return SISO_ERR_UNSUPPORTED;
    // the tile pairs block by block: blocks of SB x SB tiles, row-major inside a block
    constexpr int SB = 9;
    std::vector<uint32_t> list;
    list.reserve(static_cast<size_t>(tiles) * (tiles + 1) / (seed ? 1 : 2));
    const int cross_tiles = static_cast<int>(cross_rows / (2 * tcm::TM));
    if (cross_rows > 0) {
        if (!seed || cross_rows % (2 * tcm::TM) != 0 || cross_tiles >= tiles) return SISO_ERR_INVALID_ARG;
        for (int bi = cross_tiles; bi < tiles; bi += SB)
            for (int bt = 0; bt < cross_tiles; bt += SB)
                for (int I = bi; I < std::min(tiles, bi + SB); ++I)
                    for (int t = bt; t < std::min(cross_tiles, bt + SB); ++t)
                        list.push_back((static_cast<uint32_t>(I) << 16) | static_cast<uint32_t>(t));
    } else {
        for (int bi = 0; bi < tiles; bi += SB)
            for (int bt = 0; bt < (seed ? tiles : bi + 1); bt += SB)
                for (int I = bi; I < std::min(tiles, bi + SB); ++I)
                    for (int t = bt; t < std::min(seed ? tiles : I + 1, bt + SB); ++t)
                        list.push_back((static_cast<uint32_t>(I) << 16) | static_cast<uint32_t>(t));
    }
    const long long n_pairs = static_cast<long long>(list.size());
    uint32_t *pair_list = scr->take<uint32_t>(list.size());
    SISO_CUDA(cudaMemcpyAsync(pair_list, list.data(), sizeof(uint32_t) * list.size(), cudaMemcpyHostToDevice, s));
    const long long used = std::max<long long>(1, std::min<long long>(n_pairs, c->sm_count / 2));
    if (!c->merge_tensor_attr_set) {
        SISO_CUDA(cudaFuncSetAttribute(tcm::merge_sweep_tensor_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tcm::SMEM_BYTES));
        SISO_CUDA(cudaFuncSetAttribute(tcm::merge_sweep_tensor_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tcm::SMEM_BYTES));
        c->merge_tensor_attr_set = true;
    }
    auto kernel = split ? tcm::merge_sweep_tensor_kernel<true> : tcm::merge_sweep_tensor_kernel<false>;
    kernel<<<static_cast<unsigned>(2 * used), tcm::THREADS, tcm::SMEM_BYTES, s>>>(
        map_hi, map_lo, valid, seed, N, c->dim, pair_list, n_pairs, theta_c - margin,
        static_cast<MergeCtlView *>(ctl), static_cast<MergeCandidate *>(cand), max_cand, c->status);
    SISO_LAUNCHED(c);
    tcm::merge_verify_kernel<<<8 * c->sm_count, 256, 0, s>>>(static_cast<const MergeCtlView *>(ctl), X, c->dim, theta_c,
                                                             static_cast<MergeCandidate *>(cand), max_cand, row_count);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

siso_status_t launch_merge_sweep_tensor(Cache *c, Scratch *scr, const uint8_t *seed, float theta_c, void *ctl, void *cand,
                                        size_t max_cand, uint32_t *row_count, cudaStream_t s) {
    return launch_pair_sweep_tensor(c, scr, c->master, c->capacity, c->rows_alloc, c->valid, seed, theta_c, ctl, cand, max_cand,
                                    row_count, s, nullptr, 0);
}

}  // namespace siso
