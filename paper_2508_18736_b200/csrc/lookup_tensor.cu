// Large-batch lookup as a dense contraction on the 5th-generation tensor cores:
//     S = Q * C^T  (bf16 x bf16 -> fp32), per-row top-k and threshold fused, S never leaves the SM.
//
// One CTA owns 128 queries (the 128 TMEM lanes) and a contiguous range of 256-centroid tiles.
//   warp 0      TMA producer: per 64-element K slab one 128x64 tile of Q and one 256x64 tile of C
//               (cp.async.bulk.tensor, 128-byte swizzle) into a ring of shared-memory stages
//   warp 1      MMA issuer: tcgen05.mma (M=128, N=256, K=16) four times per slab into one of two
//               256-column TMEM accumulators; tcgen05.commit releases the stage / publishes the tile
//   warps 2-5   epilogue: tcgen05.ld the finished accumulator (thread = query row), drop empty slots,
//               keep the row's running top-k in registers, release the accumulator
// so the tensor pipe works on tile t+1 while the CUDA cores scan tile t.  Products of bf16 values are
// exact in fp32 and the accumulation is fp32, which is what the 2e-3 tolerance is derived from.
// Every wait is bounded: when one runs out the CTA raises SISO_ERR_TIMEOUT in the status word, all
// roles leave their loops, in-flight copies get time to land, TMEM is freed and the kernel returns.
#include <cuda.h>

#include <cstring>

#include "umma_pair.cuh"

namespace siso {
namespace tc {

constexpr int TM = 128;             // queries per CTA (TMEM lanes)
constexpr int TN = 256;             // centroids per MMA tile (TMEM columns per accumulator)
constexpr int TK = 64;              // K elements per stage: 128 bytes = one swizzle span
constexpr int STAGES = 4;
constexpr int ACC_STAGES = 2;
constexpr int THREADS = 192;
constexpr uint32_t A_BYTES = TM * TK * 2;     // 16 KiB
constexpr uint32_t B_BYTES = TN * TK * 2;     // 32 KiB
constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr uint32_t TMEM_COLS = ACC_STAGES * TN;   // 512: the whole tensor memory of the SM

using namespace umma2;      // PTX wrappers and the epilogue scan shared with the CTA-pair kernels

// Instruction descriptor: D fp32, A and B bf16, both K-major, N = 256, M = 128.
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(TN >> 3) << 17) |
                           (static_cast<uint32_t>(TM >> 4) << 24);

struct Barriers {
    uint64_t full[STAGES], empty[STAGES], acc_full[ACC_STAGES], acc_empty[ACC_STAGES];
    uint32_t tmem_base;
    int abort_flag;
};

template <int KMAX>
__global__ void __launch_bounds__(THREADS, 1)
lookup_tensor_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_c,
                     const uint8_t *__restrict__ valid, int64_t B, int D, int tiles_per_split, int n_tiles,
                     unsigned long long *__restrict__ partial, int splits, int stream_c, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    Barriers *bars = reinterpret_cast<Barriers *>(tiles + STAGES * STAGE_BYTES);
    volatile int *abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // blockIdx.x walks the query tiles, so CTAs that run at the same time sweep the SAME centroid range
    // and every centroid tile leaves HBM once and is then served from L2
    const int split = blockIdx.y;
    const int q0 = blockIdx.x * TM;
    const int t_begin = split * tiles_per_split;
    const int t_end = min(n_tiles, t_begin + tiles_per_split);
    const int k_slabs = (D + TK - 1) / TK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        for (int a = 0; a < ACC_STAGES; ++a) { mbar_init(&bars->acc_full[a], 1); mbar_init(&bars->acc_empty[a], 4); }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // one warp allocates all 512 TMEM columns and writes the base address to smem
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&bars->tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            const uint64_t policy = stream_c ? l2_evict_first_policy() : 0ull;
            for (int t = t_begin; t < t_end && ok; ++t) {
                const int n0 = t * TN;
                for (int ks = 0; ks < k_slabs; ++ks) {
                    if (!mbar_wait(&bars->empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t *a_dst = tiles + stage * STAGE_BYTES;
                    uint8_t *b_dst = a_dst + A_BYTES;
                    mbar_arrive_expect_tx(&bars->full[stage], STAGE_BYTES);
                    tma_load_2d(a_dst, &map_q, ks * TK, q0, &bars->full[stage]);
                    if (stream_c) tma_load_2d_hint(b_dst, &map_c, ks * TK, n0, &bars->full[stage], policy);
                    else tma_load_2d(b_dst, &map_c, ks * TK, n0, &bars->full[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
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
                    for (int kk = 0; kk < TK / 16; ++kk) {
                        // 16 bf16 = 32 bytes further along K inside the swizzle span: +2 in 16-byte units
                        umma_bf16(d_tmem, da + static_cast<uint64_t>(2 * kk), db + static_cast<uint64_t>(2 * kk), IDESC,
                                  (ks | kk) ? 1u : 0u);
                    }
                    umma_commit(&bars->empty[stage]);          // stage reusable once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit(&bars->acc_full[acc]);             // accumulator complete
                if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;                         // TMEM lanes [32*quarter, +32) belong to this warp
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
            if (lane == 0) mbar_arrive(&bars->acc_empty[acc]);
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
        // give copies still in flight time to land before the shared memory is handed back
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        if (threadIdx.x == 0) set_status(status, SISO_ERR_TIMEOUT);
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// a batch that does not fill its last tile -> whole tiles, the missing rows zero (16-byte units)
__global__ void pad_query_tile_kernel(const uint4 *__restrict__ q, uint4 *__restrict__ tile, long long have, long long total) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < total) tile[i] = i < have ? q[i] : make_uint4(0u, 0u, 0u, 0u);
}

// ---- host side ------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TensorState {
    EncodeTiledFn encode;
    CUtensorMap map_c;        // box of 256 centroid rows (single-CTA kernel)
    CUtensorMap map_c_half;   // box of 128 centroid rows (CTA-pair kernel: each CTA stages half a tile)
    bool attr_set[3];
    bool attr_set_pair[3];
    unsigned int *tail_counter;   // ticket counters of the in-sweep finalisation (one per query tile of a pair), zero between launches
};

static siso_status_t encode_map(EncodeTiledFn fn, CUtensorMap *map, const void *base, uint64_t rows, uint64_t dim,
                                uint32_t box_rows) {
    cuuint64_t gdim[2] = {dim, rows};
    cuuint64_t gstride[1] = {dim * 2};
    cuuint32_t box[2] = {static_cast<cuuint32_t>(TK), box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return check_cuda(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return SISO_OK;
}

}  // namespace tc

siso_status_t launch_lookup_tensor_pair(Cache *c, bool *attr_set3, const CUtensorMap &map_q, const CUtensorMap &map_c_half,
                                        int64_t B, int kmax, int tiles_per_split, int n_tiles, int splits, int m_tiles_even,
                                        unsigned long long *partial, unsigned int *tail_counter, const float *theta,
                                        float theta_s, int32_t *idx, float *sim, uint8_t *hit, long long *counters,
                                        cudaStream_t s);

void tensor_state_destroy(Cache *c) {
    auto *ts = static_cast<tc::TensorState *>(c->tensor_state);
    if (ts && ts->tail_counter) c->alloc.free(ts->tail_counter, c->alloc.ctx);
    delete ts;
    c->tensor_state = nullptr;
}

template <int KMAX>
static siso_status_t run_tensor(Cache *c, tc::TensorState *ts, int slot, const CUtensorMap &map_q, int64_t B,
                                int tiles_per_split, int n_tiles, int splits, int m_tiles, unsigned long long *partial,
                                cudaStream_t s) {
    auto kern = tc::lookup_tensor_kernel<KMAX>;
    if (!ts->attr_set[slot]) {
        SISO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_BYTES));
        ts->attr_set[slot] = true;
    }
    dim3 grid(m_tiles, splits);
    // one query tile: every centroid tile is read by exactly one CTA, so it need not stay in L2
    kern<<<grid, tc::THREADS, tc::SMEM_BYTES, s>>>(map_q, ts->map_c, c->valid, B, c->dim, tiles_per_split, n_tiles,
                                                   partial, splits, m_tiles == 1 ? 1 : 0, c->status);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

siso_status_t launch_lookup_tensor(Cache *c, const void *q, int64_t B, const float *theta, float theta_s, int k,
                                   int32_t *idx, float *sim, uint8_t *hit, cudaStream_t s, DeferredTop1 *defer,
                                   size_t tail_bytes, void **tail) {
    if (c->dtype != SISO_BF16) return SISO_ERR_UNSUPPORTED;
    if (defer && (k != 1 || !tail)) return SISO_ERR_INVALID_ARG;
    auto *ts = static_cast<tc::TensorState *>(c->tensor_state);
    if (!ts) {
        ts = new tc::TensorState();
        memset(ts, 0, sizeof(*ts));
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        SISO_CUDA(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres));
        if (!fn || qres != cudaDriverEntryPointSuccess) { delete ts; return check_cuda(cudaErrorNotSupported, "cuTensorMapEncodeTiled lookup"); }
        ts->encode = reinterpret_cast<tc::EncodeTiledFn>(fn);
        siso_status_t st = tc::encode_map(ts->encode, &ts->map_c, c->vecs, static_cast<uint64_t>(c->rows_alloc),
                                          static_cast<uint64_t>(c->dim), tc::TN);
        if (st == SISO_OK)
            st = tc::encode_map(ts->encode, &ts->map_c_half, c->vecs, static_cast<uint64_t>(c->rows_alloc),
                                static_cast<uint64_t>(c->dim), tc::TN / 2);
        if (st == SISO_OK) {
            ts->tail_counter = static_cast<unsigned int *>(cache_alloc_zeroed(c, 256 + 256 * sizeof(unsigned long long)));   // tickets, then one word per row
            if (!ts->tail_counter) st = SISO_ERR_OOM;
        }
        if (st != SISO_OK) { delete ts; return st; }
        c->tensor_state = ts;
    }
    const int kmax = k == 1 ? 1 : (k <= 4 ? 4 : 8);
    const int n_tiles = static_cast<int>((c->capacity + tc::TN - 1) / tc::TN);
    const int64_t m_tiles64 = (B + tc::TM - 1) / tc::TM;
    if (m_tiles64 > 0x7FFFFFFF) return SISO_ERR_UNSUPPORTED;
    const int m_tiles = static_cast<int>(m_tiles64);
    // CTA pairs (two query tiles share every centroid tile) whenever the batch has at least two query tiles
    // (an odd tile count is padded with an idle CTA: not worth it for 3, 5 or 7 query tiles)
    const bool pair = m_tiles >= 2 && (m_tiles % 2 == 0 || m_tiles >= 9) && c->tensor_pair_mode == 0;
    const int m_ctas = pair ? (m_tiles + 1) / 2 * 2 : m_tiles;
    // One CTA per SM at a time.  Few, long splits keep each row's running top-k warm (a fresh CTA inserts often
    // until its k-th best has risen) but quantise badly into waves of sm_count CTAs; try a few wave counts and
    // take the cheapest by a simple model: rounds x (tiles per CTA + a fixed start-up/drain cost in tiles).
    const int64_t units = static_cast<int64_t>(m_ctas) * n_tiles;
    const int wave_cap = static_cast<int>(std::min<int64_t>(16, std::max<int64_t>(1, units / (8ll * c->sm_count))));
    int splits = 1, tiles_per_split = n_tiles;
    int64_t best_cost = -1;
    const int candidates[] = {4, 6, 8, 12, 16};
    for (int ci = 0; ci < 5; ++ci) {
        const int w = std::min(candidates[ci], wave_cap);
        int sp = std::max(1, std::min(std::min(n_tiles, 65535), (c->sm_count * w) / m_ctas));
        const int tps = (n_tiles + sp - 1) / sp;
        sp = (n_tiles + tps - 1) / tps;
        const int64_t rounds = (static_cast<int64_t>(m_ctas) * sp + c->sm_count - 1) / c->sm_count;
        const int64_t cost = rounds * (tps + 6);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; splits = sp; tiles_per_split = tps; }
    }

    // A small batch that does not fill its last tile is copied into zero-filled whole tiles first: the sweep then reads
    // 128 real rows per load instead of rows that the copy engine has to make up (measured: up to 30 % faster for
    // 3-32 queries)
    const bool pad_q = B % tc::TM != 0 && B <= 2048;
    const int64_t padded_rows = static_cast<int64_t>(m_tiles) * tc::TM;
    const size_t pad_bytes = pad_q ? pad256(static_cast<size_t>(padded_rows) * c->dim * sizeof(__nv_bfloat16)) : 0;
    Scratch scr;
    SISO_TRY(scratch_reserve(c, pad256(sizeof(unsigned long long) * B * splits * kmax) + pad_bytes + (defer ? tail_bytes : 0), s, &scr));
    unsigned long long *partial = scr.take<unsigned long long>(static_cast<size_t>(B) * splits * kmax);
    const void *q_rows = q;
    uint64_t q_row_count = static_cast<uint64_t>(B);
    if (pad_q) {
        __nv_bfloat16 *tile = scr.take<__nv_bfloat16>(static_cast<size_t>(padded_rows) * c->dim);
        const long long n16 = padded_rows * c->dim / 8, have16 = B * c->dim / 8;      // 16-byte units
        tc::pad_query_tile_kernel<<<static_cast<unsigned>((n16 + 255) / 256), 256, 0, s>>>(
            static_cast<const uint4 *>(q), reinterpret_cast<uint4 *>(tile), have16, n16);
        SISO_LAUNCHED(c);
        q_rows = tile;
        q_row_count = static_cast<uint64_t>(padded_rows);
    }
    CUtensorMap map_q;
    SISO_TRY(tc::encode_map(ts->encode, &map_q, q_rows, q_row_count, static_cast<uint64_t>(c->dim), tc::TM));
    siso_status_t st;
    // a top-1 lookup of one CTA pair's worth of queries is finished by the sweep itself (no finalisation launch)
    const bool in_sweep = pair && kmax == 1 && m_ctas == 2 && !c->sweep_finalize_separate;
    if (pair)
        st = launch_lookup_tensor_pair(c, ts->attr_set_pair, map_q, ts->map_c_half, B, kmax, tiles_per_split, n_tiles, splits,
                                       m_ctas, partial, in_sweep ? ts->tail_counter : nullptr, theta, theta_s, idx, sim, hit,
                                       defer ? nullptr : c->counters, s);
    else
        st = kmax == 1 ? run_tensor<1>(c, ts, 0, map_q, B, tiles_per_split, n_tiles, splits, m_tiles, partial, s)
           : kmax == 4 ? run_tensor<4>(c, ts, 1, map_q, B, tiles_per_split, n_tiles, splits, m_tiles, partial, s)
                       : run_tensor<8>(c, ts, 2, map_q, B, tiles_per_split, n_tiles, splits, m_tiles, partial, s);
    SISO_TRY(st);
    if (defer) {
        defer->partial = in_sweep ? nullptr : partial;       // NULL: idx / sim / hit are already final
        defer->splits = splits;
        defer->theta = theta;
        defer->theta_s = theta_s;
        defer->sim = sim;
        *tail = scr.base + scr.off;
        return SISO_OK;
    }
    if (in_sweep) return SISO_OK;
    return launch_topk_finalize(c, partial, B, splits, kmax, k, theta, theta_s, idx, sim, hit, s);
}

}  // namespace siso
