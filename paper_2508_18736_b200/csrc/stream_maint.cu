// Maintenance of one streaming micro-batch in ONE cooperative launch: hit update, eviction of what the misses
// lack in free slots, insertion of the misses.  As separate launches these are eight small kernels whose
// launch and drain latencies add up to about as much as the lookup itself; here the phases are separated by
// grid-wide barriers instead.  The arithmetic and every ordering rule are those of update.cu and evict.cu:
//   U   CTA per row: the first hit of a slot owns the slot's group (ascending query order, fp64 sums)
//   E1  CTA 0: m = max(0, misses - free slots); strided sample of 256 live entries, sorted -> splitters
//   E2  all: bucket of every live entry (binary search among the splitters), bucket counts
//   E3  all: entries in the buckets up to the one where the cumulative count reaches m -> candidates
//   E4  all: one warp per candidate counts the candidates below it; rank < m = victim number rank
//   I1  all: free slots per CTA slice;  I2 all: first #miss free slots in ascending order
//   I3  CTA per row: miss number r takes free slot number r
// Used by siso_stream_step for batches of at most 1024 rows; larger batches take the separate kernels.
#include <cooperative_groups.h>

#include "evict_keys.cuh"

namespace cg = cooperative_groups;

namespace siso {

constexpr int SM_THREADS = 256;
constexpr int SM_WARPS = SM_THREADS / 32;
constexpr int SM_MAX_B = 1024;
constexpr int SM_SAMPLE = 256;

struct MaintCtl {
    long long m;                       // victims of this batch
    int n_sample;
    unsigned int n_cand;
    int n_miss;
    int insert_ok;
    unsigned int hist[SM_SAMPLE + 1];
};

struct MaintArgs {
    const void *Q;
    const int32_t *idx;                // [B] best slot per row (stride 1)
    const uint8_t *hit;                // [B]
    int B, D;
    long long capacity;
    void *vecs;
    float *master;
    double *size;
    uint32_t *access;
    unsigned long long *last;
    uint8_t *valid;
    long long *counters;
    int *status;
    int32_t *victims;                  // [B] or NULL
    int32_t *slots_out;                // [B] or NULL
    // scratch
    MaintCtl *ctl;
    Key3 *splitters;                   // [SM_SAMPLE]
    uint16_t *bucket;                  // [capacity]
    Key3 *cand;                        // [capacity]
    int *cta_free;                     // [grid]
    int32_t *free_list;                // [B]
};

__device__ __forceinline__ int block_exclusive_scan_256(int v, int *total, int *warp_sum) {
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
    int before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < SM_WARPS; ++w) {
        if (w < warp) before += warp_sum[w];
        all += warp_sum[w];
    }
    *total = all;
    return before + x - v;
}

template <typename T> __device__ __forceinline__ float4 maint_load4(const T *p);
template <> __device__ __forceinline__ float4 maint_load4<float>(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
template <> __device__ __forceinline__ float4 maint_load4<__nv_bfloat16>(const __nv_bfloat16 *p) {
    const uint2 u = __ldg(reinterpret_cast<const uint2 *>(p));
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xFFFF0000u));
}

struct MaintSmem {
    double red[SM_WARPS];
    int warp_sum[SM_WARPS];
    int n_members;
    int p;
    uint16_t members[SM_MAX_B];
    unsigned long long k0[SM_SAMPLE], k1[SM_SAMPLE], k2[SM_SAMPLE];
    unsigned int hist[SM_SAMPLE + 1];
};

// ---- phase U: hit update of the group that row b heads (see update_small_kernel in update.cu) ----------------
template <typename T>
__device__ void maint_update_row(const MaintArgs &a, int b, long long clock_new, double *acc, MaintSmem &sm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T *Q = static_cast<const T *>(a.Q);
    T *vecs = static_cast<T *>(a.vecs);
    bool work = false;
    long long slot = -1;
    if (a.hit[b]) {
        slot = a.idx[b];
        if (slot >= 0 && slot < a.capacity && a.valid[slot]) work = true;
        else if (tid == 0) set_status(a.status, SISO_ERR_INVALID_ARG);
    }
    int earlier = 0;
    if (work)
        for (int r = tid; r < b; r += SM_THREADS) earlier |= (a.hit[r] && a.idx[r] == slot) ? 1 : 0;
    if (__syncthreads_or(earlier) != 0) work = false;      // an earlier row owns this slot's group
    if (!work) return;                                      // uniform for the CTA
    int base_count = 0;
    for (int r0 = b; r0 < a.B; r0 += SM_THREADS) {
        const int r = r0 + tid;
        const bool mine = r < a.B && a.hit[r] && a.idx[r] == slot;
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, mine);
        if (lane == 0) sm.warp_sum[warp] = __popc(ballot);
        __syncthreads();
        int before = base_count, total = 0;
        for (int w = 0; w < SM_WARPS; ++w) { if (w < warp) before += sm.warp_sum[w]; total += sm.warp_sum[w]; }
        if (mine) sm.members[before + __popc(ballot & ((1u << lane) - 1u))] = static_cast<uint16_t>(r);
        base_count += total;
        __syncthreads();
    }
    const int count = base_count;
    const double n_old = a.size[slot];
    float *m = a.master + slot * a.D;
    for (int d = tid; d < a.D; d += SM_THREADS) acc[d] = n_old * static_cast<double>(m[d]);
    __syncthreads();
    const int quads = a.D / 4;
    constexpr int R = 8;
    for (int t = 0; t < count; t += R) {
        const int nrow = count - t < R ? count - t : R;
        const T *q[R];
#pragma unroll
        for (int r = 0; r < R; ++r) q[r] = Q + static_cast<long long>(sm.members[t + (r < nrow ? r : 0)]) * a.D;
        for (int g = tid; g < quads; g += SM_THREADS) {
            float4 v[R];
#pragma unroll
            for (int r = 0; r < R; ++r) v[r] = maint_load4<T>(q[r] + 4 * g);
            double a0 = acc[4 * g], a1 = acc[4 * g + 1], a2 = acc[4 * g + 2], a3 = acc[4 * g + 3];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (r < nrow) { a0 += v[r].x; a1 += v[r].y; a2 += v[r].z; a3 += v[r].w; }
            }
            acc[4 * g] = a0; acc[4 * g + 1] = a1; acc[4 * g + 2] = a2; acc[4 * g + 3] = a3;
        }
    }
    __syncthreads();
    double ss = 0.0;
    for (int d = tid; d < a.D; d += SM_THREADS) ss += acc[d] * acc[d];
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
    if (lane == 0) sm.red[warp] = ss;
    __syncthreads();
    double nn = 0.0;
    for (int w = 0; w < SM_WARPS; ++w) nn += sm.red[w];
    const double norm = sqrt(nn);
    T *v = vecs + slot * a.D;
    for (int d = tid; d < a.D; d += SM_THREADS) {
        const float f = static_cast<float>(acc[d] / norm);
        m[d] = f;
        if constexpr (sizeof(T) == 2) v[d] = __float2bfloat16_rn(f);
    }
    if (tid == 0) {
        a.size[slot] = n_old + static_cast<double>(count);
        const unsigned long long ac = static_cast<unsigned long long>(a.access[slot]) + static_cast<unsigned long long>(count);
        a.access[slot] = (a.access[slot] == SISO_ACCESS_INF || ac >= SISO_ACCESS_INF) ? SISO_ACCESS_INF : static_cast<uint32_t>(ac);
        a.last[slot] = static_cast<unsigned long long>(clock_new);
    }
    __syncthreads();      // acc and members are reused by the CTA's next row
}

// ---- phase E1 (CTA 0): how many victims; sample and sort the splitters ------------------------------------------
__device__ void maint_evict_sample(const MaintArgs &a, long long clock_new, MaintSmem &sm) {
    const int tid = threadIdx.x;
    const long long occupancy = a.counters[CNT_OCCUPANCY];
    int miss = 0;
    for (int b = tid; b < a.B; b += SM_THREADS) miss += a.hit[b] ? 0 : 1;
    int n_miss;
    block_exclusive_scan_256(miss, &n_miss, sm.warp_sum);
    long long m = static_cast<long long>(n_miss) - (a.capacity - occupancy);
    m = m > 0 ? m : 0;
    m = m < occupancy ? m : occupancy;
    if (a.victims)
        for (long long r = m + tid; r < a.B; r += SM_THREADS) a.victims[r] = -1;
    if (tid == 0) { a.ctl->m = m; a.ctl->n_cand = 0; a.ctl->n_miss = n_miss; }
    for (int i = tid; i <= SM_SAMPLE; i += SM_THREADS) a.ctl->hist[i] = 0;
    if (m == 0) return;
    const long long stride = (a.capacity + SM_SAMPLE - 1) / SM_SAMPLE;
    const long long lo = tid * stride, hi = min(a.capacity, lo + stride);
    const long long span = hi - lo;
    int have = 0;
    Key3 mine;
    mine.w0 = mine.w1 = mine.w2 = ~0ull;
    if (span > 0) {
        // the same window offset as evict_sample_kernel uses, which reads the clock after the update advanced it
        const long long start = static_cast<long long>((static_cast<unsigned long long>(clock_new) * 2654435761ull) % static_cast<unsigned long long>(span));
        const long long probes = span < 64 ? span : 64;
        for (long long i = 0; i < probes; ++i) {
            long long sl = lo + start + i;
            if (sl >= hi) sl -= span;
            if (a.valid[sl]) { mine = make_key(a.size[sl], a.access[sl], a.last[sl], static_cast<uint32_t>(sl)); have = 1; break; }
        }
    }
    sm.k0[tid] = mine.w0; sm.k1[tid] = mine.w1; sm.k2[tid] = mine.w2;
    int n_sample;
    block_exclusive_scan_256(have, &n_sample, sm.warp_sum);
    __syncthreads();
    for (int k = 2; k <= SM_SAMPLE; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            const int partner = tid ^ j;
            if (partner > tid) {
                Key3 x, y;
                x.w0 = sm.k0[tid]; x.w1 = sm.k1[tid]; x.w2 = sm.k2[tid];
                y.w0 = sm.k0[partner]; y.w1 = sm.k1[partner]; y.w2 = sm.k2[partner];
                const bool up = (tid & k) == 0;
                if (key_less(y, x) == up) {
                    sm.k0[tid] = y.w0; sm.k1[tid] = y.w1; sm.k2[tid] = y.w2;
                    sm.k0[partner] = x.w0; sm.k1[partner] = x.w1; sm.k2[partner] = x.w2;
                }
            }
            __syncthreads();
        }
    }
    Key3 out;
    out.w0 = sm.k0[tid]; out.w1 = sm.k1[tid]; out.w2 = sm.k2[tid];
    a.splitters[tid] = out;
    if (tid == 0) a.ctl->n_sample = n_sample;
}

// ---- phase E2 (all CTAs): bucket of every live entry ------------------------------------------------------------
__device__ void maint_evict_bucket(const MaintArgs &a, MaintSmem &sm) {
    if (a.ctl->m == 0) return;
    const int tid = threadIdx.x;
    const int n_sample = a.ctl->n_sample;
    {
        const Key3 k = a.splitters[tid];
        sm.k0[tid] = k.w0; sm.k1[tid] = k.w1; sm.k2[tid] = k.w2;
    }
    for (int i = tid; i <= SM_SAMPLE; i += SM_THREADS) sm.hist[i] = 0;
    __syncthreads();
    for (long long sl = static_cast<long long>(blockIdx.x) * SM_THREADS + tid; sl < a.capacity;
         sl += static_cast<long long>(gridDim.x) * SM_THREADS) {
        if (!a.valid[sl]) continue;
        const Key3 k = make_key(a.size[sl], a.access[sl], a.last[sl], static_cast<uint32_t>(sl));
        int lo = 0, hi = n_sample;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            Key3 sp;
            sp.w0 = sm.k0[mid]; sp.w1 = sm.k1[mid]; sp.w2 = sm.k2[mid];
            if (key_less(sp, k)) lo = mid + 1; else hi = mid;
        }
        a.bucket[sl] = static_cast<uint16_t>(lo);
        atomicAdd(&sm.hist[lo], 1u);
    }
    __syncthreads();
    for (int i = tid; i <= SM_SAMPLE; i += SM_THREADS)
        if (sm.hist[i]) atomicAdd(&a.ctl->hist[i], sm.hist[i]);
}

// ---- phase E3 (all CTAs): candidates = entries in buckets 0..p, p the first bucket where the count reaches m ----
__device__ void maint_evict_collect(const MaintArgs &a, MaintSmem &sm) {
    const long long m = a.ctl->m;
    if (m == 0) return;
    const int tid = threadIdx.x, lane = tid & 31;
    if (tid < 32) {
        long long run = 0;
        int found = SM_SAMPLE;
        for (int base = 0; base <= SM_SAMPLE && found == SM_SAMPLE; base += 32) {
            const int i = base + tid;
            long long x = i <= SM_SAMPLE ? a.ctl->hist[i] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const long long y = __shfl_up_sync(0xFFFFFFFFu, x, o);
                if (tid >= o) x += y;
            }
            const unsigned reach = __ballot_sync(0xFFFFFFFFu, run + x >= m);
            if (reach) found = base + __ffs(reach) - 1;
            run += __shfl_sync(0xFFFFFFFFu, x, 31);
        }
        if (tid == 0) sm.p = found;
    }
    __syncthreads();
    const int p = sm.p;
    for (long long base = static_cast<long long>(blockIdx.x) * SM_THREADS; base < a.capacity;
         base += static_cast<long long>(gridDim.x) * SM_THREADS) {
        const long long sl = base + tid;
        const bool take = sl < a.capacity && a.valid[sl] && a.bucket[sl] <= p;
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, take);
        if (ballot) {
            unsigned int warp_base = 0;
            if (lane == 0) warp_base = atomicAdd(&a.ctl->n_cand, static_cast<unsigned int>(__popc(ballot)));
            warp_base = __shfl_sync(0xFFFFFFFFu, warp_base, 0);
            if (take) a.cand[warp_base + __popc(ballot & ((1u << lane) - 1u))] =
                          make_key(a.size[sl], a.access[sl], a.last[sl], static_cast<uint32_t>(sl));
        }
    }
}

// ---- phase E4 (all CTAs): rank the candidates, the m lowest are the victims -------------------------------------
__device__ void maint_evict_rank(const MaintArgs &a) {
    const long long m = a.ctl->m;
    if (m == 0) return;
    const unsigned int n = a.ctl->n_cand;
    const int lane = threadIdx.x & 31;
    const unsigned int warps = gridDim.x * SM_WARPS;
    for (unsigned int i = blockIdx.x * SM_WARPS + (threadIdx.x >> 5); i < n; i += warps) {
        const Key3 mine = a.cand[i];
        unsigned int rank = 0;
        for (unsigned int j = lane; j < n; j += 32) rank += key_less(a.cand[j], mine) ? 1u : 0u;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, o);
        if (lane == 0 && rank < m) {
            const int32_t slot = static_cast<int32_t>(mine.w2 & 0xFFFFFFFFull);
            if (a.victims) a.victims[rank] = slot;
            a.valid[slot] = 0;
        }
    }
}

// ---- phases I1/I2 (all CTAs): the first n_miss free slots in ascending order ------------------------------------
// CTA g owns the contiguous slice [g * per, (g + 1) * per) of the slots; thread t owns `chunk` consecutive slots of it.
__device__ void maint_free_count(const MaintArgs &a, long long per, MaintSmem &sm) {
    const long long lo = static_cast<long long>(blockIdx.x) * per, hi = min(a.capacity, lo + per);
    int c = 0;
    for (long long sl = lo + threadIdx.x; sl < hi; sl += SM_THREADS) c += a.valid[sl] ? 0 : 1;
    int total;
    block_exclusive_scan_256(c, &total, sm.warp_sum);
    if (threadIdx.x == 0) a.cta_free[blockIdx.x] = total;
}

__device__ void maint_free_list(const MaintArgs &a, long long per, MaintSmem &sm) {
    const int tid = threadIdx.x;
    const int n_miss = a.ctl->n_miss;
    // free slots in the slices before this one, and in all slices
    int mine = 0, all = 0;
    for (int g = tid; g < static_cast<int>(gridDim.x); g += SM_THREADS) {
        const int f = a.cta_free[g];
        all += f;
        if (g < static_cast<int>(blockIdx.x)) mine += f;
    }
    int dummy;
    // two block-wide sums through the scan helper (the total is what is wanted)
    block_exclusive_scan_256(mine, &dummy, sm.warp_sum);
    const int base = dummy;
    __syncthreads();
    block_exclusive_scan_256(all, &dummy, sm.warp_sum);
    const int n_free = dummy;
    __syncthreads();
    if (blockIdx.x == 0 && tid == 0) {
        const int ok = n_miss <= n_free ? 1 : 0;
        a.ctl->insert_ok = ok;
        if (!ok) set_status(a.status, SISO_ERR_CAPACITY);
    }
    if (n_miss > n_free || base >= n_miss) return;       // nothing of this slice is needed
    const long long lo = static_cast<long long>(blockIdx.x) * per, hi = min(a.capacity, lo + per);
    const long long chunk = (per + SM_THREADS - 1) / SM_THREADS;
    const long long t_lo = lo + tid * chunk, t_hi = min(hi, t_lo + chunk);
    int c = 0;
    for (long long sl = t_lo; sl < t_hi; ++sl) c += a.valid[sl] ? 0 : 1;
    int total;
    int rank = base + block_exclusive_scan_256(c, &total, sm.warp_sum);
    for (long long sl = t_lo; sl < t_hi; ++sl) {
        if (!a.valid[sl]) {
            if (rank < n_miss) a.free_list[rank] = static_cast<int32_t>(sl);
            ++rank;
        }
    }
}

// ---- phase I3: row b, if it is a miss, takes free slot number (misses before b) ---------------------------------
template <typename T>
__device__ void maint_insert_row(const MaintArgs &a, int b, long long clock_new, MaintSmem &sm) {
    const int tid = threadIdx.x;
    const bool ok = a.ctl->insert_ok != 0;
    if (a.hit[b] || !ok) {
        if (tid == 0 && a.slots_out) a.slots_out[b] = -1;
        return;
    }
    int before = 0;
    for (int r = tid; r < b; r += SM_THREADS) before += a.hit[r] ? 0 : 1;
    int rank;
    block_exclusive_scan_256(before, &rank, sm.warp_sum);
    const int32_t slot = a.free_list[rank];
    const T *src = static_cast<const T *>(a.Q) + static_cast<long long>(b) * a.D;
    T *dv = static_cast<T *>(a.vecs) + static_cast<long long>(slot) * a.D;
    float *dm = a.master + static_cast<long long>(slot) * a.D;
    for (int d = tid; d < a.D; d += SM_THREADS) {
        const T x = src[d];
        dv[d] = x;
        if constexpr (sizeof(T) == 2) dm[d] = __bfloat162float(x);
    }
    if (tid == 0) {
        a.size[slot] = 1.0;
        a.access[slot] = SISO_ACCESS_INF;
        a.last[slot] = static_cast<unsigned long long>(clock_new);
        a.valid[slot] = 1;
        if (a.slots_out) a.slots_out[b] = slot;
    }
    __syncthreads();
}

template <typename T>
__global__ void __launch_bounds__(SM_THREADS)
stream_maint_kernel(const MaintArgs a) {
    extern __shared__ double acc[];          // [D]
    __shared__ MaintSmem sm;
    cg::grid_group grid = cg::this_grid();
    const long long clock_new = a.counters[CNT_CLOCK] + 1;      // nobody writes the clock before the first barrier
    for (int b = blockIdx.x; b < a.B; b += gridDim.x) maint_update_row<T>(a, b, clock_new, acc, sm);
    grid.sync();
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0) a.counters[CNT_CLOCK] = clock_new;
        maint_evict_sample(a, clock_new, sm);
    }
    grid.sync();
    maint_evict_bucket(a, sm);
    grid.sync();
    maint_evict_collect(a, sm);
    grid.sync();
    maint_evict_rank(a);
    const long long per = (a.capacity + gridDim.x - 1) / gridDim.x;
    grid.sync();
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        a.counters[CNT_OCCUPANCY] -= a.ctl->m;
        a.counters[CNT_EVICTIONS] += a.ctl->m;
    }
    maint_free_count(a, per, sm);
    grid.sync();
    maint_free_list(a, per, sm);
    grid.sync();
    for (int b = blockIdx.x; b < a.B; b += gridDim.x) maint_insert_row<T>(a, b, clock_new, sm);
    if (blockIdx.x == 0 && threadIdx.x == 0 && a.ctl->insert_ok) {
        a.counters[CNT_OCCUPANCY] += a.ctl->n_miss;
        a.counters[CNT_INSERTS] += a.ctl->n_miss;
    }
}

// Returns SISO_ERR_UNSUPPORTED if this batch cannot take the fused path (the caller then uses the separate kernels).
siso_status_t launch_stream_maint(Cache *c, const void *q, int64_t B, const int32_t *idx, const uint8_t *hit,
                                  int32_t *victims, int32_t *slots_out, cudaStream_t s) {
    if (B < 1 || B > SM_MAX_B) return SISO_ERR_UNSUPPORTED;
    if (c->maint_grid == 0) {
        int coop = 0;
        SISO_CUDA(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device));
        int per_sm = 0;
        const size_t smem = sizeof(double) * c->dim;
        cudaError_t e = c->dtype == SISO_F32
            ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, stream_maint_kernel<float>, SM_THREADS, smem)
            : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, stream_maint_kernel<__nv_bfloat16>, SM_THREADS, smem);
        SISO_CUDA(e);
        c->maint_grid = (coop && per_sm >= 1) ? c->sm_count * std::min(per_sm, 2) : -1;
    }
    if (c->maint_grid < 0) return SISO_ERR_UNSUPPORTED;
    const int grid = c->maint_grid;
    Scratch scr;
    const size_t need = pad256(sizeof(MaintCtl)) + pad256(sizeof(Key3) * SM_SAMPLE) + pad256(sizeof(uint16_t) * c->capacity) +
                        pad256(sizeof(Key3) * c->capacity) + pad256(sizeof(int) * grid) + pad256(sizeof(int32_t) * B);
    SISO_TRY(scratch_reserve(c, need, s, &scr));
    MaintArgs a;
    a.Q = q; a.idx = idx; a.hit = hit; a.B = static_cast<int>(B); a.D = c->dim; a.capacity = c->capacity;
    a.vecs = c->vecs; a.master = c->master; a.size = c->size; a.access = c->access; a.last = c->last; a.valid = c->valid;
    a.counters = c->counters; a.status = c->status; a.victims = victims; a.slots_out = slots_out;
    a.ctl = scr.take<MaintCtl>(1);
    a.splitters = scr.take<Key3>(SM_SAMPLE);
    a.bucket = scr.take<uint16_t>(c->capacity);
    a.cand = scr.take<Key3>(c->capacity);
    a.cta_free = scr.take<int>(grid);
    a.free_list = scr.take<int32_t>(B);
    void *args[] = {&a};
    const size_t smem = sizeof(double) * c->dim;
    const void *fn = c->dtype == SISO_F32 ? reinterpret_cast<const void *>(stream_maint_kernel<float>)
                                          : reinterpret_cast<const void *>(stream_maint_kernel<__nv_bfloat16>);
    SISO_CUDA(cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(SM_THREADS), args, smem, s));
    c->launches += 1;
    return SISO_OK;
}

}  // namespace siso
