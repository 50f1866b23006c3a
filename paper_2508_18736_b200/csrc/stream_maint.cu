// Maintenance of one streaming micro-batch in ONE cooperative launch: (top-1 finalisation of the lookup,) hit
// update, eviction of what the misses lack in free slots, insertion of the misses.  As separate launches these
// are ten small kernels whose launch and drain latencies add up to about as much as the lookup itself; here the
// phases are separated by grid-wide barriers, four of them in the steady state.  The arithmetic and every
// ordering rule are those of update.cu and evict.cu (Alg. 1 FilteringCentroids order; running-mean update):
//   F   (only when the lookup left its per-split partial results) one warp per row: best key, threshold test
//   U   CTA per row: the first hit of a slot owns the slot's group (ascending query order, fp64 sums);
//       meanwhile the last CTA draws a strided sample of 256 live entries and puts its P+1 smallest keys in
//       order -> splitters 0..P (P chosen so that about 3 m entries lie below splitter P)
//   S   CTA g owns the contiguous slice g of the slots: free slots of the slice; entries whose key is at most
//       splitter P become candidates, counted per bucket
//   R   p = first bucket where the cumulative count reaches m; every fourth CTA copies the candidates up to
//       splitter p to shared memory and ranks its share of them (one warp per candidate); rank < m = victim
//       number rank
//   I   the first #miss free slots in ascending order take the misses in ascending row order.  A full cache has
//       no free slots but the victims, so every CTA sorts the victims by slot and copies its share of the rows;
//       otherwise each CTA lists the free slots of its slice, and after one more barrier all CTAs copy
// If the sample misleads (fewer than m candidates) the selection falls back to a full sort of the sample, a full
// histogram pass and a collection pass, as evict.cu does.  Whatever the splitters are, the victims are the m
// smallest keys exactly.
// Used by siso_stream_step for batches of at most 1024 rows; larger batches take the separate kernels.
//
// Steady state of a full cache (every batch evicts exactly its misses): phases S and R and all barriers are
// replaced by a list that lives across batches.  The list holds, in eviction order, EVERY live entry whose key is
// at most a bound (about 3,000 entries after a rebuild).  The victims of a batch are the m lowest keys AFTER the
// hit update; a hit only raises a key, so with at least 2B entries in the list the m lowest are found among its
// first 2B entries (at most B of them were hit, so at least B >= m keep their key and stay below everything
// outside).  Every CTA derives the same victims from that prefix on its own (mark the hit entries with a hash of
// the batch's hit slots, give them their new keys, rank by position), so update and insertion run without a
// grid-wide barrier; a hit entry that is evicted in the same batch is not updated (its slot is overwritten by a
// miss).  The last CTA then takes the victims and the hit entries out of the list; an entry whose new key would
// still lie below the bound, or a new entry that does, cuts the list (and the bound) off just below that key, so
// the list always holds ALL live entries up to its bound.  When fewer than 2B entries are left, or another entry
// point has changed the cache, the batch takes the phases above and the list is rebuilt from a sample-chosen bound.
#include <cooperative_groups.h>

#include "evict_keys.cuh"

namespace cg = cooperative_groups;

namespace siso {

constexpr int SM_THREADS = 256;
constexpr int SM_WARPS = SM_THREADS / 32;
constexpr int SM_MAX_B = 1024;
constexpr int SM_SAMPLE = 256;
constexpr int SM_STAGE = 2048;      // candidates a CTA can hold in shared memory while ranking
constexpr int SM_SELECT = 16;       // up to this many splitters are extracted one by one instead of sorting the sample
constexpr int SM_RANK_STRIDE = 4;   // every fourth CTA ranks candidates
constexpr int SM_DENSE = 4;         // entries per sampler thread in the fine sample (4 x 256 entries)

constexpr int LOW_K = 4096;         // capacity of the eviction-order list kept across batches
constexpr int LOW_TARGET = 3072;    // entries a rebuild aims at
constexpr int LOW_UPD = 256;        // hit entries inside the examined prefix that the barrier-free path handles
constexpr int LOW_MAP_BITS = 13;
constexpr int LOW_MAP = 1 << LOW_MAP_BITS;   // open-addressing table slot -> position in the list (load at most 1/2)
constexpr int LOW_PER_THREAD = LOW_K / SM_THREADS;
constexpr unsigned int LOW_SPIN_LIMIT = 1u << 18;

// Every live entry with key <= bound (all live entries if has_bound == 0) is among k[head .. n), ascending.  An entry
// that was hit leaves the list by a mark (dead[i] = 1: its key has risen above the bound); the victims of a batch are
// the first entries that are neither marked nor hit, so evicting them moves `head` forward and nothing is copied.
// Written only by the streaming maintenance kernel; the host flag Cache::low_dirty says whether any other entry point
// has touched the cache since.
struct LowList {
    int n;                    // end of the list
    int head;                 // first entry still in it
    int n_dead;               // marked entries in [head, n), or more (it only sizes the prefix that is examined)
    int valid;
    int has_bound;
    int pad;
    Key3 bound;
    unsigned int started;     // CTAs of the running kernel that no longer read the list (reset by the writer)
    unsigned int n_cand;      // rebuild: candidates collected
    unsigned long long k0[LOW_K], k1[LOW_K], k2[LOW_K];
    uint8_t dead[LOW_K];
    unsigned long long map[LOW_MAP];   // (slot + 1) << 32 | position, 0 = empty; written by the rebuild only
};

struct MaintCtl {
    unsigned int n_cand;                 // candidates appended in phase S
    unsigned int n_cand_full;            // candidates of the fall-back collection
    int n_sample;
    unsigned int hist[SM_SAMPLE + 1];    // phase S: buckets 0..P
    unsigned int hist_full[SM_SAMPLE + 1];
};

struct MaintArgs {
    const void *Q;
    int32_t *idx;                      // [B] best slot per row (stride 1); written by phase F
    uint8_t *hit;                      // [B]
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
    // phase F (partial == NULL: idx and hit are inputs)
    int count_lookup;                  // the lookup of this batch has not been counted yet (lookups, hits)
    const unsigned long long *partial; // [B, splits] packed (similarity, slot) keys
    int splits;
    const float *theta;
    float theta_s;
    float *sim;                        // [B]
    // scratch
    MaintCtl *ctl;
    Key3 *splitters;                   // [SM_SAMPLE]
    uint16_t *bucket;                  // [capacity] (fall-back only)
    unsigned long long *cand0, *cand1, *cand2;   // [capacity] each: the candidates' key words
    int32_t *victim_buf;               // [B] victims in key order (always present, unlike `victims`)
    int *cta_free;                     // [grid]
    int32_t *free_list;                // [B]
    LowList *low;                      // eviction-order list kept across batches
    int low_ok;                        // host: nothing but this kernel has changed the cache since the list was written
};

// fixed part of the shared memory; it follows the 48 KiB that hold the fp64 row accumulator during the update and
// the candidates during ranking
struct MaintSmem {
    unsigned long long k0[SM_SAMPLE], k1[SM_SAMPLE], k2[SM_SAMPLE];    // splitters (sorting area of the sampler)
    double red[SM_WARPS];
    unsigned int hist[SM_SAMPLE + 1];
    int warp_sum[SM_WARPS];
    int32_t idx[SM_MAX_B];
    uint16_t miss_list[SM_MAX_B];
    uint16_t members[SM_MAX_B];
    uint8_t hit[SM_MAX_B];
    int n_stage;
    int p;
    // barrier-free path
    int32_t vict[SM_MAX_B];            // victims in eviction order
    int32_t by_slot[SM_MAX_B];         // victims in slot order
    uint32_t pcnt[2 * SM_MAX_B];       // hits of this batch on entry i of the prefix
    uint16_t hb[2 * SM_MAX_B + 1];     // hit entries of the list before position i
    uint8_t lflag[2 * SM_MAX_B];       // entry i of the prefix: 1 = hit in this batch, 2 = marked earlier
    unsigned long long u0[LOW_UPD], u1[LOW_UPD], u2[LOW_UPD];    // new keys of the hit entries of the prefix
    uint16_t upos[LOW_UPD];            // their positions in the list
    uint8_t uvict[LOW_UPD];            // evicted all the same
    int n_upd;
    int v_end;                         // prefix position just behind the last victim that was not hit in this batch
};
constexpr size_t SM_UNION_BYTES = 3 * sizeof(unsigned long long) * SM_STAGE;      // 48 KiB >= 8 * kMaxDim
constexpr size_t SM_SMEM_BYTES = SM_UNION_BYTES + sizeof(MaintSmem);
static_assert(SM_UNION_BYTES >= sizeof(double) * kMaxDim, "row accumulator must fit");

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

__device__ __forceinline__ int block_max_256(int v, int *warp_sum) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = v;
    __syncthreads();
    int r = warp_sum[0];
#pragma unroll
    for (int w = 1; w < SM_WARPS; ++w) r = max(r, warp_sum[w]);
    return r;
}

template <typename T> __device__ __forceinline__ float4 maint_load4(const T *p);
template <> __device__ __forceinline__ float4 maint_load4<float>(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
template <> __device__ __forceinline__ float4 maint_load4<__nv_bfloat16>(const __nv_bfloat16 *p) {
    const uint2 u = __ldg(reinterpret_cast<const uint2 *>(p));
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xFFFF0000u));
}

__device__ __forceinline__ Key3 smem_key(const MaintSmem &sm, int i) {
    Key3 k;
    k.w0 = sm.k0[i]; k.w1 = sm.k1[i]; k.w2 = sm.k2[i];
    return k;
}

// number of splitters among the first n that are smaller than k
__device__ __forceinline__ int splitter_lower_bound(const MaintSmem &sm, int n, const Key3 &k) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (key_less(smem_key(sm, mid), k)) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// ---- phase F: best key of every row over the lookup's splits, strict threshold test --------------------------
__device__ void maint_finalize(const MaintArgs &a) {
    const int lane = threadIdx.x & 31;
    const int warps = gridDim.x * SM_WARPS;
    for (int b = blockIdx.x * SM_WARPS + (threadIdx.x >> 5); b < a.B; b += warps) {
        const unsigned long long *src = a.partial + static_cast<long long>(b) * a.splits;
        unsigned long long best = 0ull;
        for (int s = lane; s < a.splits; s += 32) { const unsigned long long v = src[s]; best = v > best ? v : best; }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            const unsigned long long v = __shfl_xor_sync(0xFFFFFFFFu, best, o);
            best = v > best ? v : best;
        }
        if (lane == 0) {
            a.idx[b] = best ? key_slot(best) : -1;
            a.sim[b] = best ? key_sim(best) : -INFINITY;
            const float th = a.theta ? a.theta[b] : a.theta_s;
            a.hit[b] = (best != 0ull && key_sim(best) > th) ? 1 : 0;
        }
    }
}

// ---- phase U: hit update of the group that row b heads (see update_small_kernel in update.cu) ----------------
template <typename T>
__device__ void maint_update_row(const MaintArgs &a, int b, long long clock_new, double *acc, MaintSmem &sm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T *Q = static_cast<const T *>(a.Q);
    T *vecs = static_cast<T *>(a.vecs);
    constexpr int MR = 4;                       // master elements per thread fetched ahead (covers D <= 1024)
    long long slot = -1;
    bool work = false;
    double n_old = 0.0;
    uint32_t ac_old = 0;
    float mreg[MR];
    if (sm.hit[b]) {
        slot = sm.idx[b];
        if (slot >= 0 && slot < a.capacity) {
            // everything the update reads of the slot is requested at once, before the ownership test below
            const uint8_t live = a.valid[slot];
            n_old = a.size[slot];
            ac_old = a.access[slot];
            const float *m = a.master + slot * a.D;
#pragma unroll
            for (int j = 0; j < MR; ++j) { const int d = tid + j * SM_THREADS; mreg[j] = d < a.D ? m[d] : 0.0f; }
            work = live != 0;
        }
        if (!work && tid == 0) set_status(a.status, SISO_ERR_INVALID_ARG);
    }
    int earlier = 0;
    if (work)
        for (int r = tid; r < b; r += SM_THREADS) earlier |= (sm.hit[r] && sm.idx[r] == slot) ? 1 : 0;
    if (__syncthreads_or(earlier) != 0) work = false;      // an earlier row owns this slot's group
    if (!work) return;                                      // uniform for the CTA
    int base_count = 0;
    for (int r0 = b; r0 < a.B; r0 += SM_THREADS) {
        const int r = r0 + tid;
        const bool mine = r < a.B && sm.hit[r] && sm.idx[r] == slot;
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
    float *m = a.master + slot * a.D;
#pragma unroll
    for (int j = 0; j < MR; ++j) { const int d = tid + j * SM_THREADS; if (d < a.D) acc[d] = n_old * static_cast<double>(mreg[j]); }
    for (int d = tid + MR * SM_THREADS; d < a.D; d += SM_THREADS) acc[d] = n_old * static_cast<double>(m[d]);
    __syncthreads();
    const int quads = a.D / 4;
    constexpr int R = 16;                       // rows in flight per thread
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
        const unsigned long long ac = static_cast<unsigned long long>(ac_old) + static_cast<unsigned long long>(count);
        a.access[slot] = (ac_old == SISO_ACCESS_INF || ac >= SISO_ACCESS_INF) ? SISO_ACCESS_INF : static_cast<uint32_t>(ac);
        a.last[slot] = static_cast<unsigned long long>(clock_new);
    }
    __syncthreads();      // acc and members are reused by the CTA's next row
}

// splitter index P: entries with a key up to splitter P are looked at (about 3 m of them are expected)
__device__ __forceinline__ int maint_spec_buckets(long long m, int n_sample, long long occupancy) {
    if (n_sample == 0) return 0;
    const long long want = (3 * m * (n_sample + 1) + occupancy - 1) / occupancy + 1;
    return static_cast<int>(want < n_sample ? want : n_sample);
}

// smallest key of the CTA's 256 (each thread passes its own); all threads get it
__device__ __forceinline__ Key3 block_min_key(Key3 k, MaintSmem &sm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        Key3 y;
        y.w0 = __shfl_xor_sync(0xFFFFFFFFu, k.w0, o);
        y.w1 = __shfl_xor_sync(0xFFFFFFFFu, k.w1, o);
        y.w2 = __shfl_xor_sync(0xFFFFFFFFu, k.w2, o);
        if (key_less(y, k)) k = y;
    }
    __syncthreads();
    if (lane == 0) { sm.k0[warp] = k.w0; sm.k1[warp] = k.w1; sm.k2[warp] = k.w2; }
    __syncthreads();
    Key3 best = smem_key(sm, 0);
#pragma unroll
    for (int w = 1; w < SM_WARPS; ++w) {
        const Key3 y = smem_key(sm, w);
        if (key_less(y, best)) best = y;
    }
    return best;
}

// ---- sampler (one CTA): strided sample of live entries -> splitters ------------------------------------------
// The sample only steers the selection (which entries are looked at closely), so it may see an entry before or
// after this batch's update of it.  With `all` the whole sample is sorted; otherwise only its P+1 smallest keys
// are put in order (P as maint_spec_buckets gives it), which is all that phases S and R read.
__device__ void maint_evict_sample(const MaintArgs &a, long long clock_new, long long m, long long occupancy, bool all,
                                   MaintSmem &sm) {
    const int tid = threadIdx.x;
    const long long stride = (a.capacity + SM_SAMPLE - 1) / SM_SAMPLE;
    const long long lo = tid * stride, hi = min(a.capacity, lo + stride);
    // up to SM_DENSE live entries of this thread's window, one from each quarter of it (the first one serves the
    // 256-entry sample that is sorted in full; all of them serve the finer sample of which only the few smallest
    // keys are needed)
    Key3 k[SM_DENSE];
    int have[SM_DENSE];
    const long long sub = (stride + SM_DENSE - 1) / SM_DENSE;
#pragma unroll
    for (int d = 0; d < SM_DENSE; ++d) {
        k[d].w0 = k[d].w1 = k[d].w2 = ~0ull;
        have[d] = 0;
        const long long s_lo = min(hi, lo + d * sub), s_hi = min(hi, s_lo + sub);
        const long long span = s_hi - s_lo;
        if (span > 0) {
            const long long start = static_cast<long long>((static_cast<unsigned long long>(clock_new) * 2654435761ull) % static_cast<unsigned long long>(span));
            const long long probes = span < 16 ? span : 16;
            for (long long i = 0; i < probes; ++i) {
                long long sl = s_lo + start + i;
                if (sl >= s_hi) sl -= span;
                // the four loads do not wait for one another: a full cache answers at the first probe
                const uint8_t live = a.valid[sl];
                const double sz = a.size[sl];
                const uint32_t ac = a.access[sl];
                const unsigned long long la = a.last[sl];
                if (live) { k[d] = make_key(sz, ac, la, static_cast<uint32_t>(sl)); have[d] = 1; break; }
            }
        }
    }
    int n_dense, n_sample;
    {
        int h = 0;
#pragma unroll
        for (int d = 0; d < SM_DENSE; ++d) h += have[d];
        block_exclusive_scan_256(h, &n_dense, sm.warp_sum);
        __syncthreads();
    }
    const int P_dense = maint_spec_buckets(m, n_dense, occupancy);
    if (!all && P_dense < SM_SELECT && P_dense < n_dense) {
        // the P+1 smallest of the fine sample, one block-wide minimum at a time (keys differ in their slot word)
        n_sample = n_dense;
        for (int r = 0; r <= P_dense; ++r) {
            Key3 mine = k[0];
#pragma unroll
            for (int d = 1; d < SM_DENSE; ++d)
                if (key_less(k[d], mine)) mine = k[d];
            const Key3 best = block_min_key(mine, sm);
            if (tid == 0) a.splitters[r] = best;
#pragma unroll
            for (int d = 0; d < SM_DENSE; ++d)
                if (k[d].w0 == best.w0 && k[d].w1 == best.w1 && k[d].w2 == best.w2) k[d].w0 = k[d].w1 = k[d].w2 = ~0ull;
        }
    } else {
        // the coarse sample (one entry per thread), sorted in full
        const Key3 mine = k[0];
        block_exclusive_scan_256(have[0], &n_sample, sm.warp_sum);
        __syncthreads();
        sm.k0[tid] = mine.w0; sm.k1[tid] = mine.w1; sm.k2[tid] = mine.w2;
        __syncthreads();
        for (int k = 2; k <= SM_SAMPLE; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                const int partner = tid ^ j;
                if (partner > tid) {
                    const Key3 x = smem_key(sm, tid), y = smem_key(sm, partner);
                    const bool up = (tid & k) == 0;
                    if (key_less(y, x) == up) {
                        sm.k0[tid] = y.w0; sm.k1[tid] = y.w1; sm.k2[tid] = y.w2;
                        sm.k0[partner] = x.w0; sm.k1[partner] = x.w1; sm.k2[partner] = x.w2;
                    }
                }
                __syncthreads();
            }
        }
        a.splitters[tid] = smem_key(sm, tid);
    }
    if (tid == 0) a.ctl->n_sample = n_sample;
}

// ---- phase S (all CTAs): free slots of the slice; candidates up to splitter P ----------------------------------
struct MetaChunk {
    static constexpr int U = 4;
    uint8_t v[U];
    double sz[U];
    uint32_t ac[U];
    unsigned long long la[U];
};
__device__ __forceinline__ void maint_load_chunk(const MaintArgs &a, long long base, long long hi, MetaChunk &c) {
#pragma unroll
    for (int j = 0; j < MetaChunk::U; ++j) {
        const long long sl = base + j * SM_THREADS + threadIdx.x;
        const bool in = sl < hi;
        c.v[j] = in ? a.valid[sl] : 1;
        c.sz[j] = in ? a.size[sl] : 0.0;
        c.ac[j] = in ? a.access[sl] : 0u;
        c.la[j] = in ? a.last[sl] : 0ull;
    }
}

__device__ void maint_slice_pass(const MaintArgs &a, long long m, long long occupancy, long long per, MaintSmem &sm) {
    const int tid = threadIdx.x;
    const long long lo = min(a.capacity, static_cast<long long>(blockIdx.x) * per), hi = min(a.capacity, lo + per);
    int nfree = 0;
    if (m == 0) {
        for (long long sl = lo + tid; sl < hi; sl += SM_THREADS) nfree += a.valid[sl] ? 0 : 1;
    } else {
        MetaChunk cur;
        maint_load_chunk(a, lo, hi, cur);              // in flight while the splitters are fetched
        const int n_sample = a.ctl->n_sample;
        const int P = maint_spec_buckets(m, n_sample, occupancy);
        if (tid <= P && tid < SM_SAMPLE) {
            const Key3 k = a.splitters[tid];
            sm.k0[tid] = k.w0; sm.k1[tid] = k.w1; sm.k2[tid] = k.w2;
        }
        for (int i = tid; i <= SM_SAMPLE; i += SM_THREADS) sm.hist[i] = 0;
        __syncthreads();
        const bool has_bound = P < n_sample;
        Key3 bound;
        bound.w0 = bound.w1 = bound.w2 = ~0ull;
        if (has_bound) bound = smem_key(sm, P);
        for (long long base = lo; base < hi; base += MetaChunk::U * SM_THREADS) {
            MetaChunk nxt;
            const long long nb = base + MetaChunk::U * SM_THREADS;
            if (nb < hi) maint_load_chunk(a, nb, hi, nxt);
            // the CTA's candidates of this chunk get consecutive places: one global atomic per CTA and chunk
            if (tid == 0) sm.n_stage = 0;
            __syncthreads();
            Key3 k[MetaChunk::U];
            int place[MetaChunk::U];
#pragma unroll
            for (int j = 0; j < MetaChunk::U; ++j) {
                const long long sl = base + j * SM_THREADS + tid;
                const bool in = sl < hi;
                nfree += (in && !cur.v[j]) ? 1 : 0;
                place[j] = -1;
                if (in && cur.v[j]) {
                    k[j] = make_key(cur.sz[j], cur.ac[j], cur.la[j], static_cast<uint32_t>(sl));
                    if (!has_bound || !key_less(bound, k[j])) {
                        atomicAdd(&sm.hist[splitter_lower_bound(sm, P, k[j])], 1u);
                        place[j] = atomicAdd(&sm.n_stage, 1);
                    }
                }
            }
            __syncthreads();
            if (tid == 0 && sm.n_stage > 0) sm.p = static_cast<int>(atomicAdd(&a.ctl->n_cand, static_cast<unsigned int>(sm.n_stage)));
            __syncthreads();
            if (sm.n_stage > 0) {
                const unsigned int cta_base = static_cast<unsigned int>(sm.p);
#pragma unroll
                for (int j = 0; j < MetaChunk::U; ++j) {
                    if (place[j] >= 0) {
                        const unsigned int at = cta_base + place[j];
                        a.cand0[at] = k[j].w0; a.cand1[at] = k[j].w1; a.cand2[at] = k[j].w2;
                    }
                }
            }
            if (nb < hi) cur = nxt;
        }
        __syncthreads();
        for (int i = tid; i <= P; i += SM_THREADS)
            if (sm.hist[i]) atomicAdd(&a.ctl->hist[i], sm.hist[i]);
    }
    int total;
    block_exclusive_scan_256(nfree, &total, sm.warp_sum);
    if (tid == 0) a.cta_free[blockIdx.x] = total;
}

// first bucket in hist[0..last] where the cumulative count reaches m, or -1 (the same value in all threads)
__device__ int maint_find_bucket(const unsigned int *hist, int last, long long m, MaintSmem &sm) {
    const int tid = threadIdx.x;
    __syncthreads();
    if (tid < 32) {
        long long run = 0;
        int found = -1;
        for (int base = 0; base <= last && found < 0; base += 32) {
            const int i = base + tid;
            long long x = i <= last ? hist[i] : 0;
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
    return sm.p;
}

// ---- fall-back (all CTAs): bucket of every live entry over all splitters, then the candidates -------------------
__device__ __noinline__ void maint_full_bucket(const MaintArgs &a, MaintSmem &sm) {
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
        const int b = splitter_lower_bound(sm, n_sample, k);
        a.bucket[sl] = static_cast<uint16_t>(b);
        atomicAdd(&sm.hist[b], 1u);
    }
    __syncthreads();
    for (int i = tid; i <= SM_SAMPLE; i += SM_THREADS)
        if (sm.hist[i]) atomicAdd(&a.ctl->hist_full[i], sm.hist[i]);
}

__device__ __noinline__ void maint_full_collect(const MaintArgs &a, int p) {
    const int tid = threadIdx.x, lane = tid & 31;
    for (long long base = static_cast<long long>(blockIdx.x) * SM_THREADS; base < a.capacity;
         base += static_cast<long long>(gridDim.x) * SM_THREADS) {
        const long long sl = base + tid;
        const bool take = sl < a.capacity && a.valid[sl] && a.bucket[sl] <= p;
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, take);
        if (ballot) {
            unsigned int warp_base = 0;
            if (lane == 0) warp_base = atomicAdd(&a.ctl->n_cand_full, static_cast<unsigned int>(__popc(ballot)));
            warp_base = __shfl_sync(0xFFFFFFFFu, warp_base, 0);
            if (take) {
                const Key3 k = make_key(a.size[sl], a.access[sl], a.last[sl], static_cast<uint32_t>(sl));
                const unsigned int at = warp_base + __popc(ballot & ((1u << lane) - 1u));
                a.cand0[at] = k.w0; a.cand1[at] = k.w1; a.cand2[at] = k.w2;
            }
        }
    }
}

__device__ __forceinline__ Key3 cand_key(const MaintArgs &a, unsigned int i) {
    Key3 k;
    k.w0 = a.cand0[i]; k.w1 = a.cand1[i]; k.w2 = a.cand2[i];
    return k;
}

__device__ __forceinline__ void maint_take_victim(const MaintArgs &a, int32_t slot, unsigned int rank, long long per) {
    a.victim_buf[rank] = slot;
    if (a.victims) a.victims[rank] = slot;
    a.valid[slot] = 0;
    atomicAdd(&a.cta_free[slot / per], 1);
}

// ---- phase R (every SM_RANK_STRIDE-th CTA): rank the candidates whose key is at most `limit`; the m lowest are
// the victims.  A candidate above the limit is larger than every candidate below it, so it never counts toward
// a rank.
__device__ void maint_rank(const MaintArgs &a, long long m, unsigned int n, bool has_limit, const Key3 &limit, long long per,
                           unsigned long long *stage, MaintSmem &sm) {
    const int tid = threadIdx.x, lane = tid & 31;
    unsigned long long *s0 = stage, *s1 = stage + SM_STAGE, *s2 = stage + 2 * SM_STAGE;
    if (tid == 0) sm.n_stage = 0;
    __syncthreads();
    constexpr int SU = 6;
    for (unsigned int i0 = 0; i0 < n; i0 += SU * SM_THREADS) {
        Key3 k[SU];
#pragma unroll
        for (int u = 0; u < SU; ++u) {
            const unsigned int i = i0 + u * SM_THREADS + tid;
            if (i < n) k[u] = cand_key(a, i);
        }
#pragma unroll
        for (int u = 0; u < SU; ++u) {
            const unsigned int i = i0 + u * SM_THREADS + tid;
            if (i < n && (!has_limit || !key_less(limit, k[u]))) {
                const int j = atomicAdd(&sm.n_stage, 1);
                if (j < SM_STAGE) { s0[j] = k[u].w0; s1[j] = k[u].w1; s2[j] = k[u].w2; }
            }
        }
    }
    __syncthreads();
    const int n_stage = sm.n_stage;
    const unsigned int rankers = (gridDim.x + SM_RANK_STRIDE - 1) / SM_RANK_STRIDE;
    const unsigned int warps = rankers * SM_WARPS;
    const unsigned int me = (blockIdx.x / SM_RANK_STRIDE) * SM_WARPS + (tid >> 5);
    if (n_stage <= SM_STAGE) {
        // the copy's order differs from CTA to CTA, so the work is dealt out by slot: this warp ranks the
        // candidates whose slot is congruent to its number
        for (int j0 = 0; j0 < n_stage; j0 += 32) {
            const int j = j0 + lane;
            const bool own = j < n_stage && static_cast<uint32_t>(s2[j] & 0xFFFFFFFFull) % warps == me;
            unsigned todo = __ballot_sync(0xFFFFFFFFu, own);
            while (todo) {
                const int jj = j0 + __ffs(todo) - 1;
                todo &= todo - 1;
                Key3 mine;
                mine.w0 = s0[jj]; mine.w1 = s1[jj]; mine.w2 = s2[jj];
                unsigned int rank = 0;
                for (int t = lane; t < n_stage; t += 32) {
                    Key3 o;
                    o.w0 = s0[t]; o.w1 = s1[t]; o.w2 = s2[t];
                    rank += key_less(o, mine) ? 1u : 0u;
                }
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, o);
                if (lane == 0 && rank < m) maint_take_victim(a, static_cast<int32_t>(mine.w2 & 0xFFFFFFFFull), rank, per);
            }
        }
    } else {
        // too many for shared memory: by position in the list, against the list in global memory
#pragma unroll 1
        for (unsigned int i = me; i < n; i += warps) {
            const Key3 mine = cand_key(a, i);
            if (has_limit && key_less(limit, mine)) continue;          // the same for all lanes
            unsigned int rank = 0;
            for (unsigned int j = lane; j < n; j += 32) rank += key_less(cand_key(a, j), mine) ? 1u : 0u;
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, o);
            if (lane == 0 && rank < m) maint_take_victim(a, static_cast<int32_t>(mine.w2 & 0xFFFFFFFFull), rank, per);
        }
    }
}

// ---- phase I: row `b` (a miss) into `slot` by one warp --------------------------------------------------------
template <typename T>
__device__ __forceinline__ void maint_insert_row(const MaintArgs &a, int b, int32_t slot, long long clock_new) {
    const int lane = threadIdx.x & 31;
    const T *src = static_cast<const T *>(a.Q) + static_cast<long long>(b) * a.D;
    T *dv = static_cast<T *>(a.vecs) + static_cast<long long>(slot) * a.D;
    float *dm = a.master + static_cast<long long>(slot) * a.D;
    if constexpr (sizeof(T) == 2) {
        for (int d = lane * 8; d < a.D; d += 256) {
            const uint4 u = __ldg(reinterpret_cast<const uint4 *>(src + d));
            *reinterpret_cast<uint4 *>(dv + d) = u;
            const float4 f0 = make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u),
                                          __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xFFFF0000u));
            const float4 f1 = make_float4(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xFFFF0000u),
                                          __uint_as_float(u.w << 16), __uint_as_float(u.w & 0xFFFF0000u));
            *reinterpret_cast<float4 *>(dm + d) = f0;
            *reinterpret_cast<float4 *>(dm + d + 4) = f1;
        }
    } else {
        for (int d = lane * 4; d < a.D; d += 128)
            *reinterpret_cast<float4 *>(dv + d) = __ldg(reinterpret_cast<const float4 *>(src + d));
    }
    if (lane == 0) {
        a.size[slot] = 1.0;
        a.access[slot] = SISO_ACCESS_INF;
        a.last[slot] = static_cast<unsigned long long>(clock_new);
        a.valid[slot] = 1;
        if (a.slots_out) a.slots_out[b] = slot;
    }
}

// ==== barrier-free path: the victims from the list kept across batches ============================================
__device__ __forceinline__ uint32_t low_hash(uint32_t slot) { return (slot * 2654435761u) >> (32 - LOW_MAP_BITS); }

// position of `slot` in the list as the last rebuild wrote it, or -1.  (The caller checks that the position still
// lies in [head, n) and is not marked: the table keeps entries that have left the list since.)
__device__ __forceinline__ int low_pos_of(const LowList *low, uint32_t slot) {
    uint32_t h = low_hash(slot);
    for (int probe = 0; probe < LOW_MAP; ++probe) {
        const unsigned long long e = __ldcg(&low->map[h]);
        if (e == 0ull) return -1;
        if (static_cast<uint32_t>(e >> 32) == slot + 1u) return static_cast<int>(e & 0xFFFFFFFFull);
        h = (h + 1u) & (LOW_MAP - 1u);
    }
    return -1;
}

// the key of a list entry after `cnt` hits in the batch that ends at clock_new (what the update writes: cluster_size
// + cnt, access_count + cnt saturating at infinity, last_access = clock_new); cluster_size and access_count are
// read back from the key, because other CTAs may be updating the arrays right now
__device__ __forceinline__ Key3 low_key_after_hits(const Key3 &k, uint32_t cnt, long long clock_new) {
    const unsigned long long u = (k.w0 >> 63) ? (k.w0 & 0x7FFFFFFFFFFFFFFFull) : ~k.w0;
    const double size = __longlong_as_double(static_cast<long long>(u)) + static_cast<double>(cnt);
    const uint32_t ac_old = static_cast<uint32_t>(k.w1 >> 32);
    const unsigned long long ac = static_cast<unsigned long long>(ac_old) + cnt;
    const uint32_t ac_new = (ac_old == SISO_ACCESS_INF || ac >= SISO_ACCESS_INF) ? SISO_ACCESS_INF : static_cast<uint32_t>(ac);
    return make_key(size, ac_new, static_cast<unsigned long long>(clock_new), static_cast<uint32_t>(k.w2 & 0xFFFFFFFFull));
}

// Loads the L entries of the list from `head` on into `stage`, finds the ones hit in this batch (through the table
// slot -> position) and ranks all of them by their keys after the update; entries marked earlier take no part.  At most B <= LOW_UPD entries can have
// been hit.  sm.vict[0..m) receives the victims in eviction order.
__device__ void maint_low_select(const MaintArgs &a, int head, int L, int m, long long clock_new, unsigned long long *stage,
                                 MaintSmem &sm) {
    const int tid = threadIdx.x;
    unsigned long long *s0 = stage, *s1 = stage + SM_STAGE, *s2 = stage + 2 * SM_STAGE;
    const LowList *low = a.low;
    for (int i = tid; i < L; i += SM_THREADS) {
        s0[i] = __ldcg(&low->k0[head + i]); s1[i] = __ldcg(&low->k1[head + i]); s2[i] = __ldcg(&low->k2[head + i]);
        sm.lflag[i] = __ldcg(&low->dead[head + i]) ? 2 : 0;
    }
    for (int i = tid; i < L; i += SM_THREADS) sm.pcnt[i] = 0u;
    if (tid == 0) { sm.n_upd = 0; sm.v_end = 0; }
    __syncthreads();
    // every hit row looks its slot up in the table: a hit on an unmarked entry of the prefix is counted there
    for (int b = tid; b < a.B; b += SM_THREADS) {
        if (!sm.hit[b]) continue;
        const int32_t slot = sm.idx[b];
        if (slot < 0 || slot >= a.capacity) continue;          // reported by the update of that row
        const int pos = low_pos_of(low, static_cast<uint32_t>(slot)) - head;
        if (pos >= 0 && pos < L && sm.lflag[pos] != 2) atomicAdd(&sm.pcnt[pos], 1u);
    }
    __syncthreads();
    // hb[i] = entries before position i that were hit or marked (thread t owns a contiguous run)
    const int per = (L + SM_THREADS - 1) / SM_THREADS;
    const int lo = min(L, tid * per), hi = min(L, lo + per);
    int c = 0, c_upd = 0;
    for (int i = lo; i < hi; ++i) {
        if (sm.pcnt[i]) sm.lflag[i] = 1;
        c += sm.lflag[i] ? 1 : 0;
        c_upd += sm.lflag[i] == 1 ? 1 : 0;
    }
    int n_gone, n_upd, run, run_u;
    {
        int both;                                               // the two counts share one scan (each is at most 2048)
        const int r = block_exclusive_scan_256(c | (c_upd << 16), &both, sm.warp_sum);
        run = r & 0xFFFF; run_u = r >> 16;
        n_gone = both & 0xFFFF; n_upd = both >> 16;
    }
    for (int i = lo; i < hi; ++i) {
        sm.hb[i] = static_cast<uint16_t>(run);
        run += sm.lflag[i] ? 1 : 0;
        if (sm.lflag[i] == 1) {
            Key3 k;
            k.w0 = s0[i]; k.w1 = s1[i]; k.w2 = s2[i];
            const Key3 nk = low_key_after_hits(k, sm.pcnt[i], clock_new);
            sm.u0[run_u] = nk.w0; sm.u1[run_u] = nk.w1; sm.u2[run_u] = nk.w2;
            sm.upos[run_u] = static_cast<uint16_t>(i);
            ++run_u;
        }
    }
    if (tid == 0) { sm.hb[L] = static_cast<uint16_t>(n_gone); sm.n_upd = n_upd; }
    __syncthreads();
    // ranks after the update.  An entry that was neither hit nor marked: its position among such entries, plus the hit
    // entries whose new key is smaller.  A hit entry: the entries of the first kind below its new key (binary search
    // in the old order, minus the hit and marked entries there), plus the hit entries with a smaller new key.
    for (int i = tid; i < L; i += SM_THREADS) {
        if (sm.lflag[i]) continue;
        Key3 k;
        k.w0 = s0[i]; k.w1 = s1[i]; k.w2 = s2[i];
        int rank = i - sm.hb[i];
        for (int u = 0; u < n_upd; ++u) {
            Key3 nk;
            nk.w0 = sm.u0[u]; nk.w1 = sm.u1[u]; nk.w2 = sm.u2[u];
            rank += key_less(nk, k) ? 1 : 0;
        }
        if (rank < m) {
            sm.vict[rank] = static_cast<int32_t>(k.w2 & 0xFFFFFFFFull);
            atomicMax(&sm.v_end, i + 1);
        }
    }
    for (int u = tid; u < n_upd; u += SM_THREADS) {
        Key3 nk;
        nk.w0 = sm.u0[u]; nk.w1 = sm.u1[u]; nk.w2 = sm.u2[u];
        int lo_i = 0, hi_i = L;
        while (lo_i < hi_i) {
            const int mid = (lo_i + hi_i) >> 1;
            Key3 k;
            k.w0 = s0[mid]; k.w1 = s1[mid]; k.w2 = s2[mid];
            if (key_less(k, nk)) lo_i = mid + 1; else hi_i = mid;
        }
        int rank = lo_i - sm.hb[lo_i];
        for (int v = 0; v < n_upd; ++v) {
            Key3 ok;
            ok.w0 = sm.u0[v]; ok.w1 = sm.u1[v]; ok.w2 = sm.u2[v];
            rank += key_less(ok, nk) ? 1 : 0;
        }
        sm.uvict[u] = rank < m ? 1 : 0;
        if (rank < m) sm.vict[rank] = static_cast<int32_t>(nk.w2 & 0xFFFFFFFFull);
    }
    __syncthreads();
}

// The last CTA brings the list up to date for the next batch (see the head of the file).  It first waits, with a
// limit, until every other CTA has said that it no longer reads the list; in a cooperative launch all CTAs are
// resident and they say so a few microseconds into the kernel.  Nothing is moved: the victims that were not hit
// are the first unmarked entries, so `head` steps behind the last of them; hit entries are marked; and only if a
// moved or new key lies below the bound is the end of the list pulled in to just below that key.
__device__ void maint_low_advance(const MaintArgs &a, int head, int L, int m, long long clock_new, MaintSmem &sm) {
    const int tid = threadIdx.x;
    LowList *low = a.low;
    const int n = low->n;
    const int has_bound = low->has_bound;
    const Key3 bound = low->bound;
    const int n_dead_old = low->n_dead;
    if (tid == 0) {
        unsigned int it = 0;
        while (atomicAdd(&low->started, 0u) < gridDim.x - 1u && it < LOW_SPIN_LIMIT) { __nanosleep(100); ++it; }
        if (it >= LOW_SPIN_LIMIT) set_status(a.status, SISO_ERR_TIMEOUT);
        __threadfence();
    }
    __syncthreads();
    // the smallest key that moved or arrived: the new entries (the lowest slot gives the lowest key) ...
    Key3 cut;
    cut.w0 = cut.w1 = cut.w2 = ~0ull;
    if (m > 0) {
        int32_t lowest = sm.vict[0];
        for (int r = 1; r < m; ++r) lowest = min(lowest, sm.vict[r]);
        cut = make_key(1.0, SISO_ACCESS_INF, static_cast<unsigned long long>(clock_new), static_cast<uint32_t>(lowest));
    }
    // ... and the hit entries that stay in the cache; every hit entry of the list is marked on the way.  The first
    // row of each hit slot looks the slot up in the table (the list itself is not scanned).
    const int new_head = head + sm.v_end;
    int newly_dead = 0;
    for (int b = tid; b < a.B; b += SM_THREADS) {
        if (!sm.hit[b]) continue;
        const int32_t slot = sm.idx[b];
        if (slot < 0 || slot >= a.capacity) continue;
        const int pos = low_pos_of(low, static_cast<uint32_t>(slot));
        if (pos < new_head || pos >= n || low->dead[pos]) continue;
        int cnt = 0;
        bool first = true;
        for (int r = 0; r < a.B; ++r) {
            const bool same = sm.hit[r] && sm.idx[r] == slot;
            cnt += same ? 1 : 0;
            first = first && !(same && r < b);
        }
        if (!first) continue;
        low->dead[pos] = 1;
        ++newly_dead;
        bool evicted = false;
        if (pos - head < L) {
            for (int v = 0; v < sm.n_upd; ++v)
                if (sm.upos[v] == pos - head) evicted = sm.uvict[v] != 0;
        }
        if (!evicted) {
            Key3 k;
            k.w0 = low->k0[pos]; k.w1 = low->k1[pos]; k.w2 = low->k2[pos];
            const Key3 nk = low_key_after_hits(k, static_cast<uint32_t>(cnt), clock_new);
            if (key_less(nk, cut)) cut = nk;
        }
    }
    // hit entries in front of the new head leave with it, but one of them that stays in the cache still counts for the cut
    for (int v = tid; v < sm.n_upd; v += SM_THREADS) {
        if (sm.upos[v] < sm.v_end && !sm.uvict[v]) {
            Key3 nk;
            nk.w0 = sm.u0[v]; nk.w1 = sm.u1[v]; nk.w2 = sm.u2[v];
            if (key_less(nk, cut)) cut = nk;
        }
    }
    cut = block_min_key(cut, sm);
    int dead_total;
    block_exclusive_scan_256(newly_dead, &dead_total, sm.warp_sum);
    if (tid == 0) {
        const bool moved = (cut.w0 & cut.w1 & cut.w2) != ~0ull;
        const bool cut_off = moved && (!has_bound || key_less(cut, bound));
        int n_new = n;
        if (cut_off) {
            // first entry that is not below the cut (the list is in ascending order, marks or not)
            int lo_i = new_head, hi_i = n;
            while (lo_i < hi_i) {
                const int mid = (lo_i + hi_i) >> 1;
                Key3 k;
                k.w0 = low->k0[mid]; k.w1 = low->k1[mid]; k.w2 = low->k2[mid];
                if (key_less(k, cut)) lo_i = mid + 1; else hi_i = mid;
            }
            n_new = lo_i;
            if (n_new > new_head) {
                Key3 k;
                k.w0 = low->k0[n_new - 1]; k.w1 = low->k1[n_new - 1]; k.w2 = low->k2[n_new - 1];
                low->bound = k;
            }
            low->has_bound = 1;
        }
        low->head = new_head;
        low->n = n_new;
        // marked entries that the head has passed no longer count (hb counts hit and marked entries alike); the hit
        // entries behind the new head have just been marked (dead_total).  Entries beyond a pulled-in end stay
        // counted: too large a number only makes the next prefix longer than it has to be.
        int hit_front = 0;
        for (int v = 0; v < sm.n_upd; ++v) hit_front += sm.upos[v] < sm.v_end ? 1 : 0;
        low->n_dead = n_dead_old - (static_cast<int>(sm.hb[sm.v_end]) - hit_front) + dead_total;
        low->valid = (cut_off && n_new <= new_head) ? 0 : 1;
        low->started = 0u;
    }
}

// ==== rebuild of the list (all CTAs; the cache's state is final) ====================================================
// Collect every live entry up to the sample-chosen bound, rank all of them, store the LOW_K lowest in order.
__device__ void maint_low_collect(const MaintArgs &a, bool has_bound, const Key3 &bound) {
    const int tid = threadIdx.x, lane = tid & 31;
    for (long long base = static_cast<long long>(blockIdx.x) * SM_THREADS; base < a.capacity;
         base += static_cast<long long>(gridDim.x) * SM_THREADS) {
        const long long sl = base + tid;
        bool take = false;
        Key3 k;
        k.w0 = k.w1 = k.w2 = 0ull;
        if (sl < a.capacity && a.valid[sl]) {
            k = make_key(a.size[sl], a.access[sl], a.last[sl], static_cast<uint32_t>(sl));
            take = !has_bound || !key_less(bound, k);
        }
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, take);
        if (ballot) {
            unsigned int warp_base = 0;
            if (lane == 0) warp_base = atomicAdd(&a.low->n_cand, static_cast<unsigned int>(__popc(ballot)));
            warp_base = __shfl_sync(0xFFFFFFFFu, warp_base, 0);
            if (take) {
                const unsigned int at = warp_base + __popc(ballot & ((1u << lane) - 1u));
                a.cand0[at] = k.w0; a.cand1[at] = k.w1; a.cand2[at] = k.w2;
            }
        }
    }
}

__device__ void maint_low_rank(const MaintArgs &a, unsigned int n) {
    const int lane = threadIdx.x & 31;
    const unsigned int warps = gridDim.x * SM_WARPS;
    const unsigned int keep = n < static_cast<unsigned int>(LOW_K) ? n : static_cast<unsigned int>(LOW_K);
#pragma unroll 1
    for (unsigned int i = blockIdx.x * SM_WARPS + (threadIdx.x >> 5); i < n; i += warps) {
        const Key3 mine = cand_key(a, i);
        unsigned int rank = 0;
        for (unsigned int j0 = 0; j0 < n; j0 += 128) {
            Key3 o[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const unsigned int j = j0 + u * 32 + lane;
                o[u].w0 = o[u].w1 = o[u].w2 = ~0ull;
                if (j < n) o[u] = cand_key(a, j);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) rank += key_less(o[u], mine) ? 1u : 0u;
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, o);
        if (lane == 0 && rank < keep) {
            a.low->k0[rank] = mine.w0; a.low->k1[rank] = mine.w1; a.low->k2[rank] = mine.w2;
            a.low->dead[rank] = 0;
            const uint32_t slot = static_cast<uint32_t>(mine.w2 & 0xFFFFFFFFull);
            const unsigned long long entry = (static_cast<unsigned long long>(slot + 1u) << 32) | rank;
            uint32_t h = low_hash(slot);
            for (int probe = 0; probe < LOW_MAP; ++probe) {
                if (atomicCAS(&a.low->map[h], 0ull, entry) == 0ull) break;
                h = (h + 1u) & (LOW_MAP - 1u);
            }
            if (n > keep && rank == keep - 1) a.low->bound = mine;        // the list was cut at LOW_K entries
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(SM_THREADS, 2)
stream_maint_kernel(const MaintArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *acc = reinterpret_cast<double *>(smem_raw);                              // [D] during the update
    unsigned long long *stage = reinterpret_cast<unsigned long long *>(smem_raw);    // [3][SM_STAGE] while ranking
    int32_t *sorted = reinterpret_cast<int32_t *>(smem_raw);                         // [2][SM_MAX_B] while inserting
    MaintSmem &sm = *reinterpret_cast<MaintSmem *>(smem_raw + SM_UNION_BYTES);
    cg::grid_group grid = cg::this_grid();
    const int tid = threadIdx.x, warp = tid >> 5;
    // nobody writes the counters before the last barrier
    const long long clock_new = a.counters[CNT_CLOCK] + 1;
    const long long occupancy = a.counters[CNT_OCCUPANCY];

    if (a.partial) {
        maint_finalize(a);
        grid.sync();
    }

    // ---- every CTA: the batch's hit flags and slots, the misses in row order, the number of victims
    for (int b = tid; b < a.B; b += SM_THREADS) { sm.hit[b] = a.hit[b]; sm.idx[b] = a.idx[b]; }
    __syncthreads();
    int n_miss;
    {
        constexpr int PER = SM_MAX_B / SM_THREADS;
        int c = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) { const int b = tid * PER + j; c += (b < a.B && !sm.hit[b]) ? 1 : 0; }
        int r = block_exclusive_scan_256(c, &n_miss, sm.warp_sum);
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int b = tid * PER + j;
            if (b < a.B && !sm.hit[b]) sm.miss_list[r++] = static_cast<uint16_t>(b);
        }
    }
    const long long free0 = a.capacity - occupancy;         // free slots before this batch
    long long m = static_cast<long long>(n_miss) - free0;
    m = m > 0 ? m : 0;
    m = m < occupancy ? m : occupancy;
    __syncthreads();

    // ---- a full cache whose eviction-order list is long enough: no barrier from here on
    int L = 0, head = 0;
    bool fast = false;
    if (a.low) {
        head = a.low->head;
        const int avail = a.low->n - head, n_dead = a.low->n_dead;
        L = min(avail, 2 * a.B + n_dead);          // at least 2B unmarked entries, or all there are
        fast = a.low_ok && a.low->valid && free0 == 0 && n_miss <= occupancy && L <= 2 * SM_MAX_B && a.B <= LOW_UPD &&
               (avail - n_dead >= 2 * a.B || !a.low->has_bound);
    }
    if (fast) {
        const int G = static_cast<int>(gridDim.x);
        const bool last_cta = static_cast<int>(blockIdx.x) == G - 1;
        const int from_end = G - 2 - static_cast<int>(blockIdx.x);
        const bool ins_cta = from_end >= 0 && from_end * SM_WARPS < n_miss;
        const bool out_cta = static_cast<int>(blockIdx.x) == (a.B < G - 1 ? a.B : 0);      // a CTA without a row to update, if there is one
        // A CTA that only updates the entry of row blockIdx.x needs the victims only if that entry could be one of
        // them, i.e. if it is an unmarked entry of the examined prefix (rare: the prefix holds the coldest entries).
        bool need = last_cta || ins_cta || out_cta || a.B > G;
        if (!need) {
            int in_prefix = 0;
            const int b = blockIdx.x;
            if (tid == 0 && b < a.B && sm.hit[b] && sm.idx[b] >= 0 && sm.idx[b] < a.capacity) {
                const int pos = low_pos_of(a.low, static_cast<uint32_t>(sm.idx[b])) - head;
                in_prefix = (pos >= 0 && pos < L && !__ldcg(&a.low->dead[head + pos])) ? 1 : 0;
            }
            need = __syncthreads_or(in_prefix) != 0;
        }
        if (need) maint_low_select(a, head, L, static_cast<int>(m), clock_new, stage, sm);
        if (tid == 0 && !last_cta) atomicAdd(&a.low->started, 1u);      // this CTA has read what it needs of the list
        if (out_cta) {
            if (a.victims)
                for (int r = tid; r < a.B; r += SM_THREADS) a.victims[r] = r < m ? sm.vict[r] : -1;
            if (a.slots_out)
                for (int b = tid; b < a.B; b += SM_THREADS)
                    if (sm.hit[b]) a.slots_out[b] = -1;
        }
        // U: a hit entry that is evicted in this very batch is not updated (a miss overwrites its slot)
        for (int b = blockIdx.x; b < a.B; b += gridDim.x) {
            if (need) {
                int evicted = 0;
                if (sm.hit[b])
                    for (int r = tid; r < m; r += SM_THREADS) evicted |= sm.vict[r] == sm.idx[b] ? 1 : 0;
                if (__syncthreads_or(evicted)) continue;
            }
            maint_update_row<T>(a, b, clock_new, acc, sm);
        }
        // I: the victims' slots in ascending order take the misses in ascending row order
        // (by the CTAs counted from the far end, the last one excepted: the first ones are busy with the updates)
        const int ins_ctas = G - 1;
        if (ins_cta) {
            for (int r = tid; r < n_miss; r += SM_THREADS) {
                const int32_t mine = sm.vict[r];
                int rank = 0;
                for (int j = 0; j < n_miss; ++j) rank += sm.vict[j] < mine ? 1 : 0;
                sm.by_slot[rank] = mine;
            }
            __syncthreads();
            for (int r = from_end * SM_WARPS + warp; r < n_miss; r += ins_ctas * SM_WARPS)
                maint_insert_row<T>(a, sm.miss_list[r], sm.by_slot[r], clock_new);
        }
        if (last_cta) {
            __syncthreads();
            maint_low_advance(a, head, L, static_cast<int>(m), clock_new, sm);
            if (tid == 0) {
                a.counters[CNT_CLOCK] = clock_new;
                a.counters[CNT_EVICTIONS] += m;
                a.counters[CNT_INSERTS] += n_miss;
                if (a.count_lookup) {
                    a.counters[CNT_LOOKUPS] += a.B;
                    a.counters[CNT_HITS] += a.B - n_miss;
                }
            }
        }
        return;
    }

    // ---- U (+ sampler)
    if (blockIdx.x == 0) {
        if (tid == 0) { a.ctl->n_cand = 0; a.ctl->n_cand_full = 0; }
        for (int i = tid; i <= SM_SAMPLE; i += SM_THREADS) { a.ctl->hist[i] = 0; a.ctl->hist_full[i] = 0; }
        if (a.victims)
            for (long long r = m + tid; r < a.B; r += SM_THREADS) a.victims[r] = -1;
        if (a.slots_out)
            for (int b = tid; b < a.B; b += SM_THREADS)
                if (sm.hit[b]) a.slots_out[b] = -1;
    }
    if (m > 0 && blockIdx.x == gridDim.x - 1) maint_evict_sample(a, clock_new, m, occupancy, false, sm);
    for (int b = blockIdx.x; b < a.B; b += gridDim.x) maint_update_row<T>(a, b, clock_new, acc, sm);
    grid.sync();

    // ---- S
    const long long per = (a.capacity + gridDim.x - 1) / gridDim.x;
    maint_slice_pass(a, m, occupancy, per, sm);
    grid.sync();

    // ---- R
    if (m > 0) {
        int n_sample = a.ctl->n_sample;
        const int P = maint_spec_buckets(m, n_sample, occupancy);
        unsigned int n = a.ctl->n_cand;
        int p = maint_find_bucket(a.ctl->hist, P, m, sm);
        if (p < 0) {
            // the whole sample in order (the entries are final by now), every entry's bucket, the candidates
            if (blockIdx.x == 0) maint_evict_sample(a, clock_new, m, occupancy, true, sm);
            grid.sync();
            n_sample = a.ctl->n_sample;
            maint_full_bucket(a, sm);
            grid.sync();
            p = maint_find_bucket(a.ctl->hist_full, SM_SAMPLE, m, sm);      // m <= occupancy, so it exists
            maint_full_collect(a, p);
            grid.sync();
            n = a.ctl->n_cand_full;
            p = n_sample;                                                   // every collected entry is ranked
        }
        if (blockIdx.x % SM_RANK_STRIDE == 0) {
            const bool has_limit = p < n_sample;
            Key3 limit;
            limit.w0 = limit.w1 = limit.w2 = ~0ull;
            if (has_limit) limit = smem_key(sm, p);
            maint_rank(a, m, n, has_limit, limit, per, stage, sm);
        }
        grid.sync();
    }

    // ---- I
    bool insert_ok;
    if (free0 == 0) {
        // a full cache: the free slots are the victims; every CTA puts them in slot order
        insert_ok = n_miss <= m;
        if (insert_ok) {
            int32_t *vict = sorted, *by_slot = sorted + SM_MAX_B;
            for (int r = tid; r < n_miss; r += SM_THREADS) vict[r] = a.victim_buf[r];
            __syncthreads();
            for (int r = tid; r < n_miss; r += SM_THREADS) {
                const int32_t mine = vict[r];
                int rank = 0;
                for (int j = 0; j < n_miss; ++j) rank += vict[j] < mine ? 1 : 0;
                by_slot[rank] = mine;
            }
            __syncthreads();
            const int warps = gridDim.x * SM_WARPS;
            for (int r = blockIdx.x * SM_WARPS + warp; r < n_miss; r += warps)
                maint_insert_row<T>(a, sm.miss_list[r], by_slot[r], clock_new);
        }
    } else {
        // free slots before this CTA's slice and in all slices
        int base = 0, n_free = 0;
        {
            const int G = static_cast<int>(gridDim.x);
            const int cs = (G + SM_THREADS - 1) / SM_THREADS;
            int c = 0;
            for (int j = 0; j < cs; ++j) { const int g = tid * cs + j; c += g < G ? a.cta_free[g] : 0; }
            int run = block_exclusive_scan_256(c, &n_free, sm.warp_sum);
            __syncthreads();
            for (int j = 0; j < cs; ++j) {
                const int g = tid * cs + j;
                if (g >= G) break;
                if (g == static_cast<int>(blockIdx.x)) sm.p = run;
                run += a.cta_free[g];
            }
            __syncthreads();
            base = sm.p;
        }
        insert_ok = n_miss <= n_free;
        if (insert_ok) {          // the same in every CTA
            // the free slots of this slice that are taken, in ascending order
            const long long lo = min(a.capacity, static_cast<long long>(blockIdx.x) * per), hi = min(a.capacity, lo + per);
            const int my_need = max(0, min(a.cta_free[blockIdx.x], n_miss - base));
            if (my_need > 0) {        // uniform for the CTA
                const long long chunk = (per + SM_THREADS - 1) / SM_THREADS;
                const long long t_lo = min(hi, lo + tid * chunk), t_hi = min(hi, t_lo + chunk);
                int c = 0;
                for (long long sl = t_lo; sl < t_hi; ++sl) c += a.valid[sl] ? 0 : 1;
                int total;
                int r = block_exclusive_scan_256(c, &total, sm.warp_sum);
                for (long long sl = t_lo; sl < t_hi; ++sl) {
                    if (!a.valid[sl]) {
                        if (r < my_need) a.free_list[base + r] = static_cast<int32_t>(sl);
                        ++r;
                    }
                }
            }
            grid.sync();
            const int warps = gridDim.x * SM_WARPS;
            for (int r = blockIdx.x * SM_WARPS + warp; r < n_miss; r += warps)
                maint_insert_row<T>(a, sm.miss_list[r], a.free_list[r], clock_new);
        }
    }
    if (!insert_ok && blockIdx.x == 0) {
        if (tid == 0) set_status(a.status, SISO_ERR_CAPACITY);
        if (a.slots_out)
            for (int r = tid; r < n_miss; r += SM_THREADS) a.slots_out[sm.miss_list[r]] = -1;
    }
    if (blockIdx.x == 0 && tid == 0) {
        a.counters[CNT_CLOCK] = clock_new;
        a.counters[CNT_OCCUPANCY] = occupancy - m + (insert_ok ? n_miss : 0);
        a.counters[CNT_EVICTIONS] += m;
        if (insert_ok) a.counters[CNT_INSERTS] += n_miss;
        if (a.count_lookup) {
            a.counters[CNT_LOOKUPS] += a.B;
            a.counters[CNT_HITS] += a.B - n_miss;
        }
    }

    // ---- the eviction-order list for the batches to come: rebuilt once the cache is full, dropped otherwise
    if (a.low) {
        const long long occupancy_after = occupancy - m + (insert_ok ? n_miss : 0);
        if (occupancy_after != a.capacity) {
            // every CTA read the list's header before the first barrier of this launch
            if (blockIdx.x == 0 && tid == 0) { a.low->valid = 0; a.low->n = 0; }
            return;
        }
        grid.sync();                                             // the cache's state is final
        const long long m_equiv = LOW_TARGET / 3;                // the sampler aims at about 3 m entries below its last splitter
        if (blockIdx.x == 0) {
            if (tid == 0) a.low->n_cand = 0u;
            maint_evict_sample(a, clock_new, m_equiv, occupancy_after, false, sm);
        }
        grid.sync();
        const int n_sample = a.ctl->n_sample;
        const int P = maint_spec_buckets(m_equiv, n_sample, occupancy_after);
        const bool has_bound = P < n_sample;
        Key3 bound;
        bound.w0 = bound.w1 = bound.w2 = ~0ull;
        if (has_bound) bound = a.splitters[P];
        for (int i = blockIdx.x * SM_THREADS + tid; i < LOW_MAP; i += gridDim.x * SM_THREADS) a.low->map[i] = 0ull;
        maint_low_collect(a, has_bound, bound);
        grid.sync();
        const unsigned int n_c = a.low->n_cand;
        maint_low_rank(a, n_c);
        if (blockIdx.x == 0 && tid == 0) {
            a.low->n = static_cast<int>(n_c < static_cast<unsigned int>(LOW_K) ? n_c : static_cast<unsigned int>(LOW_K));
            a.low->head = 0;
            a.low->n_dead = 0;
            a.low->valid = n_c > 0u ? 1 : 0;
            a.low->has_bound = (has_bound || n_c > static_cast<unsigned int>(LOW_K)) ? 1 : 0;
            if (has_bound && n_c <= static_cast<unsigned int>(LOW_K)) a.low->bound = bound;
            a.low->started = 0u;
        }
    }
}

// With `deferred` the lookup's top-1 finalisation (best key over the splits, threshold test, idx/sim/hit) runs as the
// kernel's first phase; `scratch_tail` is then the part of the cache's scratch that the lookup set aside for this call.
size_t stream_maint_scratch_bytes(const Cache *c, int64_t B) {
    const int grid_cap = c->sm_count * 2;
    return pad256(sizeof(MaintCtl)) + pad256(sizeof(Key3) * SM_SAMPLE) + pad256(sizeof(uint16_t) * c->capacity) +
           3 * pad256(sizeof(unsigned long long) * c->capacity) + pad256(sizeof(int) * grid_cap) +
           2 * pad256(sizeof(int32_t) * B) + 256;
}

bool stream_maint_supported(Cache *c, int64_t B) {
    if (B < 1 || B > SM_MAX_B) return false;
    if (c->maint_grid == 0) {
        int coop = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device) != cudaSuccess) coop = 0;
        int per_sm = 0;
        const void *fn = c->dtype == SISO_F32 ? reinterpret_cast<const void *>(stream_maint_kernel<float>)
                                              : reinterpret_cast<const void *>(stream_maint_kernel<__nv_bfloat16>);
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SM_SMEM_BYTES));
        if (e == cudaSuccess)
            e = c->dtype == SISO_F32
                ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, stream_maint_kernel<float>, SM_THREADS, SM_SMEM_BYTES)
                : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, stream_maint_kernel<__nv_bfloat16>, SM_THREADS, SM_SMEM_BYTES);
        if (e != cudaSuccess) { cudaGetLastError(); per_sm = 0; }
        c->maint_grid = (coop && per_sm >= 1) ? c->sm_count * std::min(per_sm, 2) : -1;
    }
    return c->maint_grid > 0;
}

// Returns SISO_ERR_UNSUPPORTED if this batch cannot take the fused path (the caller then uses the separate kernels).
siso_status_t launch_stream_maint(Cache *c, const void *q, int64_t B, int32_t *idx, uint8_t *hit, int32_t *victims,
                                  int32_t *slots_out, const DeferredTop1 *deferred, void *scratch_tail, cudaStream_t s) {
    c->vec_epoch += 1;          // the vectors may change: derived copies (the split-bf16 parts) are stale
    if (!stream_maint_supported(c, B)) return SISO_ERR_UNSUPPORTED;
    const int grid = c->maint_grid;
    Scratch scr;
    if (scratch_tail) {
        scr.base = static_cast<char *>(scratch_tail);
        scr.off = 0;
        scr.cap = stream_maint_scratch_bytes(c, B);
    } else {
        SISO_TRY(scratch_reserve(c, stream_maint_scratch_bytes(c, B), s, &scr));
    }
    MaintArgs a;
    a.Q = q; a.idx = idx; a.hit = hit; a.B = static_cast<int>(B); a.D = c->dim; a.capacity = c->capacity;
    a.vecs = c->vecs; a.master = c->master; a.size = c->size; a.access = c->access; a.last = c->last; a.valid = c->valid;
    a.counters = c->counters; a.status = c->status; a.victims = victims; a.slots_out = slots_out;
    a.count_lookup = deferred ? 1 : 0;
    a.partial = deferred ? deferred->partial : nullptr;
    a.splits = deferred ? deferred->splits : 0;
    a.theta = deferred ? deferred->theta : nullptr;
    a.theta_s = deferred ? deferred->theta_s : 0.0f;
    a.sim = deferred ? deferred->sim : nullptr;
    a.ctl = scr.take<MaintCtl>(1);
    a.splitters = scr.take<Key3>(SM_SAMPLE);
    a.bucket = scr.take<uint16_t>(c->capacity);
    a.cand0 = scr.take<unsigned long long>(c->capacity);
    a.cand1 = scr.take<unsigned long long>(c->capacity);
    a.cand2 = scr.take<unsigned long long>(c->capacity);
    a.victim_buf = scr.take<int32_t>(B);
    a.cta_free = scr.take<int>(grid);
    a.free_list = scr.take<int32_t>(B);
    a.low = nullptr;
    if (!c->stream_list_off) {
        if (!c->low_list) c->low_list = cache_alloc_zeroed(c, sizeof(LowList));      // all zero: an empty, invalid list
        if (!c->low_list) return SISO_ERR_OOM;
        a.low = static_cast<LowList *>(c->low_list);
    }
    a.low_ok = c->low_dirty ? 0 : 1;
    void *args[] = {&a};
    const void *fn = c->dtype == SISO_F32 ? reinterpret_cast<const void *>(stream_maint_kernel<float>)
                                          : reinterpret_cast<const void *>(stream_maint_kernel<__nv_bfloat16>);
    SISO_CUDA(cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(SM_THREADS), args, SM_SMEM_BYTES, s));
    c->launches += 1;
    c->low_dirty = false;       // from here on the list on the device matches the cache, or says that it does not
    return SISO_OK;
}

}  // namespace siso
