// Hit update: running mean of every centroid that was hit in this batch, then renormalisation.
//     c_j <- normalise(cluster_size_j * c_j + sum_{b in H_j} q_b)      (H_j in ascending query order)
// The hits are grouped by slot with a stable sort, so each sum runs in one fixed order; sums and
// the norm are accumulated in fp64, the result is rounded once to the fp32 master and, for bf16
// caches, once more to the bf16 lookup copy.
#include "common.cuh"

namespace siso {

constexpr int UP_THREADS = 256;

// keys: slot of each hit row, `capacity` (sorts last) for rows that are not hits; vals: row number
__global__ void update_keys_kernel(const int32_t *__restrict__ idx, int idx_stride, const uint8_t *__restrict__ hit,
                                   const uint8_t *__restrict__ valid, int64_t B, int64_t capacity,
                                   uint32_t *__restrict__ keys, uint32_t *__restrict__ vals, long long *counters,
                                   int *status) {
    const int64_t b = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (b == 0) counters[CNT_CLOCK] += 1;      // the cache clock advances once per update call
    if (b >= B) return;
    uint32_t key = static_cast<uint32_t>(capacity);
    if (hit[b]) {
        const int64_t j = idx[b * idx_stride];
        if (j >= 0 && j < capacity && valid[j]) key = static_cast<uint32_t>(j);
        else set_status(status, SISO_ERR_INVALID_ARG);   // a hit must name a live slot; the row is skipped
    }
    keys[b] = key;
    vals[b] = static_cast<uint32_t>(b);
}

// four consecutive elements of a row as fp32 (one 8- or 16-byte load)
template <typename T> __device__ __forceinline__ float4 load4(const T *p);
template <> __device__ __forceinline__ float4 load4<float>(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
template <> __device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16 *p) {
    const uint2 u = __ldg(reinterpret_cast<const uint2 *>(p));
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xFFFF0000u));
}

__device__ __forceinline__ double block_sum_f64(double v, double *red) {
    // fixed-shape tree: the same order of additions on every run
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < UP_THREADS / 32; ++w) t += red[w];
    return t;
}

// One CTA per position of the sorted hit list.  A group (the hits of one slot, ascending query order) is cut into
// chunks of `chunk` rows; the CTA at the first row of a chunk sums that chunk in fp64.  A group of one chunk is
// finished on the spot.  Otherwise the chunk sums go to scratch and the CTA that arrives last (a counter per
// group) adds them up in chunk order and finishes, so a centroid that takes hundreds of hits is not one CTA's
// serial work and the result is still the same on every run.
template <typename T>
__global__ void __launch_bounds__(UP_THREADS)
update_apply_kernel(const uint32_t *__restrict__ keys, const uint32_t *__restrict__ rows, int64_t B, int64_t capacity,
                    int D, int chunk, const T *__restrict__ Q, float *__restrict__ master, T *__restrict__ vecs,
                    double *__restrict__ size, uint32_t *__restrict__ access, unsigned long long *__restrict__ last,
                    const long long *__restrict__ counters, double *__restrict__ partial,
                    unsigned int *__restrict__ arrived) {
    extern __shared__ double acc[];          // [D]
    __shared__ double red[UP_THREADS / 32];
    __shared__ int last_s;
    const int64_t p = blockIdx.x;
    // this position, its left neighbour and the position one chunk to the left, requested together: most CTAs
    // learn from them alone whether they start a chunk
    const uint32_t slot = keys[p];
    const uint32_t left = p > 0 ? keys[p - 1] : 0xFFFFFFFFu;
    const uint32_t far_left = p >= chunk ? keys[p - chunk] : 0xFFFFFFFFu;
    if (slot >= capacity) return;
    int64_t head = p;                        // first position of this slot in the sorted list
    if (left == slot) {
        // not the first row of the group.  If the row one chunk to the left belongs to another slot, the group began
        // less than a chunk ago and this row starts no chunk; only long groups need their first position
        if (far_left != slot) return;
        int64_t lo = 0, hi = p;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if (keys[mid] < slot) lo = mid + 1; else hi = mid;
        }
        head = lo;
        if ((p - head) % chunk != 0) return;
    }
    const bool is_head = p == head;
    // everything the CTA needs of the slot and the first rows of the chunk, requested before the chunk's end is known
    const double n_old = size[slot];
    const uint32_t access_old = access[slot];
    float *m = master + static_cast<int64_t>(slot) * D;
    constexpr int MR = 4;                    // master elements per thread fetched ahead (covers D <= 1024)
    float mreg[MR];
#pragma unroll
    for (int j = 0; j < MR; ++j) { const int d = threadIdx.x + j * UP_THREADS; mreg[j] = (is_head && d < D) ? m[d] : 0.0f; }
    uint32_t row4[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) row4[r] = p + r < B ? rows[p + r] : 0u;
    // the end of this chunk, eight positions at a time; one position beyond the chunk tells whether the group goes on
    int64_t e = p + 1;
    const int64_t limit = min(B, p + static_cast<int64_t>(chunk) + 1);
    while (e < limit) {
        uint32_t k8[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) k8[u] = e + u < limit ? keys[e + u] : 0xFFFFFFFFu;
        int same = 0;
#pragma unroll
        for (int u = 0; u < 8; ++u) same += (same == u && k8[u] == slot) ? 1 : 0;
        e += same;
        if (same < 8) break;
    }
    const bool more = e > p + chunk;
    if (more) e = p + chunk;
#pragma unroll
    for (int j = 0; j < MR; ++j) { const int d = threadIdx.x + j * UP_THREADS; if (d < D) acc[d] = is_head ? n_old * static_cast<double>(mreg[j]) : 0.0; }
    for (int d = threadIdx.x + MR * UP_THREADS; d < D; d += UP_THREADS) acc[d] = is_head ? n_old * static_cast<double>(m[d]) : 0.0;
    __syncthreads();      // the accumulation below uses a different thread-to-element mapping
    // the rows four at a time: the loads of a quartet are in flight together, additions stay in ascending order
    const int quads = D / 4;
    for (int64_t t = p; t < e; t += 4) {
        const int nrow = static_cast<int>(e - t < 4 ? e - t : 4);
        const T *q[4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
            q[r] = Q + static_cast<int64_t>(t == p ? row4[r < nrow ? r : 0] : rows[t + (r < nrow ? r : 0)]) * D;
        for (int g = threadIdx.x; g < quads; g += UP_THREADS) {
            float4 v[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) v[r] = load4<T>(q[r] + 4 * g);
            double a0 = acc[4 * g], a1 = acc[4 * g + 1], a2 = acc[4 * g + 2], a3 = acc[4 * g + 3];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                if (r < nrow) { a0 += v[r].x; a1 += v[r].y; a2 += v[r].z; a3 += v[r].w; }
            }
            acc[4 * g] = a0; acc[4 * g + 1] = a1; acc[4 * g + 2] = a2; acc[4 * g + 3] = a3;   // each thread owns its g
        }
    }
    __syncthreads();
    long long count = e - p;
    if (!(is_head && !more)) {
        // several chunks: publish this chunk's sum, the last arriver combines.  A chunk's scratch row is
        // 2 * (start / chunk) + (1 if it is the group's first chunk): unique, because chunks of one group start
        // `chunk` rows apart and a first chunk of a several-chunk group is at least `chunk` rows from the next group.
        const int64_t my_id = 2 * (p / chunk) + (is_head ? 1 : 0);
        for (int d = threadIdx.x; d < D; d += UP_THREADS) partial[my_id * D + d] = acc[d];
        int64_t glo = e, ghi = B;            // first position past the group
        while (glo < ghi) {
            const int64_t mid = (glo + ghi) >> 1;
            if (keys[mid] <= slot) glo = mid + 1; else ghi = mid;
        }
        const int64_t gend = glo;
        const int64_t n_chunks = (gend - head + chunk - 1) / chunk;
        const int64_t head_id = 2 * (head / chunk) + 1;
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) last_s = (atomicAdd(&arrived[head_id], 1u) == static_cast<unsigned int>(n_chunks - 1)) ? 1 : 0;
        __syncthreads();
        if (!last_s) return;
        __threadfence();
        for (int d = threadIdx.x; d < D; d += UP_THREADS) {
            double v = __ldcg(&partial[head_id * D + d]);
            for (int64_t cidx = 1; cidx < n_chunks; ++cidx)
                v += __ldcg(&partial[(2 * ((head + cidx * chunk) / chunk)) * D + d]);
            acc[d] = v;
        }
        __syncthreads();
        count = gend - head;
    }
    double ss = 0.0;
    for (int d = threadIdx.x; d < D; d += UP_THREADS) ss += acc[d] * acc[d];
    const double norm = sqrt(block_sum_f64(ss, red));
    T *v = vecs + static_cast<int64_t>(slot) * D;
    for (int d = threadIdx.x; d < D; d += UP_THREADS) {
        const float f = static_cast<float>(acc[d] / norm);
        m[d] = f;
        if constexpr (sizeof(T) == 2) v[d] = __float2bfloat16_rn(f);
    }
    if (threadIdx.x == 0) {
        size[slot] = n_old + static_cast<double>(count);
        const unsigned long long a = static_cast<unsigned long long>(access_old) + static_cast<unsigned long long>(count);
        access[slot] = (access_old == SISO_ACCESS_INF || a >= SISO_ACCESS_INF) ? SISO_ACCESS_INF : static_cast<uint32_t>(a);
        last[slot] = static_cast<unsigned long long>(counters[CNT_CLOCK]);
    }
}

// The same work with one WARP per chunk, for dim = 128 * NQ <= 1024.  A first kernel lists the chunks (start, slot,
// first and past-the-end position of the group) with one thread per position of the sorted hit list; then a grid of
// resident warps walks that list.  Lane l owns the element quartets l, l + 32, ..., the running sums stay in registers
// (fp64), the norm is a shuffle tree, nothing needs a CTA-wide barrier and no warp is launched only to find that it has
// nothing to do.  Chunks, their scratch rows, the arrival counter and every order of addition are those of
// update_apply_kernel; the order in which chunks are listed does not matter to any sum.
constexpr int UPW_THREADS = 128;
constexpr int UPW_SUPER = 16;            // chunks per run of the two-level combination

__global__ void __launch_bounds__(256)
update_chunks_kernel(const uint32_t *__restrict__ keys, const uint32_t *__restrict__ rows, int64_t B, int64_t capacity, int chunk,
                     int4 *__restrict__ desc, unsigned int *__restrict__ n_desc) {
    const int64_t p = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    bool start = false;
    uint32_t slot = 0xFFFFFFFFu;
    int64_t head = p, gend = p;
    if (p < B) {
        slot = keys[p];
        if (slot < capacity) {
            const uint32_t left = p > 0 ? keys[p - 1] : 0xFFFFFFFFu;
            if (left != slot) {
                start = true;
            } else if (p >= chunk && keys[p - chunk] == slot) {
                // a long group: its first position, and whether this one is a whole number of chunks away from it
                int64_t lo = 0, hi = p;
                while (lo < hi) {
                    const int64_t mid = (lo + hi) >> 1;
                    if (keys[mid] < slot) lo = mid + 1; else hi = mid;
                }
                head = lo;
                start = (p - head) % chunk == 0;
            }
        }
    }
    if (start) {
        int64_t lo = p + 1, hi = B;            // first position past the group
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if (keys[mid] <= slot) lo = mid + 1; else hi = mid;
        }
        gend = lo;
    }
    // chunks of groups that span several chunks are listed from the front, the others from the back: the warps take
    // the list front to back, so the long dependent chains (sum, publish, combine) start first and the short ones fill in
    const bool multi = start && !(head == p && gend <= p + chunk);
    const unsigned int ballot_m = __ballot_sync(0xFFFFFFFFu, multi), ballot_s = __ballot_sync(0xFFFFFFFFu, start && !multi);
    if ((ballot_m | ballot_s) == 0u) return;
    unsigned int base_m = 0, base_s = 0;
    if (lane == 0) {
        if (ballot_m) base_m = atomicAdd(&n_desc[0], static_cast<unsigned int>(__popc(ballot_m)));
        if (ballot_s) base_s = atomicAdd(&n_desc[1], static_cast<unsigned int>(__popc(ballot_s)));
    }
    base_m = __shfl_sync(0xFFFFFFFFu, base_m, 0);
    base_s = __shfl_sync(0xFFFFFFFFu, base_s, 0);
    if (start) {
        // two words of 16 bytes per chunk: where it is, and its first four rows (most chunks have no more)
        const unsigned int below = (1u << lane) - 1u;
        const unsigned int at = multi ? base_m + __popc(ballot_m & below)
                                      : static_cast<unsigned int>(B) - 1u - (base_s + __popc(ballot_s & below));
        int r[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) r[x] = static_cast<int>(rows[p + x < gend ? p + x : p]);
        desc[2 * at] = make_int4(static_cast<int>(p), static_cast<int>(slot), static_cast<int>(head), static_cast<int>(gend));
        desc[2 * at + 1] = make_int4(r[0], r[1], r[2], r[3]);
    }
}

template <typename T> struct Raw4;
template <> struct Raw4<float> { using type = float4; };
template <> struct Raw4<__nv_bfloat16> { using type = uint2; };
__device__ __forceinline__ float4 widen4(float4 v) { return v; }
__device__ __forceinline__ float4 widen4(uint2 u) {
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xFFFF0000u));
}

// rows of a chunk in flight at a time (after the first four): 12-16 KiB per warp
template <typename T> __host__ __device__ constexpr int upw_stage_rows() { return sizeof(T) == 2 ? 8 : 4; }

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
// BYTES (a multiple of 16) from global to shared memory by one warp, 16 bytes per lane and step
template <int BYTES>
__device__ __forceinline__ void warp_copy_async(void *dst_smem, const void *src, int lane) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem));
    const char *g = static_cast<const char *>(src);
#pragma unroll
    for (int o = 0; o < BYTES; o += 512) {
        const int at = o + lane * 16;
        if (at < BYTES) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d + at), "l"(g + at) : "memory");
    }
}
// shared memory of one warp: the master row as fp32, then the query rows of one stage
template <typename T> __host__ __device__ constexpr size_t upw_warp_smem(int D) { return sizeof(float) * D + upw_stage_rows<T>() * sizeof(T) * D; }

template <typename T, int NQ>
__global__ void __launch_bounds__(UPW_THREADS, 3)
update_apply_warp_kernel(const int4 *__restrict__ desc, unsigned int list_len, const unsigned int *__restrict__ n_desc,
                         unsigned int *__restrict__ ticket,
                         const uint32_t *__restrict__ rows,
                         int chunk, const T *__restrict__ Q, float *__restrict__ master, T *__restrict__ vecs,
                         double *__restrict__ size, uint32_t *__restrict__ access, unsigned long long *__restrict__ last,
                         const long long *__restrict__ counters, double *__restrict__ partial,
                         unsigned int *__restrict__ arrived, unsigned int *__restrict__ arrived_runs) {
    using raw_t = typename Raw4<T>::type;
    constexpr int D = 128 * NQ;
    constexpr int ROW_M_BYTES = D * 4, ROW_Q_BYTES = D * static_cast<int>(sizeof(T)), UPW_STAGE_ROWS = upw_stage_rows<T>();
    extern __shared__ __align__(16) unsigned char upw_smem[];
    const int lane = threadIdx.x & 31;
    float *m_s = reinterpret_cast<float *>(upw_smem + (threadIdx.x >> 5) * upw_warp_smem<T>(D));
    T *q_s = reinterpret_cast<T *>(m_s + D);
    const unsigned int n_front = n_desc[0], n = n_front + n_desc[1];
    auto place = [&](unsigned int t) { return t < n_front ? t : list_len - 1u - (t - n_front); };      // ticket -> list entry
    // chunks are handed out by a ticket counter (a long chunk delays nobody else); a warp draws its next ticket and
    // requests that chunk's description before it sums the current one
    auto draw = [&]() {
        unsigned int t = 0;
        if (lane == 0) t = atomicAdd(ticket, 1u);
        return __shfl_sync(0xFFFFFFFFu, t, 0);
    };
    unsigned int i = draw();
    if (i >= n) return;
    int4 next = desc[2 * place(i)], next_rows = desc[2 * place(i) + 1];
    while (i < n) {
        const int4 d = next, dr = next_rows;
        i = draw();
        if (i < n) { next = desc[2 * place(i)]; next_rows = desc[2 * place(i) + 1]; }
        const int64_t p = d.x, head = d.z, gend = d.w;
        const uint32_t slot = static_cast<uint32_t>(d.y);
        const bool is_head = p == head;
        const bool more = gend > p + chunk;
        const int64_t e = more ? p + chunk : gend;
        float *m = master + static_cast<int64_t>(slot) * D;
        // Everything the chunk reads travels to this warp's shared-memory buffer with asynchronous 16-byte copies, so
        // that all of a stage's bytes are in flight at once whatever the registers allow: first the master row (head
        // chunks) and the chunk's first four rows, whose numbers come with the description, then the remaining rows
        // UPW_STAGE_ROWS at a time (their numbers: one coalesced load of the whole chunk's list).  The additions run
        // from shared memory in ascending row order, as before.
        const int n_rows = static_cast<int>(e - p);
        const int first = n_rows < 4 ? n_rows : 4;
        uint32_t rid_lane = 0;
        if (n_rows > 4 && lane < n_rows) rid_lane = rows[p + lane];
        if (is_head) warp_copy_async<ROW_M_BYTES>(m_s, m, lane);
        {
            const int r4[4] = {dr.x, dr.y, dr.z, dr.w};
#pragma unroll
            for (int r = 0; r < 4; ++r)
                if (r < first) warp_copy_async<ROW_Q_BYTES>(q_s + r * D, Q + static_cast<int64_t>(r4[r]) * D, lane);
        }
        cp_async_commit();
        const double n_old = size[slot];
        const uint32_t access_old = access[slot];
        double a[NQ][4];
        cp_async_wait_all();
        __syncwarp();
#pragma unroll
        for (int j = 0; j < NQ; ++j) {
            float4 m4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (is_head) m4 = *reinterpret_cast<const float4 *>(m_s + 4 * (lane + 32 * j));
            a[j][0] = n_old * static_cast<double>(m4.x); a[j][1] = n_old * static_cast<double>(m4.y);
            a[j][2] = n_old * static_cast<double>(m4.z); a[j][3] = n_old * static_cast<double>(m4.w);
        }
        auto add_rows = [&](int n_stage) {
            for (int r = 0; r < n_stage; ++r) {
                const raw_t *src = reinterpret_cast<const raw_t *>(q_s + r * D) + lane;
#pragma unroll
                for (int j = 0; j < NQ; ++j) {
                    const float4 f = widen4(src[32 * j]);
                    a[j][0] += f.x; a[j][1] += f.y; a[j][2] += f.z; a[j][3] += f.w;
                }
            }
        };
        add_rows(first);
        for (int t = 4; t < n_rows; t += UPW_STAGE_ROWS) {
            const int n_stage = n_rows - t < UPW_STAGE_ROWS ? n_rows - t : UPW_STAGE_ROWS;
            __syncwarp();                                     // the buffer's rows have been added
            for (int r = 0; r < n_stage; ++r) {
                const uint32_t rid = __shfl_sync(0xFFFFFFFFu, rid_lane, t + r);
                warp_copy_async<ROW_Q_BYTES>(q_s + r * D, Q + static_cast<int64_t>(rid) * D, lane);
            }
            cp_async_commit();
            cp_async_wait_all();
            __syncwarp();
            add_rows(n_stage);
        }
        __syncwarp();                                         // before the next chunk's copies overwrite the buffer
        long long count = e - p;
        if (!(is_head && !more)) {
            // several chunks: publish this chunk's sum.  Chunks are combined in two levels so that a centroid with thousands
            // of hits is not one warp's serial work: the warp that arrives last among the UPW_SUPER chunks of a run adds
            // that run up in chunk order; with several runs it publishes the run's sum (in the scratch row of the run's
            // first chunk, which only it reads) and the warp that arrives last among the runs adds those up in order.
            auto chunk_id = [&](int64_t cidx) { return cidx == 0 ? 2 * (head / chunk) + 1 : 2 * ((head + cidx * chunk) / chunk); };
            auto publish = [&](double *dst_row) {
#pragma unroll
                for (int j = 0; j < NQ; ++j) {
                    double2 *dst = reinterpret_cast<double2 *>(dst_row + 4 * (lane + 32 * j));
                    dst[0] = make_double2(a[j][0], a[j][1]);
                    dst[1] = make_double2(a[j][2], a[j][3]);
                }
            };
            auto arrive = [&](unsigned int *counter, int64_t expected) {
                __threadfence();
                __syncwarp();
                int is_last = 0;
                if (lane == 0) is_last = (atomicAdd(counter, 1u) == static_cast<unsigned int>(expected - 1)) ? 1 : 0;
                is_last = __shfl_sync(0xFFFFFFFFu, is_last, 0);
                if (is_last) __threadfence();
                return is_last != 0;
            };
            auto add_up = [&](int64_t first, int64_t stop, int64_t step) {      // rows of chunks first, first + step, ... < stop
#pragma unroll
                for (int j = 0; j < NQ; ++j) {
                    const int64_t off = 4 * (lane + 32 * j);
#pragma unroll
                    for (int x = 0; x < 4; ++x) a[j][x] = __ldcg(&partial[chunk_id(first) * D + off + x]);
                }
                for (int64_t cidx = first + step; cidx < stop; cidx += step) {
                    const double *src = partial + chunk_id(cidx) * D;
#pragma unroll
                    for (int j = 0; j < NQ; ++j) {
                        const int64_t off = 4 * (lane + 32 * j);
#pragma unroll
                        for (int x = 0; x < 4; ++x) a[j][x] += __ldcg(&src[off + x]);
                    }
                }
            };
            const int64_t n_chunks = (gend - head + chunk - 1) / chunk;
            const int64_t my_chunk = (p - head) / chunk;
            const int64_t run = my_chunk / UPW_SUPER, n_runs = (n_chunks + UPW_SUPER - 1) / UPW_SUPER;
            const int64_t run_first = run * UPW_SUPER, run_stop = min(n_chunks, run_first + UPW_SUPER);
            publish(partial + chunk_id(my_chunk) * D);
            if (!arrive(&arrived[chunk_id(run_first)], run_stop - run_first)) continue;
            add_up(run_first, run_stop, 1);
            if (n_runs > 1) {
                publish(partial + chunk_id(run_first) * D);
                if (!arrive(&arrived_runs[chunk_id(0)], n_runs)) continue;
                add_up(0, n_chunks, UPW_SUPER);
            }
            count = gend - head;
        }
        double ss = 0.0;
#pragma unroll
        for (int j = 0; j < NQ; ++j) ss += a[j][0] * a[j][0] + a[j][1] * a[j][1] + a[j][2] * a[j][2] + a[j][3] * a[j][3];
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        const double norm = sqrt(ss);
        T *v = vecs + static_cast<int64_t>(slot) * D;
#pragma unroll
        for (int j = 0; j < NQ; ++j) {
            const float4 f = make_float4(static_cast<float>(a[j][0] / norm), static_cast<float>(a[j][1] / norm),
                                         static_cast<float>(a[j][2] / norm), static_cast<float>(a[j][3] / norm));
            *reinterpret_cast<float4 *>(m + 4 * (lane + 32 * j)) = f;
            if constexpr (sizeof(T) == 2) {
                const __nv_bfloat162 lo = __floats2bfloat162_rn(f.x, f.y), hi = __floats2bfloat162_rn(f.z, f.w);
                uint2 packed;
                packed.x = *reinterpret_cast<const uint32_t *>(&lo);
                packed.y = *reinterpret_cast<const uint32_t *>(&hi);
                *reinterpret_cast<uint2 *>(v + 4 * (lane + 32 * j)) = packed;
            }
        }
        if (lane == 0) {
            size[slot] = n_old + static_cast<double>(count);
            const unsigned long long acc_new = static_cast<unsigned long long>(access_old) + static_cast<unsigned long long>(count);
            access[slot] = (access_old == SISO_ACCESS_INF || acc_new >= SISO_ACCESS_INF) ? SISO_ACCESS_INF : static_cast<uint32_t>(acc_new);
            last[slot] = static_cast<unsigned long long>(counters[CNT_CLOCK]);
        }
    }
}

template <typename T>
static bool launch_update_apply_warp(int nq, unsigned blocks, cudaStream_t s, const int4 *desc, unsigned int list_len,
                                     const unsigned int *n_desc,
                                     unsigned int *ticket, const uint32_t *vs, int chunk, const T *q, float *master, T *vecs, double *size,
                                     uint32_t *access, unsigned long long *last, const long long *counters, double *partial,
                                     unsigned int *arrived, unsigned int *arrived_runs) {
#define SISO_UPW(N)                                                                                                          \
    case N: {                                                                                                                \
        const size_t smem = (UPW_THREADS / 32) * upw_warp_smem<T>(128 * N);                                                  \
        if (smem > 48 * 1024 &&                                                                                              \
            cudaFuncSetAttribute(update_apply_warp_kernel<T, N>, cudaFuncAttributeMaxDynamicSharedMemorySize,                \
                                 static_cast<int>(smem)) != cudaSuccess) {                                                   \
            cudaGetLastError();                                                                                              \
            return false;                                                                                                    \
        }                                                                                                                    \
        update_apply_warp_kernel<T, N><<<blocks, UPW_THREADS, smem, s>>>(desc, list_len, n_desc, ticket, vs, chunk, q, master, vecs, size, \
                                                                        access, last, counters, partial, arrived, arrived_runs); \
        return true;                                                                                                         \
    }
    switch (nq) {
        SISO_UPW(1) SISO_UPW(2) SISO_UPW(3) SISO_UPW(4) SISO_UPW(5) SISO_UPW(6) SISO_UPW(7) SISO_UPW(8)
        default: return false;
    }
#undef SISO_UPW
}

// Small batches (at most UPS_MAX_B rows): one launch.  CTA b looks at row b; it works only if row b is the first
// hit of its slot in the batch, then collects the later hits of that slot in ascending order (an ordered
// compaction in shared memory) and applies them exactly like update_apply_kernel.  Every CTA reads the clock
// before it signs off on a completion counter; the last CTA to sign off advances the clock, so no CTA can
// see the new value.
constexpr int UPS_MAX_B = 1024;

template <typename T>
__global__ void __launch_bounds__(UP_THREADS)
update_small_kernel(const int32_t *__restrict__ idx, int idx_stride, const uint8_t *__restrict__ hit, int B,
                    int64_t capacity, int D, const T *__restrict__ Q, float *__restrict__ master, T *__restrict__ vecs,
                    double *__restrict__ size, uint32_t *__restrict__ access, unsigned long long *__restrict__ last,
                    const uint8_t *__restrict__ valid, long long *counters, int *status) {
    extern __shared__ double acc[];          // [D]
    __shared__ double red[UP_THREADS / 32];
    __shared__ uint16_t members[UPS_MAX_B];
    __shared__ int warp_cnt[UP_THREADS / 32];
    __shared__ long long clock_s;
    __shared__ int n_members_s;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) clock_s = counters[CNT_CLOCK];
    bool work = false;
    int64_t slot = -1;
    if (hit[b]) {
        slot = idx[static_cast<int64_t>(b) * idx_stride];
        if (slot >= 0 && slot < capacity && valid[slot]) work = true;
        else if (tid == 0) set_status(status, SISO_ERR_INVALID_ARG);     // a hit must name a live slot; the row is skipped
    }
    if (work) {
        // is an earlier row a hit on the same slot?  then that row's CTA owns the group
        int earlier = 0;
        for (int r = tid; r < b; r += UP_THREADS) earlier |= (hit[r] && idx[static_cast<int64_t>(r) * idx_stride] == slot) ? 1 : 0;
        work = __syncthreads_or(earlier) == 0;
    }
    if (work) {
        // members of the group in ascending row order: rows b.. in chunks of 256, ballot-ordered
        int base_count = 0;
        for (int r0 = b; r0 < B; r0 += UP_THREADS) {
            const int r = r0 + tid;
            const bool mine = r < B && hit[r] && idx[static_cast<int64_t>(r) * idx_stride] == slot;
            const unsigned ballot = __ballot_sync(0xFFFFFFFFu, mine);
            if (lane == 0) warp_cnt[warp] = __popc(ballot);
            __syncthreads();
            int before = base_count, total = 0;
            for (int w = 0; w < UP_THREADS / 32; ++w) { if (w < warp) before += warp_cnt[w]; total += warp_cnt[w]; }
            if (mine) members[before + __popc(ballot & ((1u << lane) - 1u))] = static_cast<uint16_t>(r);
            base_count += total;
            __syncthreads();
        }
        if (tid == 0) n_members_s = base_count;
        const double n_old = size[slot];
        float *m = master + slot * D;
        for (int d = tid; d < D; d += UP_THREADS) acc[d] = n_old * static_cast<double>(m[d]);
        __syncthreads();
        const int count = n_members_s;
        const int quads = D / 4;
        constexpr int R = 8;                 // rows in flight per trip; additions stay in ascending row order
        for (int t = 0; t < count; t += R) {
            const int nrow = count - t < R ? count - t : R;
            const T *q[R];
#pragma unroll
            for (int r = 0; r < R; ++r) q[r] = Q + static_cast<int64_t>(members[t + (r < nrow ? r : 0)]) * D;
            for (int g = tid; g < quads; g += UP_THREADS) {
                float4 v[R];
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = load4<T>(q[r] + 4 * g);
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
        for (int d = tid; d < D; d += UP_THREADS) ss += acc[d] * acc[d];
        const double norm = sqrt(block_sum_f64(ss, red));
        T *v = vecs + slot * D;
        for (int d = tid; d < D; d += UP_THREADS) {
            const float f = static_cast<float>(acc[d] / norm);
            m[d] = f;
            if constexpr (sizeof(T) == 2) v[d] = __float2bfloat16_rn(f);
        }
        if (tid == 0) {
            size[slot] = n_old + static_cast<double>(count);
            const unsigned long long a = static_cast<unsigned long long>(access[slot]) + static_cast<unsigned long long>(count);
            access[slot] = (access[slot] == SISO_ACCESS_INF || a >= SISO_ACCESS_INF) ? SISO_ACCESS_INF : static_cast<uint32_t>(a);
            last[slot] = static_cast<unsigned long long>(clock_s + 1);
        }
    }
    // sign off; the last CTA advances the clock (every CTA has read it by then) and re-arms the counter
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned long long done = atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_SYNC), 1ull);
        if (done == gridDim.x - 1) {
            counters[CNT_CLOCK] = clock_s + 1;
            counters[CNT_SYNC] = 0;
        }
    }
}

siso_status_t launch_update(Cache *c, const void *q, int64_t B, const int32_t *idx, int idx_stride, const uint8_t *hit,
                            cudaStream_t s) {
    c->vec_epoch += 1;          // the vectors may change: derived copies (the split-bf16 parts) are stale
    if (B >= (1ll << 31)) return SISO_ERR_UNSUPPORTED;
    if (B >= 1 && B <= UPS_MAX_B) {
        const size_t smem_small = sizeof(double) * c->dim;
        if (c->dtype == SISO_F32)
            update_small_kernel<float><<<static_cast<unsigned>(B), UP_THREADS, smem_small, s>>>(
                idx, idx_stride, hit, static_cast<int>(B), c->capacity, c->dim, static_cast<const float *>(q), c->master,
                static_cast<float *>(c->vecs), c->size, c->access, c->last, c->valid, c->counters, c->status);
        else
            update_small_kernel<__nv_bfloat16><<<static_cast<unsigned>(B), UP_THREADS, smem_small, s>>>(
                idx, idx_stride, hit, static_cast<int>(B), c->capacity, c->dim, static_cast<const __nv_bfloat16 *>(q),
                c->master, static_cast<__nv_bfloat16 *>(c->vecs), c->size, c->access, c->last, c->valid, c->counters,
                c->status);
        SISO_LAUNCHED(c);
        return SISO_OK;
    }
    Scratch scr;
    const int chunk = static_cast<int>(std::max<int64_t>(32, (B + 4095) / 4096));
    const size_t n_ids = 2 * static_cast<size_t>(B / chunk + 1);
    const bool warp_path = c->dim % 128 == 0 && c->dim <= 1024;
    const size_t need = 4 * pad256(sizeof(uint32_t) * B) + sort_pairs_scratch_bytes(B) +
                        pad256(sizeof(double) * n_ids * c->dim) + pad256(sizeof(unsigned int) * (2 * n_ids + 4)) +
                        pad256(sizeof(int4) * 2 * B);
    SISO_TRY(scratch_reserve(c, need, s, &scr));
    uint32_t *keys = scr.take<uint32_t>(B), *vals = scr.take<uint32_t>(B);
    uint32_t *keys2 = scr.take<uint32_t>(B), *vals2 = scr.take<uint32_t>(B);
    const int threads = 256;
    // B == 0 still advances the clock
    const unsigned blocks = static_cast<unsigned>((std::max<int64_t>(B, 1) + threads - 1) / threads);
    update_keys_kernel<<<blocks, threads, 0, s>>>(idx, idx_stride, hit, c->valid, B, c->capacity, keys, vals,
                                                  c->counters, c->status);
    SISO_LAUNCHED(c);
    if (B == 0) return SISO_OK;
    int key_bits = 1;
    while ((1ll << key_bits) <= c->capacity) ++key_bits;      // keys go up to `capacity` inclusive
    uint32_t *ks, *vs;
    SISO_TRY(launch_sort_pairs(c, &scr, keys, vals, keys2, vals2, B, key_bits, &ks, &vs, s));
    const size_t smem = sizeof(double) * c->dim;
    double *partial = scr.take<double>(n_ids * c->dim);
    // arrival counters per chunk id; number of chunks listed from the front and from the back (+ one unused word); the
    // ticket counter; arrival counters of the runs
    unsigned int *arrived = scr.take<unsigned int>(2 * n_ids + 4);
    int4 *desc = scr.take<int4>(2 * B);
    SISO_CUDA(cudaMemsetAsync(arrived, 0, sizeof(unsigned int) * (2 * n_ids + 4), s));
    if (warp_path) {
        // the list of chunks, then resident warps that walk it with the sums in registers
        update_chunks_kernel<<<static_cast<unsigned>((B + 255) / 256), 256, 0, s>>>(ks, vs, B, c->capacity, chunk, desc, arrived + n_ids);
        SISO_LAUNCHED(c);
        const unsigned wblocks = static_cast<unsigned>(std::min<int64_t>((B + UPW_THREADS / 32 - 1) / (UPW_THREADS / 32), 4ll * c->sm_count));
        if (c->dtype == SISO_F32)
            launch_update_apply_warp<float>(c->dim / 128, wblocks, s, desc, static_cast<unsigned int>(B), arrived + n_ids, arrived + n_ids + 3, vs, chunk, static_cast<const float *>(q),
                                            c->master, static_cast<float *>(c->vecs), c->size, c->access, c->last, c->counters,
                                            partial, arrived, arrived + n_ids + 4);
        else
            launch_update_apply_warp<__nv_bfloat16>(c->dim / 128, wblocks, s, desc, static_cast<unsigned int>(B), arrived + n_ids, arrived + n_ids + 3, vs, chunk,
                                                    static_cast<const __nv_bfloat16 *>(q), c->master,
                                                    static_cast<__nv_bfloat16 *>(c->vecs), c->size, c->access, c->last,
                                                    c->counters, partial, arrived, arrived + n_ids + 4);
    } else if (c->dtype == SISO_F32) {
        update_apply_kernel<float><<<static_cast<unsigned>(B), UP_THREADS, smem, s>>>(
            ks, vs, B, c->capacity, c->dim, chunk, static_cast<const float *>(q), c->master, static_cast<float *>(c->vecs),
            c->size, c->access, c->last, c->counters, partial, arrived);
    } else {
        update_apply_kernel<__nv_bfloat16><<<static_cast<unsigned>(B), UP_THREADS, smem, s>>>(
            ks, vs, B, c->capacity, c->dim, chunk, static_cast<const __nv_bfloat16 *>(q), c->master,
            static_cast<__nv_bfloat16 *>(c->vecs), c->size, c->access, c->last, c->counters, partial, arrived);
    }
    SISO_LAUNCHED(c);
    return SISO_OK;
}

}  // namespace siso
