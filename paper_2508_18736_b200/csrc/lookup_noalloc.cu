// siso_lookup_small_noalloc: the small-batch streaming lookup for callers that must not allocate.
//
// Who that is: code running where a device allocation is forbidden or would stall the GPU -
// inside a latency-critical serving loop that has already handed all device memory to its own
// pools, inside a library callback that may run while another thread holds the allocator lock, or
// in a process whose memory budget was fixed at start-up.  cudaMalloc and cudaFree synchronise the
// device and can fail at an arbitrary moment; such callers need a lookup whose only device
// memory is what they pass in.
//
// The per-CTA partial results that the ordinary path keeps in scratch obtained from the cache's
// allocator live here in one file-scope device array of fixed size (kNoAllocScratchBytes, held by
// every GPU that loads the library until the process exits).  Consequences, all documented in
// include/siso.h: the batch and k are bounded, all calls share the array (calls that overlap on
// the GPU race with each other), and the first call on each device looks the array's device
// address up (a symbol lookup, not an allocation), so it should come before any stream capture.
#include <mutex>

#include "common.cuh"
#include "stream_rows.cuh"

namespace siso {
namespace noalloc {

constexpr int NA_THREADS = 256;
constexpr int NA_WARPS = NA_THREADS / 32;
constexpr int NA_MAX_Q = 8;           // queries per call
constexpr int NA_K = 8;               // list length kept per query (k <= 8)
constexpr int NA_MAX_CTAS = 1024;     // CTAs that may publish partial lists
constexpr int NA_MAX_DIM = 1024;      // NA_MAX_Q * dim * 4 bytes of shared memory (+4 KiB of lists) stays within the 48 KiB default
constexpr size_t kNoAllocScratchBytes = sizeof(unsigned long long) * NA_MAX_CTAS * NA_MAX_Q * NA_K;   // 512 KiB
static_assert(NA_MAX_Q == SISO_NOALLOC_MAX_QUERIES && NA_MAX_DIM == SISO_NOALLOC_MAX_DIM, "limits stated in siso.h");

// [cta][query][NA_K] packed (similarity, slot) keys.  Device code may name this array directly; host
// code may not pass its name to a kernel (on the host the name is only a stand-in for the symbol):
// the launcher below asks the runtime for the device address once per device.
static __device__ __align__(256) unsigned long long g_partial[NA_MAX_CTAS * NA_MAX_Q * NA_K];

template <typename T> __device__ __forceinline__ float elem(const T *p);
template <> __device__ __forceinline__ float elem<float>(const float *p) { return __ldg(p); }
template <> __device__ __forceinline__ float elem<__nv_bfloat16>(const __nv_bfloat16 *p) {
    return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short *>(p))) << 16);
}

// Each warp takes one centroid row at a time; lane l multiplies elements l, l+32, ... of the row
// with every query (fp32 FMA, queries in shared memory) and the warp sums the NA_MAX_Q partial dot
// products with shuffles.  Lane b keeps the running top-NA_K of query b (rows arrive in ascending
// order per warp, so a strict comparison keeps the lower slot on ties).
template <typename T>
__global__ void __launch_bounds__(NA_THREADS)
lookup_noalloc_kernel(const T *__restrict__ C, const uint8_t *__restrict__ valid, long long N, int D,
                      const T *__restrict__ Q, int nq, long long rows_per_cta, unsigned long long *__restrict__ partial) {
    extern __shared__ __align__(16) float qs[];        // [NA_MAX_Q][D]
    __shared__ unsigned long long lists[NA_WARPS][NA_MAX_Q][NA_K];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < NA_MAX_Q * D; i += NA_THREADS) {
        const int b = i / D;
        qs[i] = b < nq ? elem<T>(Q + static_cast<long long>(b) * D + (i - b * D)) : 0.f;
    }
    __syncthreads();
    TopK<NA_K> top;
    top.clear();
    const long long row_begin = static_cast<long long>(blockIdx.x) * rows_per_cta;
    const long long row_end = min(N, row_begin + rows_per_cta);
    for (long long n = row_begin + warp; n < row_end; n += NA_WARPS) {
        if (valid && !valid[n]) continue;
        float acc[NA_MAX_Q];
#pragma unroll
        for (int b = 0; b < NA_MAX_Q; ++b) acc[b] = 0.f;
        const T *row = C + n * D;
        for (int d = lane; d < D; d += 32) {
            const float c = elem<T>(row + d);
#pragma unroll
            for (int b = 0; b < NA_MAX_Q; ++b) acc[b] = fmaf(c, qs[b * D + d], acc[b]);
        }
#pragma unroll
        for (int b = 0; b < NA_MAX_Q; ++b) {
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) acc[b] += __shfl_xor_sync(0xFFFFFFFFu, acc[b], o);
        }
        float mine = 0.f;
#pragma unroll
        for (int b = 0; b < NA_MAX_Q; ++b) mine = (lane == b) ? acc[b] : mine;
        if (lane < nq) top.push(mine, static_cast<int32_t>(n));
    }
    if (lane < NA_MAX_Q) {
#pragma unroll
        for (int j = 0; j < NA_K; ++j) lists[warp][lane][j] = lane < nq ? top.key(j) : 0ull;
    }
    __syncthreads();
    // every launched CTA writes ALL of its entries (zeros where it found nothing), so the array never
    // needs clearing between calls: nothing read in this call was left over from an earlier one
    if (tid < NA_MAX_Q) {
        KeyList<NA_K> out;
        out.clear();
        for (int w = 0; w < NA_WARPS; ++w)
#pragma unroll
            for (int j = 0; j < NA_K; ++j) out.insert(lists[w][tid][j]);
        unsigned long long *dst = partial + (static_cast<long long>(blockIdx.x) * NA_MAX_Q + tid) * NA_K;
#pragma unroll
        for (int j = 0; j < NA_K; ++j) dst[j] = out.k[j];
    }
}

// The same sweep for matrices that allow 128-bit loads (dim a multiple of 8, base address a multiple of 16): four
// rows in flight per warp, lane l takes elements [8 l, 8 l + 8) of every stretch of 256, the 4 x BQ partial dot
// products of a step are summed across the warp by one transposing reduction, and the lane that ends up with the
// sum of (row r, query b) keeps the running top-NA_K of its rows for that query.  Rows past the end of the matrix
// are read from its last row and not counted.
template <typename T, int BQ>
__global__ void __launch_bounds__(NA_THREADS)
lookup_noalloc_vec_kernel(const T *__restrict__ C, const uint8_t *__restrict__ valid, long long N, int D,
                          const T *__restrict__ Q, int nq, long long rows_per_cta, unsigned long long *__restrict__ partial) {
    extern __shared__ __align__(16) float qs[];        // [BQ][D]; later the lists of all threads
    constexpr int ROWS = 4;
    constexpr int V = ROWS * BQ;                       // values reduced per step; value index = r * BQ + b
    constexpr int SHARE = 32 / V;                      // lanes that end up holding the same value
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < BQ * D; i += NA_THREADS) {
        const int b = i / D;
        qs[i] = b < nq ? elem<T>(Q + static_cast<long long>(b) * D + (i - b * D)) : 0.f;
    }
    __syncthreads();
    const int my_val = lane / SHARE, my_r = my_val / BQ, my_b = my_val % BQ;
    TopK<NA_K> top;
    top.clear();
    const long long row_begin = static_cast<long long>(blockIdx.x) * rows_per_cta;
    const long long row_end = min(N, row_begin + rows_per_cta);
    const int chunks = D / 8;
    for (long long n0 = row_begin + warp * ROWS; n0 < row_end; n0 += NA_WARPS * ROWS) {
        bool live[ROWS];
        const T *row[ROWS];
        bool any = false;
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const long long n = n0 + r;
            live[r] = n < row_end && (!valid || valid[n] != 0);
            row[r] = C + (n < N ? n : N - 1) * D;
            any = any || live[r];
        }
        if (!any) continue;
        float acc[V];
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = 0.f;
        for (int ch = lane; ch < chunks; ch += 32) {
            float cf[ROWS][8];
#pragma unroll
            for (int r = 0; r < ROWS; ++r) Chunk8<T>::load(row[r] + ch * 8, cf[r]);
#pragma unroll
            for (int b = 0; b < BQ; ++b) {
                const float4 q0 = *reinterpret_cast<const float4 *>(qs + b * D + ch * 8);
                const float4 q1 = *reinterpret_cast<const float4 *>(qs + b * D + ch * 8 + 4);
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    float a = acc[r * BQ + b];
                    a = fmaf(cf[r][0], q0.x, a); a = fmaf(cf[r][1], q0.y, a);
                    a = fmaf(cf[r][2], q0.z, a); a = fmaf(cf[r][3], q0.w, a);
                    a = fmaf(cf[r][4], q1.x, a); a = fmaf(cf[r][5], q1.y, a);
                    a = fmaf(cf[r][6], q1.z, a); a = fmaf(cf[r][7], q1.w, a);
                    acc[r * BQ + b] = a;
                }
            }
        }
        warp_transpose_reduce<V>(acc, lane);
        bool mine = false;
#pragma unroll
        for (int r = 0; r < ROWS; ++r) mine = (r == my_r) ? live[r] : mine;
        if ((lane % SHARE) == 0 && mine && my_b < nq) top.push(acc[0], static_cast<int32_t>(n0 + my_r));
    }
    // every thread publishes its list (empty unless it owns a (row, query) value); one thread per query merges
    __syncthreads();
    unsigned long long *lists = reinterpret_cast<unsigned long long *>(qs);     // [NA_THREADS][NA_K]
#pragma unroll
    for (int j = 0; j < NA_K; ++j) lists[tid * NA_K + j] = ((lane % SHARE) == 0 && my_b < nq) ? top.key(j) : 0ull;
    __syncthreads();
    // as in the scalar kernel every CTA writes ALL of its entries of the shared array, zeros where it has nothing
    if (tid < NA_MAX_Q) {
        KeyList<NA_K> out;
        out.clear();
        if (tid < nq) {
            for (int t = 0; t < NA_THREADS; ++t) {
                const int l = t & 31;
                if ((l % SHARE) != 0 || ((l / SHARE) % BQ) != tid) continue;
#pragma unroll
                for (int j = 0; j < NA_K; ++j) out.insert(lists[t * NA_K + j]);
            }
        }
        unsigned long long *dst = partial + (static_cast<long long>(blockIdx.x) * NA_MAX_Q + tid) * NA_K;
#pragma unroll
        for (int j = 0; j < NA_K; ++j) dst[j] = out.k[j];
    }
}

template <typename T, int BQ>
static void run_vec(const void *C, const uint8_t *valid, long long N, int D, const void *Q, int nq, long long rows_per_cta,
                    int n_ctas, unsigned long long *partial, cudaStream_t s) {
    // the query block and, afterwards, 256 lists of NA_K keys share the dynamic shared memory: at most 32 KiB, within
    // the default limit
    const size_t smem = std::max(sizeof(float) * BQ * D, sizeof(unsigned long long) * NA_THREADS * NA_K);
    lookup_noalloc_vec_kernel<T, BQ><<<n_ctas, NA_THREADS, smem, s>>>(static_cast<const T *>(C), valid, N, D,
                                                                      static_cast<const T *>(Q), nq, rows_per_cta, partial);
}
template <typename T>
static void run_vec_bq(const void *C, const uint8_t *valid, long long N, int D, const void *Q, int nq, long long rows_per_cta,
                       int n_ctas, unsigned long long *partial, cudaStream_t s) {
    if (nq <= 1) run_vec<T, 1>(C, valid, N, D, Q, nq, rows_per_cta, n_ctas, partial, s);
    else if (nq <= 2) run_vec<T, 2>(C, valid, N, D, Q, nq, rows_per_cta, n_ctas, partial, s);
    else if (nq <= 4) run_vec<T, 4>(C, valid, N, D, Q, nq, rows_per_cta, n_ctas, partial, s);
    else run_vec<T, 8>(C, valid, N, D, Q, nq, rows_per_cta, n_ctas, partial, s);
}

// One warp per query: lane l merges the lists of CTAs l, l + 32, ..., then the 32 lists are merged by a butterfly of
// shuffles (partners always hold lists of disjoint CTAs, so no key is counted twice); lane 0 writes the answer.
__global__ void __launch_bounds__(32)
lookup_noalloc_finalize_kernel(const unsigned long long *__restrict__ partial, int n_ctas, int nq, int k,
                               const float *__restrict__ theta, float theta_s,
                               int32_t *__restrict__ idx, float *__restrict__ sim,
                               uint8_t *__restrict__ hit) {
    const int b = blockIdx.x, lane = threadIdx.x;
    if (b >= nq) return;
    KeyList<NA_K> out;
    out.clear();
    for (int c = lane; c < n_ctas; c += 32) {
        const unsigned long long *src = partial + (static_cast<long long>(c) * NA_MAX_Q + b) * NA_K;
        unsigned long long v[NA_K];
#pragma unroll
        for (int j = 0; j < NA_K; ++j) v[j] = src[j];
#pragma unroll
        for (int j = 0; j < NA_K; ++j) out.insert(v[j]);
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long other[NA_K];
#pragma unroll
        for (int j = 0; j < NA_K; ++j) other[j] = __shfl_xor_sync(0xFFFFFFFFu, out.k[j], o);
#pragma unroll
        for (int j = 0; j < NA_K; ++j) out.insert(other[j]);
    }
    if (lane != 0) return;
#pragma unroll
    for (int j = 0; j < NA_K; ++j) {
        if (j < k) {
            const unsigned long long key = out.k[j];
            idx[b * k + j] = key ? key_slot(key) : -1;
            sim[b * k + j] = key ? key_sim(key) : -INFINITY;
        }
    }
    const float th = theta ? theta[b] : theta_s;
    hit[b] = (out.k[0] != 0ull && key_sim(out.k[0]) > th) ? 1 : 0;
}

// Per-device set-up: the device address of g_partial on that device and its SM count.
struct DeviceSetup {
    bool ready;
    unsigned long long *partial;
    int sm_count;
};
constexpr int kMaxDevices = 64;
static DeviceSetup g_setup[kMaxDevices];
static std::mutex g_setup_mutex;

static siso_status_t device_setup(int device, DeviceSetup *out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup &s = g_setup[device];
    if (!s.ready) {
        void *ptr = nullptr;
        // with `device` current this returns the address of THAT device's copy of the array
        SISO_CUDA(cudaGetSymbolAddress(&ptr, g_partial));
        int sms = 0;
        SISO_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
        s.partial = static_cast<unsigned long long *>(ptr);
        s.sm_count = sms;
        s.ready = true;
    }
    *out = s;
    return SISO_OK;
}

}  // namespace noalloc
}  // namespace siso

using namespace siso;
using namespace siso::noalloc;

extern "C" siso_status_t siso_lookup_small_noalloc(const void *d_centroids, const uint8_t *d_valid, int64_t n_centroids,
                                                   int32_t dim, int32_t dtype, const void *d_queries, int64_t n_queries,
                                                   const float *d_theta, float theta_scalar, int32_t k, int32_t *d_idx,
                                                   float *d_sim, uint8_t *d_hit, void *stream) {
    if (!d_centroids || !d_queries || !d_idx || !d_sim || !d_hit) return SISO_ERR_INVALID_ARG;
    if (dtype != SISO_F32 && dtype != SISO_BF16) return SISO_ERR_INVALID_ARG;
    if (n_centroids < 1 || n_centroids >= (1ll << 31) || k < 1) return SISO_ERR_INVALID_ARG;
    // the fixed scratch array bounds the batch and k; shared memory bounds dim
    if (n_queries < 1 || n_queries > NA_MAX_Q || k > NA_K || dim < 1 || dim > NA_MAX_DIM) return SISO_ERR_UNSUPPORTED;
    int device = 0;
    SISO_CUDA(cudaGetDevice(&device));
    if (device < 0 || device >= kMaxDevices) return SISO_ERR_UNSUPPORTED;
    DeviceSetup su;
    SISO_TRY(device_setup(device, &su));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int n_ctas = std::min(NA_MAX_CTAS, 4 * su.sm_count);
    const long long rows_per_cta = (n_centroids + n_ctas - 1) / n_ctas;
    n_ctas = static_cast<int>((n_centroids + rows_per_cta - 1) / rows_per_cta);
    const size_t smem = sizeof(float) * NA_MAX_Q * dim;
    const int nq = static_cast<int>(n_queries);
    // 128-bit loads need rows that start on 16-byte boundaries (and, for fp32, pairs of them: dim a multiple of 8)
    const bool vec = dim % 8 == 0 && (reinterpret_cast<uintptr_t>(d_centroids) & 15u) == 0;
    if (vec && dtype == SISO_F32)
        run_vec_bq<float>(d_centroids, d_valid, n_centroids, dim, d_queries, nq, rows_per_cta, n_ctas, su.partial, s);
    else if (vec)
        run_vec_bq<__nv_bfloat16>(d_centroids, d_valid, n_centroids, dim, d_queries, nq, rows_per_cta, n_ctas, su.partial, s);
    else if (dtype == SISO_F32)
        lookup_noalloc_kernel<float><<<n_ctas, NA_THREADS, smem, s>>>(
            static_cast<const float *>(d_centroids), d_valid, n_centroids, dim, static_cast<const float *>(d_queries),
            static_cast<int>(n_queries), rows_per_cta, su.partial);
    else
        lookup_noalloc_kernel<__nv_bfloat16><<<n_ctas, NA_THREADS, smem, s>>>(
            static_cast<const __nv_bfloat16 *>(d_centroids), d_valid, n_centroids, dim,
            static_cast<const __nv_bfloat16 *>(d_queries), static_cast<int>(n_queries), rows_per_cta, su.partial);
    SISO_CUDA(cudaGetLastError());
    lookup_noalloc_finalize_kernel<<<nq, 32, 0, s>>>(su.partial, n_ctas, nq, k, d_theta,
                                                    theta_scalar, d_idx, d_sim, d_hit);
    SISO_CUDA(cudaGetLastError());
    return SISO_OK;
}
