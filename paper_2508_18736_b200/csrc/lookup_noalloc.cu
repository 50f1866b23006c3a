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

__global__ void lookup_noalloc_finalize_kernel(const unsigned long long *__restrict__ partial, int n_ctas, int nq, int k,
                                               const float *__restrict__ theta, float theta_s,
                                               int32_t *__restrict__ idx, float *__restrict__ sim,
                                               uint8_t *__restrict__ hit) {
    const int b = threadIdx.x;
    if (b >= nq) return;
    KeyList<NA_K> out;
    out.clear();
    for (int c = 0; c < n_ctas; ++c)
#pragma unroll
        for (int j = 0; j < NA_K; ++j) out.insert(partial[(static_cast<long long>(c) * NA_MAX_Q + b) * NA_K + j]);
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
    if (dtype == SISO_F32)
        lookup_noalloc_kernel<float><<<n_ctas, NA_THREADS, smem, s>>>(
            static_cast<const float *>(d_centroids), d_valid, n_centroids, dim, static_cast<const float *>(d_queries),
            static_cast<int>(n_queries), rows_per_cta, su.partial);
    else
        lookup_noalloc_kernel<__nv_bfloat16><<<n_ctas, NA_THREADS, smem, s>>>(
            static_cast<const __nv_bfloat16 *>(d_centroids), d_valid, n_centroids, dim,
            static_cast<const __nv_bfloat16 *>(d_queries), static_cast<int>(n_queries), rows_per_cta, su.partial);
    SISO_CUDA(cudaGetLastError());
    lookup_noalloc_finalize_kernel<<<1, 32, 0, s>>>(su.partial, n_ctas, static_cast<int>(n_queries), k, d_theta,
                                                    theta_scalar, d_idx, d_sim, d_hit);
    SISO_CUDA(cudaGetLastError());
    return SISO_OK;
}
