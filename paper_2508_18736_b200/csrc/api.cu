// C ABI of libsiso: argument checking, state, scratch memory and kernel launches.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "common.cuh"

namespace siso {

static thread_local char g_last_error[512] = "";

siso_status_t check_cuda(cudaError_t e, const char *what) {
    if (e == cudaSuccess) return SISO_OK;
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, cudaGetErrorString(e));
    return e == cudaErrorMemoryAllocation ? SISO_ERR_OOM : SISO_ERR_CUDA;
}

static void *default_alloc(size_t bytes, void *, void *) {
    void *p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return p;
}
static void default_free(void *p, void *) { cudaFree(p); }

static void *cache_alloc(Cache *c, size_t bytes, cudaStream_t s) {
    return c->alloc.alloc(bytes ? bytes : 256, s, c->alloc.ctx);
}

void *cache_alloc_zeroed(Cache *c, size_t bytes) {
    void *p = cache_alloc(c, bytes, nullptr);
    if (p && cudaMemset(p, 0, bytes) != cudaSuccess) {
        cudaGetLastError();
        c->alloc.free(p, c->alloc.ctx);
        return nullptr;
    }
    return p;
}

// A block that an earlier call handed to kernels is released only once the device is idle: the kernels of earlier
// calls (on this stream or, for a handle used on several streams, on another one) may still be reading or writing it,
// and an allocator with per-stream pools (torch's) would otherwise hand the block to someone else at once.  Regrowth is
// rare (the buffers grow by a quarter more than asked and never shrink), so the wait costs nothing in the steady state.
static siso_status_t retire_block(Cache *c, void *p) {
    if (!p) return SISO_OK;
    SISO_CUDA(cudaDeviceSynchronize());
    c->alloc.free(p, c->alloc.ctx);
    return SISO_OK;
}

siso_status_t scratch_reserve(Cache *c, size_t bytes, cudaStream_t s, Scratch *out) {
    bytes += 4096;
    if (bytes > c->ws_bytes) {
        void *old = c->ws;
        c->ws = nullptr;
        c->ws_bytes = 0;
        SISO_TRY(retire_block(c, old));
        const size_t want = bytes + bytes / 4;
        c->ws = cache_alloc(c, want, s);
        if (!c->ws) return SISO_ERR_OOM;
        c->ws_bytes = want;
    }
    out->base = static_cast<char *>(c->ws);
    out->off = 0;
    out->cap = c->ws_bytes;
    return SISO_OK;
}

siso_status_t stage_reserve(Cache *c, size_t bytes, cudaStream_t s) {
    if (bytes > c->stage_bytes) {
        void *old = c->stage;
        c->stage = nullptr;
        c->stage_bytes = 0;
        SISO_TRY(retire_block(c, old));
        c->stage = cache_alloc(c, bytes, s);
        if (!c->stage) return SISO_ERR_OOM;
        c->stage_bytes = bytes;
    }
    return SISO_OK;
}

__global__ void bf16_from_master_kernel(const float *__restrict__ m, __nv_bfloat16 *__restrict__ v, long long n) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) v[i] = __float2bfloat16_rn(m[i]);
}

__global__ void import_counters_kernel(const uint8_t *__restrict__ valid, long long capacity, long long *counters,
                                       unsigned long long clock) {
    __shared__ int warp_sum[32];
    long long cnt = 0;
    for (long long i = threadIdx.x; i < capacity; i += blockDim.x) cnt += valid[i] ? 1 : 0;
    int x = static_cast<int>(cnt);
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long t = 0;
        for (int w = 0; w < static_cast<int>(blockDim.x / 32); ++w) t += warp_sum[w];
        counters[CNT_OCCUPANCY] = t;
        counters[CNT_CLOCK] = static_cast<long long>(clock);
    }
}

__global__ void normalise_valid_kernel(uint8_t *valid, long long n) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) valid[i] = valid[i] ? 1 : 0;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- checked mode (SISO_OPT_CHECKED): what the library otherwise takes on trust is verified on the device ----------
// One warp per row: the row must be a unit vector (| |x| - 1 | < 1e-2; bf16 rounding of a unit vector stays within
// 2e-3) with finite elements.  A row that is not sets SISO_ERR_INVALID_ARG in the status word; nothing traps.
template <typename T>
__global__ void __launch_bounds__(256)
check_unit_rows_kernel(const T *__restrict__ rows, long long n, int D, const uint8_t *__restrict__ skip_if_set, int *status) {
    const int lane = threadIdx.x & 31;
    const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    for (long long r = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); r < n; r += warps) {
        if (skip_if_set && skip_if_set[r]) continue;           // rows the call will not store (hits of siso_insert_misses)
        double ss = 0.0;
        for (int d = lane; d < D; d += 32) {
            float v;
            if constexpr (sizeof(T) == 2) v = __bfloat162float(rows[r * D + d]); else v = rows[r * D + d];
            ss += static_cast<double>(v) * static_cast<double>(v);
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        if (lane == 0 && !(fabs(sqrt(ss) - 1.0) < 1e-2)) set_status(status, SISO_ERR_INVALID_ARG);      // NaN fails too
    }
}

// the largest | |v| - 1 | over the live rows of the vectors that lookups read (fp64 sums), as the bit pattern of a
// non-negative float (those order like unsigned integers); a row with a NaN counts as infinitely far
template <typename T>
__global__ void __launch_bounds__(256)
norm_deviation_kernel(const T *__restrict__ rows, const uint8_t *__restrict__ valid, long long n, int D, unsigned int *out_bits) {
    const int lane = threadIdx.x & 31;
    const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    for (long long r = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); r < n; r += warps) {
        if (!valid[r]) continue;
        double ss = 0.0;
        for (int d = lane; d < D; d += 32) {
            float v;
            if constexpr (sizeof(T) == 2) v = __bfloat162float(rows[r * D + d]); else v = rows[r * D + d];
            ss += static_cast<double>(v) * static_cast<double>(v);
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        if (lane == 0) {
            const double dev = fabs(sqrt(ss) - 1.0);
            const float up = dev == dev ? __double2float_ru(dev) : __int_as_float(0x7F800000);
            atomicMax(out_bits, __float_as_uint(up));
        }
    }
}

// thresholds must be numbers; hit flags 0 or 1; slots of hits inside the cache
__global__ void check_batch_args_kernel(const float *__restrict__ theta, const uint8_t *__restrict__ hit, const int32_t *__restrict__ idx,
                                        int idx_stride, long long n, long long capacity, int *status) {
    const long long b = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (b >= n) return;
    bool ok = true;
    if (theta && !(theta[b] == theta[b])) ok = false;
    if (hit && hit[b] > 1) ok = false;
    if (hit && idx && hit[b] == 1 && (idx[b * idx_stride] < 0 || idx[b * idx_stride] >= capacity)) ok = false;
    if (!ok) set_status(status, SISO_ERR_INVALID_ARG);
}

static siso_status_t checked_rows(Cache *c, const void *rows, int64_t n, const uint8_t *skip_if_set, cudaStream_t s) {
    if (!c->checked || n <= 0) return SISO_OK;
    const unsigned blocks = static_cast<unsigned>(std::min<int64_t>((n + 7) / 8, 8ll * c->sm_count));
    if (c->dtype == SISO_F32)
        check_unit_rows_kernel<float><<<blocks, 256, 0, s>>>(static_cast<const float *>(rows), n, c->dim, skip_if_set, c->status);
    else
        check_unit_rows_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(rows), n, c->dim, skip_if_set, c->status);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

static siso_status_t checked_batch(Cache *c, const float *theta, const uint8_t *hit, const int32_t *idx, int idx_stride, int64_t n,
                                   cudaStream_t s) {
    if (!c->checked || n <= 0 || (!theta && !hit)) return SISO_OK;
    check_batch_args_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, s>>>(theta, hit, idx, idx_stride, n, c->capacity, c->status);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

}  // namespace siso

using namespace siso;

struct siso_cache : public siso::Cache {};

extern "C" {

const char *siso_status_string(siso_status_t s) {
    switch (s) {
        case SISO_OK: return "ok";
        case SISO_ERR_INVALID_ARG: return "invalid argument";
        case SISO_ERR_UNSUPPORTED: return "unsupported";
        case SISO_ERR_OOM: return "out of device memory";
        case SISO_ERR_CAPACITY: return "not enough free slots";
        case SISO_ERR_OVERFLOW: return "merge candidate buffer overflow";
        case SISO_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case SISO_ERR_CUDA: return "CUDA error";
    }
    return "unknown status";
}

const char *siso_last_cuda_error(void) { return g_last_error; }

siso_status_t siso_cache_create(siso_cache_t **out, const siso_config_t *cfg) {
    if (!out || !cfg) return SISO_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->capacity < 1 || cfg->capacity >= (1ll << 31) - siso::kRowPad) return SISO_ERR_INVALID_ARG;
    if (cfg->dim < 8 || cfg->dim > siso::kMaxDim) return SISO_ERR_UNSUPPORTED;
    if (cfg->dim % 8 != 0) return SISO_ERR_UNSUPPORTED;
    if (cfg->dtype != SISO_F32 && cfg->dtype != SISO_BF16) return SISO_ERR_INVALID_ARG;
    if ((cfg->allocator.alloc == nullptr) != (cfg->allocator.free == nullptr)) return SISO_ERR_INVALID_ARG;
    if (cfg->decay != 0.0 && !(cfg->decay > 0.0)) return SISO_ERR_INVALID_ARG;
    int n_dev = 0;
    SISO_CUDA(cudaGetDeviceCount(&n_dev));
    if (cfg->device < 0 || cfg->device >= n_dev) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(cfg->device));
    cudaDeviceProp prop;
    SISO_CUDA(cudaGetDeviceProperties(&prop, cfg->device));
    if (prop.major != 10) {
        snprintf(g_last_error, sizeof(g_last_error), "device %d is sm_%d%d; this library holds sm_100a code only",
                 cfg->device, prop.major, prop.minor);
        return SISO_ERR_UNSUPPORTED;
    }
    siso_cache *c = new (std::nothrow) siso_cache();
    if (!c) return SISO_ERR_OOM;
    memset(static_cast<siso::Cache *>(c), 0, sizeof(siso::Cache));
    c->capacity = cfg->capacity;
    c->rows_alloc = (cfg->capacity + kRowPad - 1) / kRowPad * kRowPad;
    c->dim = cfg->dim;
    c->dtype = cfg->dtype;
    c->device = cfg->device;
    c->sm_count = prop.multiProcessorCount;
    c->decay = cfg->decay == 0.0 ? 1.1 : cfg->decay;
    if (cfg->allocator.alloc) { c->alloc = cfg->allocator; c->own_alloc = false; }
    else { c->alloc.alloc = default_alloc; c->alloc.free = default_free; c->alloc.ctx = nullptr; c->own_alloc = true; }
    c->lookup_path = SISO_PATH_AUTO;
    c->stream_fused = 1;
    c->low_dirty = true;
#ifdef SISO_CHECKED
    c->checked = 1;            // a library built with -DSISO_CHECKED checks by default
#endif
    c->merge_max_cand = 16 * c->capacity + (1ll << 20);

    const size_t rows = static_cast<size_t>(c->rows_alloc), D = static_cast<size_t>(c->dim);
    const size_t esz = c->dtype == SISO_F32 ? 4 : 2;
    cudaStream_t s0 = nullptr;
    bool ok = true;
    c->master = static_cast<float *>(cache_alloc(c, rows * D * 4, s0));
    ok = ok && c->master;
    if (c->dtype == SISO_F32) c->vecs = c->master;
    else { c->vecs = cache_alloc(c, rows * D * esz, s0); ok = ok && c->vecs; }
    c->size = static_cast<double *>(cache_alloc(c, rows * 8, s0)); ok = ok && c->size;
    c->access = static_cast<uint32_t *>(cache_alloc(c, rows * 4, s0)); ok = ok && c->access;
    c->last = static_cast<unsigned long long *>(cache_alloc(c, rows * 8, s0)); ok = ok && c->last;
    c->valid = static_cast<uint8_t *>(cache_alloc(c, rows, s0)); ok = ok && c->valid;
    c->counters = static_cast<long long *>(cache_alloc(c, sizeof(long long) * CNT_N, s0)); ok = ok && c->counters;
    c->status = static_cast<int *>(cache_alloc(c, 256, s0)); ok = ok && c->status;
    if (!ok) { siso_cache_destroy(c); return SISO_ERR_OOM; }
    cudaError_t e = cudaMemset(c->master, 0, rows * D * 4);
    if (e == cudaSuccess && c->dtype != SISO_F32) e = cudaMemset(c->vecs, 0, rows * D * esz);
    if (e == cudaSuccess) e = cudaMemset(c->size, 0, rows * 8);
    if (e == cudaSuccess) e = cudaMemset(c->access, 0, rows * 4);
    if (e == cudaSuccess) e = cudaMemset(c->last, 0, rows * 8);
    if (e == cudaSuccess) e = cudaMemset(c->valid, 0, rows);
    if (e == cudaSuccess) e = cudaMemset(c->counters, 0, sizeof(long long) * CNT_N);
    if (e == cudaSuccess) e = cudaMemset(c->status, 0, 256);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { siso_status_t st = check_cuda(e, "cache initialisation"); siso_cache_destroy(c); return st; }
    *out = c;
    return SISO_OK;
}

siso_status_t siso_cache_destroy(siso_cache_t *c) {
    if (!c) return SISO_ERR_INVALID_ARG;
    cudaSetDevice(c->device);
    cudaDeviceSynchronize();
    tensor_state_destroy(c);
    void *ptrs[] = {c->dtype == SISO_F32 ? nullptr : c->vecs, c->master, c->size, c->access, c->last, c->valid,
                    c->counters, c->status, c->ws, c->stage, c->swap_plan, c->split_hi, c->split_lo, c->low_list};
    for (void *p : ptrs)
        if (p) c->alloc.free(p, c->alloc.ctx);
    delete c;
    return SISO_OK;
}

siso_status_t siso_set_option(siso_cache_t *c, int32_t key, int64_t value) {
    if (!c) return SISO_ERR_INVALID_ARG;
    switch (key) {
        case SISO_OPT_LOOKUP_PATH:
            if (value < SISO_PATH_AUTO || value > SISO_PATH_STREAM) return SISO_ERR_INVALID_ARG;
            c->lookup_path = static_cast<int32_t>(value);
            return SISO_OK;
        case SISO_OPT_TENSOR_CTA_PAIR:
            if (value != 0 && value != 1) return SISO_ERR_INVALID_ARG;
            c->tensor_pair_mode = static_cast<int32_t>(value);
            return SISO_OK;
        case SISO_OPT_STREAM_FUSED:
            if (value != 0 && value != 1) return SISO_ERR_INVALID_ARG;
            c->stream_fused = static_cast<int32_t>(value);
            return SISO_OK;
        case SISO_OPT_SWEEP_FINALIZE:
            if (value != 0 && value != 1) return SISO_ERR_INVALID_ARG;
            c->sweep_finalize_separate = static_cast<int32_t>(value);
            return SISO_OK;
        case SISO_OPT_CHECKED:
            if (value != 0 && value != 1) return SISO_ERR_INVALID_ARG;
            c->checked = static_cast<int32_t>(value);
            return SISO_OK;
        case SISO_OPT_STREAM_LIST:
            if (value != 0 && value != 1) return SISO_ERR_INVALID_ARG;
            c->stream_list_off = static_cast<int32_t>(value);
            c->low_dirty = true;
            return SISO_OK;
        case SISO_OPT_MERGE_PATH:
            if (value != SISO_PATH_AUTO && value != SISO_PATH_SIMT && value != SISO_PATH_TENSOR) return SISO_ERR_INVALID_ARG;
            c->merge_path = static_cast<int32_t>(value);
            return SISO_OK;
        case SISO_OPT_MERGE_SWEEP_PARTS:
            if (value != 1 && value != 3) return SISO_ERR_INVALID_ARG;
            c->merge_sweep_parts = static_cast<int32_t>(value);
            return SISO_OK;
        case SISO_OPT_MERGE_MAX_CANDIDATES:
            if (value < 1 || value > (1ll << 31)) return SISO_ERR_INVALID_ARG;
            c->merge_max_cand = value;
            return SISO_OK;
    }
    return SISO_ERR_INVALID_ARG;
}

siso_status_t siso_insert(siso_cache_t *c, const void *d_vecs, const double *d_sizes, int64_t n, int32_t *d_slots_out,
                          void *stream) {
    if (!c || n < 0 || (n > 0 && !d_vecs)) return SISO_ERR_INVALID_ARG;
    if (n > 0 && !aligned16(d_vecs)) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    c->low_dirty = true;        // entries or their metadata change outside the streaming maintenance kernel
    SISO_TRY(checked_rows(c, d_vecs, n, nullptr, static_cast<cudaStream_t>(stream)));
    return launch_insert(c, d_vecs, d_sizes, nullptr, n, d_slots_out, static_cast<cudaStream_t>(stream));
}

// which kernel family serves a lookup of n_queries rows
static int resolve_lookup_path(const siso_cache_t *c, int64_t n_queries) {
    int path = c->lookup_path;
    if (path == SISO_PATH_AUTO) {
        // measured on B200: with a small batch padded to a whole query tile the tensor-core kernel streams the matrix at
        // 100-104 % of the measured copy bandwidth from one query up (2 GiB matrix; 86-92 % on 384 MiB); the streaming
        // kernel holds 96 % for 1-2 queries and falls off beyond, so bf16 caches always take the tensor-core kernel
        if (c->dtype == SISO_BF16) path = SISO_PATH_TENSOR;
        // fp32: the tensor-core sweep selects, an exact rescoring decides (k <= 4; otherwise the CUDA-core sweep)
        else path = n_queries <= 4 ? SISO_PATH_STREAM : (n_queries >= 32 ? SISO_PATH_TENSOR : SISO_PATH_SIMT);
    }
    return path;
}

siso_status_t siso_lookup(siso_cache_t *c, const void *d_queries, int64_t n_queries, const float *d_theta,
                          float theta_scalar, int32_t k, int32_t *d_idx, float *d_sim, uint8_t *d_hit, void *stream) {
    if (!c || n_queries < 0 || k < 1 || k > kMaxK) return SISO_ERR_INVALID_ARG;
    if (n_queries == 0) return SISO_OK;
    if (!d_queries || !d_idx || !d_sim || !d_hit || !aligned16(d_queries)) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    SISO_TRY(checked_rows(c, d_queries, n_queries, nullptr, s));
    SISO_TRY(checked_batch(c, d_theta, nullptr, nullptr, 1, n_queries, s));
    switch (resolve_lookup_path(c, n_queries)) {
        case SISO_PATH_STREAM: return launch_lookup_stream(c, d_queries, n_queries, d_theta, theta_scalar, k, d_idx, d_sim, d_hit, s);
        case SISO_PATH_TENSOR:
            if (c->dtype == SISO_BF16) return launch_lookup_tensor(c, d_queries, n_queries, d_theta, theta_scalar, k, d_idx, d_sim, d_hit, s);
            else {
                const siso_status_t st = launch_lookup_tensor_f32(c, d_queries, n_queries, d_theta, theta_scalar, k, d_idx, d_sim, d_hit, s);
                if (st != SISO_ERR_UNSUPPORTED) return st;
            }
            return launch_lookup_simt(c, d_queries, n_queries, d_theta, theta_scalar, k, d_idx, d_sim, d_hit, s);
        default: return launch_lookup_simt(c, d_queries, n_queries, d_theta, theta_scalar, k, d_idx, d_sim, d_hit, s);
    }
}

siso_status_t siso_lookup_host(siso_cache_t *c, const void *h_queries, int64_t n_queries, const float *h_theta,
                               float theta_scalar, int32_t k, int32_t *h_idx, float *h_sim, uint8_t *h_hit,
                               void *stream) {
    if (!c || n_queries < 0 || k < 1 || k > kMaxK) return SISO_ERR_INVALID_ARG;
    if (n_queries == 0) return SISO_OK;
    if (!h_queries || !h_idx || !h_sim || !h_hit) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t esz = c->dtype == SISO_F32 ? 4 : 2;
    const size_t qb = pad256(static_cast<size_t>(n_queries) * c->dim * esz), tb = pad256(sizeof(float) * n_queries);
    const size_t ib = pad256(sizeof(int32_t) * n_queries * k), sb = pad256(sizeof(float) * n_queries * k);
    const size_t hb = pad256(static_cast<size_t>(n_queries));
    const size_t need = qb + tb + ib + sb + hb;
    SISO_TRY(stage_reserve(c, need, s));
    char *p = static_cast<char *>(c->stage);
    void *dq = p; float *dt = reinterpret_cast<float *>(p + qb);
    int32_t *di = reinterpret_cast<int32_t *>(p + qb + tb);
    float *ds = reinterpret_cast<float *>(p + qb + tb + ib);
    uint8_t *dh = reinterpret_cast<uint8_t *>(p + qb + tb + ib + sb);
    SISO_CUDA(cudaMemcpyAsync(dq, h_queries, static_cast<size_t>(n_queries) * c->dim * esz, cudaMemcpyHostToDevice, s));
    if (h_theta) SISO_CUDA(cudaMemcpyAsync(dt, h_theta, sizeof(float) * n_queries, cudaMemcpyHostToDevice, s));
    SISO_TRY(siso_lookup(c, dq, n_queries, h_theta ? dt : nullptr, theta_scalar, k, di, ds, dh, stream));
    SISO_CUDA(cudaMemcpyAsync(h_idx, di, sizeof(int32_t) * n_queries * k, cudaMemcpyDeviceToHost, s));
    SISO_CUDA(cudaMemcpyAsync(h_sim, ds, sizeof(float) * n_queries * k, cudaMemcpyDeviceToHost, s));
    SISO_CUDA(cudaMemcpyAsync(h_hit, dh, static_cast<size_t>(n_queries), cudaMemcpyDeviceToHost, s));
    return SISO_OK;
}

siso_status_t siso_update(siso_cache_t *c, const void *d_queries, int64_t n_queries, const int32_t *d_idx,
                          int32_t idx_stride, const uint8_t *d_hit, void *stream) {
    if (!c || n_queries < 0 || idx_stride < 1) return SISO_ERR_INVALID_ARG;
    if (n_queries > 0 && (!d_queries || !d_idx || !d_hit || !aligned16(d_queries))) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    c->low_dirty = true;        // entries or their metadata change outside the streaming maintenance kernel
    SISO_TRY(checked_rows(c, d_queries, n_queries, nullptr, static_cast<cudaStream_t>(stream)));
    SISO_TRY(checked_batch(c, nullptr, d_hit, d_idx, idx_stride, n_queries, static_cast<cudaStream_t>(stream)));
    return launch_update(c, d_queries, n_queries, d_idx, idx_stride, d_hit, static_cast<cudaStream_t>(stream));
}

siso_status_t siso_merge(siso_cache_t *c, const void *d_repo, const double *d_repo_sizes, int64_t n_repo, float theta_c,
                         uint32_t flags, int32_t *d_merge_map, int64_t *h_n_merged, void *stream) {
    if (!c || (flags & ~SISO_MERGE_WEIGHTED_MEAN) || !(theta_c == theta_c)) return SISO_ERR_INVALID_ARG;
    if (n_repo < 0 || (n_repo > 0 && (!d_repo || !aligned16(d_repo))) || (n_repo == 0 && (d_repo || d_repo_sizes)))
        return SISO_ERR_INVALID_ARG;
    if (n_repo >= (1ll << 31)) return SISO_ERR_UNSUPPORTED;
    SISO_CUDA(cudaSetDevice(c->device));
    c->low_dirty = true;        // entries or their metadata change outside the streaming maintenance kernel
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    SISO_TRY(checked_rows(c, d_repo, n_repo, nullptr, s));
    long long *d_n = nullptr;
    if (h_n_merged) d_n = c->counters + CNT_SPARE;
    SISO_TRY(launch_merge(c, d_repo, d_repo_sizes, n_repo, theta_c, flags, d_merge_map, d_n, s));
    if (h_n_merged) {
        long long v = 0;
        SISO_CUDA(cudaMemcpyAsync(&v, d_n, sizeof(v), cudaMemcpyDeviceToHost, s));
        SISO_CUDA(cudaStreamSynchronize(s));
        *h_n_merged = v;
        return siso_sync_status(c, stream);
    }
    return SISO_OK;
}

siso_status_t siso_lookup_keys(siso_cache_t *c, const void *d_queries, int64_t n_queries, int32_t k, int64_t slot_offset,
                               uint64_t *d_keys, void *stream) {
    if (!c || n_queries < 0 || k < 1 || k > kMaxK || slot_offset < 0) return SISO_ERR_INVALID_ARG;
    if (slot_offset + c->capacity > 0xFFFFFFFFll) return SISO_ERR_UNSUPPORTED;        // global slots are 32-bit in a key
    if (n_queries == 0) return SISO_OK;
    if (!d_queries || !d_keys) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // idx / sim / hit of the shard go to the cache's staging buffer (the lookup itself uses the scratch buffer)
    const size_t ib = pad256(sizeof(int32_t) * n_queries * k), sb = pad256(sizeof(float) * n_queries * k);
    const size_t hb = pad256(static_cast<size_t>(n_queries));
    const size_t need = ib + sb + hb;
    SISO_TRY(stage_reserve(c, need, s));
    char *p = static_cast<char *>(c->stage);
    int32_t *di = reinterpret_cast<int32_t *>(p);
    float *ds = reinterpret_cast<float *>(p + ib);
    uint8_t *dh = reinterpret_cast<uint8_t *>(p + ib + sb);
    // threshold +inf: the shard records no hit; hit or miss is decided on the combined result
    SISO_TRY(siso_lookup(c, d_queries, n_queries, nullptr, INFINITY, k, di, ds, dh, stream));
    return launch_shard_pack(c, di, ds, n_queries * k, slot_offset, reinterpret_cast<unsigned long long *>(d_keys), s);
}

siso_status_t siso_combine_keys(const uint64_t *d_keys, int64_t n_queries, int32_t n_lists, int32_t k, const float *d_theta,
                                float theta_scalar, int64_t *d_idx, float *d_sim, uint8_t *d_hit, void *stream) {
    if (n_queries < 0 || n_lists < 1 || k < 1 || k > kMaxK) return SISO_ERR_INVALID_ARG;
    if (n_queries == 0) return SISO_OK;
    if (!d_keys || !d_idx || !d_sim || !d_hit) return SISO_ERR_INVALID_ARG;
    return launch_shard_combine(reinterpret_cast<const unsigned long long *>(d_keys), n_queries, n_lists, k, d_theta,
                                theta_scalar, reinterpret_cast<long long *>(d_idx), d_sim, d_hit, static_cast<cudaStream_t>(stream));
}

siso_status_t siso_route(const int64_t *d_idx, int64_t idx_stride, const uint8_t *d_hit, int64_t n, int64_t slot_lo,
                         int64_t slot_hi, int64_t miss_skip, int64_t miss_take, int32_t *d_idx_local, uint8_t *d_update_hit,
                         uint8_t *d_insert_hit, void *stream) {
    if (n < 0 || idx_stride < 1 || slot_lo < 0 || slot_hi < slot_lo || miss_skip < 0 || miss_take < 0) return SISO_ERR_INVALID_ARG;
    if (slot_hi - slot_lo > 0x7FFFFFFFll) return SISO_ERR_UNSUPPORTED;
    if (n == 0) return SISO_OK;
    if (!d_idx || !d_hit || !d_idx_local || !d_update_hit || !d_insert_hit) return SISO_ERR_INVALID_ARG;
    return launch_shard_route(reinterpret_cast<const long long *>(d_idx), idx_stride, d_hit, n, slot_lo, slot_hi, miss_skip,
                              miss_take, d_idx_local, d_update_hit, d_insert_hit, static_cast<cudaStream_t>(stream));
}

siso_status_t siso_evict_keys(siso_cache_t *c, int64_t n, int64_t slot_offset, uint64_t *d_keys, void *stream) {
    if (!c || n < 0 || slot_offset < 0) return SISO_ERR_INVALID_ARG;
    if (slot_offset + c->capacity > 0xFFFFFFFFll) return SISO_ERR_UNSUPPORTED;
    if (n == 0) return SISO_OK;
    if (!d_keys) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    return launch_evict_keys(c, n, slot_offset, reinterpret_cast<unsigned long long *>(d_keys), static_cast<cudaStream_t>(stream));
}

siso_status_t siso_select_evict(const uint64_t *d_keys, int32_t n_lists, int64_t n, int64_t n_take, int64_t *d_victims,
                                void *stream) {
    if (n_lists < 1 || n < 0 || n_take < 0) return SISO_ERR_INVALID_ARG;
    if (n_take == 0) return SISO_OK;
    if (!d_victims || (n > 0 && !d_keys)) return SISO_ERR_INVALID_ARG;
    return launch_evict_select(reinterpret_cast<const unsigned long long *>(d_keys), n_lists, n, n_take,
                               reinterpret_cast<long long *>(d_victims), static_cast<cudaStream_t>(stream));
}

siso_status_t siso_norm_deviation(siso_cache_t *c, double *h_max_dev, void *stream) {
    if (!c || !h_max_dev) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Scratch scr;
    SISO_TRY(scratch_reserve(c, 256, s, &scr));
    unsigned int *bits = scr.take<unsigned int>(1);
    SISO_CUDA(cudaMemsetAsync(bits, 0, sizeof(unsigned int), s));
    const unsigned blocks = static_cast<unsigned>(std::min<int64_t>((c->capacity + 7) / 8, 8ll * c->sm_count));
    if (c->dtype == SISO_F32)
        norm_deviation_kernel<float><<<blocks, 256, 0, s>>>(static_cast<const float *>(c->vecs), c->valid, c->capacity, c->dim, bits);
    else
        norm_deviation_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(c->vecs), c->valid, c->capacity, c->dim, bits);
    SISO_LAUNCHED(c);
    unsigned int h = 0;
    SISO_CUDA(cudaMemcpyAsync(&h, bits, sizeof(h), cudaMemcpyDeviceToHost, s));
    SISO_CUDA(cudaStreamSynchronize(s));
    float f;
    memcpy(&f, &h, sizeof(f));
    *h_max_dev = static_cast<double>(f);
    return SISO_OK;
}

siso_status_t siso_free_slots(siso_cache_t *c, int64_t *d_free, void *stream) {
    if (!c || !d_free) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    return launch_free_slots(c, reinterpret_cast<long long *>(d_free), static_cast<cudaStream_t>(stream));
}

siso_status_t siso_shard_plan(const uint8_t *d_hit, int64_t n, const int64_t *d_free_all, int32_t world, int32_t rank,
                              int64_t *d_plan, void *stream) {
    if (n < 0 || (n > 0 && !d_hit) || !d_free_all || world < 1 || rank < 0 || rank >= world || !d_plan) return SISO_ERR_INVALID_ARG;
    return launch_shard_plan(d_hit, n, reinterpret_cast<const long long *>(d_free_all), world, rank,
                             reinterpret_cast<long long *>(d_plan), static_cast<cudaStream_t>(stream));
}

siso_status_t siso_route_planned(const int64_t *d_idx, int64_t idx_stride, const uint8_t *d_hit, int64_t n, int64_t slot_lo,
                                 int64_t slot_hi, const int64_t *d_plan, int32_t *d_idx_local, uint8_t *d_update_hit,
                                 uint8_t *d_insert_hit, void *stream) {
    if (n < 0 || idx_stride < 1 || slot_lo < 0 || slot_hi < slot_lo || !d_plan) return SISO_ERR_INVALID_ARG;
    if (slot_hi - slot_lo > 0x7FFFFFFFll) return SISO_ERR_UNSUPPORTED;
    if (n == 0) return SISO_OK;
    if (!d_idx || !d_hit || !d_idx_local || !d_update_hit || !d_insert_hit) return SISO_ERR_INVALID_ARG;
    return launch_shard_route(reinterpret_cast<const long long *>(d_idx), idx_stride, d_hit, n, slot_lo, slot_hi, 0, 0, d_idx_local,
                              d_update_hit, d_insert_hit, static_cast<cudaStream_t>(stream), reinterpret_cast<const long long *>(d_plan));
}

siso_status_t siso_select_evict_planned(const uint64_t *d_keys, int32_t n_lists, int64_t n, const int64_t *d_plan,
                                        int64_t *d_victims, void *stream) {
    if (n_lists < 1 || n < 0 || !d_plan) return SISO_ERR_INVALID_ARG;
    if (n == 0) return SISO_OK;
    if (!d_victims || !d_keys) return SISO_ERR_INVALID_ARG;
    return launch_evict_select(reinterpret_cast<const unsigned long long *>(d_keys), n_lists, n, n, reinterpret_cast<long long *>(d_victims),
                               static_cast<cudaStream_t>(stream), reinterpret_cast<const long long *>(d_plan));
}

siso_status_t siso_evict_slots(siso_cache_t *c, const int64_t *d_victims, int64_t n, int64_t slot_offset, uint32_t flags,
                               void *stream) {
    if (!c || n < 0 || slot_offset < 0 || (n > 0 && !d_victims) || (flags & ~SISO_EVICT_DECAY)) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    c->low_dirty = true;        // entries or their metadata change outside the streaming maintenance kernel
    return launch_evict_slots(c, reinterpret_cast<const long long *>(d_victims), n, slot_offset, flags,
                              static_cast<cudaStream_t>(stream));
}

siso_status_t siso_cache_copy(siso_cache_t *dst, siso_cache_t *src, void *stream) {
    if (!dst || !src || dst == src) return SISO_ERR_INVALID_ARG;
    if (dst->dim != src->dim || dst->dtype != src->dtype || dst->device != src->device) return SISO_ERR_INVALID_ARG;
    if (dst->capacity < src->capacity) return SISO_ERR_CAPACITY;
    SISO_CUDA(cudaSetDevice(dst->device));
    dst->low_dirty = true;
    return launch_cache_copy(dst, src, static_cast<cudaStream_t>(stream));
}

siso_status_t siso_update_centroids(siso_cache_t *cur, siso_cache_t *c_new, int64_t first_slot, int64_t n_slots, void *stream) {
    if (!cur || !c_new || cur == c_new || first_slot < 0 || n_slots < 0) return SISO_ERR_INVALID_ARG;
    if (cur->dim != c_new->dim || cur->dtype != c_new->dtype || cur->device != c_new->device) return SISO_ERR_INVALID_ARG;
    if (first_slot > cur->capacity) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(cur->device));
    cur->low_dirty = true;
    return launch_update_centroids(cur, c_new, first_slot, n_slots, static_cast<cudaStream_t>(stream));
}

siso_status_t siso_cluster(siso_cache_t *c, const void *d_vecs, int64_t n, float theta_c, int32_t *d_label, int32_t *d_centres,
                           double *d_sizes, void *d_centroids, int64_t *h_n_clusters, void *stream) {
    if (!c || n < 0 || !(theta_c == theta_c)) return SISO_ERR_INVALID_ARG;
    if (n == 0) {
        if (h_n_clusters) *h_n_clusters = 0;
        return SISO_OK;
    }
    if (!d_vecs || !aligned16(d_vecs)) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    long long *d_n = h_n_clusters ? c->counters + CNT_SPARE : nullptr;
    SISO_TRY(launch_cluster(c, d_vecs, n, theta_c, d_label, d_centres, d_sizes, d_centroids, d_n, s));
    if (h_n_clusters) {
        long long v = 0;
        SISO_CUDA(cudaMemcpyAsync(&v, d_n, sizeof(v), cudaMemcpyDeviceToHost, s));
        SISO_CUDA(cudaStreamSynchronize(s));
        *h_n_clusters = v;
        return siso_sync_status(c, stream);
    }
    return SISO_OK;
}

siso_status_t siso_evict(siso_cache_t *c, int64_t n_evict, uint32_t flags, int32_t *d_victims, void *stream) {
    if (!c || n_evict < 0 || (flags & ~SISO_EVICT_DECAY)) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    c->low_dirty = true;        // entries or their metadata change outside the streaming maintenance kernel
    return launch_evict(c, n_evict, nullptr, 0, flags, d_victims, n_evict, static_cast<cudaStream_t>(stream));
}

siso_status_t siso_make_room(siso_cache_t *c, const uint8_t *d_hit, int64_t n, uint32_t flags, int32_t *d_victims,
                             void *stream) {
    if (!c || n < 0 || (n > 0 && !d_hit) || (flags & ~SISO_EVICT_DECAY)) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    c->low_dirty = true;        // entries or their metadata change outside the streaming maintenance kernel
    return launch_evict(c, -1, d_hit, n, flags, d_victims, n, static_cast<cudaStream_t>(stream));
}

siso_status_t siso_insert_misses(siso_cache_t *c, const void *d_queries, int64_t n, const uint8_t *d_hit,
                                 int32_t *d_slots_out, void *stream) {
    if (!c || n < 0 || (n > 0 && (!d_queries || !d_hit || !aligned16(d_queries)))) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    c->low_dirty = true;        // entries or their metadata change outside the streaming maintenance kernel
    SISO_TRY(checked_rows(c, d_queries, n, d_hit, static_cast<cudaStream_t>(stream)));
    SISO_TRY(checked_batch(c, nullptr, d_hit, nullptr, 1, n, static_cast<cudaStream_t>(stream)));
    return launch_insert(c, d_queries, nullptr, d_hit, n, d_slots_out, static_cast<cudaStream_t>(stream));
}

siso_status_t siso_stream_step(siso_cache_t *c, const void *d_queries, int64_t n, const float *d_theta,
                               float theta_scalar, int32_t *d_idx, float *d_sim, uint8_t *d_hit, int32_t *d_victims,
                               int32_t *d_slots_out, void *stream) {
    if (!c || n < 0) return SISO_ERR_INVALID_ARG;
    if (n == 0) return SISO_OK;
    if (!d_queries || !d_idx || !d_sim || !d_hit || !aligned16(d_queries)) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (c->checked && c->stream_fused && c->dtype == SISO_BF16) {      // (the other branches go through siso_lookup, which checks)
        SISO_TRY(checked_rows(c, d_queries, n, nullptr, s));
        SISO_TRY(checked_batch(c, d_theta, nullptr, nullptr, 1, n, s));
    }
    // small batches: update, make-room and insertion in one cooperative launch, which also finishes the lookup
    // (best key over the splits, threshold test) when the tensor-core kernel produced it
    if (c->stream_fused && stream_maint_supported(c, n)) {
        if (c->dtype == SISO_BF16 && resolve_lookup_path(c, n) == SISO_PATH_TENSOR) {
            DeferredTop1 top1;
            void *tail = nullptr;
            SISO_TRY(launch_lookup_tensor(c, d_queries, n, d_theta, theta_scalar, 1, d_idx, d_sim, d_hit, s, &top1,
                                          stream_maint_scratch_bytes(c, n), &tail));
            return launch_stream_maint(c, d_queries, n, d_idx, d_hit, d_victims, d_slots_out, &top1, tail, s);
        }
        SISO_TRY(siso_lookup(c, d_queries, n, d_theta, theta_scalar, 1, d_idx, d_sim, d_hit, stream));
        return launch_stream_maint(c, d_queries, n, d_idx, d_hit, d_victims, d_slots_out, nullptr, nullptr, s);
    }
    SISO_TRY(siso_lookup(c, d_queries, n, d_theta, theta_scalar, 1, d_idx, d_sim, d_hit, stream));
    SISO_TRY(siso_update(c, d_queries, n, d_idx, 1, d_hit, stream));
    SISO_TRY(siso_make_room(c, d_hit, n, 0, d_victims, stream));
    return siso_insert_misses(c, d_queries, n, d_hit, d_slots_out, stream);
}

siso_status_t siso_export(siso_cache_t *c, void *d_vecs, float *d_master, double *d_sizes, uint32_t *d_access,
                          uint64_t *d_last, uint8_t *d_valid, void *stream) {
    if (!c) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t n = static_cast<size_t>(c->capacity), D = static_cast<size_t>(c->dim);
    const size_t esz = c->dtype == SISO_F32 ? 4 : 2;
    if (d_vecs) SISO_CUDA(cudaMemcpyAsync(d_vecs, c->vecs, n * D * esz, cudaMemcpyDeviceToDevice, s));
    if (d_master) SISO_CUDA(cudaMemcpyAsync(d_master, c->master, n * D * 4, cudaMemcpyDeviceToDevice, s));
    if (d_sizes) SISO_CUDA(cudaMemcpyAsync(d_sizes, c->size, n * 8, cudaMemcpyDeviceToDevice, s));
    if (d_access) SISO_CUDA(cudaMemcpyAsync(d_access, c->access, n * 4, cudaMemcpyDeviceToDevice, s));
    if (d_last) SISO_CUDA(cudaMemcpyAsync(d_last, c->last, n * 8, cudaMemcpyDeviceToDevice, s));
    if (d_valid) SISO_CUDA(cudaMemcpyAsync(d_valid, c->valid, n, cudaMemcpyDeviceToDevice, s));
    return SISO_OK;
}

siso_status_t siso_import(siso_cache_t *c, const float *d_master, const double *d_sizes, const uint32_t *d_access,
                          const uint64_t *d_last, const uint8_t *d_valid, uint64_t clock, void *stream) {
    if (!c || !d_master || !d_sizes || !d_access || !d_last || !d_valid) return SISO_ERR_INVALID_ARG;
    c->vec_epoch += 1;          // the vectors may change: derived copies (the split-bf16 parts) are stale
    SISO_CUDA(cudaSetDevice(c->device));
    c->low_dirty = true;        // entries or their metadata change outside the streaming maintenance kernel
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t n = static_cast<size_t>(c->capacity), D = static_cast<size_t>(c->dim);
    SISO_CUDA(cudaMemcpyAsync(c->master, d_master, n * D * 4, cudaMemcpyDeviceToDevice, s));
    SISO_CUDA(cudaMemcpyAsync(c->size, d_sizes, n * 8, cudaMemcpyDeviceToDevice, s));
    SISO_CUDA(cudaMemcpyAsync(c->access, d_access, n * 4, cudaMemcpyDeviceToDevice, s));
    SISO_CUDA(cudaMemcpyAsync(c->last, d_last, n * 8, cudaMemcpyDeviceToDevice, s));
    SISO_CUDA(cudaMemcpyAsync(c->valid, d_valid, n, cudaMemcpyDeviceToDevice, s));
    normalise_valid_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, s>>>(c->valid, static_cast<long long>(n));
    SISO_LAUNCHED(c);
    if (c->dtype == SISO_BF16) {
        const long long total = static_cast<long long>(n * D);
        bf16_from_master_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, s>>>(
            c->master, static_cast<__nv_bfloat16 *>(c->vecs), total);
        SISO_LAUNCHED(c);
    }
    import_counters_kernel<<<1, 1024, 0, s>>>(c->valid, c->capacity, c->counters, clock);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

siso_status_t siso_get_stats(siso_cache_t *c, int64_t *h_counts, void *stream) {
    if (!c || !h_counts) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    long long tmp[CNT_N];
    SISO_CUDA(cudaMemcpyAsync(tmp, c->counters, sizeof(tmp), cudaMemcpyDeviceToHost, s));
    SISO_CUDA(cudaStreamSynchronize(s));
    for (int i = 0; i < 8; ++i) h_counts[i] = i < CNT_SPARE ? tmp[i] : 0;
    h_counts[7] = tmp[CNT_RESCANS];
    return SISO_OK;
}

siso_status_t siso_sync_status(siso_cache_t *c, void *stream) {
    if (!c) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int st = 0;
    SISO_CUDA(cudaMemcpyAsync(&st, c->status, sizeof(int), cudaMemcpyDeviceToHost, s));
    SISO_CUDA(cudaStreamSynchronize(s));
    if (st != 0) SISO_CUDA(cudaMemsetAsync(c->status, 0, sizeof(int), s));
    return static_cast<siso_status_t>(st);
}

int64_t siso_launch_count(const siso_cache_t *c) { return c ? c->launches : 0; }

}  // extern "C"
