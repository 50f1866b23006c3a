// Internal declarations shared by the kernels of libsiso (never installed; the public
// interface is include/siso.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "../../include/siso.h"

namespace siso {

constexpr int kRowPad = 256;        // vector arrays are allocated in multiples of this many rows, zero-filled
constexpr int kMaxDim = 4096;
constexpr int kMaxK = 8;
constexpr uint32_t kNoSlot = 0xFFFFFFFFu;

// device counters, int64 each
enum Counter { CNT_OCCUPANCY = 0, CNT_LOOKUPS, CNT_HITS, CNT_INSERTS, CNT_EVICTIONS, CNT_MERGES, CNT_CLOCK, CNT_SPARE, CNT_SYNC, CNT_RESCANS, CNT_N };

struct Cache {
    int64_t capacity;
    int64_t rows_alloc;    // capacity rounded up to kRowPad
    int32_t dim;
    int32_t dtype;
    int32_t device;
    int32_t sm_count;
    double decay;
    siso_allocator_t alloc;
    bool own_alloc;

    void *vecs;            // [rows_alloc, dim] lookup copy in the cache dtype (for fp32 caches this IS the master)
    float *master;         // [rows_alloc, dim] fp32 master
    double *size;          // [rows_alloc] cluster_size
    uint32_t *access;      // [rows_alloc] access_count
    unsigned long long *last;  // [rows_alloc] last_access
    uint8_t *valid;        // [rows_alloc]
    long long *counters;   // [CNT_N]
    int *status;           // device status word (first error wins)

    // scratch, grown on demand
    void *ws;
    size_t ws_bytes;
    // staging for the host-buffer lookup
    void *stage;
    size_t stage_bytes;

    int32_t lookup_path;
    int32_t stream_fused;       // 1: siso_stream_step uses the fused maintenance kernel for small batches
    int32_t tensor_pair_mode;   // 0: CTA pairs when the batch spans two query tiles; 1: single-CTA kernel only
    int64_t merge_max_cand;
    int64_t launches;
    void *tensor_state;    // owned by lookup_tensor.cu
    // large-shared-memory opt-in is a per-device function attribute: remembered per cache, not per process
    bool simt_attr_set[2][3];   // [dtype][k class] of lookup_simt_kernel
    bool merge_attr_set;
    bool split_attr_set;
    // fp32 caches: the bf16 parts (hi, lo) of the vectors for the tensor-core lookup, valid while split_epoch == vec_epoch
    void *split_hi, *split_lo;
    unsigned long long vec_epoch, split_epoch;
    bool merge_tensor_attr_set;
    int merge_resolve_grid;     // CTAs of the grid-wide merge resolution (0: not yet asked, -1: unavailable)
    int32_t merge_path;         // SISO_PATH_AUTO, SISO_PATH_SIMT or SISO_PATH_TENSOR for the pairwise sweep of siso_merge
    int32_t merge_sweep_parts;  // 3: the tensor-core sweep of fp32 rows multiplies three bf16 parts; otherwise one part as a filter
    void *swap_plan;            // UpdateCentroids: slot of the d-th live entry, when this cache serves as C_new
    int maint_grid;             // CTAs of the fused streaming maintenance kernel (0: not yet asked, -1: unavailable)
    int32_t sweep_finalize_separate;   // 1: never finish a top-1 lookup inside the sweep kernel
    int32_t checked;                   // 1: inputs are verified on the device (SISO_OPT_CHECKED)
    int32_t stream_list_off;           // 1: the streaming maintenance kernel never uses the list below
    void *low_list;             // eviction-order list that the streaming maintenance kernel keeps across batches
    bool low_dirty;             // an entry point other than that kernel has changed entries or their metadata since
};

// ---- scratch bump allocator -------------------------------------------------
struct Scratch {
    char *base;
    size_t off, cap;
    template <typename T> T *take(size_t n) {
        size_t bytes = (n * sizeof(T) + 255) & ~size_t(255);
        T *p = reinterpret_cast<T *>(base + off);
        off += bytes;
        return p;
    }
};
inline size_t pad256(size_t b) { return (b + 255) & ~size_t(255); }
siso_status_t scratch_reserve(Cache *c, size_t bytes, cudaStream_t s, Scratch *out);
siso_status_t stage_reserve(Cache *c, size_t bytes, cudaStream_t s);   // c->stage of at least `bytes`
// memory that lives as long as the cache, set to zero; NULL if the allocator fails
void *cache_alloc_zeroed(Cache *c, size_t bytes);
siso_status_t check_cuda(cudaError_t e, const char *what);
#define SISO_CUDA(expr)                                                  \
    do {                                                                 \
        siso_status_t st__ = ::siso::check_cuda((expr), #expr);          \
        if (st__ != SISO_OK) return st__;                                \
    } while (0)
#define SISO_TRY(expr)                                                   \
    do {                                                                 \
        siso_status_t st__ = (expr);                                     \
        if (st__ != SISO_OK) return st__;                                \
    } while (0)
#define SISO_LAUNCHED(c)                                                 \
    do {                                                                 \
        (c)->launches += 1;                                              \
        SISO_CUDA(cudaGetLastError());                                   \
    } while (0)

// ---- launchers implemented in the .cu files -----------------------------------
siso_status_t launch_lookup_simt(Cache *c, const void *q, int64_t B, const float *theta, float theta_s, int k,
                                 int32_t *idx, float *sim, uint8_t *hit, cudaStream_t s);
siso_status_t launch_lookup_stream(Cache *c, const void *q, int64_t B, const float *theta, float theta_s, int k,
                                   int32_t *idx, float *sim, uint8_t *hit, cudaStream_t s);
// A top-1 lookup whose last step (best key over the splits, threshold test) is left to a later kernel.
struct DeferredTop1 {
    const unsigned long long *partial;     // [B, splits] packed (similarity, slot) keys, 0 = no entry
    int splits;
    const float *theta;
    float theta_s;
    float *sim;                            // [B] out
};
// With `defer` (k must be 1) the finalisation kernel is not launched; *defer receives the partial results and
// *tail points to `tail_bytes` of the cache's scratch that stay untouched by the lookup.
siso_status_t launch_lookup_tensor(Cache *c, const void *q, int64_t B, const float *theta, float theta_s, int k,
                                   int32_t *idx, float *sim, uint8_t *hit, cudaStream_t s,
                                   DeferredTop1 *defer = nullptr, size_t tail_bytes = 0, void **tail = nullptr);
void tensor_state_destroy(Cache *c);
// fp32 caches on the tensor cores (split-bf16 selection, exact rescoring); SISO_ERR_UNSUPPORTED for bf16 caches or k > 4
siso_status_t launch_lookup_tensor_f32(Cache *c, const void *q, int64_t B, const float *theta, float theta_s, int k,
                                       int32_t *idx, float *sim, uint8_t *hit, cudaStream_t s);
siso_status_t launch_split_bf16(Cache *c, const float *x, __nv_bfloat16 *hi, __nv_bfloat16 *lo, long long n4, cudaStream_t s);
siso_status_t launch_topk_finalize(Cache *c, const unsigned long long *partial, int64_t B, int splits, int kmax, int k,
                                   const float *theta, float theta_s, int32_t *idx, float *sim, uint8_t *hit,
                                   cudaStream_t s);
siso_status_t launch_update(Cache *c, const void *q, int64_t B, const int32_t *idx, int idx_stride, const uint8_t *hit,
                            cudaStream_t s);
siso_status_t launch_merge(Cache *c, const void *repo, const double *repo_sizes, int64_t n_repo, float theta_c,
                           uint32_t flags, int32_t *merge_map, long long *d_n_merged, cudaStream_t s);
siso_status_t launch_merge_resolve_global(Cache *c, const void *cand, int64_t n_cand, const uint8_t *valid, int64_t N,
                                          int32_t *merge_map, long long *d_n_merged, cudaStream_t s);
siso_status_t launch_pair_sweep_block(Cache *c, int64_t own_offset, const void *d_peer_rows, const uint8_t *d_peer_valid, int64_t n_peer,
                                      int64_t peer_offset, float theta_c, int32_t *d_cand, int64_t max_cand, int64_t *d_n_cand,
                                      bool lookup_copies, cudaStream_t s);
size_t merge_tensor_scratch_bytes(const Cache *c);
size_t pair_sweep_tensor_scratch_bytes(int64_t n, int64_t rows, int dim);
siso_status_t launch_pair_sweep_tensor(Cache *c, Scratch *scr, const float *X, int64_t N, int64_t rows, const uint8_t *valid,
                                       const uint8_t *seed, float theta_c, void *ctl, void *cand, size_t max_cand,
                                       uint32_t *row_count, cudaStream_t s, const void *rows_bf16, int64_t cross_rows = 0);
siso_status_t launch_merge_resolve(Cache *c, void *ctl, int64_t N, const uint8_t *valid, const uint8_t *seed,
                                   const uint32_t *row_off, const uint32_t *row_count, const int32_t *csr_j,
                                   const float *csr_sim, uint8_t *state, int32_t *target, unsigned int *undecided,
                                   cudaStream_t s);
siso_status_t launch_shard_pack(Cache *c, const int32_t *idx, const float *sim, int64_t n, int64_t slot_offset,
                                unsigned long long *keys, cudaStream_t s);
siso_status_t launch_shard_combine(const unsigned long long *keys, int64_t n, int n_lists, int k, const float *theta,
                                   float theta_s, long long *idx, float *sim, uint8_t *hit, cudaStream_t s);
siso_status_t launch_cache_copy(Cache *dst, const Cache *src, cudaStream_t s);
siso_status_t launch_update_centroids(Cache *cur, Cache *c_new, int64_t first, int64_t n, cudaStream_t s);
siso_status_t launch_cluster(Cache *c, const void *vecs, int64_t n, float theta_c, int32_t *label, int32_t *centres,
                             double *sizes, void *centroids, long long *d_n_clusters, cudaStream_t s);
siso_status_t launch_merge_sweep_tensor(Cache *c, Scratch *scr, const uint8_t *seed, float theta_c, void *ctl, void *cand,
                                        size_t max_cand, uint32_t *row_count, cudaStream_t s);
siso_status_t launch_evict(Cache *c, int64_t n_evict, const uint8_t *hit, int64_t n_hit, uint32_t flags,
                           int32_t *victims, int64_t n_victims_out, cudaStream_t s);
siso_status_t launch_insert(Cache *c, const void *vecs, const double *sizes, const uint8_t *hit, int64_t n,
                            int32_t *slots_out, cudaStream_t s);
siso_status_t launch_evict_keys(Cache *c, int64_t n, int64_t slot_offset, unsigned long long *keys_out, cudaStream_t s);
siso_status_t launch_evict_select(const unsigned long long *keys, int n_lists, int64_t n, int64_t n_take, long long *victims,
                                  cudaStream_t s, const long long *plan = nullptr);
siso_status_t launch_shard_plan(const uint8_t *hit, int64_t n, const long long *free_all, int world, int rank, long long *plan,
                                cudaStream_t s);
siso_status_t launch_free_slots(Cache *c, long long *out, cudaStream_t s);
siso_status_t launch_evict_slots(Cache *c, const long long *victims, int64_t n, int64_t slot_offset, uint32_t flags, cudaStream_t s);
siso_status_t launch_shard_route(const long long *idx, long long idx_stride, const uint8_t *hit, int64_t n, int64_t slot_lo,
                                 int64_t slot_hi, int64_t skip, int64_t take, int32_t *idx_local, uint8_t *upd_hit,
                                 uint8_t *ins_hit, cudaStream_t s, const long long *plan = nullptr);
siso_status_t launch_sort_pairs(Cache *c, Scratch *scr, uint32_t *keys, uint32_t *vals, uint32_t *keys_tmp,
                                uint32_t *vals_tmp, int64_t n, int key_bits, uint32_t **keys_out, uint32_t **vals_out,
                                cudaStream_t s);
size_t sort_pairs_scratch_bytes(int64_t n);
bool stream_maint_supported(Cache *c, int64_t B);
size_t stream_maint_scratch_bytes(const Cache *c, int64_t B);
siso_status_t launch_stream_maint(Cache *c, const void *q, int64_t B, int32_t *idx, uint8_t *hit, int32_t *victims,
                                  int32_t *slots_out, const DeferredTop1 *deferred, void *scratch_tail, cudaStream_t s);
siso_status_t launch_exclusive_scan_u32(Cache *c, uint32_t *a, int64_t n, cudaStream_t s);

#ifdef __CUDACC__
// ---- device helpers ------------------------------------------------------------
// Order-preserving map fp32 -> u32, and the packed (similarity, slot) key whose maximum is the
// best match with ties going to the lower slot.  Key 0 means "no entry".
__device__ __forceinline__ uint32_t f32_sortable(float f) {
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float sortable_f32(uint32_t s) {
    uint32_t u = (s & 0x80000000u) ? (s & 0x7FFFFFFFu) : ~s;
    return __uint_as_float(u);
}
__device__ __forceinline__ unsigned long long pack_key(float sim, uint32_t slot) {
    return (static_cast<unsigned long long>(f32_sortable(sim)) << 32) | (0xFFFFFFFFu - slot);
}
__device__ __forceinline__ float key_sim(unsigned long long k) { return sortable_f32(static_cast<uint32_t>(k >> 32)); }
__device__ __forceinline__ int32_t key_slot(unsigned long long k) {
    return static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(k));
}

// Sorted (descending) list of K packed keys in registers; insert keeps the K largest.
template <int K> struct KeyList {
    unsigned long long k[K];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int i = 0; i < K; ++i) k[i] = 0ull;
    }
    __device__ __forceinline__ void insert(unsigned long long v) {
        if (v > k[K - 1]) {
            k[K - 1] = v;
#pragma unroll
            for (int i = K - 1; i > 0; --i) {
                if (k[i] > k[i - 1]) {
                    unsigned long long t = k[i];
                    k[i] = k[i - 1];
                    k[i - 1] = t;
                }
            }
        }
    }
};

// Per-thread running top-K over a stream of (similarity, slot) pairs that arrive in ASCENDING slot
// order: a later pair with an equal similarity never displaces an earlier one, so a strict float
// comparison implements "ties to the lower slot".
template <int K> struct TopK {
    float s[K];
    int32_t i[K];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int j = 0; j < K; ++j) { s[j] = -INFINITY; i[j] = -1; }
    }
    __device__ __forceinline__ void push(float v, int32_t slot) {
        if (v > s[K - 1]) {          // empty places hold -inf, so any finite similarity enters
            s[K - 1] = v;
            i[K - 1] = slot;
#pragma unroll
            for (int j = K - 1; j > 0; --j) {
                if (s[j] > s[j - 1]) {
                    float ts = s[j]; s[j] = s[j - 1]; s[j - 1] = ts;
                    int32_t ti = i[j]; i[j] = i[j - 1]; i[j - 1] = ti;
                }
            }
        }
    }
    __device__ __forceinline__ unsigned long long key(int j) const { return i[j] < 0 ? 0ull : pack_key(s[j], (uint32_t)i[j]); }
};

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t b) { return __uint_as_float(b << 16); }

__device__ __forceinline__ void set_status(int *status, int code) { atomicCAS(status, 0, code); }
#endif  // __CUDACC__

}  // namespace siso
