/*
 * siso.h - C ABI of the B200 semantic-cache hot path (SISO, arXiv 2508.18736).
 *
 * A cache is a slot-indexed array of unit-norm centroid vectors with, per slot, the
 * paper's two replacement fields cluster_size and access_count (Sec. 4.2, the cache manager) plus a last_access stamp and a valid flag.  Every entry
 * point below runs hand-written sm_100a kernels; there is no CPU path.
 *
 * Conventions
 *   - d_* arguments are DEVICE pointers owned by the caller; the library never frees
 *     them and never keeps them after the call returns.  h_* are HOST pointers.
 *   - stream is a cudaStream_t passed as void*.  Calls are asynchronous on it unless
 *     stated otherwise; calls on one handle must be issued on one stream (or be
 *     ordered by the caller).  A handle is not thread-safe; handles are independent.
 *   - Argument errors are detected on the host, return at once and modify nothing.
 *     Conditions only the device can see (capacity exhausted, candidate buffer
 *     overflow, a bounded wait that ran out) are written to a device status word that
 *     siso_sync_status() returns; the call that hit them modifies nothing.
 *   - Vectors are row-major [rows, dim], fp32 or bfloat16 (raw 16-bit patterns), and
 *     MUST be L2-normalised by the caller: similarity = dot product = cosine.
 *     dim % 8 == 0 and 16-byte aligned base pointers are required (else
 *     SISO_ERR_UNSUPPORTED / SISO_ERR_INVALID_ARG).
 *   - Ties in similarity go to the lower slot; the hit and merge tests are strict
 *     ('>' as printed in Algorithm 1, MergeCentroids).
 *   - access_count "infinity" (Algorithm 1, else-branch of MergeCentroids) is
 *     0xFFFFFFFF; additions saturate there.
 */
#ifndef SISO_H_
#define SISO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct siso_cache siso_cache_t; /* opaque host-side handle */

typedef enum {
    SISO_OK = 0,
    SISO_ERR_INVALID_ARG = 1,
    SISO_ERR_UNSUPPORTED = 2,
    SISO_ERR_OOM = 3,
    SISO_ERR_CAPACITY = 4, /* insert: fewer free slots than rows to insert; nothing modified */
    SISO_ERR_OVERFLOW = 5, /* merge: candidate buffer too small; nothing modified           */
    SISO_ERR_TIMEOUT = 6,  /* a bounded device-side wait gave up                            */
    SISO_ERR_CUDA = 7
} siso_status_t;

typedef enum { SISO_F32 = 0, SISO_BF16 = 1 } siso_dtype_t;

#define SISO_ACCESS_INF 0xFFFFFFFFu

/* merge flags */
#define SISO_MERGE_SIZES_ONLY 0u    /* Algorithm 1 as printed: only cluster_size moves             */
#define SISO_MERGE_WEIGHTED_MEAN 1u /* survivors become the cluster_size-weighted mean, renormalised */
/* evict flags */
#define SISO_EVICT_DECAY 1u /* afterwards cluster_size /= decay, access_count = 0 (Algorithm 1, FilteringCentroids) */

/* lookup kernel selection (siso_set_option key SISO_OPT_LOOKUP_PATH) */
#define SISO_OPT_LOOKUP_PATH 1
#define SISO_OPT_MERGE_MAX_CANDIDATES 2 /* capacity of the merge candidate buffer, in pairs */
#define SISO_OPT_STREAM_FUSED 4         /* 1 (default): siso_stream_step fuses update, make-room and insertion of batches
                                           of at most 1024 rows into one cooperative launch; 0: separate kernels */
#define SISO_OPT_MERGE_PATH 5           /* pairwise sweep of siso_merge: SISO_PATH_AUTO (default: tensor cores from 4096
                                           entries), SISO_PATH_SIMT or SISO_PATH_TENSOR; the results are the same */
#define SISO_OPT_SWEEP_FINALIZE 6       /* 0 (default): a top-1 tensor-core lookup of at most 256 queries picks its results inside the
                                         * sweep kernel; 1: always by a separate finalisation launch */
#define SISO_OPT_STREAM_LIST 7          /* 0 (default): on a full cache the fused streaming step takes its victims from an
                                         * eviction-order list kept across batches (no grid-wide barrier); 1: never */
#define SISO_OPT_MERGE_SWEEP_PARTS 8    /* tensor-core pairwise sweep over fp32 rows (MergeCentroids, clustering).  1 (default): the rows
                                         * rounded to bf16 are multiplied once, as a filter whose margin (8.1e-3 + 1e-8 dim)
                                         * bounds the rounding for rows of norm <= 1.01, and every pair above the filter is then
                                         * decided by its exact fp32 similarity; 3: three products of bf16 parts reproduce the
                                         * fp32 product to 1e-4 before the same exact decision.  The results are the same. */
#define SISO_OPT_CHECKED 9              /* 1: checked mode.  What the library otherwise takes on trust is verified on the device before
                                         * the call's own kernels run: query, insert and repository rows must be unit vectors
                                         * (| |x| - 1 | < 1e-2) with finite elements, thresholds must be numbers, hit flags 0 or 1,
                                         * slots of hits inside the cache.  A violation sets SISO_ERR_INVALID_ARG in the status
                                         * word (read it with siso_sync_status); nothing traps and the call still runs.  0
                                         * (default) unless the library was built with -DSISO_CHECKED. */
#define SISO_OPT_TENSOR_CTA_PAIR 3      /* 0 (default): tensor-core lookup runs CTA pairs for >= 2 query tiles; 1: never */
#define SISO_PATH_AUTO 0
#define SISO_PATH_SIMT 1   /* CUDA-core tiled sweep (fp32 accumulate of exact products)        */
#define SISO_PATH_TENSOR 2 /* tcgen05 tensor-core sweep (fp32 caches: split-bf16 selection + exact rescoring, k <= 4) */
#define SISO_PATH_STREAM 3 /* small-batch streaming sweep, one pass over the centroid matrix   */

/* Device memory for the cache's own state and scratch comes from here.  alloc returns a
 * device pointer aligned to 256 bytes or NULL; both may be NULL to use cudaMalloc/cudaFree. */
typedef struct {
    void *(*alloc)(size_t bytes, void *stream, void *ctx);
    void (*free)(void *ptr, void *ctx);
    void *ctx;
} siso_allocator_t;

typedef struct {
    int64_t capacity; /* number of slots: the capacity M of Algorithm 1, counted in entries */
    int32_t dim;      /* embedding dimension, multiple of 8                                            */
    int32_t dtype;    /* siso_dtype_t: storage type of cached vectors AND of query/insert arguments    */
    int32_t device;   /* CUDA device ordinal                                                           */
    int32_t reserved;
    double decay; /* divisor of cluster_size in FilteringCentroids (Algorithm 1: 1.1); 0 selects 1.1 */
    siso_allocator_t allocator;
} siso_config_t;

/* Create an empty cache (all slots invalid, clock 0).  Synchronous. */
siso_status_t siso_cache_create(siso_cache_t **out, const siso_config_t *cfg);
/* Synchronises the device, then releases everything obtained through the allocator. */
siso_status_t siso_cache_destroy(siso_cache_t *c);

/* Set a tuning option (SISO_OPT_*).  Host-side only. */
siso_status_t siso_set_option(siso_cache_t *c, int32_t key, int64_t value);

/* Bulk promotion of n centroids into the cache (the else-branch of MergeCentroids, Algorithm 1:
 * a new entry gets access_count = infinity).  Rows take the free slots in ascending slot order.
 * d_vecs [n, dim] in the cache dtype; d_sizes [n] cluster_size per row or NULL (= 1);
 * d_slots_out [n] receives the slot of each row, or NULL.  Too few free slots:
 * SISO_ERR_CAPACITY in the status word and nothing is modified. */
siso_status_t siso_insert(siso_cache_t *c, const void *d_vecs, const double *d_sizes, int64_t n,
                          int32_t *d_slots_out, void *stream);

/* FindClosestCentroid + CosineSimilarity for a batch (Algorithm 1; the cache search of Sec. 4.3), exact, and the hit test against the retrieval threshold theta_R (Sec. 3.1), which is
 * an input because it is adjusted at run time (Sec. 4.3, threshold adjustment under load).
 *   d_queries [n_queries, dim] in the cache dtype, unit-norm
 *   d_theta   [n_queries] per-query thresholds, or NULL to use theta_scalar for all
 *   k         in [1, 8]: number of best entries returned per query
 *   d_idx     [n_queries, k] slots by (similarity desc, slot asc); -1 where fewer than k entries exist
 *   d_sim     [n_queries, k] fp32 similarities (-inf beside idx = -1)
 *   d_hit     [n_queries] 1 if d_sim[.,0] > theta, else 0 (empty cache: all 0)
 * Reads the cache, modifies only its lookup/hit statistics. */
siso_status_t siso_lookup(siso_cache_t *c, const void *d_queries, int64_t n_queries, const float *d_theta,
                          float theta_scalar, int32_t k, int32_t *d_idx, float *d_sim, uint8_t *d_hit,
                          void *stream);

/* Same as siso_lookup with HOST buffers (pinned memory recommended): copies queries and
 * thresholds to the device, runs the lookup, copies the three results back, all on `stream`. */
siso_status_t siso_lookup_host(siso_cache_t *c, const void *h_queries, int64_t n_queries, const float *h_theta,
                               float theta_scalar, int32_t k, int32_t *h_idx, float *h_sim, uint8_t *h_hit,
                               void *stream);

/* Hit update: Sec. 3.1 describes a centroid as the mean point of its group of vectors; here it is kept as
 * a running mean.  For every slot j hit by the set H_j of this batch (ascending query order):
 *     c_j <- normalise(cluster_size_j * c_j + sum_{b in H_j} q_b),  cluster_size_j += |H_j|,
 *     access_count_j += |H_j| (saturating; Sec. 4.2 counts references made while the entry is
 *     cached),  last_access_j <- clock.
 * The cache clock advances by one per call.  d_idx is read with stride idx_stride (column 0 of a
 * lookup result: pass k).  Rows with d_hit == 0 are ignored.  bf16 caches keep an fp32 master copy and
 * re-round the lookup copy. */
siso_status_t siso_update(siso_cache_t *c, const void *d_queries, int64_t n_queries, const int32_t *d_idx,
                          int32_t idx_stride, const uint8_t *d_hit, void *stream);

/* MergeCentroids (Algorithm 1).
 * d_repo == NULL, n_repo == 0: the cache is merged with itself.  Entries are taken in ascending slot order, each
 * is compared with the survivors before it (vectors as they were when the call began) and joins the most
 * similar one if that similarity is > theta_c (cluster_size added, slot freed), else survives.
 * d_repo != NULL: Algorithm 1 as printed, with C_cur = the entries live at the call and C_repo = the n_repo rows
 * of d_repo [n_repo, dim] (cache dtype, unit-norm) with cluster sizes d_repo_sizes [n_repo] (NULL = 1).  The rows
 * first take the free slots in ascending order (as siso_insert: access_count = infinity), then each is compared,
 * in row order, with C_cur and with the repository rows that survived before it; it joins the most similar one
 * above theta_c (ties: a member of C_cur first, then the lower slot) and frees its slot, else stays.  Members of
 * C_cur are never merged with each other.  Fewer than n_repo free slots: SISO_ERR_CAPACITY, nothing modified.
 *   flags        SISO_MERGE_SIZES_ONLY or SISO_MERGE_WEIGHTED_MEAN
 *   d_merge_map  [capacity] slot -> surviving slot (own slot for survivors, -1 for empty slots), or NULL
 *   h_n_merged   host pointer receiving the number of entries merged away, or NULL.  When not NULL the
 *                call synchronises `stream` and returns the device status (SISO_ERR_OVERFLOW if the
 *                pairs above theta_c did not fit the candidate buffer; then nothing was modified). */
siso_status_t siso_merge(siso_cache_t *c, const void *d_repo, const double *d_repo_sizes, int64_t n_repo,
                         float theta_c, uint32_t flags, int32_t *d_merge_map, int64_t *h_n_merged, void *stream);

/* FilteringCentroids (Algorithm 1): remove the n_evict entries that come first in ascending
 * (cluster_size, access_count, last_access, slot) order; with SISO_EVICT_DECAY every remaining entry then
 * gets cluster_size /= decay and access_count = 0.  d_victims [n_evict] receives the removed slots in that
 * order (-1 padding if the cache held fewer entries), or NULL. */
siso_status_t siso_evict(siso_cache_t *c, int64_t n_evict, uint32_t flags, int32_t *d_victims, void *stream);

/* Spare-space caching of individual query vectors (Sec. 5.2.5: space left over after the centroids holds
 * single query vectors under LRU).  siso_make_room evicts exactly as many entries as the
 * misses of this batch lack free slots for (max(0, #miss - #free), decided on the device);
 * d_victims [n] receives them (-1 padding) or NULL.  siso_insert_misses then stores every row with
 * d_hit == 0, in ascending row order into ascending free slots, as a new entry (cluster_size 1,
 * access_count infinity, last_access = clock); d_slots_out [n] receives the slot or -1 for hits. */
siso_status_t siso_make_room(siso_cache_t *c, const uint8_t *d_hit, int64_t n, uint32_t flags,
                             int32_t *d_victims, void *stream);
siso_status_t siso_insert_misses(siso_cache_t *c, const void *d_queries, int64_t n, const uint8_t *d_hit,
                                 int32_t *d_slots_out, void *stream);

/* One micro-batch of the streaming cache: lookup (k = 1), update, make_room, insert_misses, in this
 * order on `stream`.  Output arrays as in the four calls; d_victims / d_slots_out may be NULL. */
siso_status_t siso_stream_step(siso_cache_t *c, const void *d_queries, int64_t n, const float *d_theta,
                               float theta_scalar, int32_t *d_idx, float *d_sim, uint8_t *d_hit,
                               int32_t *d_victims, int32_t *d_slots_out, void *stream);

/* Small-batch lookup for callers that cannot allocate device memory.  The paper has no counterpart: this
 * entry point exists for integration reasons only.  Some callers of this library run where cudaMalloc
 * and cudaFree are off limits - a serving loop whose device memory was handed out at start-up, a callback
 * that may run while another thread holds an allocator lock, a process with a fixed memory budget -
 * because those calls synchronise the device and can fail at any moment.  This call allocates nothing,
 * neither through CUDA nor through the cache's allocator, and needs no cache handle: the caller passes
 * the centroid matrix and every output.
 *   d_centroids [n_centroids, dim] row-major in `dtype` (siso_dtype_t), unit-norm; 1 <= dim <= 1024
 *   d_valid     [n_centroids] 1 = live entry, 0 = skip; NULL = all live
 *   d_queries   [n_queries, dim] in `dtype`; 1 <= n_queries <= SISO_NOALLOC_MAX_QUERIES
 *   d_theta / theta_scalar, k (1..8), d_idx, d_sim, d_hit: as in siso_lookup
 * Its scratch (per-CTA partial top-k lists, 512 KiB) is a fixed array inside the library image that
 * every GPU loading the library holds until the process exits.  That fixes the limits above; sizes
 * beyond them return SISO_ERR_UNSUPPORTED and launch nothing.  All calls share that array and it keeps
 * the previous call's contents; each call overwrites every entry it later reads, so calls issued in
 * order on one stream are independent, but two calls that may run on the GPU at the same time
 * (different streams, different threads) race on it and must be ordered by the caller.
 * The first call on each device looks up the array's device address (with that device current, which
 * is the caller's current device); make that first call before starting any stream capture.
 * Asynchronous on `stream`; runs on the calling thread's current device. */
#define SISO_NOALLOC_MAX_QUERIES 8
#define SISO_NOALLOC_MAX_DIM 1024
siso_status_t siso_lookup_small_noalloc(const void *d_centroids, const uint8_t *d_valid, int64_t n_centroids,
                                        int32_t dim, int32_t dtype, const void *d_queries, int64_t n_queries,
                                        const float *d_theta, float theta_scalar, int32_t k, int32_t *d_idx,
                                        float *d_sim, uint8_t *d_hit, void *stream);

/* Lookup over a cache whose rows are partitioned across several GPUs (one handle per GPU, each holding a contiguous
 * range of the global slots).  FindClosestCentroid over the whole cache = the best of the shards' best, so every GPU
 * scores the full query batch against its own rows and the shards' top-k lists are combined after one exchange.
 * siso_lookup_keys is the similarity sweep and the top-k selection on one shard: d_keys [n_queries, k] receives packed 64-bit keys,
 * (order-preserving similarity bits << 32) | (2^32 - 1 - (slot + slot_offset)), 0 where the shard has fewer than k
 * entries; a larger key is a better match, ties go to the lower global slot.  The shard's hit statistics are not
 * touched.  slot_offset + capacity must stay below 2^32.
 * siso_combine_keys (needs no handle; runs on the current device): d_keys [n_queries, n_lists, k], e.g. the all-gathered
 * lists of n_lists shards brought into that layout; per query the k largest keys give d_idx [n_queries, k] (int64 global
 * slot, -1 where none), d_sim [n_queries, k] and the strict threshold test d_hit [n_queries] on the best one (d_theta
 * per query, or theta_scalar if NULL).  The result is the same for any number and order of shards.
 * Both are asynchronous on `stream`. */
siso_status_t siso_lookup_keys(siso_cache_t *c, const void *d_queries, int64_t n_queries, int32_t k, int64_t slot_offset,
                               uint64_t *d_keys, void *stream);
siso_status_t siso_combine_keys(const uint64_t *d_keys, int64_t n_queries, int32_t n_lists, int32_t k, const float *d_theta,
                                float theta_scalar, int64_t *d_idx, float *d_sim, uint8_t *d_hit, void *stream);

/* Maintenance of a cache partitioned across GPUs: updates, insertions and evictions go to the shard that owns the slot,
 * and the whole behaves as one cache over the global slots (same victims, same slots for new entries).
 *   siso_route         no handle.  From the combined result of a batch (d_idx int64 global slots read with stride idx_stride,
 *                      d_hit [n]) what the shard owning global slots [slot_lo, slot_hi) has to do: d_idx_local [n] (local
 *                      slot of a hit on its rows, else -1) and d_update_hit [n] (1 there, else 0) are the arguments of
 *                      siso_update, which every shard calls once per batch so that the clocks agree; d_insert_hit [n] is
 *                      the d_hit argument of siso_insert_misses: 0 exactly for the misses number miss_skip ..
 *                      miss_skip + miss_take - 1, counted in ascending row order (the misses that land in this shard's
 *                      free slots when the shards before it have miss_skip free slots and it has miss_take).
 *   siso_evict_keys    the n lowest entries of this shard in FilteringCentroids order, ascending, as keys of three
 *                      64-bit words [n, 3] (order-preserving cluster_size; access_count and last_access; last_access and
 *                      slot + slot_offset), padded with all-ones words where the shard holds fewer; nothing is evicted.
 *   siso_select_evict  no handle.  d_keys [n_lists, n, 3], every list as siso_evict_keys wrote it: the n_take lowest of
 *                      all keys give d_victims [n_take] (int64 global slots in eviction order, -1 padding).  n_take <= n
 *                      makes the result the exact global selection.
 *   siso_evict_slots   drops the victims that lie in [slot_offset, slot_offset + capacity) from this shard (others are
 *                      ignored), then the decay pass if SISO_EVICT_DECAY is set.
 * All asynchronous on `stream`; device pointers. */
siso_status_t siso_route(const int64_t *d_idx, int64_t idx_stride, const uint8_t *d_hit, int64_t n, int64_t slot_lo,
                         int64_t slot_hi, int64_t miss_skip, int64_t miss_take, int32_t *d_idx_local, uint8_t *d_update_hit,
                         uint8_t *d_insert_hit, void *stream);
siso_status_t siso_evict_keys(siso_cache_t *c, int64_t n, int64_t slot_offset, uint64_t *d_keys, void *stream);
siso_status_t siso_select_evict(const uint64_t *d_keys, int32_t n_lists, int64_t n, int64_t n_take, int64_t *d_victims,
                                void *stream);
siso_status_t siso_evict_slots(siso_cache_t *c, const int64_t *d_victims, int64_t n, int64_t slot_offset, uint32_t flags,
                               void *stream);

/* The same steps with every count kept on the device, so that a streaming step of the partitioned cache needs no host read:
 *   siso_free_slots           d_free[0] = free slots of this shard (capacity - occupancy).
 *   siso_shard_plan           d_hit [n] of the combined result and d_free_all [world] (the gathered free counts) ->
 *                             d_plan[4] = { misses of the batch, entries to evict over the whole cache (misses - all free
 *                             slots, at least 0), free slots on the shards before `rank`, free slots on this shard }.
 *   siso_route_planned        siso_route with miss_skip / miss_take taken from d_plan[2], d_plan[3].
 *   siso_select_evict_planned siso_select_evict with n_take = min(d_plan[1], n); d_victims [n], -1 beyond the victims. */
siso_status_t siso_free_slots(siso_cache_t *c, int64_t *d_free, void *stream);
siso_status_t siso_shard_plan(const uint8_t *d_hit, int64_t n, const int64_t *d_free_all, int32_t world, int32_t rank,
                              int64_t *d_plan, void *stream);
siso_status_t siso_route_planned(const int64_t *d_idx, int64_t idx_stride, const uint8_t *d_hit, int64_t n, int64_t slot_lo,
                                 int64_t slot_hi, const int64_t *d_plan, int32_t *d_idx_local, uint8_t *d_update_hit,
                                 uint8_t *d_insert_hit, void *stream);
siso_status_t siso_select_evict_planned(const uint64_t *d_keys, int32_t n_lists, int64_t n, const int64_t *d_plan,
                                        int64_t *d_victims, void *stream);

/* Locality-ordered exact search, k = 1 (the exact-search counterpart of Sec. 4.3, "Searching for vectors in semantic
 * cache": entries with strong semantic locality are searched first and most queries end there).  The cache is held as
 * two handles: a small hot tier and the cold rest.  A query whose best hot similarity s exceeds exit_sim needs no cold
 * search: if every hot/cold pair of entries has similarity <= sep, then by the triangle inequality on angles no cold
 * entry can reach s once angle(q, hot) < acos(sep) / 2.  The result equals the top-1 over the whole cache.
 *   siso_tier_exit_sim  (host arithmetic) the exit similarity for a separation bound `sep_sim` when all norms lie in
 *                       [1 - norm_slack, 1 + norm_slack]; includes 1e-5 for the rounding of computed similarities;
 *                       +infinity when no exit is possible (sep too close to 1, bad arguments).
 *   siso_tier_select    d_hot_keys [n_queries] = siso_lookup_keys(hot tier, k = 1, slot_offset 0).  d_rows [n_queries]
 *                       receives, ascending, the rows whose key is 0 or whose similarity is not above exit_sim;
 *                       *d_count (device int64) their number; d_cold_queries [n_queries, row_bytes] those rows of
 *                       d_queries, densely packed (row_bytes = dim * element size, a multiple of 16).
 *   siso_tier_finish    d_cold_keys [n_cold] = siso_lookup_keys(cold tier, k = 1, slot_offset 0) of the packed rows;
 *                       d_hot_slot / d_cold_slot (device int32, or NULL for identity) map a tier's slot to the slot
 *                       reported; per query the better of the two keys (ties to the lower reported slot) gives
 *                       d_idx [n_queries] (int32, -1 where both tiers are empty), d_sim, and d_hit by the strict
 *                       threshold test (d_theta per query, or theta_scalar if NULL).  exit_sim as given to select.
 * All device pointers, no handle, current device, asynchronous on `stream`; the caller reads *d_count (one 8-byte copy)
 * to size the cold lookup.  SISO_ERR_INVALID_ARG on bad sizes or NULL pointers, nothing written. */
double siso_tier_exit_sim(double sep_sim, double norm_slack);
/* *h_max_dev = the largest | |v| - 1 | over the live entries, taken on the vectors that lookups read (fp64 sums, rounded
 * up; +infinity if an entry holds a NaN; 0 for an empty cache): the smallest norm_slack that is true of the entries.
 * Synchronises `stream`. */
siso_status_t siso_norm_deviation(siso_cache_t *c, double *h_max_dev, void *stream);
siso_status_t siso_tier_select(const uint64_t *d_hot_keys, int64_t n_queries, float exit_sim, const void *d_queries,
                               int64_t row_bytes, void *d_cold_queries, int32_t *d_rows, int64_t *d_count, void *stream);
siso_status_t siso_tier_finish(const uint64_t *d_hot_keys, int64_t n_queries, float exit_sim, const uint64_t *d_cold_keys,
                               const int32_t *d_rows, int64_t n_cold, const int32_t *d_hot_slot, const int32_t *d_cold_slot,
                               const float *d_theta, float theta_scalar, int32_t *d_idx, float *d_sim, uint8_t *d_hit,
                               void *stream);

/* The locality-ordered search as two calls (Sec. 4.3, "Searching for vectors in semantic cache", exact counterpart).
 *   siso_tier_build   Splits `cache` (left untouched) into the HOT tier - the hot_rows entries FilteringCentroids would
 *                     evict last - and the COLD rest, written into the handles `hot` and `cold` (same dim, dtype and
 *                     device; capacities at least hot_rows and occupancy - hot_rows, else SISO_ERR_CAPACITY; what they
 *                     held is dropped).  Entries keep their vectors and metadata and are laid out in ascending slot of
 *                     `cache`; d_hot_slot / d_cold_slot [capacity of the tier] receive the slot of `cache` each place
 *                     came from.  h_counts[0], [1] = entries in the hot and the cold tier.  If sep_sim is not NaN, every
 *                     hot/cold pair is also checked against it (tensor-core sweep + exact fp64 check) and h_counts[2]
 *                     receives the number of pairs MORE similar than sep_sim (at least 65 if there are more than 64):
 *                     the exit rule of siso_tier_exit_sim(sep_sim, ...) is only valid if that is 0.  h_counts[2] = -1 if
 *                     the check was not asked for.  Synchronises `stream`.
 *   siso_tier_lookup  Top-1 over both tiers, equal to siso_lookup(k = 1) on the cache the tiers were built from: the
 *                     whole batch against the hot tier, the queries whose best hot similarity does not exceed exit_sim
 *                     packed and scored against the cold tier, the better of the two per query (ties to the lower slot),
 *                     strict threshold.  d_idx are slots of the original cache.  d_work: siso_tier_work_bytes() bytes of
 *                     device memory, 256-byte aligned.  *h_settled (may be NULL) = queries that ended in the hot tier.
 *                     Synchronises `stream` once in the middle (one 8-byte read sizes the cold sweep). */
siso_status_t siso_tier_build(siso_cache_t *cache, int64_t hot_rows, double sep_sim, siso_cache_t *hot, siso_cache_t *cold,
                              int32_t *d_hot_slot, int32_t *d_cold_slot, int64_t *h_counts, void *stream);
int64_t siso_tier_work_bytes(int64_t n_queries, int32_t dim, int32_t dtype);
siso_status_t siso_tier_lookup(siso_cache_t *hot, siso_cache_t *cold, const int32_t *d_hot_slot, const int32_t *d_cold_slot,
                               const void *d_queries, int64_t n_queries, float exit_sim, const float *d_theta, float theta_scalar,
                               void *d_work, int32_t *d_idx, float *d_sim, uint8_t *d_hit, int64_t *h_settled, void *stream);

/* Algorithm 1 as a whole (Sec. 4.2): C_new <- MergeCentroids(C_cur, C_repo, theta_C); C_new <- FilteringCentroids(C_new, M);
 * UpdateCentroids(C_cur, C_new).  With a second handle as C_new the steps are
 *     siso_cache_copy(c_new, cur)                       "C_new <- C_cur", the first line of MergeCentroids
 *     siso_merge(c_new, d_repo, d_repo_sizes, ...)      the rest of MergeCentroids (c_new needs n_repo free slots)
 *     siso_evict(c_new, occupancy - M, SISO_EVICT_DECAY)   FilteringCentroids
 *     siso_update_centroids(cur, c_new, g, group) for g = 0, group, 2 group, ... < capacity of cur
 * and the cache `cur` serves lookups all the while.
 *
 * siso_cache_copy: every slot of src (vector, cluster_size, access_count, last_access, live flag) into the same slot of
 * dst, the counters and the clock too; dst must have the same dim, dtype and device and at least src's capacity (its
 * further slots become empty), else SISO_ERR_INVALID_ARG / SISO_ERR_CAPACITY.
 *
 * siso_update_centroids is the update step: "progressively replaces small groups of centroids one at a time" so that
 * the cache stays available (the paper gives no group size; 256 slots is a reasonable one).  The live entries of c_new,
 * in ascending slot order, are numbered 0, 1, ...; slot d of cur, first_slot <= d < first_slot + n_slots, receives entry
 * number d, or becomes empty if c_new has no such entry.  The numbering is taken when first_slot == 0 is copied, so
 * c_new must not change until the last group is done; groups may be issued in any order after that first one.  A lookup
 * ordered between two groups sees every slot either as it was or as it will be.  If c_new holds more live entries than
 * cur has slots nothing is copied and the device status becomes SISO_ERR_CAPACITY.  Asynchronous on `stream`. */
siso_status_t siso_cache_copy(siso_cache_t *dst, siso_cache_t *src, void *stream);
siso_status_t siso_update_centroids(siso_cache_t *cur, siso_cache_t *c_new, int64_t first_slot, int64_t n_slots, void *stream);

/* Clustering of logged query vectors into centroids (Sec. 4.1, SISO-Cluster: community detection at the clustering
 * threshold theta_C, which yields for every cluster a centroid and cluster_size, "the number of vectors in the
 * cluster").  The paper names the method without stating its steps; the reading built here: two vectors are neighbours
 * if their cosine is strictly above theta_c; vectors are visited by neighbourhood size, largest first, ties by index;
 * a visited vector that belongs to no community founds one and takes every neighbour that belongs to none.
 * d_vecs [n, dim] in the cache's dtype, unit norm, 16-byte aligned, n < 2^24; the cache's own contents are neither
 * read nor written (the handle supplies dim, dtype, device, allocator and scratch memory).
 * Outputs, each optional (NULL), all caller-owned device memory:
 *   d_label     [n] int32   index of the centre of the vector's community (a centre labels itself)
 *   d_centres   [n] int32   the centres in founding order; the first *h_n_clusters entries are written
 *   d_sizes     [n] fp64    cluster_size of the communities, in the same order
 *   d_centroids [n, dim]    cache dtype: per community the mean of its members (fp64 sums in ascending index), scaled
 *                           to unit length (Sec. 3.1: a centroid is the mean point of its group); rows beyond the
 *                           number of communities are not written.  The rows can be handed to siso_merge as C_repo
 *                           with d_sizes as their cluster_size.
 * h_n_clusters (host, optional): number of communities; if given the call synchronises the stream and returns the
 * device status (SISO_ERR_OVERFLOW if the pairs above the threshold exceed the candidate buffer, whose size is the
 * larger of SISO_OPT_MERGE_MAX_CANDIDATES and 16 n + 2^20; the outputs are then undefined). */
siso_status_t siso_cluster(siso_cache_t *c, const void *d_vecs, int64_t n, float theta_c, int32_t *d_label,
                           int32_t *d_centres, double *d_sizes, void *d_centroids, int64_t *h_n_clusters, void *stream);

/* Threshold control (Sec. 4.3, the part on adjusting theta_R to meet the SLO).
 * siso_t2h builds the threshold-to-hit-ratio table: it looks up a sample of queries (k = 1, exact, no hit is
 * recorded in the statistics) and counts, for every threshold of the grid, the queries whose best similarity
 * is strictly above it.  d_queries [n_queries, dim] in the cache dtype; d_thetas [n_thetas] fp32 (the paper
 * sweeps 0.98 down to 0.6; at most 1024 values); d_hits [n_thetas] int64 receives the counts (hit ratio =
 * count / n_queries).  Asynchronous on `stream`. */
siso_status_t siso_t2h(siso_cache_t *c, const void *d_queries, int64_t n_queries, const float *d_thetas,
                       int32_t n_thetas, int64_t *d_hits, void *stream);
/* Eq. 1 with E = L (1 - h) (Eq. 2): mean waiting time of the M/D/1 queue in front of the LLM,
 * W = E + lambda E^2 / (2 (1 - lambda E)); +infinity if lambda E >= 1.  Host arithmetic only. */
double siso_md1_wait(double llm_latency, double arrival_rate, double hit_ratio);
/* Index of the highest threshold of the table whose W is below the SLO (strictly), or -1; *h_wait_out (may be
 * NULL) receives that W.  Host arrays. */
int32_t siso_choose_theta(const float *h_thetas, const double *h_hit_ratio, int32_t n_thetas, double llm_latency,
                          double arrival_rate, double slo, double *h_wait_out);
/* Correction step of Sec. 4.3: if the measured waiting time differs from the estimate by more than 10 % (relative to
 * the measured one), move to the next lower threshold of the table when the measured time is the longer one,
 * to the next higher when it is the shorter; otherwise, or if there is no such entry, keep `chosen`. */
int32_t siso_correct_theta(const float *h_thetas, int32_t n_thetas, int32_t chosen, double wait_estimated,
                           double wait_measured);

/* Copy the state out (checkpoint, parity checks).  Any pointer may be NULL.
 *   d_vecs   [capacity, dim] lookup copy in the cache dtype     d_master [capacity, dim] fp32 master
 *   d_sizes  [capacity] fp64   d_access [capacity] u32   d_last [capacity] u64   d_valid [capacity] u8 */
siso_status_t siso_export(siso_cache_t *c, void *d_vecs, float *d_master, double *d_sizes, uint32_t *d_access,
                          uint64_t *d_last, uint8_t *d_valid, void *stream);
/* Replace the whole state (restore a checkpoint).  d_master (fp32) is required; the lookup copy is
 * re-derived from it.  clock becomes `clock`. */
siso_status_t siso_import(siso_cache_t *c, const float *d_master, const double *d_sizes, const uint32_t *d_access,
                          const uint64_t *d_last, const uint8_t *d_valid, uint64_t clock, void *stream);

/* h_counts[8] = occupancy, lookups, hits, inserts, evictions, merges, clock, rescans (queries of fp32 tensor-core
 * lookups that the exact rescoring could not settle and that were scanned again).  Synchronises `stream`. */
siso_status_t siso_get_stats(siso_cache_t *c, int64_t *h_counts, void *stream);
/* Synchronise `stream`, return the device status word (SISO_OK if clear) and clear it. */
siso_status_t siso_sync_status(siso_cache_t *c, void *stream);
/* MergeCentroids (Algorithm 1, Sec. 4.2 merge step) over a cache whose rows are partitioned across several GPUs: one
 * handle per GPU holds a contiguous block of the global slots [own_offset, own_offset + capacity).  The double loop of
 * MergeCentroids is a pairwise sweep over the whole cache; by blocks it falls into one sweep of every block with itself
 * and one sweep of every unordered pair of blocks, done on one of the two owners after the other block's rows have been
 * copied into that GPU's own memory (the caller moves them: NCCL send/recv or a peer copy; the library reads local
 * memory only).  Every GPU then holds the same candidates and runs the same resolution, so all merge maps agree.
 *   siso_pair_sweep_block   Pairs with similarity > theta_c (exact: fp64 over the fp32 vectors) between the rows of this
 *                           block and (d_peer_master == NULL) the earlier rows of the same block, or the rows of a peer
 *                           block d_peer_master [n_peer, dim] fp32 with live flags d_peer_valid [n_peer] at global slots
 *                           peer_offset + row.  Records (i, j, similarity) of three 32-bit words, global slots, j < i,
 *                           are APPENDED to d_cand [max_cand][3] at *d_n_cand (a device counter the caller zeroes once);
 *                           more than max_cand records: SISO_ERR_OVERFLOW in the status word.
 *   siso_merge_resolve      d_cand [n_cand][3] (records of all GPUs in any order; i = -1 marks an unused place), d_valid
 *                           [n_total] live flags of all global slots -> d_merge_map [n_total]: the survivor every slot
 *                           joins (itself for survivors, -1 for empty slots), exactly as siso_merge over one cache would
 *                           resolve it (closest earlier survivor, ties to the lower slot); *d_n_merged (device) = slots
 *                           merged away.  The handle only lends its scratch memory.
 *   siso_merge_pack         This block's merged rows in ascending slot: d_meta [pack_capacity][2] int32 (global slot,
 *                           survivor; slot -1 in unused places), d_sizes [pack_capacity] cluster_size, d_rows
 *                           [pack_capacity, dim] fp32 vectors (NULL in sizes-only mode), *d_n_pack (device) their number.
 *   siso_merge_apply_shard  d_meta / d_sizes / d_rows [n_places]: the packs of all GPUs one after the other in rank order
 *                           (so ascending global slot, unused places skipped).  Every survivor of this block takes its
 *                           members: cluster_size added, and with SISO_MERGE_WEIGHTED_MEAN the vector becomes
 *                           normalise(cluster_size_s c_s + sum of cluster_size_m c_m), vectors as at the start of the
 *                           merge; this block's merged rows leave the cache.
 * All asynchronous on `stream`; device pointers. */
siso_status_t siso_pair_sweep_block(siso_cache_t *c, int64_t own_offset, const float *d_peer_master, const uint8_t *d_peer_valid,
                                    int64_t n_peer, int64_t peer_offset, float theta_c, int32_t *d_cand, int64_t max_cand,
                                    int64_t *d_n_cand, void *stream);
siso_status_t siso_merge_resolve(siso_cache_t *c, const int32_t *d_cand, int64_t n_cand, const uint8_t *d_valid, int64_t n_total,
                                 int32_t *d_merge_map, int64_t *d_n_merged, void *stream);
siso_status_t siso_merge_pack(siso_cache_t *c, const int32_t *d_merge_map, int64_t own_offset, int64_t pack_capacity,
                              int32_t *d_meta, double *d_sizes, float *d_rows, int64_t *d_n_pack, void *stream);
siso_status_t siso_merge_apply_shard(siso_cache_t *c, const int32_t *d_merge_map, int64_t own_offset, const int32_t *d_meta,
                                     const double *d_sizes, const float *d_rows, int64_t n_places, uint32_t flags, void *stream);

/* Diagnostics (no passage of the paper: they serve the error model and the measurements of this library).
 *   siso_selftest_wait_timeout  Every device-side wait of the tensor-core kernels is bounded; when one runs out the
 *                      kernel records SISO_ERR_TIMEOUT in the status word and returns normally.  This call exercises
 *                      exactly that path without touching a real sweep: one warp waits, with the kernels' own wait
 *                      routine, at most poll_limit polls (1 .. 2^20) on a barrier that nothing arrives on and with no
 *                      copy or tensor-core operation in flight.  Afterwards siso_sync_status returns SISO_ERR_TIMEOUT
 *                      once and the handle is usable as before.  d_gave_up (device int32, may be NULL) receives 1 if
 *                      the wait gave up.  Asynchronous on `stream`.
 *   siso_measure_fp32_fma       FP32 fused multiply-add throughput of the device's CUDA cores in TFLOP/s (2 flop per
 *                      FMA; best of three timed launches of a register-only kernel): the roof of the CUDA-core
 *                      sweeps.  Synchronises `stream`. */
siso_status_t siso_selftest_wait_timeout(siso_cache_t *c, uint32_t poll_limit, int32_t *d_gave_up, void *stream);
siso_status_t siso_measure_fp32_fma(siso_cache_t *c, double *h_tflops, void *stream);

/* Number of kernels this handle has launched so far (host-side count). */
int64_t siso_launch_count(const siso_cache_t *c);
const char *siso_status_string(siso_status_t s);
/* Text of the last CUDA error seen by this library in the calling process ("" if none). */
const char *siso_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SISO_H_ */
