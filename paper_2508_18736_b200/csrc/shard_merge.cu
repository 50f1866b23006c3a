// MergeCentroids (Algorithm 1) over a cache whose rows are partitioned across several GPUs.
//
// The double loop of MergeCentroids - every entry against the earlier entries of C_new - is a pairwise similarity
// sweep over the whole cache.  With the rows in blocks, one per GPU, the sweep falls into block products: every GPU
// sweeps its own block against itself, and every unordered pair of blocks is swept once, on one of its two owners,
// after the other block has been COPIED INTO THAT GPU'S OWN MEMORY (a ring of plain copies; the tensor maps of the
// sweep kernel never cover another GPU's memory).  What comes out are candidate pairs (i, j, exact similarity) in
// global slots; all GPUs gather all candidates and each runs the same resolution over them, so every GPU holds the
// same merge map.  The grouping step then needs the merged rows at the owner of their survivor: every GPU packs its
// merged rows (slot, survivor, cluster_size, vector), the packs are gathered, and every GPU applies those that join
// one of its own survivors, survivor first, members in ascending global slot.
//
//   siso_pair_sweep_block    own block x own block (lower triangle), or own block x one peer block
//   siso_merge_resolve       candidates of all GPUs -> merge map over the global slots
//   siso_merge_pack          this GPU's merged rows, ascending slot
//   siso_merge_apply_shard   gathered packs -> this GPU's survivors and flags
#include "common.cuh"

namespace siso {

namespace {

struct PairRecord {      // the candidate record of the sweep (merge_tensor.cu, merge.cu)
    int32_t i, j;
    float sim;
};
struct SweepCtl {        // same layout as MergeCtl
    unsigned long long n_cand;
    int overflow;
    int n_merged;
};

// local row of the sweep's array -> global slot, larger slot first; confirmed pairs are appended to `out`
__global__ void sweep_to_global_kernel(const SweepCtl *ctl, const PairRecord *__restrict__ cand, unsigned long long max_cand,
                                       long long peer_rows_pad, long long peer_offset, long long own_offset,
                                       PairRecord *__restrict__ out, long long out_cap, unsigned long long *n_out, int *status) {
    if (ctl->overflow) { if (blockIdx.x == 0 && threadIdx.x == 0) set_status(status, SISO_ERR_OVERFLOW); return; }
    const unsigned long long n = ctl->n_cand < max_cand ? ctl->n_cand : max_cand;
    const int lane = threadIdx.x & 31;
    for (unsigned long long e0 = static_cast<unsigned long long>(blockIdx.x) * blockDim.x; e0 < n;
         e0 += static_cast<unsigned long long>(gridDim.x) * blockDim.x) {
        const unsigned long long e = e0 + threadIdx.x;
        PairRecord cd;
        cd.i = -1; cd.j = -1; cd.sim = 0.f;
        if (e < n) cd = cand[e];
        const bool take = cd.i >= 0;
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, take);
        if (!ballot) continue;
        unsigned long long base = 0;
        if (lane == 0) base = atomicAdd(n_out, static_cast<unsigned long long>(__popc(ballot)));
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        if (take) {
            const long long gi = cd.i < peer_rows_pad ? peer_offset + cd.i : own_offset + (cd.i - peer_rows_pad);
            const long long gj = cd.j < peer_rows_pad ? peer_offset + cd.j : own_offset + (cd.j - peer_rows_pad);
            const long long at = static_cast<long long>(base) + __popc(ballot & ((1u << lane) - 1u));
            if (at < out_cap) {
                PairRecord o;
                o.i = static_cast<int32_t>(gi > gj ? gi : gj);
                o.j = static_cast<int32_t>(gi > gj ? gj : gi);
                o.sim = cd.sim;
                out[at] = o;
            } else {
                set_status(status, SISO_ERR_OVERFLOW);
            }
        }
    }
}

__global__ void block_flags_kernel(const uint8_t *__restrict__ peer_valid, long long n_peer, long long peer_rows_pad,
                                   const uint8_t *__restrict__ own_valid, long long n_own, uint8_t *__restrict__ valid,
                                   uint8_t *__restrict__ seed) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= peer_rows_pad + n_own) return;
    if (i < peer_rows_pad) {
        valid[i] = (i < n_peer && peer_valid[i]) ? 1 : 0;
        seed[i] = 1;
    } else {
        valid[i] = own_valid[i - peer_rows_pad] ? 1 : 0;
        seed[i] = 0;
    }
}

// bf16 rows -> fp32, eight elements per thread
__global__ void widen_rows_kernel(const uint4 *__restrict__ src, float4 *__restrict__ dst, long long n8) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    const uint4 u = __ldg(src + i);
    dst[2 * i] = make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u), __uint_as_float(u.y << 16),
                             __uint_as_float(u.y & 0xFFFF0000u));
    dst[2 * i + 1] = make_float4(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xFFFF0000u), __uint_as_float(u.w << 16),
                                 __uint_as_float(u.w & 0xFFFF0000u));
}

// flag[i] = 1 if local row i is live and merged away (merge_map names another slot)
__global__ void pack_flags_kernel(const int32_t *__restrict__ merge_map, long long own_offset, long long n_own,
                                  const uint8_t *__restrict__ valid, uint32_t *__restrict__ flag) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i > n_own) return;
    flag[i] = (i < n_own && valid[i] && merge_map[own_offset + i] >= 0 && merge_map[own_offset + i] != own_offset + i) ? 1u : 0u;
}

// pos = exclusive scan of the flags: merged row i goes to place pos[i] of the pack (ascending slot)
__global__ void pack_rows_kernel(const int32_t *__restrict__ merge_map, long long own_offset, long long n_own,
                                 const uint8_t *__restrict__ valid, const uint32_t *__restrict__ pos,
                                 const float *__restrict__ master, const double *__restrict__ size, int D, long long cap,
                                 int32_t *__restrict__ meta, double *__restrict__ sizes, float *__restrict__ rows,
                                 long long *n_pack, int *status) {
    const long long i = blockIdx.x;
    if (i == 0 && threadIdx.x == 0) {
        *n_pack = pos[n_own];
        if (static_cast<long long>(pos[n_own]) > cap) set_status(status, SISO_ERR_OVERFLOW);
    }
    const long long g = own_offset + i;
    if (!(valid[i] && merge_map[g] >= 0 && merge_map[g] != g)) return;
    const long long at = pos[i];
    if (at >= cap) return;
    if (threadIdx.x == 0) {
        meta[2 * at] = static_cast<int32_t>(g);
        meta[2 * at + 1] = merge_map[g];
        sizes[at] = size[i];
    }
    if (rows) {
        const float4 *src = reinterpret_cast<const float4 *>(master + i * D);
        float4 *dst = reinterpret_cast<float4 *>(rows + at * D);
        for (int q = threadIdx.x; q < D / 4; q += blockDim.x) dst[q] = src[q];
    }
}

// One CTA per place of the gathered packs.  A place whose survivor lives here and which is the first place naming
// that survivor does the survivor's whole group: cluster_size of the survivor plus the members' in ascending slot,
// and in weighted-mean mode normalise(size_s c_s + sum of size_m c_m) in fp64.
template <typename T>
__global__ void __launch_bounds__(256)
shard_apply_kernel(const int32_t *__restrict__ meta, const double *__restrict__ sizes, const float *__restrict__ rows,
                   long long n_places, long long own_offset, long long n_own, int D, int weighted, float *__restrict__ master,
                   T *__restrict__ vecs, double *__restrict__ size) {
    extern __shared__ double acc[];
    __shared__ double red[8];
    const long long p = blockIdx.x;
    const int32_t slot = meta[2 * p], sv = meta[2 * p + 1];
    if (slot < 0 || sv < own_offset || sv >= own_offset + n_own) return;
    int earlier = 0;
    for (long long t = threadIdx.x; t < p; t += 256) earlier |= (meta[2 * t] >= 0 && meta[2 * t + 1] == sv) ? 1 : 0;
    if (__syncthreads_or(earlier)) return;
    const long long ls = sv - own_offset;
    float *m = master + ls * D;
    const double own = size[ls];
    double total = own;
    if (weighted)
        for (int d = threadIdx.x; d < D; d += 256) acc[d] = own * static_cast<double>(m[d]);
    for (long long t = p; t < n_places; ++t) {
        if (meta[2 * t] < 0 || meta[2 * t + 1] != sv) continue;         // the same decision in every thread
        const double w = sizes[t];
        total += w;
        if (weighted) {
            const float *mv = rows + t * D;
            for (int d = threadIdx.x; d < D; d += 256) acc[d] += w * static_cast<double>(mv[d]);
        }
    }
    if (weighted) {
        double ss = 0.0;
        for (int d = threadIdx.x; d < D; d += 256) ss += acc[d] * acc[d];
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        double nn = 0.0;
        for (int w = 0; w < 8; ++w) nn += red[w];
        nn = sqrt(nn);
        T *v = vecs + ls * D;
        for (int d = threadIdx.x; d < D; d += 256) {
            const float f = static_cast<float>(acc[d] / nn);
            m[d] = f;
            if constexpr (sizeof(T) == 2) v[d] = __float2bfloat16_rn(f);
        }
    }
    if (threadIdx.x == 0) size[ls] = total;
}

// this GPU's merged rows leave the cache
__global__ void shard_drop_kernel(const int32_t *__restrict__ merge_map, long long own_offset, long long n_own,
                                  uint8_t *__restrict__ valid, long long *counters) {
    __shared__ int dropped;
    if (threadIdx.x == 0) dropped = 0;
    __syncthreads();
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n_own && valid[i]) {
        const int32_t t = merge_map[own_offset + i];
        if (t >= 0 && t != own_offset + i) { valid[i] = 0; atomicAdd(&dropped, 1); }
    }
    __syncthreads();
    if (threadIdx.x == 0 && dropped) {
        atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_MERGES), static_cast<unsigned long long>(dropped));
        atomicAdd(reinterpret_cast<unsigned long long *>(counters + CNT_OCCUPANCY), static_cast<unsigned long long>(-static_cast<long long>(dropped)));
    }
}

}  // namespace

}  // namespace siso

using namespace siso;

// `lookup_copies`: compare the vectors that lookups read (for a bf16 cache its bf16 copies, widened; d_peer_rows is
// then a bf16 array too) instead of the fp32 masters.  Used to certify the separation of the two tiers of the
// locality-ordered search, whose exit rule is about the vectors that lookups see.
siso_status_t siso::launch_pair_sweep_block(Cache *c, int64_t own_offset, const void *d_peer_rows, const uint8_t *d_peer_valid,
                                            int64_t n_peer, int64_t peer_offset, float theta_c, int32_t *d_cand, int64_t max_cand,
                                            int64_t *d_n_cand, bool lookup_copies, cudaStream_t s) {
    if (!c || own_offset < 0 || !d_cand || max_cand < 1 || !d_n_cand || !(theta_c == theta_c)) return SISO_ERR_INVALID_ARG;
    if ((d_peer_rows != nullptr) != (n_peer > 0) || (n_peer > 0 && (!d_peer_valid || peer_offset < 0))) return SISO_ERR_INVALID_ARG;
    if (n_peer > 0 && (reinterpret_cast<uintptr_t>(d_peer_rows) & 15u)) return SISO_ERR_INVALID_ARG;
    const bool widen = lookup_copies && c->dtype == SISO_BF16;
    if (widen && n_peer == 0) return SISO_ERR_UNSUPPORTED;
    const int64_t n_own = c->capacity;
    const int64_t peer_pad = (n_peer + 255) / 256 * 256;
    if (own_offset + n_own >= (1ll << 31) || peer_offset + n_peer >= (1ll << 31) || peer_pad + c->rows_alloc >= (1ll << 24)) return SISO_ERR_UNSUPPORTED;
    SISO_CUDA(cudaSetDevice(c->device));
    const size_t tmp_cand = static_cast<size_t>(c->merge_max_cand);
    const int64_t rows = peer_pad + c->rows_alloc, N = peer_pad + n_own;
    const size_t D = static_cast<size_t>(c->dim);
    Scratch scr;
    const size_t need = pad256(sizeof(SweepCtl)) + pad256(sizeof(PairRecord) * tmp_cand) + pair_sweep_tensor_scratch_bytes(N, rows, c->dim) +
                        (n_peer > 0 ? pad256(static_cast<size_t>(rows) * D * sizeof(float)) + 2 * pad256(static_cast<size_t>(N)) : 0) + 1024;
    SISO_TRY(scratch_reserve(c, need, s, &scr));
    SweepCtl *ctl = scr.take<SweepCtl>(1);
    PairRecord *cand = scr.take<PairRecord>(tmp_cand);
    SISO_CUDA(cudaMemsetAsync(ctl, 0, sizeof(SweepCtl), s));
    if (n_peer == 0) {
        SISO_TRY(launch_pair_sweep_tensor(c, &scr, c->master, n_own, c->rows_alloc, c->valid, nullptr, theta_c, ctl, cand, tmp_cand,
                                          nullptr, s, nullptr, 0));
    } else {
        // the peer block (rounded up to whole tiles of 256 rows, the rest zero and not live) and then the own block, in
        // one array in this GPU's memory; the peer rows play the part of C_cur: they are compared with, never merged
        float *X = scr.take<float>(static_cast<size_t>(rows) * D);
        uint8_t *valid = scr.take<uint8_t>(static_cast<size_t>(N)), *seed = scr.take<uint8_t>(static_cast<size_t>(N));
        if (widen) {
            const long long p8 = static_cast<long long>(n_peer) * D / 8, o8 = static_cast<long long>(c->rows_alloc) * D / 8;
            widen_rows_kernel<<<static_cast<unsigned>((p8 + 255) / 256), 256, 0, s>>>(static_cast<const uint4 *>(d_peer_rows),
                                                                                      reinterpret_cast<float4 *>(X), p8);
            widen_rows_kernel<<<static_cast<unsigned>((o8 + 255) / 256), 256, 0, s>>>(static_cast<const uint4 *>(c->vecs),
                                                                                      reinterpret_cast<float4 *>(X + static_cast<size_t>(peer_pad) * D), o8);
            c->launches += 2;
        } else {
            SISO_CUDA(cudaMemcpyAsync(X, d_peer_rows, static_cast<size_t>(n_peer) * D * sizeof(float), cudaMemcpyDeviceToDevice, s));
            SISO_CUDA(cudaMemcpyAsync(X + static_cast<size_t>(peer_pad) * D, c->master, static_cast<size_t>(c->rows_alloc) * D * sizeof(float),
                                      cudaMemcpyDeviceToDevice, s));
        }
        if (peer_pad > n_peer)
            SISO_CUDA(cudaMemsetAsync(X + static_cast<size_t>(n_peer) * D, 0, static_cast<size_t>(peer_pad - n_peer) * D * sizeof(float), s));
        block_flags_kernel<<<static_cast<unsigned>((N + 255) / 256), 256, 0, s>>>(d_peer_valid, n_peer, peer_pad, c->valid, n_own, valid, seed);
        SISO_LAUNCHED(c);
        SISO_TRY(launch_pair_sweep_tensor(c, &scr, X, N, rows, valid, seed, theta_c, ctl, cand, tmp_cand, nullptr, s, nullptr, peer_pad));
    }
    sweep_to_global_kernel<<<4 * c->sm_count, 256, 0, s>>>(ctl, cand, tmp_cand, n_peer > 0 ? peer_pad : 0, peer_offset, own_offset,
                                                           reinterpret_cast<PairRecord *>(d_cand), max_cand,
                                                           reinterpret_cast<unsigned long long *>(d_n_cand), c->status);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

extern "C" siso_status_t siso_pair_sweep_block(siso_cache_t *h, int64_t own_offset, const float *d_peer_master,
                                               const uint8_t *d_peer_valid, int64_t n_peer, int64_t peer_offset, float theta_c,
                                               int32_t *d_cand, int64_t max_cand, int64_t *d_n_cand, void *stream) {
    return launch_pair_sweep_block(reinterpret_cast<Cache *>(h), own_offset, d_peer_master, d_peer_valid, n_peer, peer_offset, theta_c,
                                   d_cand, max_cand, d_n_cand, false, static_cast<cudaStream_t>(stream));
}

extern "C" siso_status_t siso_merge_resolve(siso_cache_t *h, const int32_t *d_cand, int64_t n_cand, const uint8_t *d_valid,
                                            int64_t n_total, int32_t *d_merge_map, int64_t *d_n_merged, void *stream) {
    Cache *c = reinterpret_cast<Cache *>(h);
    if (!c || n_cand < 0 || (n_cand > 0 && !d_cand) || !d_valid || n_total < 1 || !d_merge_map || !d_n_merged) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    return launch_merge_resolve_global(c, d_cand, n_cand, d_valid, n_total, d_merge_map, reinterpret_cast<long long *>(d_n_merged),
                                       static_cast<cudaStream_t>(stream));
}

extern "C" siso_status_t siso_merge_pack(siso_cache_t *h, const int32_t *d_merge_map, int64_t own_offset, int64_t pack_capacity,
                                         int32_t *d_meta, double *d_sizes, float *d_rows, int64_t *d_n_pack, void *stream) {
    Cache *c = reinterpret_cast<Cache *>(h);
    if (!c || !d_merge_map || own_offset < 0 || pack_capacity < 1 || !d_meta || !d_sizes || !d_n_pack) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t n_own = c->capacity;
    Scratch scr;
    SISO_TRY(scratch_reserve(c, pad256(sizeof(uint32_t) * (n_own + 1)) + 256, s, &scr));
    uint32_t *pos = scr.take<uint32_t>(n_own + 1);
    pack_flags_kernel<<<static_cast<unsigned>((n_own + 1 + 255) / 256), 256, 0, s>>>(d_merge_map, own_offset, n_own, c->valid, pos);
    SISO_LAUNCHED(c);
    SISO_TRY(launch_exclusive_scan_u32(c, pos, n_own + 1, s));
    SISO_CUDA(cudaMemsetAsync(d_meta, 0xFF, sizeof(int32_t) * 2 * pack_capacity, s));        // unused places: slot -1
    pack_rows_kernel<<<static_cast<unsigned>(n_own), 128, 0, s>>>(d_merge_map, own_offset, n_own, c->valid, pos, c->master, c->size, c->dim,
                                                                pack_capacity, d_meta, d_sizes, d_rows,
                                                                reinterpret_cast<long long *>(d_n_pack), c->status);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

extern "C" siso_status_t siso_merge_apply_shard(siso_cache_t *h, const int32_t *d_merge_map, int64_t own_offset, const int32_t *d_meta,
                                                const double *d_sizes, const float *d_rows, int64_t n_places, uint32_t flags,
                                                void *stream) {
    Cache *c = reinterpret_cast<Cache *>(h);
    if (!c || !d_merge_map || own_offset < 0 || n_places < 0 || (flags & ~SISO_MERGE_WEIGHTED_MEAN)) return SISO_ERR_INVALID_ARG;
    const int weighted = (flags & SISO_MERGE_WEIGHTED_MEAN) ? 1 : 0;
    if (n_places > 0 && (!d_meta || !d_sizes || (weighted && !d_rows))) return SISO_ERR_INVALID_ARG;
    SISO_CUDA(cudaSetDevice(c->device));
    c->low_dirty = true;
    c->vec_epoch += 1;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t n_own = c->capacity;
    if (n_places > 0) {
        const size_t smem = sizeof(double) * c->dim;
        if (c->dtype == SISO_F32)
            shard_apply_kernel<float><<<static_cast<unsigned>(n_places), 256, smem, s>>>(d_meta, d_sizes, d_rows, n_places, own_offset, n_own,
                                                                                         c->dim, weighted, c->master,
                                                                                         static_cast<float *>(c->vecs), c->size);
        else
            shard_apply_kernel<__nv_bfloat16><<<static_cast<unsigned>(n_places), 256, smem, s>>>(
                d_meta, d_sizes, d_rows, n_places, own_offset, n_own, c->dim, weighted, c->master,
                static_cast<__nv_bfloat16 *>(c->vecs), c->size);
        SISO_LAUNCHED(c);
    }
    shard_drop_kernel<<<static_cast<unsigned>((n_own + 255) / 256), 256, 0, s>>>(d_merge_map, own_offset, n_own, c->valid, c->counters);
    SISO_LAUNCHED(c);
    return SISO_OK;
}
