// Clustering of a set of vectors by community detection at the clustering threshold theta_C (Sec. 4.1: SISO-Cluster
// turns the logged query vectors into centroids with a cluster_size each).  The paper names the method only; the
// steps taken here:
//   neighbours   u ~ v if their cosine is strictly above theta_C (every vector is its own neighbour)
//   order        vectors are visited by neighbourhood size, largest first, ties by index
//   communities  a visited vector that belongs to no community founds one and takes every neighbour that belongs to
//                none; a vector that belongs to one already is passed over
// Written that way the procedure is sequential, but its outcome has a closed description: v founds a community exactly
// if none of its neighbours EARLIER in the visiting order founds one, and otherwise joins the earliest founder among
// its neighbours.  That is the dependency structure of MergeCentroids' resolution with "earlier in the visiting order"
// in place of "lower slot" and "earliest founder" in place of "most similar survivor", so the same kernels serve:
//   sweep     all pairs on the tensor cores (split-bf16 filter, exact fp64 check): merge_tensor.cu
//   degrees   neighbourhood sizes from the confirmed pairs; a stable radix sort by descending size gives the order
//   graph     for every vector the neighbours earlier in the order, as a CSR list whose "similarity" field holds
//             minus the neighbour's position in the order (the largest = the earliest)
//   resolve   the grid-wide resolution of merge.cu
//   output    label (centre of each vector), centres in founding order, sizes, and optionally the mean of each
//             community's members (ascending index, fp64) scaled to unit length (Sec. 3.1: the mean point of the group)
#include "common.cuh"

namespace siso {

namespace {

struct PairRec {           // layout of the sweep's candidate records
    int32_t i, j;
    float sim;
};
struct SweepCtl {          // layout of the sweep's control block
    unsigned long long n_cand;
    int overflow;
    int n_merged;
};

template <typename T>
__global__ void cluster_widen_kernel(const T *__restrict__ in, float *__restrict__ out, long long n) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) {
        if constexpr (sizeof(T) == 2) out[i] = __bfloat162float(in[i]);
        else out[i] = in[i];
    }
}

__global__ void cluster_fill_kernel(uint8_t *p, long long n, uint8_t v) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}

__global__ void cluster_check_kernel(const SweepCtl *ctl, int *status) {
    if (ctl->overflow) set_status(status, SISO_ERR_OVERFLOW);
}

// neighbourhood sizes (the vector itself not counted: it shifts every size by one and leaves the order alone)
__global__ void cluster_degree_kernel(const SweepCtl *ctl, const PairRec *__restrict__ cand, uint32_t *__restrict__ deg) {
    if (ctl->overflow) return;
    const unsigned long long n = ctl->n_cand;
    for (unsigned long long e = static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x; e < n;
         e += static_cast<unsigned long long>(gridDim.x) * blockDim.x) {
        const PairRec r = cand[e];
        if (r.i < 0) continue;
        atomicAdd(&deg[r.i], 1u);
        atomicAdd(&deg[r.j], 1u);
    }
}

__global__ void cluster_order_keys_kernel(const uint32_t *__restrict__ deg, int64_t n, uint32_t *__restrict__ keys,
                                          uint32_t *__restrict__ vals) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    keys[i] = static_cast<uint32_t>(n - 1) - deg[i];       // ascending key = descending size; the sort is stable
    vals[i] = static_cast<uint32_t>(i);
}

__global__ void cluster_rank_kernel(const uint32_t *__restrict__ sorted, int64_t n, uint32_t *__restrict__ rank) {
    const int64_t pos = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (pos < n) rank[sorted[pos]] = static_cast<uint32_t>(pos);
}

// pass 0: count, for the later vector of each pair, one earlier neighbour; pass 1: write it
template <int PASS>
__global__ void cluster_graph_kernel(const SweepCtl *ctl, const PairRec *__restrict__ cand, const uint32_t *__restrict__ rank,
                                     uint32_t *__restrict__ row_count, const uint32_t *__restrict__ row_off,
                                     uint32_t *__restrict__ row_cursor, int32_t *__restrict__ csr_j, float *__restrict__ csr_key) {
    if (ctl->overflow) return;
    const unsigned long long n = ctl->n_cand;
    for (unsigned long long e = static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x; e < n;
         e += static_cast<unsigned long long>(gridDim.x) * blockDim.x) {
        const PairRec r = cand[e];
        if (r.i < 0) continue;
        const bool i_later = rank[r.i] > rank[r.j];
        const int32_t later = i_later ? r.i : r.j, earlier = i_later ? r.j : r.i;
        if (PASS == 0) {
            atomicAdd(&row_count[later], 1u);
        } else {
            const uint32_t pos = row_off[later] + atomicAdd(&row_cursor[later], 1u);
            csr_j[pos] = earlier;
            csr_key[pos] = -static_cast<float>(rank[earlier]);      // exact below 2^24 vectors
        }
    }
}

// in visiting order: 1 where the vector founded a community
__global__ void cluster_founder_flags_kernel(const SweepCtl *ctl, const uint32_t *__restrict__ sorted, const uint8_t *__restrict__ state,
                                             int64_t n, uint32_t *__restrict__ flag) {
    const int64_t pos = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (pos > n) return;
    flag[pos] = (pos < n && !ctl->overflow && state[sorted[pos]] == 1) ? 1u : 0u;
}

// flag_scan = exclusive scan of the founder flags: the founder at position pos is community number flag_scan[pos]
__global__ void cluster_emit_kernel(const SweepCtl *ctl, const uint32_t *__restrict__ sorted, const uint8_t *__restrict__ state,
                                    const uint32_t *__restrict__ flag_scan, int64_t n, int32_t *__restrict__ centres,
                                    uint32_t *__restrict__ ordinal, long long *n_clusters) {
    const int64_t pos = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (pos == 0 && n_clusters) *n_clusters = ctl->overflow ? 0 : static_cast<long long>(flag_scan[n]);
    if (pos >= n || ctl->overflow) return;
    const uint32_t v = sorted[pos];
    if (state[v] == 1) {
        const uint32_t c = flag_scan[pos];
        if (centres) centres[c] = static_cast<int32_t>(v);
        ordinal[v] = c;
    }
}

__global__ void cluster_label_kernel(const SweepCtl *ctl, const int32_t *__restrict__ target, const uint32_t *__restrict__ ordinal,
                                     int64_t n, int32_t *__restrict__ label, uint32_t *__restrict__ member_count,
                                     uint32_t *__restrict__ keys, uint32_t *__restrict__ vals) {
    const int64_t v = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (v >= n || ctl->overflow) return;
    const int32_t centre = target[v];
    if (label) label[v] = centre;
    const uint32_t c = ordinal[centre];
    atomicAdd(&member_count[c], 1u);
    keys[v] = c;                      // members are grouped by community with a stable sort: ascending index inside
    vals[v] = static_cast<uint32_t>(v);
}

__global__ void cluster_sizes_kernel(const SweepCtl *ctl, const uint32_t *__restrict__ member_count, const uint32_t *__restrict__ flag_scan,
                                     int64_t n, double *__restrict__ sizes) {
    const int64_t c = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (ctl->overflow || c >= static_cast<int64_t>(flag_scan[n])) return;
    sizes[c] = static_cast<double>(member_count[c]);
}

// One CTA per community: mean of the members (fp64 sums in ascending index), scaled to unit length.
template <typename T>
__global__ void __launch_bounds__(256)
cluster_centroid_kernel(const SweepCtl *ctl, const uint32_t *__restrict__ flag_scan, int64_t n, const uint32_t *__restrict__ member_off,
                        const uint32_t *__restrict__ members, const float *__restrict__ X, int D, T *__restrict__ out) {
    extern __shared__ double acc[];
    __shared__ double red[8];
    if (ctl->overflow) return;
    const int64_t k = flag_scan[n];
    for (int64_t c = blockIdx.x; c < k; c += gridDim.x) {
        for (int d = threadIdx.x; d < D; d += 256) acc[d] = 0.0;
        const uint32_t lo = member_off[c], hi = member_off[c + 1];
        for (uint32_t t = lo; t < hi; ++t) {
            const float *row = X + static_cast<int64_t>(members[t]) * D;
            for (int d = threadIdx.x; d < D; d += 256) acc[d] += static_cast<double>(row[d]);
        }
        double ss = 0.0;
        for (int d = threadIdx.x; d < D; d += 256) ss += acc[d] * acc[d];
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        double nn = 0.0;
        for (int w = 0; w < 8; ++w) nn += red[w];
        nn = sqrt(nn);
        T *o = out + c * D;
        for (int d = threadIdx.x; d < D; d += 256) {
            const float f = static_cast<float>(acc[d] / nn);
            if constexpr (sizeof(T) == 2) o[d] = __float2bfloat16_rn(f);
            else o[d] = f;
        }
        __syncthreads();
    }
}

}  // namespace

siso_status_t launch_cluster(Cache *c, const void *vecs, int64_t n, float theta_c, int32_t *label, int32_t *centres,
                             double *sizes, void *centroids, long long *d_n_clusters, cudaStream_t s) {
    if (n >= (1ll << 24)) return SISO_ERR_UNSUPPORTED;       // positions in the order are held exactly in fp32
    const int D = c->dim;
    const size_t max_cand = static_cast<size_t>(std::max<int64_t>(c->merge_max_cand, 16 * n + (1ll << 20)));
    const size_t n1 = static_cast<size_t>(n) + 1;
    size_t need = pair_sweep_tensor_scratch_bytes(n, n, D) + pad256(sizeof(float) * n * D) + pad256(n) + pad256(sizeof(SweepCtl)) +
                  pad256(sizeof(PairRec) * max_cand) + 8 * pad256(sizeof(uint32_t) * n1) + pad256(sizeof(int32_t) * max_cand) +
                  pad256(sizeof(float) * max_cand) + pad256(n) + pad256(sizeof(int32_t) * n) + 6 * pad256(sizeof(uint32_t) * n1) +
                  2 * sort_pairs_scratch_bytes(n) + 4096;
    Scratch scr;
    SISO_TRY(scratch_reserve(c, need, s, &scr));
    const unsigned nblk = static_cast<unsigned>((n + 255) / 256), nblk1 = static_cast<unsigned>((n + 256) / 256);
    // fp32 copy of the vectors (the exact check and the centroids read it)
    const float *X;
    if (c->dtype == SISO_F32) {
        X = static_cast<const float *>(vecs);
    } else {
        float *xw = scr.take<float>(static_cast<size_t>(n) * D);
        const long long total = static_cast<long long>(n) * D;
        cluster_widen_kernel<__nv_bfloat16><<<static_cast<unsigned>((total + 255) / 256), 256, 0, s>>>(
            static_cast<const __nv_bfloat16 *>(vecs), xw, total);
        SISO_LAUNCHED(c);
        X = xw;
    }
    uint8_t *all_live = scr.take<uint8_t>(n);
    cluster_fill_kernel<<<nblk, 256, 0, s>>>(all_live, n, 1);
    SISO_LAUNCHED(c);
    SweepCtl *ctl = scr.take<SweepCtl>(1);
    PairRec *cand = scr.take<PairRec>(max_cand);
    uint32_t *deg = scr.take<uint32_t>(n1), *rank = scr.take<uint32_t>(n1);
    uint32_t *row_count = scr.take<uint32_t>(n1), *row_off = scr.take<uint32_t>(n1), *row_cursor = scr.take<uint32_t>(n1);
    uint32_t *flag = scr.take<uint32_t>(n1), *ordinal = scr.take<uint32_t>(n1), *member_count = scr.take<uint32_t>(n1);
    int32_t *csr_j = scr.take<int32_t>(max_cand);
    float *csr_key = scr.take<float>(max_cand);
    uint8_t *state = scr.take<uint8_t>(n);
    int32_t *target = scr.take<int32_t>(n);
    uint32_t *k1 = scr.take<uint32_t>(n1), *v1 = scr.take<uint32_t>(n1), *k2 = scr.take<uint32_t>(n1), *v2 = scr.take<uint32_t>(n1);
    uint32_t *k3 = scr.take<uint32_t>(n1), *v3 = scr.take<uint32_t>(n1);
    unsigned int *undecided = scr.take<unsigned int>(3);
    SISO_CUDA(cudaMemsetAsync(ctl, 0, sizeof(SweepCtl), s));
    SISO_CUDA(cudaMemsetAsync(deg, 0, sizeof(uint32_t) * n1, s));
    SISO_CUDA(cudaMemsetAsync(row_count, 0, sizeof(uint32_t) * n1, s));
    SISO_CUDA(cudaMemsetAsync(row_cursor, 0, sizeof(uint32_t) * n1, s));
    SISO_CUDA(cudaMemsetAsync(member_count, 0, sizeof(uint32_t) * n1, s));

    // all pairs j < i above the threshold
    SISO_TRY(launch_pair_sweep_tensor(c, &scr, X, n, n, all_live, nullptr, theta_c, ctl, cand, max_cand, nullptr, s,
                                      c->dtype == SISO_BF16 ? vecs : nullptr));
    cluster_check_kernel<<<1, 1, 0, s>>>(ctl, c->status);
    SISO_LAUNCHED(c);
    // visiting order
    const unsigned wide = 4 * c->sm_count;
    cluster_degree_kernel<<<wide, 256, 0, s>>>(ctl, cand, deg);
    SISO_LAUNCHED(c);
    cluster_order_keys_kernel<<<nblk, 256, 0, s>>>(deg, n, k1, v1);
    SISO_LAUNCHED(c);
    int key_bits = 1;
    while ((1ll << key_bits) <= n) ++key_bits;
    uint32_t *ks, *sorted;
    SISO_TRY(launch_sort_pairs(c, &scr, k1, v1, k2, v2, n, key_bits, &ks, &sorted, s));
    cluster_rank_kernel<<<nblk, 256, 0, s>>>(sorted, n, rank);
    SISO_LAUNCHED(c);
    // earlier neighbours of every vector
    cluster_graph_kernel<0><<<wide, 256, 0, s>>>(ctl, cand, rank, row_count, nullptr, nullptr, nullptr, nullptr);
    SISO_LAUNCHED(c);
    SISO_CUDA(cudaMemcpyAsync(row_off, row_count, sizeof(uint32_t) * n1, cudaMemcpyDeviceToDevice, s));
    SISO_TRY(launch_exclusive_scan_u32(c, row_off, static_cast<int64_t>(n1), s));
    cluster_graph_kernel<1><<<wide, 256, 0, s>>>(ctl, cand, rank, row_count, row_off, row_cursor, csr_j, csr_key);
    SISO_LAUNCHED(c);
    // founders and members
    SISO_TRY(launch_merge_resolve(c, ctl, n, all_live, nullptr, row_off, row_count, csr_j, csr_key, state, target, undecided, s));
    cluster_founder_flags_kernel<<<nblk1, 256, 0, s>>>(ctl, sorted, state, n, flag);
    SISO_LAUNCHED(c);
    SISO_TRY(launch_exclusive_scan_u32(c, flag, static_cast<int64_t>(n1), s));
    cluster_emit_kernel<<<nblk, 256, 0, s>>>(ctl, sorted, state, flag, n, centres, ordinal, d_n_clusters);
    SISO_LAUNCHED(c);
    // the sort above may have left its result in k1/v1 or k2/v2; the member grouping uses the third pair
    cluster_label_kernel<<<nblk, 256, 0, s>>>(ctl, target, ordinal, n, label, member_count, k3, v3);
    SISO_LAUNCHED(c);
    if (sizes) {
        cluster_sizes_kernel<<<nblk, 256, 0, s>>>(ctl, member_count, flag, n, sizes);
        SISO_LAUNCHED(c);
    }
    if (centroids) {
        uint32_t *kt = (sorted == v1) ? k2 : k1, *vt = (sorted == v1) ? v2 : v1;      // the pair the order does not live in
        uint32_t *gk, *members;
        SISO_TRY(launch_sort_pairs(c, &scr, k3, v3, kt, vt, n, key_bits, &gk, &members, s));
        SISO_TRY(launch_exclusive_scan_u32(c, member_count, static_cast<int64_t>(n1), s));
        const size_t smem = sizeof(double) * D;
        const unsigned grid = static_cast<unsigned>(std::min<int64_t>(n, 8ll * c->sm_count));
        if (c->dtype == SISO_F32)
            cluster_centroid_kernel<float><<<grid, 256, smem, s>>>(ctl, flag, n, member_count, members, X, D, static_cast<float *>(centroids));
        else
            cluster_centroid_kernel<__nv_bfloat16><<<grid, 256, smem, s>>>(ctl, flag, n, member_count, members, X, D,
                                                                           static_cast<__nv_bfloat16 *>(centroids));
        SISO_LAUNCHED(c);
    }
    return SISO_OK;
}

}  // namespace siso
