// MergeCentroids (Algorithm 1) over the cache itself, in ascending slot order.
//
//   sweep    blocked pairwise similarity of the fp32 master vectors (lower triangle only); every
//            pair (i, j), j < i, with similarity > theta_c becomes a candidate record
//   group    candidates are grouped by row i (count, scan, scatter)
//   resolve  entry i joins the most similar SURVIVOR among its candidates (ties: lowest slot), else
//            survives.  Whether j survives is known once all of j's own candidates are decided, so
//            one CTA iterates rounds until every row is decided; each decision is final and equals
//            the sequential algorithm's, whatever the timing of the rounds
//   apply    merged entries are grouped by survivor with a stable sort; each survivor adds the
//            members' cluster_size in ascending slot order and, in weighted-mean mode, becomes
//            normalise(sum of cluster_size * vector over itself and its members)
// The similarity used is that of the vectors as they were when the call began: nothing is written
// before the sweep has finished.  If the candidates do not fit their buffer the status word gets
// SISO_ERR_OVERFLOW and every later kernel of the call returns without writing.
#include <cooperative_groups.h>

#include "sweep_simt.cuh"

namespace siso {

using namespace sweep;

struct Candidate {
    int32_t i, j;
    float sim;
};

struct MergeCtl {
    unsigned long long n_cand;   // candidates found (may exceed the buffer: overflow)
    int overflow;
    int n_merged;
};

// grid = (tile pairs of the lower triangle incl. diagonal).  blockIdx.x -> (ti, tj), tj <= ti.
__global__ void __launch_bounds__(THREADS, 2)
merge_sweep_kernel(const float *__restrict__ C, const uint8_t *__restrict__ valid, const uint8_t *__restrict__ seed,
                   int64_t N, int D, float theta, MergeCtl *ctl, Candidate *__restrict__ cand,
                   unsigned long long max_cand, uint32_t *__restrict__ row_count) {
    extern __shared__ __align__(16) float smem[];
    __shared__ uint8_t valid_i[BM], valid_j[BN];     // bit 0: live, bit 1: member of C_cur (two-set mode)
    if (ctl->overflow) return;
    const long long p = blockIdx.x;
    long long ti, tj;
    if (seed) {                                       // two sets: the whole matrix of tiles
        const long long tiles = (N + BM - 1) / BM;
        ti = p / tiles;
        tj = p - ti * tiles;
    } else {                                          // one set: invert p = ti*(ti+1)/2 + tj
        ti = static_cast<long long>((sqrt(8.0 * static_cast<double>(p) + 1.0) - 1.0) * 0.5);
        while (ti * (ti + 1) / 2 > p) --ti;
        while ((ti + 1) * (ti + 2) / 2 <= p) ++ti;
        tj = p - ti * (ti + 1) / 2;
    }
    const int64_t i0 = ti * BM, j0 = tj * BN;
    const int tid = threadIdx.x;
    tile_to_smem<float>(C, N, i0, C, N, j0, D, smem);
    if (tid < BM) {
        const int64_t g = i0 + tid;
        valid_i[tid] = g < N ? ((valid[g] ? 1 : 0) | ((seed && seed[g]) ? 2 : 0)) : 0;
    } else if (tid < BM + BN) {
        const int64_t g = j0 + tid - BM;
        valid_j[tid - BM] = g < N ? ((valid[g] ? 1 : 0) | ((seed && seed[g]) ? 2 : 0)) : 0;
    }
    __syncthreads();
    const int row = tid >> 1, par = tid & 1, lane = tid & 31;
    const float *srow = smem + row * S_STRIDE;
    const int64_t gi = i0 + row;
    for (int it = 0; it < BN / 2; ++it) {
        const int cidx = par + 2 * it;
        const int64_t gj = j0 + cidx;
        const float v = srow[cidx];
        // entry i is compared with j if j comes before it in C_new: any member of C_cur, or an earlier entry of
        // the set being merged; members of C_cur are never rows
        const uint8_t fi = valid_i[row], fj = valid_j[cidx];
        const bool take = (fi & 1) && !(fi & 2) && (fj & 1) && ((fj & 2) || gj < gi) && gi != gj && v > theta;
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, take);
        if (ballot) {
            unsigned long long base = 0;
            if (lane == 0) base = atomicAdd(&ctl->n_cand, static_cast<unsigned long long>(__popc(ballot)));
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            if (take) {
                const unsigned long long pos = base + __popc(ballot & ((1u << lane) - 1u));
                if (pos < max_cand) {
                    Candidate cd;
                    cd.i = static_cast<int32_t>(gi); cd.j = static_cast<int32_t>(gj); cd.sim = v;
                    cand[pos] = cd;
                    atomicAdd(&row_count[gi], 1u);
                } else {
                    ctl->overflow = 1;
                }
            }
        }
    }
}

__global__ void merge_check_kernel(MergeCtl *ctl, int *status) {
    if (ctl->overflow == 1) set_status(status, SISO_ERR_OVERFLOW);     // 2 = insertion failed: status already set
}

// in: row_off = exclusive scan of row_count.  Scatter candidates into row-grouped order.
__global__ void merge_scatter_kernel(const MergeCtl *ctl, const Candidate *__restrict__ cand,
                                     const uint32_t *__restrict__ row_off, uint32_t *__restrict__ row_cursor,
                                     int32_t *__restrict__ csr_j, float *__restrict__ csr_sim) {
    if (ctl->overflow) return;
    const unsigned long long n = ctl->n_cand;        // no overflow here, so every one of them is in the buffer
    for (unsigned long long e = static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x; e < n;
         e += static_cast<unsigned long long>(gridDim.x) * blockDim.x) {
        const Candidate cd = cand[e];
        if (cd.i < 0) continue;          // a pair the tensor-core filter proposed and the exact check rejected
        const uint32_t pos = row_off[cd.i] + atomicAdd(&row_cursor[cd.i], 1u);
        csr_j[pos] = cd.j;
        csr_sim[pos] = cd.sim;
    }
}

// state: 0 undecided, 1 survivor, 2 merged, 3 empty slot
__global__ void __launch_bounds__(1024)
merge_resolve_kernel(MergeCtl *ctl, int64_t N, const uint8_t *__restrict__ valid, const uint8_t *__restrict__ seed,
                     const uint32_t *__restrict__ row_off,
                     const uint32_t *__restrict__ row_count, const int32_t *__restrict__ csr_j,
                     const float *__restrict__ csr_sim, volatile uint8_t *state, int32_t *__restrict__ target) {
    if (ctl->overflow) return;
    __shared__ int undecided_s;
    const int tid = threadIdx.x;
    for (int64_t i = tid; i < N; i += 1024) {
        state[i] = valid[i] ? (row_count[i] == 0 ? 1 : 0) : 3;
        target[i] = valid[i] ? static_cast<int32_t>(i) : -1;
    }
    __threadfence_block();
    __syncthreads();
    // every round decides at least the lowest undecided row, so at most N rounds are needed
    for (int64_t round = 0; round <= N; ++round) {
        if (tid == 0) undecided_s = 0;
        __syncthreads();
        int left = 0;
        for (int64_t i = tid; i < N; i += 1024) {
            if (state[i] != 0) continue;
            const uint32_t o = row_off[i], cnt = row_count[i];
            bool ready = true;
            unsigned long long best = 0ull;
            for (uint32_t e = 0; e < cnt; ++e) {
                const int32_t j = csr_j[o + e];
                const uint8_t sj = state[j];
                if (sj == 0) { ready = false; break; }
                if (sj == 1) {
                    // ties go to the earliest entry of C_new: members of C_cur first, then by slot
                    const uint32_t order = static_cast<uint32_t>(j) | ((seed && seed[j]) ? 0u : 0x80000000u);
                    const unsigned long long key = pack_key(csr_sim[o + e], order);
                    best = key > best ? key : best;
                }
            }
            if (!ready) { ++left; continue; }
            if (best) { target[i] = key_slot(best) & 0x7FFFFFFF; state[i] = 2; }
            else state[i] = 1;
        }
        __threadfence_block();
        if (left) atomicAdd(&undecided_s, left);
        __syncthreads();
        const int any = undecided_s;
        __syncthreads();
        if (!any) break;
    }
}

// The same resolution spread over the whole GPU: a cooperative launch, one thread per row at a time, a grid-wide
// barrier per round.  A chain of k entries that each merge into the previous survivor needs k rounds; a round costs
// a barrier plus a few memory round trips instead of one CTA's walk over all rows.
namespace cgm = cooperative_groups;
constexpr int RESOLVE_LOOKS = 32;
__global__ void __launch_bounds__(256)
merge_resolve_grid_kernel(MergeCtl *ctl, int64_t N, const uint8_t *__restrict__ valid, const uint8_t *__restrict__ seed,
                          const uint32_t *__restrict__ row_off, const uint32_t *__restrict__ row_count,
                          const int32_t *__restrict__ csr_j, const float *__restrict__ csr_sim, volatile uint8_t *state,
                          int32_t *__restrict__ target, unsigned int *undecided /* [3], zeroed */) {
    cgm::grid_group grid = cgm::this_grid();
    if (ctl->overflow) return;                      // the same in every CTA
    __shared__ int warp_left[8];
    const int64_t first = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * 256;
    for (int64_t i = first; i < N; i += stride) {
        state[i] = valid[i] ? (row_count[i] == 0 ? 1 : 0) : 3;
        target[i] = valid[i] ? static_cast<int32_t>(i) : -1;
    }
    grid.sync();
    for (int64_t round = 0; round <= N; ++round) {
        int left = 0;
        // a row whose candidates are still undecided is looked at again a few times before the grid-wide barrier: the
        // rows it waits for are being decided by other threads in this very round, and another look costs a memory
        // round trip where a round costs a barrier as well (the outcome does not depend on who decides when)
        for (int look = 0; look < RESOLVE_LOOKS; ++look) {
        left = 0;
        for (int64_t i = first; i < N; i += stride) {
            if (state[i] != 0) continue;
            const uint32_t o = row_off[i], cnt = row_count[i];
            bool ready = true;
            unsigned long long best = 0ull;
            // eight candidates at a time, so that their loads are in flight together
            for (uint32_t e0 = 0; e0 < cnt && ready; e0 += 8) {
                int32_t j[8];
                uint8_t sj[8];
                float sv[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) j[u] = e0 + u < cnt ? csr_j[o + e0 + u] : -1;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    sj[u] = j[u] >= 0 ? state[j[u]] : 3;
                    sv[u] = j[u] >= 0 ? csr_sim[o + e0 + u] : 0.0f;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    if (sj[u] == 0) ready = false;
                    if (sj[u] == 1) {
                        const uint32_t order = static_cast<uint32_t>(j[u]) | ((seed && seed[j[u]]) ? 0u : 0x80000000u);
                        const unsigned long long key = pack_key(sv[u], order);
                        best = key > best ? key : best;
                    }
                }
            }
            if (!ready) { ++left; continue; }
            if (best) { target[i] = key_slot(best) & 0x7FFFFFFF; state[i] = 2; }
            else state[i] = 1;
        }
        if (left == 0) break;
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) left += __shfl_xor_sync(0xFFFFFFFFu, left, o);
        if ((threadIdx.x & 31) == 0) warp_left[threadIdx.x >> 5] = left;
        __syncthreads();
        if (threadIdx.x == 0) {
            int t = 0;
            for (int w = 0; w < 8; ++w) t += warp_left[w];
            if (t) atomicAdd(&undecided[round % 3], static_cast<unsigned int>(t));
            // the counter of the round after this one was last read two barriers ago
            if (blockIdx.x == 0) undecided[(round + 1) % 3] = 0;
        }
        grid.sync();
        const unsigned int any = *reinterpret_cast<volatile unsigned int *>(&undecided[round % 3]);
        if (!any) break;
    }
}

// keys for the grouping sort: survivor slot for merged rows, N (sorts last) otherwise
__global__ void merge_keys_kernel(const MergeCtl *ctl, int64_t N, const volatile uint8_t *state,
                                  const int32_t *__restrict__ target, uint32_t *__restrict__ keys,
                                  uint32_t *__restrict__ vals) {
    if (ctl->overflow) return;
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= N) return;
    keys[i] = state[i] == 2 ? static_cast<uint32_t>(target[i]) : static_cast<uint32_t>(N);
    vals[i] = static_cast<uint32_t>(i);
}

// One CTA per position of the sorted (survivor, member) list; the head of a group does the group.
template <typename T>
__global__ void __launch_bounds__(256)
merge_apply_kernel(MergeCtl *ctl, const uint32_t *__restrict__ keys, const uint32_t *__restrict__ members, int64_t N,
                   int D, int weighted, float *__restrict__ master, T *__restrict__ vecs, double *__restrict__ size,
                   uint8_t *__restrict__ valid) {
    if (ctl->overflow) return;
    extern __shared__ double acc[];
    __shared__ double red[8];
    const int64_t p = blockIdx.x;
    const uint32_t sv = keys[p];
    if (sv >= N) return;
    if (p > 0 && keys[p - 1] == sv) return;
    int64_t e = p;
    while (e < N && keys[e] == sv) ++e;
    const double own = size[sv];
    double total = own;
    for (int64_t t = p; t < e; ++t) total += size[members[t]];       // ascending member slot: fixed order
    if (weighted) {
        float *m = master + static_cast<int64_t>(sv) * D;
        for (int d = threadIdx.x; d < D; d += 256) acc[d] = own * static_cast<double>(m[d]);
        for (int64_t t = p; t < e; ++t) {
            const uint32_t mb = members[t];
            const double w = size[mb];
            const float *mv = master + static_cast<int64_t>(mb) * D;
            for (int d = threadIdx.x; d < D; d += 256) acc[d] += w * static_cast<double>(mv[d]);
        }
        double ss = 0.0;
        for (int d = threadIdx.x; d < D; d += 256) ss += acc[d] * acc[d];
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        double nn = 0.0;
        for (int w = 0; w < 8; ++w) nn += red[w];
        nn = sqrt(nn);
        T *v = vecs + static_cast<int64_t>(sv) * D;
        for (int d = threadIdx.x; d < D; d += 256) {
            const float f = static_cast<float>(acc[d] / nn);
            m[d] = f;
            if constexpr (sizeof(T) == 2) v[d] = __float2bfloat16_rn(f);
        }
    }
    __syncthreads();      // every read of member sizes is done before they could be reused
    if (threadIdx.x == 0) size[sv] = total;
    for (int64_t t = p + threadIdx.x; t < e; t += 256) valid[members[t]] = 0;
    if (threadIdx.x == 0) atomicAdd(&ctl->n_merged, static_cast<int>(e - p));
}

// two-set mode: the repository rows were inserted first; if that failed for lack of free slots the whole merge is off
__global__ void merge_begin_kernel(MergeCtl *ctl, const int32_t *__restrict__ repo_slots) {
    if (repo_slots[0] < 0) ctl->overflow = 2;
}

// two-set mode, candidate overflow: take the inserted repository rows out again so that nothing is modified
__global__ void merge_rollback_kernel(const MergeCtl *ctl, int64_t N, uint8_t *__restrict__ valid,
                                      const uint8_t *__restrict__ seed, long long n_repo, long long *counters) {
    if (ctl->overflow != 1) return;
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < N && valid[i] && !seed[i]) valid[i] = 0;
    if (i == 0) {
        counters[CNT_OCCUPANCY] -= n_repo;
        counters[CNT_INSERTS] -= n_repo;
    }
}

__global__ void merge_finish_kernel(MergeCtl *ctl, int64_t N, const int32_t *__restrict__ target,
                                    int32_t *__restrict__ merge_map, long long *counters, long long *n_merged_out) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (ctl->overflow) {
        if (i == 0 && n_merged_out) *n_merged_out = 0;
        return;
    }
    if (merge_map && i < N) merge_map[i] = target[i];
    if (i == 0) {
        counters[CNT_OCCUPANCY] -= ctl->n_merged;
        counters[CNT_MERGES] += ctl->n_merged;
        if (n_merged_out) *n_merged_out = ctl->n_merged;
    }
}

// Resolution of the candidate graph: state[i] = 1 survivor / 2 merged / 3 empty, target[i] = the survivor that i joins
// (itself for survivors, -1 for empty slots).  `ctl` is a MergeCtl (only its overflow flag is read).
siso_status_t launch_merge_resolve(Cache *c, void *ctl_v, int64_t N, const uint8_t *valid, const uint8_t *seed,
                                   const uint32_t *row_off, const uint32_t *row_count, const int32_t *csr_j,
                                   const float *csr_sim, uint8_t *state, int32_t *target, unsigned int *undecided,
                                   cudaStream_t s) {
    MergeCtl *ctl = static_cast<MergeCtl *>(ctl_v);
    if (c->merge_resolve_grid == 0) {
        int coop = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device) != cudaSuccess) coop = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, merge_resolve_grid_kernel, 256, 0) != cudaSuccess) {
            cudaGetLastError();
            per_sm = 0;
        }
        c->merge_resolve_grid = (coop && per_sm >= 1) ? c->sm_count * std::min(per_sm, 4) : -1;
    }
    if (c->merge_resolve_grid > 0) {
        SISO_CUDA(cudaMemsetAsync(undecided, 0, 3 * sizeof(unsigned int), s));
        const uint8_t *valid_p = valid;
        const uint8_t *seed_p = seed;
        int64_t n_arg = N;
        volatile uint8_t *state_p = state;
        void *args[] = {&ctl, &n_arg, &valid_p, &seed_p, &row_off, &row_count, &csr_j, &csr_sim, &state_p, &target, &undecided};
        const int grid = static_cast<int>(std::min<int64_t>(c->merge_resolve_grid, (N + 255) / 256));
        SISO_CUDA(cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(merge_resolve_grid_kernel), dim3(grid), dim3(256),
                                              args, 0, s));
        c->launches += 1;
    } else {
        merge_resolve_kernel<<<1, 1024, 0, s>>>(ctl, N, valid, seed, row_off, row_count, csr_j, csr_sim, state, target);
        SISO_LAUNCHED(c);
    }
    return SISO_OK;
}

// ---- resolution over candidates that were found elsewhere (a cache partitioned over several GPUs) ----------------
__global__ void merge_count_rows_kernel(const Candidate *__restrict__ cand, unsigned long long n, int64_t N,
                                        uint32_t *__restrict__ row_count, int *status) {
    for (unsigned long long e = static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x; e < n;
         e += static_cast<unsigned long long>(gridDim.x) * blockDim.x) {
        const Candidate cd = cand[e];
        if (cd.i < 0) continue;
        if (cd.i >= N || cd.j < 0 || cd.j >= cd.i) { set_status(status, SISO_ERR_INVALID_ARG); continue; }
        atomicAdd(&row_count[cd.i], 1u);
    }
}

__global__ void merge_map_out_kernel(int64_t N, const volatile uint8_t *state, const int32_t *__restrict__ target,
                                     int32_t *__restrict__ merge_map, unsigned long long *n_merged) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const bool merged = i < N && state[i] == 2;
    if (i < N) merge_map[i] = target[i];
    const unsigned ballot = __ballot_sync(0xFFFFFFFFu, merged);
    if (ballot && (threadIdx.x & 31) == 0) atomicAdd(n_merged, static_cast<unsigned long long>(__popc(ballot)));
}

// cand [n_cand]: records (i, j, similarity) with j < i over rows 0..N-1, i = -1 for unused places; valid [N].
// merge_map [N] receives, for every row, the survivor it joins (itself for survivors, -1 for empty rows), as the
// resolution inside siso_merge would give it; *d_n_merged the number of rows merged away.
siso_status_t launch_merge_resolve_global(Cache *c, const void *cand_v, int64_t n_cand, const uint8_t *valid, int64_t N,
                                          int32_t *merge_map, long long *d_n_merged, cudaStream_t s) {
    if (N >= (1ll << 31) - 1 || n_cand < 0) return SISO_ERR_UNSUPPORTED;
    const Candidate *cand = static_cast<const Candidate *>(cand_v);
    const size_t nc = static_cast<size_t>(std::max<int64_t>(n_cand, 1));
    Scratch scr;
    const size_t need = pad256(sizeof(MergeCtl)) + 3 * pad256(sizeof(uint32_t) * (N + 1)) + pad256(sizeof(int32_t) * nc) +
                        pad256(sizeof(float) * nc) + pad256(N) + pad256(sizeof(int32_t) * N) + 256 + 256;
    SISO_TRY(scratch_reserve(c, need, s, &scr));
    MergeCtl *ctl = scr.take<MergeCtl>(1);
    uint32_t *row_count = scr.take<uint32_t>(N + 1);
    uint32_t *row_off = scr.take<uint32_t>(N + 1);
    uint32_t *row_cursor = scr.take<uint32_t>(N + 1);
    int32_t *csr_j = scr.take<int32_t>(nc);
    float *csr_sim = scr.take<float>(nc);
    uint8_t *state = scr.take<uint8_t>(N);
    int32_t *target = scr.take<int32_t>(N);
    unsigned int *undecided = scr.take<unsigned int>(3);
    MergeCtl h = {};
    h.n_cand = static_cast<unsigned long long>(n_cand);
    SISO_CUDA(cudaMemcpyAsync(ctl, &h, sizeof(h), cudaMemcpyHostToDevice, s));      // pageable source: copied before the call returns
    SISO_CUDA(cudaMemsetAsync(row_count, 0, sizeof(uint32_t) * (N + 1), s));
    SISO_CUDA(cudaMemsetAsync(row_cursor, 0, sizeof(uint32_t) * (N + 1), s));
    SISO_CUDA(cudaMemsetAsync(d_n_merged, 0, sizeof(long long), s));
    if (n_cand > 0) {
        merge_count_rows_kernel<<<4 * c->sm_count, 256, 0, s>>>(cand, static_cast<unsigned long long>(n_cand), N, row_count, c->status);
        SISO_LAUNCHED(c);
    }
    SISO_CUDA(cudaMemcpyAsync(row_off, row_count, sizeof(uint32_t) * (N + 1), cudaMemcpyDeviceToDevice, s));
    SISO_TRY(launch_exclusive_scan_u32(c, row_off, N + 1, s));
    if (n_cand > 0) {
        merge_scatter_kernel<<<4 * c->sm_count, 256, 0, s>>>(ctl, cand, row_off, row_cursor, csr_j, csr_sim);
        SISO_LAUNCHED(c);
    }
    SISO_TRY(launch_merge_resolve(c, ctl, N, valid, nullptr, row_off, row_count, csr_j, csr_sim, state, target, undecided, s));
    merge_map_out_kernel<<<static_cast<unsigned>((N + 255) / 256), 256, 0, s>>>(N, state, target, merge_map,
                                                                               reinterpret_cast<unsigned long long *>(d_n_merged));
    SISO_LAUNCHED(c);
    return SISO_OK;
}

siso_status_t launch_merge(Cache *c, const void *repo, const double *repo_sizes, int64_t n_repo, float theta_c,
                           uint32_t flags, int32_t *merge_map, long long *d_n_merged, cudaStream_t s) {
    c->vec_epoch += 1;          // the vectors may change: derived copies (the split-bf16 parts) are stale
    const int64_t N = c->capacity;
    if (N >= (1ll << 31) - 1) return SISO_ERR_UNSUPPORTED;
    const int64_t tiles = (N + BM - 1) / BM;
    const bool two_sets = n_repo > 0;
    const int64_t pairs = two_sets ? tiles * tiles : tiles * (tiles + 1) / 2;
    if (pairs > 0x7FFFFFFFll) return SISO_ERR_UNSUPPORTED;
    const size_t max_cand = static_cast<size_t>(c->merge_max_cand);
    Scratch scr;
    // the tensor-core sweep pays off once the matrix of pairs is large; small caches take the CUDA-core sweep
    const bool tensor = c->merge_path == SISO_PATH_TENSOR || (c->merge_path == SISO_PATH_AUTO && N >= 4096);
    size_t need = (tensor ? merge_tensor_scratch_bytes(c) : 0) + pad256(sizeof(MergeCtl)) + pad256(sizeof(Candidate) * max_cand) + 3 * pad256(sizeof(uint32_t) * (N + 1)) +
                  pad256(sizeof(int32_t) * max_cand) + pad256(sizeof(float) * max_cand) + pad256(N) +
                  pad256(sizeof(int32_t) * N) + 4 * pad256(sizeof(uint32_t) * N) + sort_pairs_scratch_bytes(N) +
                  pad256(N) + pad256(sizeof(int32_t) * (n_repo + 1)) + 256;
    SISO_TRY(scratch_reserve(c, need, s, &scr));
    MergeCtl *ctl = scr.take<MergeCtl>(1);
    Candidate *cand = scr.take<Candidate>(max_cand);
    uint32_t *row_count = scr.take<uint32_t>(N + 1);
    uint32_t *row_off = scr.take<uint32_t>(N + 1);
    uint32_t *row_cursor = scr.take<uint32_t>(N + 1);
    int32_t *csr_j = scr.take<int32_t>(max_cand);
    float *csr_sim = scr.take<float>(max_cand);
    uint8_t *state = scr.take<uint8_t>(N);
    int32_t *target = scr.take<int32_t>(N);
    uint32_t *keys = scr.take<uint32_t>(N), *vals = scr.take<uint32_t>(N);
    uint32_t *keys2 = scr.take<uint32_t>(N), *vals2 = scr.take<uint32_t>(N);
    unsigned int *undecided = scr.take<unsigned int>(3);
    uint8_t *seed = nullptr;
    if (two_sets) {
        // C_cur = what is live now; the repository rows then take free slots (new entries: access_count = infinity).
        // The insertion borrows the low end of this scratch buffer, which is only initialised afterwards; the
        // mask and the slot list sit beyond what it touches.
        seed = scr.take<uint8_t>(N);
        int32_t *repo_slots = scr.take<int32_t>(n_repo + 1);
        SISO_CUDA(cudaMemcpyAsync(seed, c->valid, static_cast<size_t>(N), cudaMemcpyDeviceToDevice, s));
        SISO_TRY(launch_insert(c, repo, repo_sizes, nullptr, n_repo, repo_slots, s));
        SISO_CUDA(cudaMemsetAsync(ctl, 0, sizeof(MergeCtl), s));
        merge_begin_kernel<<<1, 1, 0, s>>>(ctl, repo_slots);
        SISO_LAUNCHED(c);
    } else {
        SISO_CUDA(cudaMemsetAsync(ctl, 0, sizeof(MergeCtl), s));
    }
    SISO_CUDA(cudaMemsetAsync(row_count, 0, sizeof(uint32_t) * (N + 1), s));
    SISO_CUDA(cudaMemsetAsync(row_cursor, 0, sizeof(uint32_t) * (N + 1), s));
    if (tensor) {
        SISO_TRY(launch_merge_sweep_tensor(c, &scr, seed, theta_c, ctl, cand, max_cand, row_count, s));
    } else {
        if (!c->merge_attr_set) {
            SISO_CUDA(cudaFuncSetAttribute(merge_sweep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
            c->merge_attr_set = true;
        }
        merge_sweep_kernel<<<static_cast<unsigned>(pairs), THREADS, SMEM_BYTES, s>>>(c->master, c->valid, seed, N, c->dim,
                                                                                    theta_c, ctl, cand, max_cand, row_count);
        SISO_LAUNCHED(c);
    }
    merge_check_kernel<<<1, 1, 0, s>>>(ctl, c->status);
    SISO_LAUNCHED(c);
    if (two_sets) {
        merge_rollback_kernel<<<static_cast<unsigned>((N + 255) / 256), 256, 0, s>>>(ctl, N, c->valid, seed, n_repo, c->counters);
        SISO_LAUNCHED(c);
    }
    SISO_CUDA(cudaMemcpyAsync(row_off, row_count, sizeof(uint32_t) * (N + 1), cudaMemcpyDeviceToDevice, s));
    SISO_TRY(launch_exclusive_scan_u32(c, row_off, N + 1, s));
    merge_scatter_kernel<<<4 * c->sm_count, 256, 0, s>>>(ctl, cand, row_off, row_cursor, csr_j, csr_sim);
    SISO_LAUNCHED(c);
    SISO_TRY(launch_merge_resolve(c, ctl, N, c->valid, seed, row_off, row_count, csr_j, csr_sim, state, target, undecided, s));
    const unsigned nblk = static_cast<unsigned>((N + 255) / 256);
    merge_keys_kernel<<<nblk, 256, 0, s>>>(ctl, N, state, target, keys, vals);
    SISO_LAUNCHED(c);
    int key_bits = 1;
    while ((1ll << key_bits) <= N) ++key_bits;
    uint32_t *ks, *vs;
    SISO_TRY(launch_sort_pairs(c, &scr, keys, vals, keys2, vals2, N, key_bits, &ks, &vs, s));
    const int weighted = (flags & SISO_MERGE_WEIGHTED_MEAN) ? 1 : 0;
    const size_t smem = sizeof(double) * c->dim;
    if (c->dtype == SISO_F32)
        merge_apply_kernel<float><<<static_cast<unsigned>(N), 256, smem, s>>>(ctl, ks, vs, N, c->dim, weighted, c->master,
                                                                              static_cast<float *>(c->vecs), c->size, c->valid);
    else
        merge_apply_kernel<__nv_bfloat16><<<static_cast<unsigned>(N), 256, smem, s>>>(
            ctl, ks, vs, N, c->dim, weighted, c->master, static_cast<__nv_bfloat16 *>(c->vecs), c->size, c->valid);
    SISO_LAUNCHED(c);
    merge_finish_kernel<<<nblk, 256, 0, s>>>(ctl, N, target, merge_map, c->counters, d_n_merged);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

}  // namespace siso
