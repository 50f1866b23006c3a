/*
 * CPU oracle for the centroid semantic cache hot path (SISO, arXiv 2508.18736).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of what
 * the GPU library must compute.  It shares no code, header, table or helper with
 * the CUDA path and must never be called from it; only the tests, the smoke check
 * and the benchmark's CPU-baseline leg use it.
 *
 * Every routine widens its inputs (fp32 or bfloat16 bit patterns) to binary64
 * exactly and then works in binary64 with sums taken in index order.  OpenMP is
 * used only across independent outer iterations (queries; candidate survivors of
 * one FindClosestCentroid), never inside a sum.
 *
 * What follows which passage of the paper:
 *   lookup        FindClosestCentroid / CosineSimilarity of Algorithm 1 (closest =
 *                 largest cosine) and the retrieval threshold theta_R of Sec. 3.1,
 *                 which decides hit or miss; cosine = dot product because stored
 *                 centroids and queries are unit-norm by contract.
 *   update        the running-mean reading of Sec. 3.1, where a centroid is the mean
 *                 point of its group of vectors, plus the access_count
 *                 bookkeeping of Sec. 4.2 (merge step).
 *   merge         MergeCentroids of Algorithm 1, in the listed order.
 *   evict         FilteringCentroids of Algorithm 1: remove the smallest
 *                 (cluster_size, access_count) entry while over capacity, then
 *                 cluster_size /= 1.1 and access_count = 0 for the rest.
 *   cluster       the clustering step of Sec. 4.1 (community detection at theta_C); the
 *                 paper names the method without stating it, so the steps are a reading:
 *                 see siso_oracle_cluster.
 *   insert        the else-branch of MergeCentroids (new entry, access_count =
 *                 infinity) used for spare-space caching of individual vectors
 *                 (Sec. 5.2.5: left-over space holds single vectors under LRU).
 *
 * Readings taken where the paper is silent (ties to the lowest index, strict '>'
 * for both tests, (cluster_size, access_count, last_access, slot) as the full
 * eviction key, 0xFFFFFFFF as infinity with saturating adds) are listed in the
 * repository's design notes.
 *
 * Pins: tests/test_oracle_*.py check every routine against closed forms, the
 * hand-computed four-centroid example under tests/golden/, brute force written
 * independently in numpy, and invariants.  The streaming composition (lookup,
 * update, evict what the misses lack, insert per micro-batch) is pinned by a second
 * hand-computed example (two batches on a cache of four slots, every output and the
 * whole state after each batch) that five planted mistakes in the composition each
 * fail.  What no pin can fix are the hit ratios of a synthetic stream: the paper
 * prints none for such data ("parity unpinned" for those numbers only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1
#define ORACLE_F64 2
#define ACCESS_INF 0xFFFFFFFFu

static inline double widen(const void *p, int dtype, size_t i) {
    if (dtype == ORACLE_F32) return (double)((const float *)p)[i];
    if (dtype == ORACLE_F64) return ((const double *)p)[i];
    uint32_t u = ((uint32_t)((const uint16_t *)p)[i]) << 16; /* bfloat16 = top half of an fp32 */
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* dot product of row a of A with row b of B, summed in index order in binary64 */
static double dot_rows(const void *A, int a_dtype, size_t a, const void *B, int b_dtype, size_t b, int D) {
    double s = 0.0;
    size_t ao = a * (size_t)D, bo = b * (size_t)D;
    for (int d = 0; d < D; ++d) s += widen(A, a_dtype, ao + d) * widen(B, b_dtype, bo + d);
    return s;
}

/* ---------------------------------------------------------------------------
 * Round binary64 to bfloat16, one rounding, ties to even.  bfloat16 keeps 8
 * significant bits with the fp32 exponent range.
 * ------------------------------------------------------------------------- */
static uint16_t round_to_bf16(double x) {
    double r;
    if (x == 0.0 || isnan(x) || isinf(x)) {
        r = x;
    } else if (fabs(x) < ldexp(1.0, -126)) { /* subnormal range: fixed spacing 2^-133 */
        r = ldexp(rint(ldexp(x, 133)), -133);
    } else {
        int e;
        double m = frexp(x, &e);               /* x = m * 2^e, 0.5 <= |m| < 1 */
        r = ldexp(rint(ldexp(m, 8)), e - 8);   /* rint: current mode = nearest-even */
    }
    float f = (float)r;                        /* exact: every bfloat16 is an fp32 */
    uint32_t u;
    memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
}

void siso_oracle_round_bf16(const double *in, uint16_t *out, int64_t n) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = round_to_bf16(in[i]);
}

/* ---------------------------------------------------------------------------
 * O1  lookup: for each query the k most similar valid centroids, ordered by
 * (similarity descending, slot ascending); hit = best similarity > theta.
 * Fewer than k valid entries: idx = -1, sim = -inf in the tail.
 * ------------------------------------------------------------------------- */
int siso_oracle_lookup(const void *C, int c_dtype, const uint8_t *valid, int64_t N, int D,
                       const void *Q, int q_dtype, int64_t B, const float *theta, int k,
                       int32_t *idx, double *sim, uint8_t *hit) {
    if (k < 1 || D < 1 || N < 0 || B < 0) return 1;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t b = 0; b < B; ++b) {
        double *s = (double *)malloc(sizeof(double) * (size_t)(N > 0 ? N : 1));
        uint8_t *taken = (uint8_t *)calloc((size_t)(N > 0 ? N : 1), 1);
        if (!s || !taken) { fail = 1; free(s); free(taken); continue; }
        for (int64_t n = 0; n < N; ++n)
            if (!valid || valid[n]) s[n] = dot_rows(Q, q_dtype, (size_t)b, C, c_dtype, (size_t)n, D);
        for (int j = 0; j < k; ++j) {
            int64_t best = -1;
            for (int64_t n = 0; n < N; ++n) {
                if ((valid && !valid[n]) || taken[n]) continue;
                if (best < 0 || s[n] > s[best]) best = n; /* strict '>' keeps the lowest slot on ties */
            }
            if (best >= 0) {
                taken[best] = 1;
                idx[b * k + j] = (int32_t)best;
                sim[b * k + j] = s[best];
            } else {
                idx[b * k + j] = -1;
                sim[b * k + j] = -INFINITY;
            }
        }
        hit[b] = (idx[b * k] >= 0 && sim[b * k] > (double)theta[b]) ? 1 : 0;
        free(s);
        free(taken);
    }
    return fail;
}

/* ---------------------------------------------------------------------------
 * O2  hit update.  clock_now is the cache clock AFTER this call's increment.
 * For each slot j with hit set H_j (ascending query index):
 *     v = n_j * c_j + sum_{b in H_j} q_b ;  c_j = v / |v| ;  n_j += |H_j| ;
 *     access_j = min(inf, access_j + |H_j|) ;  last_j = clock_now.
 * All lookups of the batch saw the pre-batch cache, so the order of slots does
 * not matter; within a slot the queries are added in ascending b.
 * ------------------------------------------------------------------------- */
int siso_oracle_update(double *master, double *size, uint32_t *access, uint64_t *last, const uint8_t *valid,
                       int64_t N, int D, const void *Q, int q_dtype, int64_t B, const int32_t *idx,
                       int64_t idx_stride, const uint8_t *hit, uint64_t clock_now) {
    int64_t *count = (int64_t *)calloc((size_t)(N > 0 ? N : 1), sizeof(int64_t));
    if (!count) return 1;
    for (int64_t b = 0; b < B; ++b) {   /* reject bad input before touching anything */
        if (!hit[b]) continue;
        int64_t j = idx[b * idx_stride];
        if (j < 0 || j >= N || (valid && !valid[j])) { free(count); return 2; }
    }
    for (int64_t b = 0; b < B; ++b) {
        if (!hit[b]) continue;
        int64_t j = idx[b * idx_stride];
        double *c = master + (size_t)j * D;
        if (count[j] == 0)
            for (int d = 0; d < D; ++d) c[d] = size[j] * c[d];      /* v starts as n_j * c_j */
        for (int d = 0; d < D; ++d) c[d] += widen(Q, q_dtype, (size_t)b * D + d);
        count[j] += 1;
    }
    for (int64_t j = 0; j < N; ++j) {
        if (count[j] == 0) continue;
        double *c = master + (size_t)j * D;
        double nn = 0.0;
        for (int d = 0; d < D; ++d) nn += c[d] * c[d];
        nn = sqrt(nn);
        for (int d = 0; d < D; ++d) c[d] = c[d] / nn;
        size[j] += (double)count[j];
        uint64_t a = (uint64_t)access[j] + (uint64_t)count[j];
        access[j] = (access[j] == ACCESS_INF || a >= ACCESS_INF) ? ACCESS_INF : (uint32_t)a;
        last[j] = clock_now;
    }
    free(count);
    return 0;
}

/* ---------------------------------------------------------------------------
 * O3  MergeCentroids over one slot array.  Valid slots whose seed_mask is set form
 * C_cur: they are survivors unconditionally, are never compared with each other and
 * head the survivor list in ascending slot order.  The other valid slots are the
 * repository entries, taken in ascending slot
 * i: find the closest current survivor (largest dot product with the survivor's
 * vector AS IT WAS AT ENTRY; ties to the earliest survivor); if that similarity
 * is > theta_c the entry joins it (merge_map[i] = survivor, survivor's size grows
 * by the entry's size at entry, the entry's slot becomes invalid), otherwise the
 * entry becomes a survivor itself.  seed_mask = NULL is the self-merge of one set.
 * After the pass, with weighted_mean != 0, each survivor's vector becomes
 * normalise(size_s(entry)*c_s(entry) + sum over its other members m in ascending slot of
 * size_m(entry)*c_m(entry)); otherwise vectors are untouched.
 * new_access_inf != 0 sets access = infinity for surviving repository entries
 * (the else-branch of the algorithm); 0 leaves their counters as they are.
 * merge_map: -1 for invalid slots, own slot for survivors.  Returns #merged.
 * ------------------------------------------------------------------------- */
int64_t siso_oracle_merge(double *vec, double *size, uint32_t *access, uint8_t *valid, int64_t N, int D,
                          const uint8_t *seed_mask, double theta_c, int weighted_mean, int new_access_inf,
                          int32_t *merge_map) {
    int64_t *surv = (int64_t *)malloc(sizeof(int64_t) * (size_t)(N > 0 ? N : 1));
    double *s = (double *)malloc(sizeof(double) * (size_t)(N > 0 ? N : 1));
    double *size0 = (double *)malloc(sizeof(double) * (size_t)(N > 0 ? N : 1));
    if (!surv || !s || !size0) { free(surv); free(s); free(size0); return -1; }
    memcpy(size0, size, sizeof(double) * (size_t)N);
    int64_t n_surv = 0, n_merged = 0;
    for (int64_t i = 0; i < N; ++i)              /* C_new <- C_cur */
        if (valid[i] && seed_mask && seed_mask[i]) { merge_map[i] = (int32_t)i; surv[n_surv++] = i; }
    for (int64_t i = 0; i < N; ++i) {
        if (!valid[i]) { merge_map[i] = -1; continue; }
        if (seed_mask && seed_mask[i]) continue;
        /* FindClosestCentroid over the survivors so far; vec[] is not modified until the pass ends */
#pragma omp parallel for schedule(static)
        for (int64_t t = 0; t < n_surv; ++t) s[t] = dot_rows(vec, ORACLE_F64, (size_t)i, vec, ORACLE_F64, (size_t)surv[t], D);
        int64_t best = -1;
        for (int64_t t = 0; t < n_surv; ++t)
            if (best < 0 || s[t] > s[best]) best = t;
        if (best >= 0 && s[best] > theta_c) {
            merge_map[i] = (int32_t)surv[best];
            size[surv[best]] += size0[i];
            n_merged += 1;
        } else {
            merge_map[i] = (int32_t)i;
            surv[n_surv++] = i;
            if (new_access_inf) access[i] = ACCESS_INF;
        }
    }
    if (weighted_mean) {
        double *acc = (double *)malloc(sizeof(double) * (size_t)D);
        if (!acc) { free(surv); free(s); free(size0); return -1; }
        for (int64_t t = 0; t < n_surv; ++t) {
            int64_t sv = surv[t];
            int members = 0;
            for (int d = 0; d < D; ++d) acc[d] = size0[sv] * vec[(size_t)sv * D + d];
            members = 1;
            for (int64_t m = 0; m < N; ++m) {
                if (m == sv || !valid[m] || merge_map[m] != (int32_t)sv) continue;
                for (int d = 0; d < D; ++d) acc[d] += size0[m] * vec[(size_t)m * D + d];
                members += 1;
            }
            if (members > 1) {
                double nn = 0.0;
                for (int d = 0; d < D; ++d) nn += acc[d] * acc[d];
                nn = sqrt(nn);
                /* A survivor is a member of its own group only and merged rows are never written, so
                   storing the new vector now cannot change an input of a later group. */
                for (int d = 0; d < D; ++d) vec[(size_t)sv * D + d] = acc[d] / nn;
            }
        }
        free(acc);
    }
    for (int64_t i = 0; i < N; ++i)
        if (valid[i] && merge_map[i] != (int32_t)i) valid[i] = 0;
    free(surv);
    free(s);
    free(size0);
    return n_merged;
}

/* ---------------------------------------------------------------------------
 * O4  FilteringCentroids: n_evict times remove the valid entry that comes first
 * in ascending (cluster_size, access_count, last_access, slot) order, recording
 * it; then, if decay_flag, cluster_size = cluster_size / decay (binary64
 * division) and access_count = 0 for every remaining entry.
 * Removing the first element of a freshly sorted list is removing the minimum.
 * Returns the number actually evicted (less than n_evict if the cache empties).
 * ------------------------------------------------------------------------- */
static int key_less(const double *size, const uint32_t *access, const uint64_t *last, int64_t a, int64_t b) {
    if (size[a] != size[b]) return size[a] < size[b];
    if (access[a] != access[b]) return access[a] < access[b];
    if (last[a] != last[b]) return last[a] < last[b];
    return a < b;
}

int64_t siso_oracle_evict(double *size, uint32_t *access, const uint64_t *last, uint8_t *valid, int64_t N,
                          int64_t n_evict, int decay_flag, double decay, int32_t *victims) {
    int64_t done = 0;
    for (; done < n_evict; ++done) {
        int64_t first = -1;
        for (int64_t i = 0; i < N; ++i) {
            if (!valid[i]) continue;
            if (first < 0 || key_less(size, access, last, i, first)) first = i;
        }
        if (first < 0) break;
        valid[first] = 0;
        victims[done] = (int32_t)first;
    }
    for (int64_t r = done; r < n_evict; ++r) victims[r] = -1;
    if (decay_flag) {
        for (int64_t i = 0; i < N; ++i) {
            if (!valid[i]) continue;
            size[i] = size[i] / decay;
            access[i] = 0;
        }
    }
    return done;
}

/* ---------------------------------------------------------------------------
 * O5  insert: rows b with (hit == NULL or hit[b] == 0), in ascending b, take the
 * free slots in ascending slot order.  New entry: vector = the row's bits widened,
 * cluster_size = sizes_in[b] (1 if NULL), access = infinity, last = clock_now.
 * slots_out[b] = slot, or -1 for rows that are hits.  If there are fewer free
 * slots than rows to insert nothing is modified and -1 is returned; otherwise the
 * number inserted.
 * ------------------------------------------------------------------------- */
int64_t siso_oracle_insert(double *master, double *size, uint32_t *access, uint64_t *last, uint8_t *valid,
                           int64_t N, int D, const void *Q, int q_dtype, int64_t B, const uint8_t *hit,
                           const double *sizes_in, uint64_t clock_now, int32_t *slots_out) {
    int64_t want = 0, free_slots = 0;
    for (int64_t b = 0; b < B; ++b) want += (!hit || !hit[b]) ? 1 : 0;
    for (int64_t i = 0; i < N; ++i) free_slots += valid[i] ? 0 : 1;
    if (free_slots < want) return -1;
    int64_t slot = 0, n_ins = 0;
    for (int64_t b = 0; b < B; ++b) {
        if (hit && hit[b]) { slots_out[b] = -1; continue; }
        while (valid[slot]) ++slot;
        for (int d = 0; d < D; ++d) master[(size_t)slot * D + d] = widen(Q, q_dtype, (size_t)b * D + d);
        size[slot] = sizes_in ? sizes_in[b] : 1.0;
        access[slot] = ACCESS_INF;
        last[slot] = clock_now;
        valid[slot] = 1;
        slots_out[b] = (int32_t)slot;
        n_ins += 1;
    }
    return n_ins;
}

/* ---------------------------------------------------------------------------
 * Threshold control (Sec. 4.3, "Adjusting theta_R to meet SLO").
 *
 * T2H table: for each threshold of a grid, the hit ratio of a sample of queries,
 * h(theta) = #{queries whose best similarity > theta} / n  (the same strict test
 * as lookup).  best[] holds the best similarity of each sampled query.
 * ------------------------------------------------------------------------- */
void siso_oracle_t2h(const double *best, int64_t n, const float *thetas, int n_thetas, int64_t *hits, double *ratio) {
    for (int t = 0; t < n_thetas; ++t) {
        int64_t c = 0;
        for (int64_t i = 0; i < n; ++i) c += (best[i] > (double)thetas[t]) ? 1 : 0;
        hits[t] = c;
        ratio[t] = n > 0 ? (double)c / (double)n : 0.0;
    }
}

/* Eq. 1 with E = L (1 - h) (Eq. 2): mean waiting time of the M/D/1 queue,
 *     W = E + lambda E^2 / (2 (1 - lambda E)),
 * +infinity when the queue is not stable (lambda E >= 1). */
double siso_oracle_md1_wait(double L, double lambda, double h) {
    double E = L * (1.0 - h);
    double rho = lambda * E;
    if (rho >= 1.0) return INFINITY;
    return E + lambda * E * E / (2.0 * (1.0 - rho));
}

/* The highest threshold of the table whose estimated W is below the SLO S
 * ("find the highest theta_R ... that satisfies S > W").  Returns its index,
 * or -1 if no entry qualifies.  W of the chosen entry goes to *w_out. */
int siso_oracle_choose_theta(const float *thetas, const double *ratio, int n_thetas, double L, double lambda,
                             double slo, double *w_out) {
    int best = -1;
    for (int t = 0; t < n_thetas; ++t) {
        double W = siso_oracle_md1_wait(L, lambda, ratio[t]);
        if (W < slo && (best < 0 || thetas[t] > thetas[best])) best = t;
    }
    if (w_out) *w_out = best >= 0 ? siso_oracle_md1_wait(L, lambda, ratio[best]) : INFINITY;
    return best;
}

/* Correction step of Sec. 4.3: when the estimate W and the measured W' differ by more than 10 % (of W'), theta_R
 * moves one table entry further: down if W' is the longer (less traffic to the LLM), up if it is the shorter. */
int siso_oracle_correct_theta(const float *thetas, int n_thetas, int chosen, double w_est, double w_meas) {
    if (chosen < 0 || chosen >= n_thetas || !(w_meas > 0.0)) return chosen;
    if (fabs(w_est - w_meas) / w_meas <= 0.10) return chosen;
    int next = -1;
    for (int t = 0; t < n_thetas; ++t) {
        if (w_meas > w_est) {            /* next lower threshold */
            if (thetas[t] < thetas[chosen] && (next < 0 || thetas[t] > thetas[next])) next = t;
        } else {                          /* next higher threshold */
            if (thetas[t] > thetas[chosen] && (next < 0 || thetas[t] < thetas[next])) next = t;
        }
    }
    return next < 0 ? chosen : next;
}

/* ---------------------------------------------------------------------------
 * Clustering of Sec. 4.1: community detection at the clustering threshold
 * theta_C.  The paper only names the method; the reading taken here:
 *   - u and v are neighbours if their cosine (dot product of unit vectors, summed
 *     in index order in binary64) is strictly above theta_C; every vector is its
 *     own neighbour;
 *   - vectors are visited by neighbourhood size, largest first, ties by index;
 *   - a visited vector that belongs to no community yet founds one: it is the
 *     centre, and every neighbour that belongs to no community yet joins it;
 *     a visited vector that already belongs to a community is passed over.
 * So every vector ends in exactly one community (possibly alone), communities
 * are disjoint, and cluster_size is the number of members (Sec. 4.1: "the number
 * of vectors in the cluster").
 * Outputs: label[v] = index of the centre of v's community; centres[] in the order
 * they were founded; sizes[] alongside; if centroids != NULL, row c = the mean of
 * the members of community c (members added in ascending index) scaled to unit
 * length (Sec. 3.1: a centroid is the mean point of its group).  Returns the
 * number of communities.
 * ------------------------------------------------------------------------- */
typedef struct { int64_t degree; int64_t index; } visit_t;
static int visit_cmp(const void *a, const void *b) {
    const visit_t *x = (const visit_t *)a, *y = (const visit_t *)b;
    if (x->degree != y->degree) return x->degree > y->degree ? -1 : 1;
    return x->index < y->index ? -1 : (x->index > y->index ? 1 : 0);
}

int64_t siso_oracle_cluster(const void *V, int dtype, int64_t n, int D, double theta, int32_t *label,
                            int32_t *centres, double *sizes, double *centroids) {
    uint8_t *nb = (uint8_t *)calloc((size_t)n * (size_t)n, 1);   /* neighbour matrix */
    visit_t *order = (visit_t *)malloc(sizeof(visit_t) * (size_t)n);
    if (!nb || !order) { free(nb); free(order); return -1; }
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t u = 0; u < n; ++u)
        for (int64_t v = 0; v < n; ++v)
            nb[u * n + v] = (u == v) || (dot_rows(V, dtype, (size_t)u, V, dtype, (size_t)v, D) > theta);
    for (int64_t v = 0; v < n; ++v) {
        int64_t deg = 0;
        for (int64_t u = 0; u < n; ++u) deg += nb[v * n + u];    /* symmetric: both directions multiply and add alike */
        order[v].degree = deg;
        order[v].index = v;
        label[v] = -1;
    }
    qsort(order, (size_t)n, sizeof(visit_t), visit_cmp);
    int64_t n_comm = 0;
    for (int64_t k = 0; k < n; ++k) {
        const int64_t v = order[k].index;
        if (label[v] >= 0) continue;
        int64_t members = 0;
        for (int64_t u = 0; u < n; ++u)
            if (nb[v * n + u] && label[u] < 0) { label[u] = (int32_t)v; ++members; }
        centres[n_comm] = (int32_t)v;
        sizes[n_comm] = (double)members;
        ++n_comm;
    }
    if (centroids) {
        for (int64_t c = 0; c < n_comm; ++c) {
            double *row = centroids + (size_t)c * (size_t)D;
            for (int d = 0; d < D; ++d) row[d] = 0.0;
            for (int64_t u = 0; u < n; ++u)
                if (label[u] == centres[c])
                    for (int d = 0; d < D; ++d) row[d] += widen(V, dtype, (size_t)u * (size_t)D + (size_t)d);
            double ss = 0.0;
            for (int d = 0; d < D; ++d) ss += row[d] * row[d];
            const double norm = sqrt(ss);
            for (int d = 0; d < D; ++d) row[d] /= norm;
        }
    }
    free(nb);
    free(order);
    return n_comm;
}
