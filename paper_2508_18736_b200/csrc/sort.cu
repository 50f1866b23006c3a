// Stable sort of (key, value) pairs of 32-bit integers.  It groups the hits of a batch by centroid
// with the query order kept inside each group, and the merged entries by surviving slot, so that
// every later floating-point sum is taken in one fixed order (bitwise reproducible results).
//   n <= SMALL_N : one CTA, rank by counting over packed 64-bit (key, position) words
//   otherwise    : least-significant-digit radix sort, 8 or 9 bits per pass (9 where that saves a pass: 17- and 18-bit
//                  keys, e.g. the slots of a 65,536-entry cache, sort in two passes), three kernels per pass
//                  (two up to 131,072 items: the scatter kernel then scans the small histogram itself)
#include "common.cuh"

namespace siso {

constexpr int SMALL_N = 2048;
constexpr int RS_THREADS = 256;
constexpr int RS_ITEMS = 4;                       // rounds per tile
constexpr int RS_TILE = RS_THREADS * RS_ITEMS;    // items per CTA
constexpr int RS_MAX_BINS = 512;                  // 9 bits
constexpr int RS_FUSED_TILES = 128;               // up to here the scatter kernel scans the histogram itself

__global__ void __launch_bounds__(1024)
sort_small_kernel(const uint32_t *__restrict__ keys, const uint32_t *__restrict__ vals, int n,
                  uint32_t *__restrict__ keys_out, uint32_t *__restrict__ vals_out) {
    __shared__ unsigned long long w[SMALL_N];
    for (int i = threadIdx.x; i < n; i += blockDim.x) w[i] = (static_cast<unsigned long long>(keys[i]) << 32) | (uint32_t)i;
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const unsigned long long mine = w[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (w[j] < mine) ? 1 : 0;
        keys_out[rank] = static_cast<uint32_t>(mine >> 32);
        vals_out[rank] = vals[i];
    }
}

// pass 1: per-tile digit histogram, stored digit-major for the scan kernel, hist[digit * n_tiles + tile], or tile-major,
// hist[tile * bins + digit], when the scatter kernel reads it raw (its threads then walk the tiles with coalesced loads)
__global__ void __launch_bounds__(RS_THREADS)
radix_hist_kernel(const uint32_t *__restrict__ keys, int64_t n, int shift, int bins, int n_tiles, int tile_major,
                  uint32_t *__restrict__ hist) {
    __shared__ uint32_t h[RS_MAX_BINS];
    const uint32_t mask = static_cast<uint32_t>(bins - 1);
    for (int d = threadIdx.x; d < bins; d += RS_THREADS) h[d] = 0;
    __syncthreads();
    const int64_t base = static_cast<int64_t>(blockIdx.x) * RS_TILE;
#pragma unroll
    for (int r = 0; r < RS_ITEMS; ++r) {
        const int64_t i = base + r * RS_THREADS + threadIdx.x;
        if (i < n) atomicAdd(&h[(keys[i] >> shift) & mask], 1u);
    }
    __syncthreads();
    for (int d = threadIdx.x; d < bins; d += RS_THREADS)
        hist[tile_major ? static_cast<int64_t>(blockIdx.x) * bins + d : static_cast<int64_t>(d) * n_tiles + blockIdx.x] = h[d];
}

// pass 2: exclusive scan of the histogram in place (one CTA; the array has bins * n_tiles entries).  A block of
// 1024 * SCAN_PER elements per trip: every warp owns a contiguous stretch of 32 * SCAN_PER elements, reads it with
// coalesced loads that are all in flight together, scans it with shuffles, and the warps' totals and the running total
// of the earlier blocks are added on the way out: one trip (two barriers) per 16,384 elements instead of per 1,024.
constexpr int SCAN_PER = 16;
__global__ void __launch_bounds__(1024) exclusive_scan_u32_kernel(uint32_t *__restrict__ a, int64_t n) {
    __shared__ uint32_t warp_sum[32];
    __shared__ uint32_t carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int64_t base = 0; base < n; base += 1024 * SCAN_PER) {
        const int64_t wbase = base + static_cast<int64_t>(warp) * 32 * SCAN_PER + lane;
        uint32_t v[SCAN_PER], incl[SCAN_PER];
#pragma unroll
        for (int u = 0; u < SCAN_PER; ++u) v[u] = wbase + u * 32 < n ? a[wbase + u * 32] : 0u;
        uint32_t run = 0;
#pragma unroll
        for (int u = 0; u < SCAN_PER; ++u) {
            uint32_t x = v[u];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o);
                if (lane >= o) x += y;
            }
            incl[u] = run + x;
            run += __shfl_sync(0xFFFFFFFFu, x, 31);
        }
        if (lane == 0) warp_sum[warp] = run;
        __syncthreads();
        if (warp == 0) {
            uint32_t s = warp_sum[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, s, o);
                if (lane >= o) s += y;
            }
            warp_sum[lane] = s;          // inclusive over warps
        }
        __syncthreads();
        const uint32_t carry = carry_s;
        const uint32_t before = carry + (warp ? warp_sum[warp - 1] : 0u);
#pragma unroll
        for (int u = 0; u < SCAN_PER; ++u)
            if (wbase + u * 32 < n) a[wbase + u * 32] = before + incl[u] - v[u];
        __syncthreads();
        if (tid == 0) carry_s = carry + warp_sum[31];
        __syncthreads();
    }
}

// pass 3: stable scatter.  Items of a tile are visited in 8 rounds of 256 in index order; inside a
// round the rank of an item among equal digits is (equal digits in earlier warps) + (in earlier lanes).
__global__ void __launch_bounds__(RS_THREADS)
radix_scatter_kernel(const uint32_t *__restrict__ keys, const uint32_t *__restrict__ vals, int64_t n, int shift, int bins,
                     int n_tiles, const uint32_t *__restrict__ hist_scanned, int raw_hist, uint32_t *__restrict__ keys_out,
                     uint32_t *__restrict__ vals_out) {
    __shared__ uint32_t base_s[RS_MAX_BINS];
    __shared__ uint32_t cnt_s[RS_THREADS / 32][RS_MAX_BINS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t mask = static_cast<uint32_t>(bins - 1);
    if (!raw_hist) {
        for (int d = tid; d < bins; d += RS_THREADS) base_s[d] = hist_scanned[static_cast<int64_t>(d) * n_tiles + blockIdx.x];
    } else {
        // few tiles: no scan kernel ran and the histogram is tile-major.  Every CTA works its bases out itself: thread t
        // takes digits t and t + 256, sums each digit's counts over all tiles (and over the tiles before its own) with
        // loads that are coalesced across the threads, and a block scan over the digit totals gives where each digit
        // starts (digits t < 256 first, then t + 256).
        __shared__ uint32_t warp_tot[2][RS_THREADS / 32];
        uint32_t tot[2] = {0u, 0u}, before[2] = {0u, 0u};
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int d = tid + j * RS_THREADS;
            if (d < bins) {
                // 32 loads in flight at a time: the sums wait for L2 once per 32 tiles, not once per tile
                for (int t0 = 0; t0 < n_tiles; t0 += 32) {
                    uint32_t v[32];
#pragma unroll
                    for (int u = 0; u < 32; ++u) v[u] = t0 + u < n_tiles ? __ldg(hist_scanned + static_cast<int64_t>(t0 + u) * bins + d) : 0u;
#pragma unroll
                    for (int u = 0; u < 32; ++u) {
                        tot[j] += v[u];
                        before[j] += t0 + u < static_cast<int>(blockIdx.x) ? v[u] : 0u;
                    }
                }
            }
        }
        uint32_t incl[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            uint32_t x = tot[j];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o);
                if (lane >= o) x += y;
            }
            incl[j] = x;
            if (lane == 31) warp_tot[j][warp] = x;
        }
        __syncthreads();
        uint32_t lower_half = 0;                                   // all digits below 256
        for (int w = 0; w < RS_THREADS / 32; ++w) lower_half += warp_tot[0][w];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int d = tid + j * RS_THREADS;
            uint32_t start = incl[j] - tot[j] + (j ? lower_half : 0u);
            for (int w = 0; w < warp; ++w) start += warp_tot[j][w];
            if (d < bins) base_s[d] = start + before[j];
        }
    }
    const int64_t base = static_cast<int64_t>(blockIdx.x) * RS_TILE;
    for (int r = 0; r < RS_ITEMS; ++r) {
        for (int d = tid; d < bins; d += RS_THREADS) {
#pragma unroll
            for (int w = 0; w < RS_THREADS / 32; ++w) cnt_s[w][d] = 0;
        }
        __syncthreads();
        const int64_t i = base + r * RS_THREADS + tid;
        const bool live = i < n;
        uint32_t key = 0, digit = static_cast<uint32_t>(bins + lane);     // dead lanes never match anything
        if (live) { key = keys[i]; digit = (key >> shift) & mask; }
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, digit);
        const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
        if (live && rank_in_warp == 0) cnt_s[warp][digit] = __popc(peers);
        __syncthreads();
        if (live) {
            uint32_t pos = base_s[digit] + rank_in_warp;
            for (int w = 0; w < warp; ++w) pos += cnt_s[w][digit];
            keys_out[pos] = key;
            vals_out[pos] = vals[i];
        }
        __syncthreads();
        for (int d = tid; d < bins; d += RS_THREADS) {
            uint32_t total = 0;
#pragma unroll
            for (int w = 0; w < RS_THREADS / 32; ++w) total += cnt_s[w][d];
            base_s[d] += total;
        }
        __syncthreads();
    }
}

siso_status_t launch_exclusive_scan_u32(Cache *c, uint32_t *a, int64_t n, cudaStream_t s) {
    exclusive_scan_u32_kernel<<<1, 1024, 0, s>>>(a, n);
    SISO_LAUNCHED(c);
    return SISO_OK;
}

size_t sort_pairs_scratch_bytes(int64_t n) {
    const int64_t n_tiles = (n + RS_TILE - 1) / RS_TILE;
    return pad256(sizeof(uint32_t) * RS_MAX_BINS * static_cast<size_t>(n_tiles > 0 ? n_tiles : 1));
}

// Sorts n pairs by the low key_bits of the key, stably.  The result lands either in the input
// arrays or in the *_tmp arrays; *keys_out / *vals_out say which.
siso_status_t launch_sort_pairs(Cache *c, Scratch *scr, uint32_t *keys, uint32_t *vals, uint32_t *keys_tmp,
                                uint32_t *vals_tmp, int64_t n, int key_bits, uint32_t **keys_out, uint32_t **vals_out,
                                cudaStream_t s) {
    if (n <= SMALL_N) {
        sort_small_kernel<<<1, 1024, 0, s>>>(keys, vals, static_cast<int>(n), keys_tmp, vals_tmp);
        SISO_LAUNCHED(c);
        *keys_out = keys_tmp;
        *vals_out = vals_tmp;
        return SISO_OK;
    }
    const int n_tiles = static_cast<int>((n + RS_TILE - 1) / RS_TILE);
    uint32_t *hist = scr->take<uint32_t>(RS_MAX_BINS * static_cast<size_t>(n_tiles));
    uint32_t *ka = keys, *va = vals, *kb = keys_tmp, *vb = vals_tmp;
    // 9-bit digits where they save a pass over 8-bit ones
    const int bits = (key_bits + 8) / 9 < (key_bits + 7) / 8 ? 9 : 8;
    const int bins = 1 << bits;
    for (int shift = 0; shift < key_bits; shift += bits) {
        radix_hist_kernel<<<n_tiles, RS_THREADS, 0, s>>>(ka, n, shift, bins, n_tiles, n_tiles <= RS_FUSED_TILES ? 1 : 0, hist);
        SISO_LAUNCHED(c);
        // up to 128 tiles (131,072 items) the scatter CTAs read the raw histogram themselves (256 KiB each, from L2):
        // cheaper than a one-CTA scan kernel and the launch around it
        const int raw_hist = n_tiles <= RS_FUSED_TILES ? 1 : 0;
        if (!raw_hist) {
            exclusive_scan_u32_kernel<<<1, 1024, 0, s>>>(hist, bins * static_cast<int64_t>(n_tiles));
            SISO_LAUNCHED(c);
        }
        radix_scatter_kernel<<<n_tiles, RS_THREADS, 0, s>>>(ka, va, n, shift, bins, n_tiles, hist, raw_hist, kb, vb);
        SISO_LAUNCHED(c);
        uint32_t *t = ka; ka = kb; kb = t;
        t = va; va = vb; vb = t;
    }
    *keys_out = ka;
    *vals_out = va;
    return SISO_OK;
}

}  // namespace siso
