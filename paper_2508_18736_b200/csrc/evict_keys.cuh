// Eviction order as integer keys, shared by the eviction kernels (evict.cu) and the fused streaming-step
// maintenance kernel (stream_maint.cu).
#pragma once

#include "common.cuh"

namespace siso {

// (cluster_size, access_count, last_access, slot) as three 64-bit words whose lexicographic order is the
// eviction order of FilteringCentroids plus the tie-breaks; the fp64 cluster_size maps to an order-preserving
// unsigned integer.
struct Key3 {
    unsigned long long w0, w1, w2;
};
__device__ __forceinline__ bool key_less(const Key3 &a, const Key3 &b) {
    if (a.w0 != b.w0) return a.w0 < b.w0;
    if (a.w1 != b.w1) return a.w1 < b.w1;
    return a.w2 < b.w2;
}
__device__ __forceinline__ Key3 make_key(double size, uint32_t access, unsigned long long last, uint32_t slot) {
    const unsigned long long u = static_cast<unsigned long long>(__double_as_longlong(size));
    Key3 k;
    k.w0 = (u >> 63) ? ~u : (u | 0x8000000000000000ull);          // order-preserving for every finite double
    k.w1 = (static_cast<unsigned long long>(access) << 32) | (last >> 32);
    k.w2 = (last << 32) | slot;
    return k;
}

}  // namespace siso
