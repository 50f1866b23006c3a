// PTX wrappers of the tensor-core kernels: mbarriers with bounded waits, TMA tile loads, tcgen05 MMA and commit,
// tensor-memory loads, the shared-memory operand descriptor, and the epilogue's scan of one chunk of accumulator
// columns.  Two forms where they differ: one CTA drives a tile (cta_group::1), or two CTAs of a cluster drive one
// tile (cta_group::2: cluster addressing, loads that report to the leader CTA's barrier, commits that signal both
// CTAs, the M=256 MMA).  Shared by the lookup kernels (single CTA, CTA pair, fp32 split) and the merge sweep.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace siso {
namespace umma2 {

constexpr uint32_t SPIN_LIMIT = 4u << 20;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
// address of the same shared-memory location in CTA `rank` of the cluster (shared::cluster window)
__device__ __forceinline__ uint32_t cluster_addr(uint32_t local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_address) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_address) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// the same test with the default (CTA-scope) acquire: for barriers completed by this CTA's own asynchronous work
// (TMA bytes, tcgen05.commit), whose results the waiting thread does not read through generic loads of a peer's memory
__device__ __forceinline__ bool mbar_try_wait_cta(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if `limit` polls ran out (the flag is then set) or another role has already given up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint32_t limit = SPIN_LIMIT) {
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    *abort_flag = 1;
    return false;
}
// Bounded wait of a role that expects to wait long (an epilogue warp waiting for a whole tile): it sleeps between polls,
// so that it takes no issue slots from the MMA-issuing warp that shares its scheduler.  At most limit / 16 polls.
__device__ __forceinline__ bool mbar_wait_idle(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint32_t limit = SPIN_LIMIT) {
    for (uint32_t it = 0; it < limit / 16u; ++it) {
        if (mbar_try_wait_cta(bar, parity)) return true;
        __nanosleep(96);
        if ((it & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// this CTA's tile into its own shared memory; the bytes are reported to the barrier at `bar_cluster_addr`,
// which lives in the leader CTA
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *map, int c0, int c1, uint32_t bar_cluster_addr) {
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_cluster_addr)
                 : "memory");
}
// the same load with an L2 eviction policy (centroid tiles that no other cluster will read again)
__device__ __forceinline__ void tma_load_2d_pair_hint(void *dst, const CUtensorMap *map, int c0, int c1, uint32_t bar_cluster_addr,
                                                      uint64_t policy) {
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_cluster_addr), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Arrive, once all MMAs issued so far have completed, on the barrier at this shared-memory offset in BOTH
// CTAs of the pair (a commit that signals two barriers; no data is copied by it).
__device__ __forceinline__ void umma_commit_both(uint64_t *bar) {
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(both) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp receives row (lane base + i).  The load is
// asynchronous: the registers hold the data only after tmem_ld_fence() on the same array.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
// Wait for all tensor-memory loads issued so far.  The registers pass through the statement as in/out operands,
// so the compiler cannot schedule any use of them before the wait.
__device__ __forceinline__ void tmem_ld_fence(uint32_t (&r)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}
// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes and 128-byte swizzled
// (what the TMA writes): 8-row groups 1024 bytes apart; descriptor version 1; layout type 2 = 128B swizzle.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);          // start address, 16-byte units
    d |= static_cast<uint64_t>(1) << 16;                         // leading byte offset (unused for swizzled K-major)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                 // stride byte offset: 8 rows x 128 B
    d |= static_cast<uint64_t>(1) << 46;                         // descriptor version
    d |= static_cast<uint64_t>(2) << 61;                         // SWIZZLE_128B
    return d;
}

// ---- one CTA per tile ----------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(smem_u32(bar))
                 : "memory");
}
// the same load with an L2 eviction policy: used for centroid tiles that no other CTA will read again, so that the
// one-pass stream does not push the queries, the cache's metadata and the kernels' code out of L2
__device__ __forceinline__ void tma_load_2d_hint(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar, uint64_t policy) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(smem_u32(bar)), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}

// ---- epilogue of the lookup kernels ----------------------------------------------------------------------------
// One thread owns one query row: r holds 32 consecutive accumulator columns of that row (similarities of slots
// first_slot .. first_slot + 31), `live` says which of those slots hold an entry (the same for the whole warp).
// The columns are taken in groups of 4: a group is looked at value by value only if its maximum beats the row's
// k-th best.  A warp pays for that path when ANY of its 32 rows takes it, so small groups keep the common case
// (nothing to insert) down to 3 max operations and one comparison per group.  Insertion is in ascending slot order.
template <int KMAX>
__device__ __forceinline__ void scan_chunk32(uint32_t (&r)[32], uint32_t live, int first_slot, TopK<KMAX> &top) {
    if (live == 0u) return;
    if (live != 0xFFFFFFFFu) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if (!((live >> j) & 1u)) r[j] = 0xFF800000u;      // -inf: never enters a list
    }
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        float m = __uint_as_float(r[g * 4]);
#pragma unroll
        for (int j = 1; j < 4; ++j) m = fmaxf(m, __uint_as_float(r[g * 4 + j]));
        if (m > top.s[KMAX - 1]) {
#pragma unroll
            for (int j = 0; j < 4; ++j) top.push(__uint_as_float(r[g * 4 + j]), first_slot + g * 4 + j);
        }
    }
}

// Drains one finished accumulator of TN columns for this thread's row (tensor-memory address `taddr`): vflags bit ch
// says whether slot first_slot + 32 ch + lane holds an entry.  Two register buffers: while one chunk of 32 columns
// is scanned the next is in flight from tensor memory.  The loop stays rolled (two chunks per trip): unrolled eight
// times the scan code no longer fits the instruction cache.
template <int KMAX, int TN>
__device__ __forceinline__ void drain_accumulator(uint32_t taddr, unsigned long long vflags, int first_slot, TopK<KMAX> &top) {
    uint32_t ra[32], rb[32];
    tmem_ld_32x32(taddr, ra);
#pragma unroll 1
    for (int ch = 0; ch < TN / 32; ch += 2) {
        tmem_ld_fence(ra);
        tmem_ld_32x32(taddr + (ch + 1) * 32, rb);
        scan_chunk32<KMAX>(ra, __ballot_sync(0xFFFFFFFFu, ((vflags >> ch) & 1ull) != 0ull), first_slot + ch * 32, top);
        tmem_ld_fence(rb);
        if (ch + 2 < TN / 32) tmem_ld_32x32(taddr + (ch + 2) * 32, ra);
        scan_chunk32<KMAX>(rb, __ballot_sync(0xFFFFFFFFu, ((vflags >> (ch + 1)) & 1ull) != 0ull), first_slot + (ch + 1) * 32, top);
    }
}
}  // namespace umma2
}  // namespace siso
