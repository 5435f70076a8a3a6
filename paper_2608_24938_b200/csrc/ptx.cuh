// Inline-PTX wrappers for sm_100a: mbarrier, TMA (cp.async.bulk.tensor), tcgen05 (UMMA + TMEM).
// Every wait is bounded: it returns false once a wall-clock limit passes or another thread
// of the CTA (or another CTA, through the status word) has already given up.
#pragma once
#include <cuda.h>
#include <stdint.h>

#include "common.cuh"

namespace exfold {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// ------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.b32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s per wait, far above any legitimate wait here

// Bounded wait. `abort_flag` is a CTA-local shared word set by whoever gives up first.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          DeviceStatus* st, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 0u) {
            if (*abort_flag) return false;
            if (((volatile int*)&st->code)[0] != 0) {
                *abort_flag = 1;
                return false;
            }
            uint64_t now = globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                report_timeout(st, where);
                return false;
            }
        }
    }
}

// ------------------------------------------------------------------ TMA
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
// 2-D tiled load, completion counted in bytes on `bar`. c0 = innermost (element) coordinate, which
// must be a multiple of 8 for 16-bit types; c1 = row coordinate (may be out of range: zero fill).
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(m), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* gptr) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(gptr));
}

// ------------------------------------------------------------------ tcgen05 / TMEM
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {  // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {  // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// One k-block of the main loop in a single instruction sequence: issue kGemmBK/16 K=16 MMAs on this stage's operands,
// with a poll of `next_full` (the NEXT stage's operands) before the last of them (descriptor low words advance by 32 bytes = 2 per MMA;
// `desc_hi` is the shared high word), commit to `empty`, and only then read the poll's predicate, so that the
// poll's round trip overlaps the MMA issue. Returns whether the next stage was already complete.
__device__ __forceinline__ bool umma_kblock_bf16(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                                 uint32_t idesc, uint32_t acc_first, uint64_t* empty,
                                                 uint64_t* next_full, uint32_t next_parity) {
    uint32_t ready;
    asm volatile(
        "{\n"
        ".reg .pred pr, pa;\n"
        ".reg .b64 da, db;\n"
        ".reg .b32 la, lb;\n"
        "setp.ne.b32 pa, %6, 0;\n"
        "mov.b64 da, {%2, %4};\n"
        "mov.b64 db, {%3, %4};\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%1], da, db, %5, pa;\n"
        "add.u32 la, %2, 2;\n"
        "add.u32 lb, %3, 2;\n"
        "mov.b64 da, {la, %4};\n"
        "mov.b64 db, {lb, %4};\n"
#if EXFOLD_BK != 64
        "mbarrier.try_wait.parity.shared::cta.b64 pr, [%8], %9;\n"
#endif
        "tcgen05.mma.cta_group::1.kind::f16 [%1], da, db, %5, 1;\n"
#if EXFOLD_BK == 64
        "add.u32 la, %2, 4;\n"
        "add.u32 lb, %3, 4;\n"
        "mov.b64 da, {la, %4};\n"
        "mov.b64 db, {lb, %4};\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%1], da, db, %5, 1;\n"
        "add.u32 la, %2, 6;\n"
        "add.u32 lb, %3, 6;\n"
        "mov.b64 da, {la, %4};\n"
        "mov.b64 db, {lb, %4};\n"
        "mbarrier.try_wait.parity.shared::cta.b64 pr, [%8], %9;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%1], da, db, %5, 1;\n"
#endif
        "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%7];\n"
        "selp.b32 %0, 1, 0, pr;\n"
        "}\n"
        : "=r"(ready)
        : "r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first), "r"(smem_u32(empty)),
          "r"(smem_u32(next_full)), "r"(next_parity)
        : "memory");
    return ready != 0;
}
// ------------------------------------------------------------------ CTA pairs (cta_group::2)
// A cluster of two CTAs issues MMAs that span both CTAs' tensor cores and tensor memory: each CTA stages its own
// 128 A rows and its half of B at the same shared-memory offsets, the leader (cluster rank 0) issues.
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;  // clears the CTA-rank bit of a shared::cluster address: CTA 0's copy
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {  // same warp in both CTAs
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {  // same warp in both CTAs
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// 2-D tiled load into this CTA's shared memory; the bytes are counted on the LEADER CTA's barrier at `bar`'s offset
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(m), "r"(smem_u32(bar) & kPeerBitMask), "r"(c0), "r"(c1)
        : "memory");
}
// Arrive on the barrier at `bar`'s offset in every CTA of `cta_mask` once the MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar, uint16_t cta_mask) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(smem_u32(bar)), "h"(cta_mask)
        : "memory");
}
// Arrive on the leader CTA's barrier at `bar`'s offset (from either CTA of the pair)
__device__ __forceinline__ void mbar_arrive_leader(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(smem_u32(bar) & kPeerBitMask) : "memory");
}
// The pair form of umma_kblock_bf16 (K = 64 per stage): four M256 MMAs over both CTAs, the commit frees the stage in
// both CTAs (`empty` at the same offset in each).
__device__ __forceinline__ bool umma_kblock_bf16_pair(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                                      uint32_t idesc, uint32_t acc_first, uint64_t* empty,
                                                      uint64_t* next_full, uint32_t next_parity) {
    uint32_t ready;
    const uint16_t both = 3;
    asm volatile(
        "{\n"
        ".reg .pred pr, pa;\n"
        ".reg .b64 da, db;\n"
        ".reg .b32 la, lb;\n"
        "setp.ne.b32 pa, %6, 0;\n"
        "mov.b64 da, {%2, %4};\n"
        "mov.b64 db, {%3, %4};\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], da, db, %5, pa;\n"
        "add.u32 la, %2, 2;\n"
        "add.u32 lb, %3, 2;\n"
        "mov.b64 da, {la, %4};\n"
        "mov.b64 db, {lb, %4};\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], da, db, %5, 1;\n"
        "add.u32 la, %2, 4;\n"
        "add.u32 lb, %3, 4;\n"
        "mov.b64 da, {la, %4};\n"
        "mov.b64 db, {lb, %4};\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], da, db, %5, 1;\n"
        "add.u32 la, %2, 6;\n"
        "add.u32 lb, %3, 6;\n"
        "mov.b64 da, {la, %4};\n"
        "mov.b64 db, {lb, %4};\n"
        "mbarrier.try_wait.parity.shared::cta.b64 pr, [%8], %9;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], da, db, %5, 1;\n"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%7], %10;\n"
        "selp.b32 %0, 1, 0, pr;\n"
        "}\n"
        : "=r"(ready)
        : "r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first), "r"(smem_u32(empty)),
          "r"(smem_u32(next_full)), "r"(next_parity), "h"(both)
        : "memory");
    return ready != 0;
}
// Arrive on `bar` once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// Warp-wide read of 32 lanes x 32 consecutive fp32 columns: thread l gets row (lane base + l).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor for a K-major bf16 tile stored as rows of kGemmBK elements (128 or 64 bytes)
// with the swizzle TMA applies (SWIZZLE_128B / SWIZZLE_64B): 8-row groups are 8 rows apart (1024 / 512 bytes).
// The tile base must be aligned to that group size. Advancing by 16 elements along K adds 32 bytes (>>4 = 2)
// to the start-address field.
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
    constexpr uint32_t group_bytes = 8u * kGemmBK * 2u;
    uint64_t desc = 0;
    desc |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);   // start address, bits [0,14)
    desc |= (uint64_t)0 << 16;                         // leading byte offset: unused for swizzled K-major
    desc |= (uint64_t)(group_bytes >> 4) << 32;        // stride byte offset between 8-row groups
    desc |= (uint64_t)1 << 46;                         // descriptor version for sm_100
    desc |= (uint64_t)(kGemmBK == 64 ? 2 : 4) << 61;   // layout type: SWIZZLE_128B = 2, SWIZZLE_64B = 4
    return desc;
}

// Instruction descriptor: D fp32, A and B bf16, both K-major, shape M x N (K is 16 per instruction).
__device__ __host__ constexpr uint32_t make_idesc_bf16(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

}  // namespace ptx

}  // namespace exfold
