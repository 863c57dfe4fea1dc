// Primitives of the 5th-generation tensor-core kernels (sm_100a): bounded mbarrier waits, L2 eviction
// policies, TMA tiled loads, shared-memory / instruction descriptors, tcgen05.mma / commit / ld wrappers for
// one CTA and for a CTA pair, and the few cluster-scope operations the pair kernels need.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "head_stream.cuh"   // mbarrier helpers

namespace coral {

constexpr int kTcEpilogueWarps = 8;
constexpr int kTcEpilogueThreads = kTcEpilogueWarps * 32;
constexpr int kTcThreads = (2 + kTcEpilogueWarps) * 32;   // warp 0 = producer, warp 1 = MMA issuer, 8 epilogue warps
constexpr int kTcSub = 128;          // rows of one operand tile / columns of one accumulator
constexpr int kTcK = 64;             // columns per stage (one 128-byte swizzle atom of bf16)
constexpr int kTcTileBytes = kTcSub * kTcK * 2;   // 16 KiB: one 128 x 64 bf16 operand tile
constexpr int kTcTmemCols = 512;
constexpr int kTcSpin = 1 << 22;     // bound of every wait

__device__ __forceinline__ void tc_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, DeviceState* st) {
    if (mbar_try_wait(bar, parity)) return;                  // the common case costs one instruction
    const int limit = *abort_flag ? 64 : kTcSpin;
    for (int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return;
    *abort_flag = 1;
    set_status(st, -5);
}

// L2 eviction policies for the operand loads: the weights of a group are streamed once per pass (evict first,
// unless a later pass reads them again), the gathered hidden rows are re-read for every batch of the entry
// (evict last), so the weight stream does not push them out of L2.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x0, int x1, uint32_t bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, "
        "%3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(x0), "r"(x1), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int x0, int x1, int x2, int x3,
                                            int x4, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, "
        "%3, %4, %5, %6}], [%7], %8;"
        ::"r"(dst), "l"(map), "r"(x0), "r"(x1), "r"(x2), "r"(x3), "r"(x4), "r"(bar), "l"(policy) : "memory");
}

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D = f32, A = B = bf16, both K-major, D of m x n (m rows over the CTAs of the
// instruction, n columns).
__host__ __device__ constexpr uint32_t tc_idesc(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
constexpr uint32_t kTcIdesc = tc_idesc(128, 128);

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kTcIdesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// ---- CTA pair (cluster of two CTAs, tcgen05 cta_group::2) ---------------------------------------------------
// One MMA of the pair spans both CTAs: rows 0..127 of A and of D belong to the CTA of rank 0, rows 128..255 to
// rank 1, and each CTA holds half of B's rows; the operands of both are read from the same shared-memory
// offsets.  The instruction is issued by one thread of the rank-0 CTA.
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address, in the cluster's shared window, of the location `addr` (a shared::cta address) in CTA `rank`.
__device__ __forceinline__ uint32_t cluster_map_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Arrive on a barrier of the other CTA.  What the arrival orders is work of the asynchronous units (a landed bulk
// copy, finished tensor-memory reads), not data written by this thread, so the barrier's default semantics
// are enough; cluster-scope release / acquire qualifiers here cost a memory fence per arrival and per wait.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// All threads of both CTAs.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The operands are given by the low words of their shared-memory descriptors (tc_smem_desc_lo); the high word
// is the same for every tile of this layout.  The single issuing thread is the pair's critical path, so the
// instruction stream per MMA is kept to the two register pairs and the instruction itself.
constexpr uint32_t kTcDescHi = 64u | (1u << 14) | (2u << 29);          // bits 32..63 of tc_smem_desc
__device__ __forceinline__ uint32_t tc_smem_desc_lo(uint32_t saddr) { return ((saddr >> 4) & 0x3FFFu) | (1u << 16); }
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint32_t adesc_lo, uint32_t bdesc_lo, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(adesc_lo), "r"(bdesc_lo), "r"(idesc), "r"(accumulate), "r"(kTcDescHi) : "memory");
}
// Arrives, once the pair's MMAs issued so far have completed, on the barrier at this shared-memory offset in
// both CTAs.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}

}  // namespace coral
