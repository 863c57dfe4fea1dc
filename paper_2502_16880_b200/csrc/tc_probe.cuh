// Measurement aid: how fast can tcgen05.mma be issued and executed by a CTA pair?  The same instruction forms
// as head_tc_kernel (cta_group::2, kind::f16, M = 256, descriptors of K-major 128-byte-swizzled tiles) on zeroed
// shared memory, from one or two issuing threads, `per_commit` MMAs followed by one tcgen05.commit per round.
// Nothing is loaded and nothing is read back, so the time per round is what the issuing thread(s) and the
// tensor pipe cost by themselves: the floor under the mainloop of the tensor-core path.
#pragma once
#include "tc_prims.cuh"

namespace coral {

constexpr int kTcProbeOperandBytes = 96 * 1024;     // two 16 KiB A tiles, up to 32 KiB of B rows per CTA, zeroed

// grid = 2 * pairs CTAs of 128 threads in clusters of two.  out[0] = nanoseconds the first pair's first issuer
// spent issuing `rounds` rounds, out[1] = until its last MMA had completed.
__global__ void __launch_bounds__(128, 1) tc_issue_probe_kernel(int n, int per_commit, int rounds, int issuers,
                                                                unsigned long long* __restrict__ out, DeviceState* st) {
    extern __shared__ unsigned char probe_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(probe_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kTcProbeOperandBytes);     // [0..1] done, [2..3] per-round
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_ctarank();
    for (int i = threadIdx.x; i < kTcProbeOperandBytes / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (threadIdx.x == 0) {
        for (int s = 0; s < 4; ++s) mbar_init(smem_u32(&bars[s]), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTcTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (warp >= 1 && warp <= issuers && lane == 0 && rank == 0) {
        const int a = warp - 1;
        const uint32_t a_lo = tc_smem_desc_lo(smem_u32(smem)) + a * (kTcTileBytes >> 4);
        const uint32_t b_lo = tc_smem_desc_lo(smem_u32(smem)) + (2 * kTcTileBytes >> 4);
        const uint32_t idesc = tc_idesc(256, n);
        const uint32_t acc = tmem_base + a * 256;
        unsigned long long t0, t1, t2;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        for (int r = 0; r < rounds; ++r) {
            for (int k = 0; k < per_commit; ++k)
                tc_mma_pair(acc, a_lo + 2 * (k & 3), b_lo + 2 * (k & 3), idesc, (r | k) ? 1u : 0u);
            tc_commit_pair(smem_u32(&bars[2 + a]));          // nobody waits on it: the cost of the commit is the point
        }
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        tc_commit_pair(smem_u32(&bars[a]));
        tc_wait(smem_u32(&bars[a]), 0, abort_flag, st);
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t2));
        if (blockIdx.x == 0 && a == 0) { out[0] = t1 - t0; out[1] = t2 - t0; }
    }
    tc_fence_before();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols) : "memory");
    }
}

}  // namespace coral
