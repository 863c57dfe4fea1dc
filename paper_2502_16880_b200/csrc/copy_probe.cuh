// Measurement aid: how fast can this GPU bring `chunks` x 16 KiB of the packed head into shared memory when
// nothing is done with them?  One thread per CTA issues contiguous 16 KiB bulk copies, `stages` in flight,
// chunk k of CTA b = b + k * grid (the CTAs sweep the buffer together); the region is swept `repeats` times
// (sweeps after the first find a region smaller than L2 still cached, so the difference between two repeat
// counts is the L2 -> shared-memory rate).  The time of this kernel for the bytes a draft call reads is the
// floor of that call's weight-streaming kernel: a one-shot read of a few hundred megabytes from a cold L2 does
// not reach the bandwidth of a long copy.
#pragma once
#include "common.cuh"
#include "head_stream.cuh"   // mbarrier and bulk-copy helpers

namespace coral {

constexpr int kCopyStages = 8;          // default number of copies in flight per SM
constexpr int kCopyMaxStages = 13;      // 13 x 16 KiB = 208 KiB of shared memory
constexpr int kCopyChunk = 16384;
constexpr int kCopySpin = 1 << 22;

__global__ void __launch_bounds__(32) copy_probe_kernel(const unsigned char* __restrict__ buf, long long chunks,
                                                        int stages, int repeats, DeviceState* state,
                                                        unsigned* __restrict__ sink) {
    extern __shared__ __align__(128) unsigned char copy_smem[];
    __shared__ uint64_t full[kCopyMaxStages];
    if (threadIdx.x != 0) return;
    for (int s = 0; s < stages; ++s) mbar_init(smem_u32(&full[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    long long mine = 0;
    for (long long cidx = blockIdx.x; cidx < chunks; cidx += gridDim.x) ++mine;
    const long long total = mine * repeats;
    long long issued = 0, done = 0;
    unsigned acc = 0;
    while (done < total) {
        while (issued < total && issued < done + stages) {
            const int s = (int)(issued % stages);
            const uint32_t bar = smem_u32(&full[s]);
            mbar_expect_tx(bar, kCopyChunk);
            bulk_g2s(smem_u32(copy_smem + s * kCopyChunk),
                     buf + ((long long)blockIdx.x + (issued % mine) * gridDim.x) * kCopyChunk, kCopyChunk, bar);
            ++issued;
        }
        const int s = (int)(done % stages);
        const uint32_t parity = (uint32_t)((done / stages) & 1);
        int spins = 0;
        while (!mbar_try_wait(smem_u32(&full[s]), parity)) {
            if (++spins > kCopySpin) {              // give up: report, let the copies in flight land, leave
                set_status(state, -5);
                for (long long d = done + 1; d < issued; ++d) {
                    const uint32_t b2 = smem_u32(&full[d % stages]);
                    for (int i = 0; i < (1 << 16) && !mbar_try_wait(b2, (uint32_t)((d / stages) & 1)); ++i) {}
                }
                return;
            }
        }
        acc += copy_smem[s * kCopyChunk];
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the read above before the slot's next bulk copy
        ++done;
    }
    sink[blockIdx.x] = acc;
}

// Failure-detection self-test: one warp polls, with the primitive every wait in the kernels is built on
// (mbarrier.try_wait under an iteration bound), a barrier that nothing will ever complete.  The bound runs
// out, the status word gets CORAL_ERR_TIMEOUT and the kernel returns normally: no trap, no endless loop, the
// context stays usable.  (A shorter bound than the kernels' own, so that the test takes milliseconds.)
constexpr int kSelfTestSpin = 1 << 14;
__global__ void __launch_bounds__(32) wait_expiry_kernel(DeviceState* state) {
    __shared__ uint64_t never;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&never), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    for (int i = 0; i < kSelfTestSpin; ++i)
        if (mbar_try_wait(smem_u32(&never), 0)) return;
    set_status(state, -5);
}

}  // namespace coral
