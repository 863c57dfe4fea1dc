// Router stage: gate scores, per-row top-n groups, rows bucketed by group.
// (CORAL Section 3.3: the router scores N groups and only the top-n are
// activated; Appendix B: with several candidate rows, the union of their
// groups is what has to be read.)
#pragma once
#include "common.cuh"

namespace coral {

constexpr int kGateRows = 8;       // query rows per gate block
constexpr int kGateThreads = 256;

// g[m][n] = W_gate[n] . h[m].  grid (N, ceil(M / kGateRows)); the block's
// threads split H, every thread accumulates its slice for up to 8 rows.
__global__ void __launch_bounds__(kGateThreads) gate_kernel(CallView c, float* __restrict__ gate_tap) {
    const int n = blockIdx.x;
    const int m0 = blockIdx.y * kGateRows;
    const int rows = min(kGateRows, c.M - m0);
    const int chunks = c.H >> 3;
    const uint4* __restrict__ wg = reinterpret_cast<const uint4*>(c.w_gate + (size_t)n * c.H);
    const uint4* __restrict__ hid = reinterpret_cast<const uint4*>(c.hidden + (size_t)m0 * c.H);
    float acc[kGateRows];
#pragma unroll
    for (int r = 0; r < kGateRows; ++r) acc[r] = 0.f;
    for (int ch = threadIdx.x; ch < chunks; ch += kGateThreads) {
        const uint4 w = __ldg(wg + ch);
#pragma unroll
        for (int r = 0; r < kGateRows; ++r) {
            if (r < rows) acc[r] = dot8(w, __ldg(hid + (size_t)r * chunks + ch), acc[r]);
        }
    }
    __shared__ float red[kGateThreads / 32][kGateRows];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int r = 0; r < kGateRows; ++r) {
        const float s = warp_sum(acc[r]);
        if (lane == 0) red[warp][r] = s;
    }
    __syncthreads();
    if (threadIdx.x < rows) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kGateThreads / 32; ++w) s += red[w][threadIdx.x];
        c.gate[(size_t)(m0 + threadIdx.x) * c.N + n] = s;
        if (gate_tap) gate_tap[(size_t)(m0 + threadIdx.x) * c.N + n] = s;
    }
}

// One warp per row: the k_groups best gate scores (descending, equal -> lower
// index), or the caller's forced groups.  Writes sel[m][*] and slot_of[m][*].
constexpr int kSelectWarps = 4;
__global__ void __launch_bounds__(kSelectWarps * 32) select_kernel(CallView c, const int32_t* __restrict__ forced,
                                                                   int32_t* __restrict__ groups_tap) {
    const int lane = threadIdx.x & 31;
    const int m = blockIdx.x * kSelectWarps + (threadIdx.x >> 5);
    if (m >= c.M) return;
    constexpr int kPer = kMaxGroups / 32;
    float val[kPer];
    int slot[kPer];
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int n = lane + 32 * i;
        val[i] = (n < c.N) ? c.gate[(size_t)m * c.N + n] : kNegInf;
        slot[i] = -1;
    }
    for (int s = 0; s < c.k_groups; ++s) {
        int pick;
        if (forced) {
            pick = forced[(size_t)m * c.k_groups + s];
            if (pick < 0 || pick >= c.N) {           // never index with it; report and fall back to group 0
                if (lane == 0) set_status(c.state, -6);
                pick = 0;
            }
        } else {
            float bv = kNegInf;
            int bk = kNoToken;
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                const int n = lane + 32 * i;
                if (n < c.N && slot[i] < 0 && better(val[i], n, bv, bk)) { bv = val[i]; bk = n; }
            }
            warp_argbest(bv, bk);
            pick = bk;
        }
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            if (lane + 32 * i == pick) {
                if (slot[i] >= 0) set_status(c.state, -6);   // a forced group named twice
                slot[i] = s;
            }
        }
        if (lane == 0) {
            c.sel[(size_t)m * c.k_groups + s] = pick;
            if (groups_tap) groups_tap[(size_t)m * c.k_groups + s] = pick;
        }
    }
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int n = lane + 32 * i;
        if (n < c.N) c.slot_of[(size_t)m * c.N + n] = (int16_t)slot[i];
    }
}

// One block.  Counting sort of the (row, slot) pairs by group: group_count,
// group_offset (exclusive scan), bucket_row / bucket_slot with the rows of each
// group in ascending order, and the union size.
constexpr int kBucketThreads = 1024;
__global__ void __launch_bounds__(kBucketThreads) bucket_kernel(CallView c) {
    __shared__ int s_count[kMaxGroups];
    __shared__ int s_offset[kMaxGroups + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kBucketThreads / 32;
    for (int n = warp; n < c.N; n += kWarps) {
        int cnt = 0;
        for (int m0 = 0; m0 < c.M; m0 += 32) {
            const int m = m0 + lane;
            const bool in = m < c.M && c.slot_of[(size_t)m * c.N + n] >= 0;
            cnt += __popc(__ballot_sync(0xffffffffu, in));
        }
        if (lane == 0) s_count[n] = cnt;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0, uni = 0, virt = 0;
        for (int n = 0; n < c.N; ++n) {
            s_offset[n] = run;
            run += s_count[n];
            if (c.union_rank) c.union_rank[n] = s_count[n] > 0 ? virt : -1;
            if (s_count[n] > 0) {
                const int passes = c.pass_rows > 0 ? (s_count[n] + c.pass_rows - 1) / c.pass_rows : 1;
                for (int p = 0; p < passes; ++p)
                    if (c.union_list && virt + p < c.union_cap) c.union_list[virt + p] = n | (p << 16);
                virt += passes;
                ++uni;
            }
        }
        s_offset[c.N] = run;
        c.state->n_union = uni;
        c.state->n_virtual = min(virt, c.union_cap);
    }
    __syncthreads();
    for (int n = threadIdx.x; n <= c.N; n += kBucketThreads) {
        c.group_offset[n] = s_offset[n];
        if (n < c.N) c.group_count[n] = s_count[n];
    }
    for (int n = warp; n < c.N; n += kWarps) {
        int pos = s_offset[n];
        for (int m0 = 0; m0 < c.M; m0 += 32) {
            const int m = m0 + lane;
            const int sl = (m < c.M) ? (int)c.slot_of[(size_t)m * c.N + n] : -1;
            const unsigned bal = __ballot_sync(0xffffffffu, sl >= 0);
            if (sl >= 0) {
                const int p = pos + __popc(bal & ((1u << lane) - 1u));
                c.bucket_row[p] = m;
                c.bucket_slot[p] = sl;
                if (c.bucket_pos) c.bucket_pos[(size_t)m * c.k_groups + sl] = p - s_offset[n];
            }
            pos += __popc(bal);
        }
    }
}

}  // namespace coral
