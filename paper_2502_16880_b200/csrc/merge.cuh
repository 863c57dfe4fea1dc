// Per-row merge of the tile partials: joint log-sum-exp over the row's active
// logits and the k_tokens best tokens (CORAL Section 3.3 softmax over the
// activated groups; Appendix B top candidates), emitted as log-probabilities
// sorted in descending order with equal values ordered by token id.
#pragma once
#include "common.cuh"

namespace coral {

constexpr int kMergeThreads = 128;

__global__ void __launch_bounds__(kMergeThreads) merge_kernel(CallView c, int32_t* __restrict__ out_ids,
                                                              float* __restrict__ out_logprobs,
                                                              float* __restrict__ lse_tap) {
    const int m = blockIdx.x;
    if (call_is_poisoned(c.state)) return;        // the partials were not written: emit nothing (the status says why)
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kMergeThreads / 32;
    __shared__ float s_f[kWarps];
    __shared__ int s_i[kWarps];
    __shared__ float s_lse;
    const int P = c.k_groups * c.T;
    const float* pmax = c.part_max + (size_t)m * P;
    const float* psum = c.part_sum + (size_t)m * P;

    float mx = kNegInf;
    for (int p = threadIdx.x; p < P; p += kMergeThreads) mx = fmaxf(mx, pmax[p]);
    mx = warp_max(mx);
    if (lane == 0) s_f[warp] = mx;
    __syncthreads();
    mx = s_f[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) mx = fmaxf(mx, s_f[w]);
    __syncthreads();
    float sum = 0.f;
    for (int p = threadIdx.x; p < P; p += kMergeThreads) sum += psum[p] * expf(pmax[p] - mx);
    sum = warp_sum(sum);
    if (lane == 0) s_f[warp] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot += s_f[w];
        s_lse = mx + logf(tot);
        if (lse_tap) lse_tap[m] = s_lse;
    }
    __syncthreads();
    const float lse = s_lse;

    // Token ids are unique across the candidates, so "strictly after the last
    // pick in (value desc, id asc) order" selects the next one without marking.
    const int C = P * c.k_tokens;
    const float* cval = c.part_val + (size_t)m * C;
    const int32_t* cid = c.part_id + (size_t)m * C;
    float last_v = __builtin_huge_valf();
    int last_id = -1;
    for (int k = 0; k < c.k_tokens; ++k) {
        float bv = kNegInf;
        int bk = kNoToken;
        for (int i = threadIdx.x; i < C; i += kMergeThreads) {
            const float v = cval[i];
            const int id = cid[i];
            const bool after = v < last_v || (v == last_v && id > last_id);
            if (after && better(v, id, bv, bk)) { bv = v; bk = id; }
        }
        warp_argbest(bv, bk);
        __syncthreads();
        if (lane == 0) { s_f[warp] = bv; s_i[warp] = bk; }
        __syncthreads();
        bv = s_f[0]; bk = s_i[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w)
            if (better(s_f[w], s_i[w], bv, bk)) { bv = s_f[w]; bk = s_i[w]; }
        if (threadIdx.x == 0) {
            out_ids[(size_t)m * c.k_tokens + k] = bk;
            out_logprobs[(size_t)m * c.k_tokens + k] = bv - lse;
        }
        last_v = bv;
        last_id = bk;
    }
}

}  // namespace coral
