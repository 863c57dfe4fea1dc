// Tree-expansion score step that consumes the draft head's outputs (CORAL Section 2.2: several candidates per
// timestep give a tree of drafts; Section 4.1: depth 6, 60 candidate tokens; Appendix B: top 10 candidates per
// node).  For every sequence: child score = parent's cumulative log-score + the candidate's log-probability;
// the K best children (score descending, equal -> lower flat (node, candidate) index) become the next level.
// The same kernel re-ranks a pool of nodes (k_tokens = 1, no log-probabilities) to keep the best 60.
#pragma once
#include "common.cuh"

namespace coral {

constexpr int kTreeThreads = 256;
constexpr int kTreeMaxCand = 2048;    // nodes * k_tokens per sequence
constexpr int kTreeMaxK = 256;

// grid = n_seq blocks.  Rank by counting: child i goes to output position (number of children that beat it).
__global__ void __launch_bounds__(kTreeThreads) tree_expand_kernel(const float* __restrict__ parent_scores,
                                                                   const int32_t* __restrict__ cand_ids,
                                                                   const float* __restrict__ cand_logprobs, int nodes,
                                                                   int k_tokens, int K, int32_t* __restrict__ out_parent,
                                                                   int32_t* __restrict__ out_token,
                                                                   float* __restrict__ out_score) {
    __shared__ float s_score[kTreeMaxCand];
    const int seq = blockIdx.x;
    const int C = nodes * k_tokens;
    const float* ps = parent_scores + (size_t)seq * nodes;
    const float* lp = cand_logprobs ? cand_logprobs + (size_t)seq * C : nullptr;
    for (int i = threadIdx.x; i < C; i += kTreeThreads)
        s_score[i] = lp ? __fadd_rn(ps[i / k_tokens], lp[i]) : ps[i / k_tokens];
    __syncthreads();
    for (int i = threadIdx.x; i < C; i += kTreeThreads) {
        const float v = s_score[i];
        int rank = 0;
        for (int j = 0; j < C; ++j) rank += better(s_score[j], j, v, i) ? 1 : 0;
        if (rank < K) {
            out_parent[(size_t)seq * K + rank] = i / k_tokens;
            out_token[(size_t)seq * K + rank] = cand_ids ? cand_ids[(size_t)seq * C + i] : i;
            out_score[(size_t)seq * K + rank] = v;
        }
    }
}

}  // namespace coral
