// Gathered GEMV for few query rows (M <= 8), streaming version.
//
// Every touched group's vocab rows are read exactly once: a producer thread
// issues bulk asynchronous copies (cp.async.bulk, mbarrier completion) of whole
// packed rows into a shared-memory ring; eight consumer warps split the hidden
// dimension between them, keep their slice of the group's hidden rows in fp32
// registers, and accumulate the dot products with fp32 FMAs.  Per 16-row item
// the warps' partial sums are combined in shared memory, and one warp per
// hidden row folds the 16 logits into a running (max, sum-exp, top-k) that is
// written once per (CTA, group) segment.  (CORAL Section 3.3: logits only for
// the activated groups, softmax over them; Appendix B: top candidates per row.)
//
// Work split: the touched groups' rows form n_union * T items of 16 rows; CTA b
// owns the contiguous run [b*per, (b+1)*per), so it changes group at most
// seg_max - 1 times and all CTAs stream the same number of bytes.
#pragma once
#include "common.cuh"

namespace coral {

constexpr int kStreamTile = 16;                 // vocab rows per item
constexpr int kStreamWarps = 8;                 // consumer warps
constexpr int kStreamConsumers = kStreamWarps * 32;
constexpr int kStreamThreads = 32 + kStreamConsumers;   // warp 0 = producer
constexpr int kStreamMaxR = 8;                  // hidden rows per group on this path (M <= 8)
constexpr int kStreamMaxH = 4096;               // two 16-byte chunks per consumer thread
constexpr int kStreamSpin = 1 << 20;            // bound of every mbarrier wait
constexpr int kStreamSpinAfterAbort = 1 << 8;

struct StreamGeom {
    int grid;         // CTAs launched
    int stage_rows;   // vocab rows per ring stage (divides kStreamTile)
    int n_stages;     // ring depth
    int seg_max;      // most groups one CTA's run can overlap
    int T;            // items per group = ceil(v / kStreamTile)
};

// One partial per (CTA, segment, hidden row of the group).
struct StreamPartials {
    float* pmax;      // [grid][seg_max][kStreamMaxR]
    float* psum;
    float* pval;      // [...][k_tokens]
    int32_t* pid;
};

// ---- mbarrier / bulk-copy primitives (shared::cta addresses as 32-bit) ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  On expiry the device status word is set, the CTA-wide abort
// flag raised, and the caller carries on (all indices stay in bounds; results
// of the call are then meaningless and the status says so).  After an abort
// later waits give up quickly so the kernel still ends promptly.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, DeviceState* st) {
    const int limit = *abort_flag ? kStreamSpinAfterAbort : kStreamSpin;
    for (int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return;
    *abort_flag = 1;
    set_status(st, -5);
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kStreamConsumers) : "memory"); }

__device__ __forceinline__ void unpack8(const uint4& q, float* f) {
    f[0] = bf16_lo(q.x); f[1] = bf16_hi(q.x); f[2] = bf16_lo(q.y); f[3] = bf16_hi(q.y);
    f[4] = bf16_lo(q.z); f[5] = bf16_hi(q.z); f[6] = bf16_lo(q.w); f[7] = bf16_hi(q.w);
}

struct StreamShared {
    unsigned char* ring;      // n_stages * stage_bytes
    float* zpart;             // [kStreamWarps][kStreamTile][kStreamMaxR]
    float* z;                 // [kStreamMaxR][kStreamTile]
    uint64_t* full;           // [n_stages]
    uint64_t* empty;          // [n_stages]
    volatile int* abort_flag;
};

// Consumer side of one segment: items [lo, hi) of the run, all inside union group j (group n, R hidden rows).
template <int R>
__device__ __forceinline__ void stream_segment(const CallView& c, const StreamGeom& g, const StreamShared& sh,
                                               const StreamPartials& pp, float* __restrict__ logits_tap, int n,
                                               int j, int lo, int hi, int seg, int& stage, uint32_t& phase) {
    const int ct = threadIdx.x - 32, cw = ct >> 5, lane = ct & 31;
    const int chunks = c.H >> 3;
    const int off = c.group_offset[n];
    const bool v0 = ct < chunks, v1 = ct + kStreamConsumers < chunks;
    const int stage_bytes = g.stage_rows * c.H * 2;
    const int row_bytes = c.H * 2;

    float hreg[R][16];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const uint4* hp = reinterpret_cast<const uint4*>(c.hidden + (size_t)c.bucket_row[off + r] * c.H);
        uint4 q0 = make_uint4(0, 0, 0, 0), q1 = make_uint4(0, 0, 0, 0);
        if (v0) q0 = __ldg(hp + ct);
        if (v1) q1 = __ldg(hp + ct + kStreamConsumers);
        unpack8(q0, &hreg[r][0]);
        unpack8(q1, &hreg[r][8]);
    }
    // running statistics of hidden row r = cw (warps cw < R); list entry i lives in lane i
    float run_max = kNegInf, run_sum = 0.f, lv = kNegInf;
    int lid = kNoToken;
    const int my_m = (cw < R) ? c.bucket_row[off + cw] : 0;
    const int my_slot = (cw < R) ? c.bucket_slot[off + cw] : 0;

    for (int item = lo; item < hi; ++item) {
        const int t = item - j * g.T;
        const int row0 = t * kStreamTile;
        const int rows = min(kStreamTile, c.v - row0);
        for (int s0 = 0; s0 < rows; s0 += g.stage_rows) {
            const int nrows = min(g.stage_rows, rows - s0);
            mbar_wait(smem_u32(&sh.full[stage]), phase, sh.abort_flag, c.state);
            const unsigned char* sp = sh.ring + (size_t)stage * stage_bytes;
            for (int rr = 0; rr < nrows; rr += 2) {
                const bool two = rr + 1 < nrows;
                float acc0[R], acc1[R];
#pragma unroll
                for (int r = 0; r < R; ++r) { acc0[r] = 0.f; acc1[r] = 0.f; }
                const uint4* w0p = reinterpret_cast<const uint4*>(sp + (size_t)rr * row_bytes);
                const uint4* w1p = reinterpret_cast<const uint4*>(sp + (size_t)(rr + (two ? 1 : 0)) * row_bytes);
                if (v0) {
                    float a[8], b[8];
                    unpack8(w0p[ct], a);
                    unpack8(w1p[ct], b);
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            acc0[r] = fmaf(a[e], hreg[r][e], acc0[r]);
                            acc1[r] = fmaf(b[e], hreg[r][e], acc1[r]);
                        }
                }
                if (v1) {
                    float a[8], b[8];
                    unpack8(w0p[ct + kStreamConsumers], a);
                    unpack8(w1p[ct + kStreamConsumers], b);
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            acc0[r] = fmaf(a[e], hreg[r][8 + e], acc0[r]);
                            acc1[r] = fmaf(b[e], hreg[r][8 + e], acc1[r]);
                        }
                }
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float s0v = warp_sum(acc0[r]);
                    const float s1v = warp_sum(acc1[r]);
                    if (lane == 0) {
                        sh.zpart[(cw * kStreamTile + s0 + rr) * kStreamMaxR + r] = s0v;
                        if (two) sh.zpart[(cw * kStreamTile + s0 + rr + 1) * kStreamMaxR + r] = s1v;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.empty[stage]));
            if (++stage == g.n_stages) { stage = 0; phase ^= 1u; }
        }
        consumer_bar();
        if (ct < R * kStreamTile) {
            const int r = ct / kStreamTile, row = ct - r * kStreamTile;
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kStreamWarps; ++w) s += sh.zpart[(w * kStreamTile + row) * kStreamMaxR + r];
            sh.z[r * kStreamTile + row] = s;
        }
        consumer_bar();
        if (cw < R) {
            const bool have = lane < rows;
            const float zv = have ? sh.z[cw * kStreamTile + lane] : kNegInf;
            const int tok = have ? __ldg(c.group_tokens + (size_t)n * c.v + row0 + lane) : kNoToken;
            if (logits_tap && have) logits_tap[((size_t)my_m * c.k_groups + my_slot) * c.v + row0 + lane] = zv;
            const float tmax = warp_max(zv);
            const float nmax = fmaxf(run_max, tmax);
            const float add = warp_sum(have ? __expf(zv - nmax) : 0.f);
            run_sum = run_sum * __expf(run_max - nmax) + add;     // exp(-inf) = 0 on the first item
            run_max = nmax;
            const float kth = __shfl_sync(0xffffffffu, lv, c.k_tokens - 1);
            const int kth_id = __shfl_sync(0xffffffffu, lid, c.k_tokens - 1);
            if (kth_id == kNoToken || tmax >= kth) {
                // merge the sorted list (lane i: entry i) with the new values (lane i: row i)
                float a = lv, b = zv;
                int ai = lid, bi = tok;
                float ov = kNegInf;
                int oi = kNoToken;
                for (int k = 0; k < c.k_tokens; ++k) {
                    float bv;
                    int bk;
                    if (better(a, ai, b, bi)) { bv = a; bk = ai; } else { bv = b; bk = bi; }
                    warp_argbest(bv, bk);
                    if (bk != kNoToken) {
                        if (ai == bk) { a = kNegInf; ai = kNoToken; }
                        if (bi == bk) { b = kNegInf; bi = kNoToken; }
                    }
                    if (lane == k) { ov = bv; oi = bk; }
                }
                lv = ov;
                lid = oi;
            }
        }
    }
    if (cw < R) {
        const size_t p = ((size_t)blockIdx.x * g.seg_max + seg) * kStreamMaxR + cw;
        if (lane == 0) { pp.pmax[p] = run_max; pp.psum[p] = run_sum; }
        if (lane < c.k_tokens) { pp.pval[p * c.k_tokens + lane] = lv; pp.pid[p * c.k_tokens + lane] = lid; }
    }
}

// grid = g.grid CTAs of kStreamThreads threads; dynamic shared memory laid out as StreamShared.
__global__ void __launch_bounds__(kStreamThreads, 1) head_stream_kernel(CallView c, StreamGeom g, StreamPartials pp,
                                                                        float* __restrict__ logits_tap) {
    extern __shared__ __align__(128) unsigned char stream_smem_raw[];
    unsigned char* smem_raw = stream_smem_raw;
    const int stage_bytes = g.stage_rows * c.H * 2;
    StreamShared sh;
    sh.ring = smem_raw;
    size_t o = (size_t)g.n_stages * stage_bytes;
    sh.zpart = reinterpret_cast<float*>(smem_raw + o);
    o += sizeof(float) * kStreamWarps * kStreamTile * kStreamMaxR;
    sh.z = reinterpret_cast<float*>(smem_raw + o);
    o += sizeof(float) * kStreamMaxR * kStreamTile;
    sh.full = reinterpret_cast<uint64_t*>(smem_raw + o);
    o += sizeof(uint64_t) * g.n_stages;
    sh.empty = reinterpret_cast<uint64_t*>(smem_raw + o);
    o += sizeof(uint64_t) * g.n_stages;
    sh.abort_flag = reinterpret_cast<volatile int*>(smem_raw + o);

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.n_stages; ++s) {
            mbar_init(smem_u32(&sh.full[s]), 1);
            mbar_init(smem_u32(&sh.empty[s]), kStreamWarps);
        }
        *sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int n_union = c.state->n_union;
    const int n_items = n_union * g.T;
    const int per = (n_items + g.grid - 1) / g.grid;
    const int lo = min(n_items, (int)blockIdx.x * per);
    const int hi = min(n_items, lo + per);
    if (lo >= hi) return;

    if (threadIdx.x < 32) {
        if (threadIdx.x != 0) return;
        // producer: one bulk copy per ring stage, rows of one group are contiguous in the packed copy
        int stage = 0;
        uint32_t phase = 0;
        for (int item = lo; item < hi; ++item) {
            const int j = item / g.T, t = item - j * g.T;
            const int n = c.union_list[j];
            const int row0 = t * kStreamTile;
            const int rows = min(kStreamTile, c.v - row0);
            for (int s0 = 0; s0 < rows; s0 += g.stage_rows) {
                const int nrows = min(g.stage_rows, rows - s0);
                mbar_wait(smem_u32(&sh.empty[stage]), phase ^ 1u, sh.abort_flag, c.state);
                const uint32_t bytes = (uint32_t)nrows * c.H * 2;
                const uint32_t bar = smem_u32(&sh.full[stage]);
                mbar_expect_tx(bar, bytes);
                bulk_g2s(smem_u32(sh.ring + (size_t)stage * stage_bytes),
                         c.packed + ((size_t)n * c.v + row0 + s0) * c.H, bytes, bar);
                if (++stage == g.n_stages) { stage = 0; phase ^= 1u; }
            }
        }
        return;
    }

    // consumers: walk the run segment by segment (one union group each)
    int stage = 0;
    uint32_t phase = 0;
    const int j_first = lo / g.T;
    for (int pos = lo; pos < hi;) {
        const int j = pos / g.T;
        const int seg_hi = min(hi, (j + 1) * g.T);
        const int n = c.union_list[j];
        const int R = min(c.group_count[n], kStreamMaxR);
        const int seg = j - j_first;
        switch (R) {
            case 1: stream_segment<1>(c, g, sh, pp, logits_tap, n, j, pos, seg_hi, seg, stage, phase); break;
            case 2: stream_segment<2>(c, g, sh, pp, logits_tap, n, j, pos, seg_hi, seg, stage, phase); break;
            case 3: stream_segment<3>(c, g, sh, pp, logits_tap, n, j, pos, seg_hi, seg, stage, phase); break;
            case 4: stream_segment<4>(c, g, sh, pp, logits_tap, n, j, pos, seg_hi, seg, stage, phase); break;
            case 5: stream_segment<5>(c, g, sh, pp, logits_tap, n, j, pos, seg_hi, seg, stage, phase); break;
            case 6: stream_segment<6>(c, g, sh, pp, logits_tap, n, j, pos, seg_hi, seg, stage, phase); break;
            case 7: stream_segment<7>(c, g, sh, pp, logits_tap, n, j, pos, seg_hi, seg, stage, phase); break;
            default: stream_segment<8>(c, g, sh, pp, logits_tap, n, j, pos, seg_hi, seg, stage, phase); break;
        }
        pos = seg_hi;
    }
}

// Merge for the streaming path: block per row.  The pieces of row m, slot s are the partials that the
// CTAs overlapping that slot's group wrote for the row's position in the group's bucket.
constexpr int kMergeStreamThreads = 256;
__global__ void __launch_bounds__(kMergeStreamThreads) merge_stream_kernel(CallView c, StreamGeom g, StreamPartials pp,
                                                                           float* __restrict__ cand_val_scratch,
                                                                           int32_t* __restrict__ cand_id_scratch,
                                                                           int cand_cap, int smem_cands,
                                                                           int32_t* __restrict__ out_ids,
                                                                           float* __restrict__ out_logprobs,
                                                                           float* __restrict__ lse_tap) {
    extern __shared__ __align__(16) unsigned char msm[];
    const int m = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kMergeStreamThreads / 32;
    __shared__ float s_f[kWarps];
    __shared__ int s_i[kWarps];
    __shared__ float s_lse;
    __shared__ int s_first[kMaxGroups], s_cnt[kMaxGroups], s_base[kMaxGroups + 1], s_rpos[kMaxGroups], s_j[kMaxGroups];

    const int n_union = c.state->n_union;
    const int n_items = n_union * g.T;
    const int per = (n_items + g.grid - 1) / g.grid;
    for (int s = threadIdx.x; s < c.k_groups; s += kMergeStreamThreads) {
        const int n = c.sel[(size_t)m * c.k_groups + s];
        const int j = c.union_rank[n];
        const int fb = (j * g.T) / per;
        const int lb = ((j + 1) * g.T - 1) / per;
        s_first[s] = fb;
        s_cnt[s] = lb - fb + 1;
        s_j[s] = j;
        s_rpos[s] = c.bucket_pos[(size_t)m * c.k_groups + s];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int s = 0; s < c.k_groups; ++s) { s_base[s] = run; run += s_cnt[s]; }
        s_base[c.k_groups] = run;
    }
    __syncthreads();
    const int P = s_base[c.k_groups];
    const int C = P * c.k_tokens;
    float* cv = (C <= smem_cands) ? reinterpret_cast<float*>(msm) : cand_val_scratch + (size_t)m * cand_cap;
    int32_t* ci = (C <= smem_cands) ? reinterpret_cast<int32_t*>(msm + sizeof(float) * smem_cands)
                                    : cand_id_scratch + (size_t)m * cand_cap;

    // piece q -> (slot s, CTA b) by search over the (few) slots; gather max/sum and the candidate lists
    float mx = kNegInf;
    for (int q = threadIdx.x; q < P; q += kMergeStreamThreads) {
        int s = 0;
        while (s + 1 < c.k_groups && s_base[s + 1] <= q) ++s;
        const int b = s_first[s] + (q - s_base[s]);
        const int seg = s_j[s] - (b * per) / g.T;
        const size_t p = ((size_t)b * g.seg_max + seg) * kStreamMaxR + s_rpos[s];
        mx = fmaxf(mx, pp.pmax[p]);
        for (int i = 0; i < c.k_tokens; ++i) {
            cv[q * c.k_tokens + i] = pp.pval[p * c.k_tokens + i];
            ci[q * c.k_tokens + i] = pp.pid[p * c.k_tokens + i];
        }
    }
    mx = warp_max(mx);
    if (lane == 0) s_f[warp] = mx;
    __syncthreads();
    mx = s_f[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) mx = fmaxf(mx, s_f[w]);
    __syncthreads();
    float sum = 0.f;
    for (int q = threadIdx.x; q < P; q += kMergeStreamThreads) {
        int s = 0;
        while (s + 1 < c.k_groups && s_base[s + 1] <= q) ++s;
        const int b = s_first[s] + (q - s_base[s]);
        const int seg = s_j[s] - (b * per) / g.T;
        const size_t p = ((size_t)b * g.seg_max + seg) * kStreamMaxR + s_rpos[s];
        sum += pp.psum[p] * expf(pp.pmax[p] - mx);
    }
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

    float last_v = __builtin_huge_valf();
    int last_id = -1;
    for (int k = 0; k < c.k_tokens; ++k) {
        float bv = kNegInf;
        int bk = kNoToken;
        for (int i = threadIdx.x; i < C; i += kMergeStreamThreads) {
            const float v = cv[i];
            const int id = ci[i];
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
