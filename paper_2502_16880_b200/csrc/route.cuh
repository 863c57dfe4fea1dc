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
        if (val[i] != val[i]) {                      // NaN orders against nothing: rank it last and report
            val[i] = kNegInf;
            set_status(c.state, -8);
        }
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
            if (c.shard_world > 1) c.slot_desc[(size_t)m * c.k_groups + s] = -1;   // stays -1 for another GPU's group
            if (groups_tap) groups_tap[(size_t)m * c.k_groups + s] = pick;
        }
    }
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int n = lane + 32 * i;
        if (n < c.N) c.slot_of[(size_t)m * c.N + n] = (int16_t)slot[i];
    }
}

// Groups of row m by one warp (NPER = groups per lane); bit `bit` of s_rowmask[n] is set for every selected group n.  Rank selection: slot of a group = number of groups
// that beat it (higher score, or equal score and lower index).  Forced groups take their listed order.
template <int NPER>
__device__ __forceinline__ void route_select_row(const CallView& c, const int32_t* __restrict__ forced,
                                                 int32_t* __restrict__ groups_tap, int m, int lane, float* s_val,
                                                 int16_t* s_slot_row, unsigned* s_rowmask, int bit,
                                                 bool from_smem = false) {
    int slot[NPER];
#pragma unroll
    for (int i = 0; i < NPER; ++i) slot[i] = -1;
    if (forced) {
        for (int s = 0; s < c.k_groups; ++s) {
            int pick = forced[(size_t)m * c.k_groups + s];
            if (pick < 0 || pick >= c.N) {           // never index with it; report and fall back to group 0
                if (lane == 0) set_status(c.state, -6);
                pick = 0;
            }
#pragma unroll
            for (int i = 0; i < NPER; ++i) {
                if (lane + 32 * i == pick) {
                    if (slot[i] >= 0) set_status(c.state, -6);   // a forced group named twice
                    slot[i] = s;
                }
            }
        }
    } else {
        float val[NPER];
#pragma unroll
        for (int i = 0; i < NPER; ++i) {
            const int n = lane + 32 * i;
            val[i] = n >= c.N ? kNegInf : from_smem ? s_val[n] : __ldcg(c.gate + (size_t)m * c.N + n);   // s_val: the row's scores, already there
            if (val[i] != val[i]) {                  // NaN orders against nothing: rank it last and report, so that
                val[i] = kNegInf;                    // every row still gets exactly k_groups distinct groups
                set_status(c.state, -8);
            }
            if (n < c.N) s_val[n] = val[i];
        }
        __syncwarp();
        int rank[NPER];
#pragma unroll
        for (int i = 0; i < NPER; ++i) rank[i] = 0;
#pragma unroll 4
        for (int j = 0; j < c.N; ++j) {
            const float vj = s_val[j];
#pragma unroll
            for (int i = 0; i < NPER; ++i) rank[i] += better(vj, j, val[i], lane + 32 * i) ? 1 : 0;
        }
#pragma unroll
        for (int i = 0; i < NPER; ++i)
            if (lane + 32 * i < c.N && rank[i] < c.k_groups) slot[i] = rank[i];
        __syncwarp();
    }
#pragma unroll
    for (int i = 0; i < NPER; ++i) {
        const int n = lane + 32 * i;
        if (n < c.N) {
            s_slot_row[n] = (int16_t)slot[i];
            c.slot_of[(size_t)m * c.N + n] = (int16_t)slot[i];
            if (slot[i] >= 0) {
                atomicOr(&s_rowmask[n], 1u << bit);
                c.sel[(size_t)m * c.k_groups + slot[i]] = n;
                if (c.shard_world > 1) c.slot_desc[(size_t)m * c.k_groups + slot[i]] = -1;   // stays -1 for another GPU's group
                if (groups_tap) groups_tap[(size_t)m * c.k_groups + slot[i]] = n;
            }
        }
    }
}

// Router stage in one launch for few rows (M <= kRouteFusedMaxM).  grid = N CTAs: CTA n computes the gate
// scores of group n (threads split H), then takes a ticket; the CTA that draws the last ticket - nobody
// waits for anybody - selects the groups of every row, buckets the rows by group and writes the union
// list.  Same outputs as gate_kernel + select_kernel + bucket_kernel.
// Selection is by rank: a group's slot is the number of groups that beat it (higher score, or equal score
// and lower index), so the cost does not grow with k_groups.
constexpr int kRouteFusedMaxM = 32;
constexpr int kRouteThreads = 256;

__global__ void __launch_bounds__(kRouteThreads)
    route_fused_kernel(CallView c, const int32_t* __restrict__ forced, int32_t* __restrict__ groups_tap,
                       float* __restrict__ gate_tap) {
    __shared__ int16_t s_slot[kRouteFusedMaxM][kMaxGroups];
    __shared__ float s_val[kRouteThreads / 32][kMaxGroups];
    __shared__ unsigned s_rowmask[kMaxGroups];     // bit m: row m selected the group
    __shared__ int s_warp_tot[kRouteThreads / 32];
    __shared__ float s_red[kRouteThreads / 32][8];
    __shared__ int s_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kRouteThreads / 32;
    const int chunks = c.H >> 3;
    pdl_wait();                   // with the two-layer router this grid follows the kernel that writes router_in
    pdl_launch_dependents();      // the next kernel may set itself up; it waits for this grid before reading

    {
        const int n = blockIdx.x;
        const uint4* __restrict__ wg = reinterpret_cast<const uint4*>(c.w_gate + (size_t)n * c.H);
        for (int m0 = 0; m0 < c.M; m0 += 8) {
            const int rows = min(8, c.M - m0);
            const uint4* __restrict__ hid = reinterpret_cast<const uint4*>(c.hidden + (size_t)m0 * c.H);
            float acc[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) acc[r] = 0.f;
            if (c.router_in) {             // Eq. 7: the gate reads act(W1 h) + h, kept in fp32
                for (int ch = threadIdx.x; ch < chunks; ch += kRouteThreads) {
                    const uint4 q = __ldg(wg + ch);
                    const float w[8] = {bf16_lo(q.x), bf16_hi(q.x), bf16_lo(q.y), bf16_hi(q.y),
                                        bf16_lo(q.z), bf16_hi(q.z), bf16_lo(q.w), bf16_hi(q.w)};
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        if (r < rows) {
                            const float4* up = reinterpret_cast<const float4*>(c.router_in + (size_t)(m0 + r) * c.H) + 2 * ch;
                            const float4 a = __ldcg(up), b = __ldcg(up + 1);
                            acc[r] = fmaf(w[0], a.x, acc[r]); acc[r] = fmaf(w[1], a.y, acc[r]);
                            acc[r] = fmaf(w[2], a.z, acc[r]); acc[r] = fmaf(w[3], a.w, acc[r]);
                            acc[r] = fmaf(w[4], b.x, acc[r]); acc[r] = fmaf(w[5], b.y, acc[r]);
                            acc[r] = fmaf(w[6], b.z, acc[r]); acc[r] = fmaf(w[7], b.w, acc[r]);
                        }
                    }
                }
            } else
            for (int ch = threadIdx.x; ch < chunks; ch += kRouteThreads) {
                const uint4 w = __ldg(wg + ch);
                uint4 hv[8];                       // all loads first, so they are in flight together
#pragma unroll
                for (int r = 0; r < 8; ++r)
                    hv[r] = r < rows ? __ldg(hid + (size_t)r * chunks + ch) : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int r = 0; r < 8; ++r) acc[r] = dot8(w, hv[r], acc[r]);
            }
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const float sum = warp_sum(acc[r]);
                if (lane == 0) s_red[warp][r] = sum;
            }
            __syncthreads();
            if (threadIdx.x < rows) {
                float sum = 0.f;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) sum += s_red[w][threadIdx.x];
                c.gate[(size_t)(m0 + threadIdx.x) * c.N + n] = sum;
                if (gate_tap) gate_tap[(size_t)(m0 + threadIdx.x) * c.N + n] = sum;
            }
            __syncthreads();
        }
    }
    // ticket: the scores above are published before the ticket is drawn; the last CTA sees all of them
    if (threadIdx.x == 0) {
        __threadfence();
        const int ticket = atomicAdd(&c.state->ticket, 1);
        s_last = ticket == (int)gridDim.x - 1;
        if (s_last) c.state->ticket = 0;          // ready for the next call on this handle
        __threadfence();
    }
    s_rowmask[threadIdx.x] = 0;                     // kRouteThreads == kMaxGroups
    __syncthreads();
    if (!s_last) return;

    // groups of every row: one warp per row
    for (int m = warp; m < c.M; m += kWarps) {
        if (c.N <= 32) route_select_row<1>(c, forced, groups_tap, m, lane, s_val[warp], s_slot[m], s_rowmask, m);
        else if (c.N <= 64) route_select_row<2>(c, forced, groups_tap, m, lane, s_val[warp], s_slot[m], s_rowmask, m);
        else if (c.N <= 128) route_select_row<4>(c, forced, groups_tap, m, lane, s_val[warp], s_slot[m], s_rowmask, m);
        else route_select_row<8>(c, forced, groups_tap, m, lane, s_val[warp], s_slot[m], s_rowmask, m);
    }
    __syncthreads();

    // One thread per group: rows that selected it, passes over its weights, and (by a block-wide exclusive
    // scan of both counts, packed in one word) its place in the bucket array and in the union list.
    const int n = threadIdx.x;
    const unsigned mask = (n < c.N && group_is_local(c, n)) ? s_rowmask[n] : 0u;
    const int cnt = __popc(mask);
    const int passes = cnt == 0 ? 0 : (c.pass_rows > 0 ? (cnt + c.pass_rows - 1) / c.pass_rows : 1);
    const int packed = cnt | (passes << 16);
    int incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += a;
    }
    if (lane == 31) s_warp_tot[warp] = incl;
    const int n_union = __syncthreads_count(cnt > 0);
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const int t = s_warp_tot[w];
        if (w < warp) before += t;
        total += t;
    }
    const int excl = before + incl - packed;
    const int off = excl & 0xffff, virt = excl >> 16;
    if (n < c.N) {
        c.group_offset[n] = off;
        c.group_count[n] = cnt;
        c.union_rank[n] = cnt > 0 ? virt : -1;
        for (int p = 0; p < passes; ++p)
            if (virt + p < c.union_cap) c.union_list[virt + p] = n | (p << 16);
        unsigned left = mask;
        for (int pos = 0; left; ++pos) {
            const int m = __ffs(left) - 1;
            left &= left - 1;
            const int sl = s_slot[m][n];
            if (!CORAL_IDX_OK(off + pos, c.cap_pairs, c.state) || !CORAL_IDX_OK(m * c.k_groups + sl, c.cap_pairs, c.state)) continue;
            c.bucket_row[off + pos] = m;
            c.bucket_slot[off + pos] = sl;
            const int pass = c.pass_rows > 0 ? pos / c.pass_rows : 0;
            c.slot_desc[(size_t)m * c.k_groups + sl] = ((virt + pass) << 8) | ((pos - pass * max(c.pass_rows, 1)) & 255);
            if (c.bucket_dst && c.pass_rows == kTcPassRows)
                c.bucket_dst[off + pos] = tc_entry_row(off + pass * kTcPassRows, virt + pass) + pos - pass * kTcPassRows;
        }
    }
    if (threadIdx.x == 0) {
        c.group_offset[c.N] = total & 0xffff;
        c.state->n_union = n_union;
        c.state->n_virtual = min(total >> 16, c.union_cap);
    }
}


// ---- router stage for many rows (M > kRouteFusedMaxM): three short kernels --------------------------------

// Gate scores for a tile of 8 groups x 8 rows per block, so that every hidden row is read N/8 times and
// every gate row M/8 times (from L2).  grid (ceil(N/8), ceil(M/8)).  Block (0,0) also clears the per-group
// row counters that select_count_kernel accumulates.
constexpr int kGateTile = 8;
__global__ void __launch_bounds__(256) gate_tile_kernel(CallView c, float* __restrict__ gate_tap) {
    __shared__ float s_red[8][kGateTile * kGateTile];
    const int n0 = blockIdx.x * kGateTile, m0 = blockIdx.y * kGateTile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = c.H >> 3;
    if (blockIdx.x == 0 && blockIdx.y == 0)
        for (int n = threadIdx.x; n < c.N; n += 256) c.group_count[n] = 0;
    float acc[kGateTile][kGateTile];
#pragma unroll
    for (int g = 0; g < kGateTile; ++g)
#pragma unroll
        for (int r = 0; r < kGateTile; ++r) acc[g][r] = 0.f;
    for (int ch = threadIdx.x; ch < chunks; ch += 256) {
        float hf[kGateTile][8];
#pragma unroll
        for (int r = 0; r < kGateTile; ++r) {
            const uint4 q = (m0 + r < c.M) ? __ldg(reinterpret_cast<const uint4*>(c.hidden + (size_t)(m0 + r) * c.H) + ch)
                                           : make_uint4(0, 0, 0, 0);
            hf[r][0] = bf16_lo(q.x); hf[r][1] = bf16_hi(q.x); hf[r][2] = bf16_lo(q.y); hf[r][3] = bf16_hi(q.y);
            hf[r][4] = bf16_lo(q.z); hf[r][5] = bf16_hi(q.z); hf[r][6] = bf16_lo(q.w); hf[r][7] = bf16_hi(q.w);
        }
#pragma unroll
        for (int g = 0; g < kGateTile; ++g) {
            const uint4 q = (n0 + g < c.N) ? __ldg(reinterpret_cast<const uint4*>(c.w_gate + (size_t)(n0 + g) * c.H) + ch)
                                           : make_uint4(0, 0, 0, 0);
            const float w[8] = {bf16_lo(q.x), bf16_hi(q.x), bf16_lo(q.y), bf16_hi(q.y),
                                bf16_lo(q.z), bf16_hi(q.z), bf16_lo(q.w), bf16_hi(q.w)};
#pragma unroll
            for (int r = 0; r < kGateTile; ++r)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[g][r] = fmaf(w[e], hf[r][e], acc[g][r]);
        }
    }
#pragma unroll
    for (int g = 0; g < kGateTile; ++g)
#pragma unroll
        for (int r = 0; r < kGateTile; ++r) {
            const float sum = warp_sum(acc[g][r]);
            if (lane == 0) s_red[warp][g * kGateTile + r] = sum;
        }
    __syncthreads();
    if (threadIdx.x < kGateTile * kGateTile) {
        const int g = threadIdx.x / kGateTile, r = threadIdx.x % kGateTile;
        if (n0 + g < c.N && m0 + r < c.M) {
            float sum = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) sum += s_red[w][threadIdx.x];
            c.gate[(size_t)(m0 + r) * c.N + n0 + g] = sum;
            if (gate_tap) gate_tap[(size_t)(m0 + r) * c.N + n0 + g] = sum;
        }
    }
}

// Gate scores on the warp-level tensor cores for many rows: a block computes a 16-group x 8-row tile, its 8 warps
// splitting H in blocks of 32 columns (mma.sync m16n8k16, bf16 x bf16 -> fp32; groups on the M axis, rows on N).
// Every lane loads 16 bytes of two gate rows and of one hidden row per block of 32 columns; the column order
// inside a block is permuted the same way for both operands, which leaves the dot products unchanged.
// H a multiple of 32.
// With `part` set the block covers only the 32-column blocks [kb_lo, kb_hi) of H (several blocks split H between
// them) and writes its 16 x 8 partial sums there, element (group g, row r) at part[g * 8 + r]; whoever finishes
// the band adds the parts up in a fixed order.
__device__ __forceinline__ void gate_mma_tile(const CallView& c, float* __restrict__ gate_tap, int n0, int m0,
                                              float (*s_part)[16 * 8], int kb_lo, int kb_hi, float* __restrict__ part) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, tq = lane & 3;
    const bool a_lo = n0 + gq < c.N, a_hi = n0 + gq + 8 < c.N, b_ok = m0 + gq < c.M;
    const uint16_t* wlo = c.w_gate + (size_t)(a_lo ? n0 + gq : 0) * c.H + tq * 8;
    const uint16_t* whi = c.w_gate + (size_t)(a_hi ? n0 + gq + 8 : 0) * c.H + tq * 8;
    const uint16_t* hb = c.hidden + (size_t)(b_ok ? m0 + gq : 0) * c.H + tq * 8;
    float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
    const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll 4
    for (int kb = kb_lo + warp; kb < kb_hi; kb += 8) {
        const uint4 a = a_lo ? __ldg(reinterpret_cast<const uint4*>(wlo + kb * 32)) : zero;
        const uint4 b = a_hi ? __ldg(reinterpret_cast<const uint4*>(whi + kb * 32)) : zero;
        const uint4 h = b_ok ? __ldg(reinterpret_cast<const uint4*>(hb + kb * 32)) : zero;
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                     : "+f"(acc0[0]), "+f"(acc0[1]), "+f"(acc0[2]), "+f"(acc0[3])
                     : "r"(a.x), "r"(b.x), "r"(a.y), "r"(b.y), "r"(h.x), "r"(h.y));
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                     : "+f"(acc1[0]), "+f"(acc1[1]), "+f"(acc1[2]), "+f"(acc1[3])
                     : "r"(a.z), "r"(b.z), "r"(a.w), "r"(b.w), "r"(h.z), "r"(h.w));
    }
    // accumulator layout: [0],[1] = group gq, rows 2*tq, 2*tq+1; [2],[3] = group gq + 8
    float* sp = s_part[warp];
    sp[gq * 8 + 2 * tq] = acc0[0] + acc1[0];
    sp[gq * 8 + 2 * tq + 1] = acc0[1] + acc1[1];
    sp[(gq + 8) * 8 + 2 * tq] = acc0[2] + acc1[2];
    sp[(gq + 8) * 8 + 2 * tq + 1] = acc0[3] + acc1[3];
    __syncthreads();
    if (threadIdx.x < 128) {
        const int g = threadIdx.x >> 3, r = threadIdx.x & 7;
        if (n0 + g < c.N && m0 + r < c.M) {
            float sum = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) sum += s_part[w][threadIdx.x];
            if (part) {
                part[threadIdx.x] = sum;
            } else {
                c.gate[(size_t)(m0 + r) * c.N + n0 + g] = sum;
                if (gate_tap) gate_tap[(size_t)(m0 + r) * c.N + n0 + g] = sum;
            }
        }
    }
}

// Router stage in one launch for a medium number of rows (kRouteFusedMaxM < M <= kRouteMidMaxM, M * N <=
// kRouteMidMaxCells, H a multiple of 32).  grid (ceil(N/16), ceil(M/8)): a block computes one 16-group x 8-row tile of scores (gate_mma_tile).  Nobody waits for
// anybody: the blocks of one 8-row band draw tickets from the band's counter and the last one selects the
// groups of the band's rows (one warp per row) and ORs them into per-group row masks in global memory; these
// band-finishers draw a second ticket and the last of them buckets the rows by group (one thread per group)
// and writes the union list and the merge descriptors.  With finish = 0 (any number of rows) the
// band-finishers only add their rows to per-group counters and bucket_group_kernel, launched next, does the
// bucketing.  band_ticket: one counter per 8-row band; rowmask: four mask words per group; count_acc: one
// counter per group; all zero between calls (whoever uses them last clears them).
constexpr int kRouteMidMaxM = 128;
constexpr int kRouteMidBands = kRouteMidMaxM / 8;
constexpr int kRouteMidMaxCells = 8192;       // M * N slots staged in shared memory by the last block
constexpr int kRouteMidSplitMax = 4;          // blocks that share one tile's H
__global__ void __launch_bounds__(256)
    route_mid_kernel(CallView c, const int32_t* __restrict__ forced, int32_t* __restrict__ groups_tap,
                     float* __restrict__ gate_tap, unsigned* __restrict__ band_ticket, unsigned* __restrict__ rowmask,
                     int* __restrict__ count_acc, int finish, float* __restrict__ gate_part) {
    __shared__ float s_part[8][16 * 8];
    __shared__ float s_val[8][kMaxGroups];
    __shared__ int16_t s_slot_row[8][kMaxGroups];
    __shared__ unsigned s_mask[kMaxGroups];
    __shared__ int16_t s_slot[kRouteMidMaxCells];      // last finisher: every row's slot of every group
    __shared__ int s_warp_tot[8];
    __shared__ int s_flag;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int m0 = blockIdx.y * 8;
    pdl_launch_dependents();      // the next kernel may set itself up; it waits for this grid before reading

    // gridDim.z > 1 (few rows, hence few tiles): the blocks of a tile split H between them, so that every load of
    // a block is in flight at once, and leave partial sums for the band's finisher
    const int KS = (int)gridDim.z, kblocks = c.H >> 5;
    float* part = KS > 1 ? gate_part + ((((size_t)blockIdx.y * gridDim.x + blockIdx.x) * KS + blockIdx.z) << 7) : nullptr;
    gate_mma_tile(c, gate_tap, blockIdx.x * 16, m0, s_part, (int)((long long)kblocks * blockIdx.z / KS),
                  (int)((long long)kblocks * (blockIdx.z + 1) / KS), part);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned t = atomicAdd(&band_ticket[blockIdx.y], 1u);
        s_flag = t == gridDim.x * gridDim.z - 1;
        if (s_flag) band_ticket[blockIdx.y] = 0;
        __threadfence();
    }
    s_mask[threadIdx.x] = 0;                        // 256 threads == kMaxGroups
    __syncthreads();
    if (!s_flag) return;

    // this block saw the band's last ticket: every score (or partial sum) of rows m0 .. m0 + 7 is published
    if (KS > 1) {
        // add the parts of every score in the order of the column ranges: the same sum whoever finishes
        for (int e = threadIdx.x; e < 8 * c.N; e += 256) {
            const int r = e & 7, n = e >> 3;
            const float* p = gate_part + ((((size_t)blockIdx.y * gridDim.x + (n >> 4)) * KS) << 7) + (n & 15) * 8 + r;
            float sum = 0.f;
            for (int z = 0; z < KS; ++z) sum += __ldcg(p + ((size_t)z << 7));
            s_val[r][n] = sum;
            if (m0 + r < c.M) {
                c.gate[(size_t)(m0 + r) * c.N + n] = sum;
                if (gate_tap) gate_tap[(size_t)(m0 + r) * c.N + n] = sum;
            }
        }
        __syncthreads();
    }
    {
        const int m = m0 + warp;
        const bool sm = KS > 1;
        if (m < c.M) {
            if (c.N <= 32) route_select_row<1>(c, forced, groups_tap, m, lane, s_val[warp], s_slot_row[warp], s_mask, warp, sm);
            else if (c.N <= 64) route_select_row<2>(c, forced, groups_tap, m, lane, s_val[warp], s_slot_row[warp], s_mask, warp, sm);
            else if (c.N <= 128) route_select_row<4>(c, forced, groups_tap, m, lane, s_val[warp], s_slot_row[warp], s_mask, warp, sm);
            else route_select_row<8>(c, forced, groups_tap, m, lane, s_val[warp], s_slot_row[warp], s_mask, warp, sm);
        }
    }
    __syncthreads();
    if (!finish) {                                  // many rows: only count; bucket_group_kernel does the rest
        if (threadIdx.x < c.N && s_mask[threadIdx.x] && group_is_local(c, threadIdx.x))
            atomicAdd(&count_acc[threadIdx.x], __popc(s_mask[threadIdx.x]));
        return;
    }
    if (threadIdx.x < c.N && s_mask[threadIdx.x])
        atomicOr(&rowmask[threadIdx.x * 4 + (m0 >> 5)], s_mask[threadIdx.x] << (m0 & 31));
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int t = atomicAdd(&c.state->ticket, 1);
        s_flag = t == (int)gridDim.y - 1;
        if (s_flag) c.state->ticket = 0;
        __threadfence();
    }
    __syncthreads();
    if (!s_flag) return;

    // last band-finisher: every row's selection is published.  Stage the slots, then one thread per group.
    for (int i = threadIdx.x; i < c.M * c.N; i += 256) s_slot[i] = __ldcg(c.slot_of + i);
    const int n = threadIdx.x;
    unsigned mask[4] = {0u, 0u, 0u, 0u};
    if (n < c.N) {
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            mask[w] = group_is_local(c, n) ? __ldcg(rowmask + n * 4 + w) : 0u;
            rowmask[n * 4 + w] = 0;                 // ready for the next call
        }
    }
    const int cnt = __popc(mask[0]) + __popc(mask[1]) + __popc(mask[2]) + __popc(mask[3]);
    // Adaptive call: the streaming kernel reads a group once per pass_rows rows, the tensor-core kernel once
    // per pass_rows_tc rows but costs more per read and has a fixed extra cost (gathering the rows, a longer
    // tail).  Compare the two totals (cost per pass in units of 10 ns, measured on the Llama3-8B shape) and
    // record the choice for the kernels launched after this one.
    int pr = c.pass_rows, ucap = c.union_cap;
    if (c.adaptive) {
        const int ps = cnt == 0 ? 0 : (cnt + c.pass_rows - 1) / c.pass_rows;
        const int pt = cnt == 0 ? 0 : (cnt + c.pass_rows_tc - 1) / c.pass_rows_tc;
        int both = ps | (pt << 16);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) both += __shfl_xor_sync(0xffffffffu, both, o);
        if (lane == 0) s_warp_tot[warp] = both;
        __syncthreads();
        int tot2 = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot2 += s_warp_tot[w];
        __syncthreads();
        const bool use_tc = (tot2 & 0xffff) * 330 > (tot2 >> 16) * 345 + 1200;
        if (use_tc) { pr = c.pass_rows_tc; ucap = c.union_cap_tc; }
        if (threadIdx.x == 0) c.state->path_choice = use_tc ? 2 : 1;
    }
    const int passes = cnt == 0 ? 0 : (pr > 0 ? (cnt + pr - 1) / pr : 1);
    const int packed = cnt | (passes << 16);
    int incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += a;
    }
    if (lane == 31) s_warp_tot[warp] = incl;
    const int n_union = __syncthreads_count(cnt > 0);
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        const int t = s_warp_tot[w];
        if (w < warp) before += t;
        total += t;
    }
    const int excl = before + incl - packed;
    const int off = excl & 0xffff, virt = excl >> 16;
    if (n < c.N) {
        c.group_offset[n] = off;
        c.group_count[n] = cnt;
        c.union_rank[n] = cnt > 0 ? virt : -1;
        for (int p = 0; p < passes; ++p)
            if (virt + p < ucap) c.union_list[virt + p] = n | (p << 16);
        int pos = 0;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            unsigned left = mask[w];
            for (; left; ++pos) {
                const int m = w * 32 + __ffs(left) - 1;
                left &= left - 1;
                const int sl = s_slot[m * c.N + n];
                if (!CORAL_IDX_OK(off + pos, c.cap_pairs, c.state) || !CORAL_IDX_OK(m * c.k_groups + sl, c.cap_pairs, c.state)) continue;
                c.bucket_row[off + pos] = m;
                c.bucket_slot[off + pos] = sl;
                const int pass = pr > 0 ? pos / pr : 0;
                c.slot_desc[(size_t)m * c.k_groups + sl] = ((virt + pass) << 8) | ((pos - pass * max(pr, 1)) & 255);
                if (c.bucket_dst && pr == kTcPassRows)
                    c.bucket_dst[off + pos] = tc_entry_row(off + pass * kTcPassRows, virt + pass) + pos - pass * kTcPassRows;
            }
        }
    }
    if (threadIdx.x == 0) {
        c.group_offset[c.N] = total & 0xffff;
        c.state->n_union = n_union;
        c.state->n_virtual = min(total >> 16, ucap);
    }
}

// select_kernel plus per-group row counts (integer atomics: the totals do not depend on their order).
__global__ void __launch_bounds__(kSelectWarps * 32) count_groups_kernel(CallView c) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < c.M * c.k_groups && group_is_local(c, c.sel[i])) atomicAdd(&c.group_count[c.sel[i]], 1);
}

// One block per group: the group's place in the bucket array and in the union list (prefix sums over the
// per-group counts, recomputed by every block), then an ordered compaction of the rows that selected it.
__global__ void __launch_bounds__(256) bucket_group_kernel(CallView c, int* __restrict__ count_acc) {
    __shared__ int s_cnt[kMaxGroups], s_pass[kMaxGroups];
    __shared__ int s_warp[8];
    const int n = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_wait();                   // (launched over the tail of the kernel that selects and counts)
    pdl_launch_dependents();
    {
        // counts: group_count (filled by count_groups_kernel), or the accumulators of route_mid_kernel, which
        // the last block to have read them clears for the next call
        const int t = threadIdx.x;
        const int cnt = t < c.N ? (count_acc ? __ldcg(count_acc + t) : c.group_count[t]) : 0;
        s_cnt[t] = cnt;
        s_pass[t] = cnt == 0 ? 0 : (c.pass_rows > 0 ? (cnt + c.pass_rows - 1) / c.pass_rows : 1);
    }
    __syncthreads();
    int off = 0, virt = 0, uni = 0, tot = 0, vtot = 0;
    for (int t = 0; t < c.N; ++t) {           // N <= 256 shared-memory reads, same in every thread
        if (t < n) { off += s_cnt[t]; virt += s_pass[t]; }
        tot += s_cnt[t];
        vtot += s_pass[t];
        uni += s_cnt[t] > 0;
    }
    const int cnt = s_cnt[n], passes = s_pass[n];
    if (threadIdx.x == 0) {
        c.group_offset[n] = off;
        if (count_acc) {
            c.group_count[n] = cnt;
            const int ticket = atomicAdd(&c.state->ticket, 1);     // every block has read all counters by now
            if (ticket == (int)gridDim.x - 1) {
                for (int t = 0; t < c.N; ++t) count_acc[t] = 0;
                c.state->ticket = 0;
            }
        }
        c.union_rank[n] = cnt > 0 ? virt : -1;
        for (int p = 0; p < passes; ++p)
            if (virt + p < c.union_cap) c.union_list[virt + p] = n | (p << 16);
        if (n == 0) {
            c.group_offset[c.N] = tot;
            c.state->n_union = uni;
            c.state->n_virtual = min(vtot, c.union_cap);
        }
    }
    int running = 0;
    for (int m0 = 0; m0 < c.M; m0 += 256) {
        const int m = m0 + threadIdx.x;
        const int sl = (m < c.M && cnt > 0) ? (int)c.slot_of[(size_t)m * c.N + n] : -1;   // cnt = 0: not this GPU's group
        const unsigned bal = __ballot_sync(0xffffffffu, sl >= 0);
        if (lane == 0) s_warp[warp] = __popc(bal);
        __syncthreads();
        int before = 0, all = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            if (w < warp) before += s_warp[w];
            all += s_warp[w];
        }
        if (sl >= 0) {
            const int pos = running + before + __popc(bal & ((1u << lane) - 1u));
            if (CORAL_IDX_OK(off + pos, c.cap_pairs, c.state) && CORAL_IDX_OK(m * c.k_groups + sl, c.cap_pairs, c.state)) {
            c.bucket_row[off + pos] = m;
            c.bucket_slot[off + pos] = sl;
            const int pass = c.pass_rows > 0 ? pos / c.pass_rows : 0;
            c.slot_desc[(size_t)m * c.k_groups + sl] = ((virt + pass) << 8) | ((pos - pass * max(c.pass_rows, 1)) & 255);
            if (c.bucket_dst && c.pass_rows == kTcPassRows)
                c.bucket_dst[off + pos] = tc_entry_row(off + pass * kTcPassRows, virt + pass) + pos - pass * kTcPassRows;
            }
        }
        running += all;
        __syncthreads();
    }
}


// ---- two-layer router of the paper's Eq. 7: scores = W2 (act(W1 h) + h), act = SiLU ---------------------------

// u[m][i] = SiLU(W1[i] . h[m]) + h[m][i] in fp32, for a tile of 8 output columns x 8 rows per block.
// grid (ceil(H/8), ceil(M/8)).
__global__ void __launch_bounds__(256) router_hidden_kernel(CallView c, const uint16_t* __restrict__ W1,
                                                            float* __restrict__ u) {
    __shared__ float s_red[8][kGateTile * kGateTile];
    const int i0 = blockIdx.x * kGateTile, m0 = blockIdx.y * kGateTile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = c.H >> 3;
    float acc[kGateTile][kGateTile];
#pragma unroll
    for (int g = 0; g < kGateTile; ++g)
#pragma unroll
        for (int r = 0; r < kGateTile; ++r) acc[g][r] = 0.f;
    for (int ch = threadIdx.x; ch < chunks; ch += 256) {
        float hf[kGateTile][8];
#pragma unroll
        for (int r = 0; r < kGateTile; ++r) {
            const uint4 q = (m0 + r < c.M) ? __ldg(reinterpret_cast<const uint4*>(c.hidden + (size_t)(m0 + r) * c.H) + ch)
                                           : make_uint4(0, 0, 0, 0);
            hf[r][0] = bf16_lo(q.x); hf[r][1] = bf16_hi(q.x); hf[r][2] = bf16_lo(q.y); hf[r][3] = bf16_hi(q.y);
            hf[r][4] = bf16_lo(q.z); hf[r][5] = bf16_hi(q.z); hf[r][6] = bf16_lo(q.w); hf[r][7] = bf16_hi(q.w);
        }
#pragma unroll
        for (int g = 0; g < kGateTile; ++g) {
            const uint4 q = (i0 + g < c.H) ? __ldg(reinterpret_cast<const uint4*>(W1 + (size_t)(i0 + g) * c.H) + ch)
                                           : make_uint4(0, 0, 0, 0);
            const float w[8] = {bf16_lo(q.x), bf16_hi(q.x), bf16_lo(q.y), bf16_hi(q.y),
                                bf16_lo(q.z), bf16_hi(q.z), bf16_lo(q.w), bf16_hi(q.w)};
#pragma unroll
            for (int r = 0; r < kGateTile; ++r)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[g][r] = fmaf(w[e], hf[r][e], acc[g][r]);
        }
    }
#pragma unroll
    for (int g = 0; g < kGateTile; ++g)
#pragma unroll
        for (int r = 0; r < kGateTile; ++r) {
            const float sum = warp_sum(acc[g][r]);
            if (lane == 0) s_red[warp][g * kGateTile + r] = sum;
        }
    __syncthreads();
    if (threadIdx.x < kGateTile * kGateTile) {
        const int g = threadIdx.x / kGateTile, r = threadIdx.x % kGateTile;
        if (i0 + g < c.H && m0 + r < c.M) {
            float a = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) a += s_red[w][threadIdx.x];
            const float hv = __uint_as_float((uint32_t)c.hidden[(size_t)(m0 + r) * c.H + i0 + g] << 16);
            u[(size_t)(m0 + r) * c.H + i0 + g] = a / (1.f + expf(-a)) + hv;
        }
    }
}

// The same on the warp-level tensor cores (H a multiple of 32): a block owns 16 columns i of u (16 rows of W1) and
// walks over the query rows 32 at a time (four n-tiles sharing every load of W1), its 8 warps splitting H in
// blocks of 32 columns (mma.sync m16n8k16, bf16 x bf16 -> fp32; W1 rows on the M axis, query rows on N, the same
// column permutation in both operands).  The block's 128 KiB of W1 come from HBM once and from L1/L2 for the
// further row tiles.  grid H / 16.
constexpr int kRouterHiddenNT = 4;
__global__ void __launch_bounds__(256) router_hidden_mma_kernel(CallView c, const uint16_t* __restrict__ W1,
                                                                float* __restrict__ u) {
    __shared__ float s_part[8][kRouterHiddenNT * 16 * 8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, tq = lane & 3;
    const int i0 = blockIdx.x * 16;
    pdl_launch_dependents();
    const bool a_lo = i0 + gq < c.H, a_hi = i0 + gq + 8 < c.H;
    const uint16_t* wlo = W1 + (size_t)(a_lo ? i0 + gq : 0) * c.H + tq * 8;
    const uint16_t* whi = W1 + (size_t)(a_hi ? i0 + gq + 8 : 0) * c.H + tq * 8;
    const int kblocks = c.H >> 5;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    for (int m0 = 0; m0 < c.M; m0 += 8 * kRouterHiddenNT) {
        const uint16_t* hb[kRouterHiddenNT];
        bool b_ok[kRouterHiddenNT];
#pragma unroll
        for (int t = 0; t < kRouterHiddenNT; ++t) {
            b_ok[t] = m0 + t * 8 + gq < c.M;
            hb[t] = c.hidden + (size_t)(b_ok[t] ? m0 + t * 8 + gq : 0) * c.H + tq * 8;
        }
        float acc[kRouterHiddenNT][2][4];
#pragma unroll
        for (int t = 0; t < kRouterHiddenNT; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) { acc[t][0][e] = 0.f; acc[t][1][e] = 0.f; }
#pragma unroll 2
        for (int kb = warp; kb < kblocks; kb += 8) {
            const uint4 a = a_lo ? __ldg(reinterpret_cast<const uint4*>(wlo + kb * 32)) : zero;
            const uint4 b = a_hi ? __ldg(reinterpret_cast<const uint4*>(whi + kb * 32)) : zero;
            uint4 h[kRouterHiddenNT];
#pragma unroll
            for (int t = 0; t < kRouterHiddenNT; ++t)
                h[t] = b_ok[t] ? __ldg(reinterpret_cast<const uint4*>(hb[t] + kb * 32)) : zero;
#pragma unroll
            for (int t = 0; t < kRouterHiddenNT; ++t) {
                asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                             : "+f"(acc[t][0][0]), "+f"(acc[t][0][1]), "+f"(acc[t][0][2]), "+f"(acc[t][0][3])
                             : "r"(a.x), "r"(b.x), "r"(a.y), "r"(b.y), "r"(h[t].x), "r"(h[t].y));
                asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                             : "+f"(acc[t][1][0]), "+f"(acc[t][1][1]), "+f"(acc[t][1][2]), "+f"(acc[t][1][3])
                             : "r"(a.z), "r"(b.z), "r"(a.w), "r"(b.w), "r"(h[t].z), "r"(h[t].w));
            }
        }
        // accumulator layout: [0],[1] = W1 row gq, query rows 2*tq, 2*tq+1 of the n-tile; [2],[3] = W1 row gq + 8
        float* sp = s_part[warp];
#pragma unroll
        for (int t = 0; t < kRouterHiddenNT; ++t) {
            sp[t * 128 + gq * 8 + 2 * tq] = acc[t][0][0] + acc[t][1][0];
            sp[t * 128 + gq * 8 + 2 * tq + 1] = acc[t][0][1] + acc[t][1][1];
            sp[t * 128 + (gq + 8) * 8 + 2 * tq] = acc[t][0][2] + acc[t][1][2];
            sp[t * 128 + (gq + 8) * 8 + 2 * tq + 1] = acc[t][0][3] + acc[t][1][3];
        }
        __syncthreads();
        for (int e = threadIdx.x; e < kRouterHiddenNT * 128; e += 256) {
            const int t = e >> 7, g = (e >> 3) & 15, r = e & 7;
            const int m = m0 + t * 8 + r;
            if (i0 + g < c.H && m < c.M) {
                float a = 0.f;
#pragma unroll
                for (int w = 0; w < 8; ++w) a += s_part[w][e];
                const float hv = __uint_as_float((uint32_t)c.hidden[(size_t)m * c.H + i0 + g] << 16);
                u[(size_t)m * c.H + i0 + g] = a / (1.f + expf(-a)) + hv;
            }
        }
        __syncthreads();
    }
}

// g[m][n] = W_gate[n] . u[m] with u in fp32.  grid (N, ceil(M/8)); block (0,0) clears the per-group counters.
__global__ void __launch_bounds__(kGateThreads) gate_f32_kernel(CallView c, float* __restrict__ gate_tap) {
    const int n = blockIdx.x;
    const int m0 = blockIdx.y * kGateRows;
    const int rows = min(kGateRows, c.M - m0);
    const int chunks = c.H >> 3;
    pdl_wait();                   // router_in is complete from here on
    if (blockIdx.x == 0 && blockIdx.y == 0)
        for (int t = threadIdx.x; t < c.N; t += kGateThreads) c.group_count[t] = 0;
    const uint4* __restrict__ wg = reinterpret_cast<const uint4*>(c.w_gate + (size_t)n * c.H);
    float acc[kGateRows];
#pragma unroll
    for (int r = 0; r < kGateRows; ++r) acc[r] = 0.f;
    for (int ch = threadIdx.x; ch < chunks; ch += kGateThreads) {
        const uint4 q = __ldg(wg + ch);
        const float w[8] = {bf16_lo(q.x), bf16_hi(q.x), bf16_lo(q.y), bf16_hi(q.y),
                            bf16_lo(q.z), bf16_hi(q.z), bf16_lo(q.w), bf16_hi(q.w)};
#pragma unroll
        for (int r = 0; r < kGateRows; ++r) {
            if (r < rows) {
                const float4* up = reinterpret_cast<const float4*>(c.router_in + (size_t)(m0 + r) * c.H) + 2 * ch;
                const float4 a = __ldg(up), b = __ldg(up + 1);
                acc[r] = fmaf(w[0], a.x, acc[r]); acc[r] = fmaf(w[1], a.y, acc[r]);
                acc[r] = fmaf(w[2], a.z, acc[r]); acc[r] = fmaf(w[3], a.w, acc[r]);
                acc[r] = fmaf(w[4], b.x, acc[r]); acc[r] = fmaf(w[5], b.y, acc[r]);
                acc[r] = fmaf(w[6], b.z, acc[r]); acc[r] = fmaf(w[7], b.w, acc[r]);
            }
        }
    }
    __shared__ float red[kGateThreads / 32][kGateRows];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int r = 0; r < kGateRows; ++r) {
        const float sum = warp_sum(acc[r]);
        if (lane == 0) red[warp][r] = sum;
    }
    __syncthreads();
    if (threadIdx.x < rows) {
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < kGateThreads / 32; ++w) sum += red[w][threadIdx.x];
        c.gate[(size_t)(m0 + threadIdx.x) * c.N + n] = sum;
        if (gate_tap) gate_tap[(size_t)(m0 + threadIdx.x) * c.N + n] = sum;
    }
}

}  // namespace coral
