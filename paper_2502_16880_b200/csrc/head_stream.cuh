// Gathered GEMV / small grouped GEMM for the draft step, streaming version.
//
// Every touched group's vocab rows are read exactly once per pass: a producer
// warp issues one bulk asynchronous copy (cp.async.bulk, mbarrier completion)
// per 16-row x kc-column slab (16 KiB, contiguous in the packed layout) into a
// shared-memory ring.  Eight MMA warps split each slab's columns between them and
// multiply it with their slice of the
// group's hidden rows, which they keep in registers as bf16 MMA operands
// (mma.sync m16n8k16, fp32 accumulators: vocab rows on the M axis, up to 16
// hidden rows on the N axis).  Per 16-row item the MMA warps drop their partial
// sums into one of four shared-memory buffers and carry on; three further warps
// pick the buffers up, add the eight partials and fold the 16 logits of every
// hidden row into a running (max, sum-exp, top-k) that is written once per
// (CTA, group) segment.  The MMA warps therefore never wait for the statistics.
// (CORAL Section 3.3: logits only for the activated groups, softmax over them;
// Appendix B: top candidates per row, union of the rows' groups.)
//
// A group selected by more than 16 rows is streamed in ceil(R/16) passes; each
// (group, pass) is a "virtual group" of the union list.
// Work split: the virtual groups' rows form n_virtual * T items of 16 rows; CTA b
// owns the contiguous run [b*per, (b+1)*per), so all CTAs stream the same bytes.
#pragma once
#include "common.cuh"

namespace coral {

constexpr int kStreamTile = 16;                 // vocab rows per item (the MMA's M)
constexpr int kStreamWarps = 8;                 // MMA warps (warps 0..7)
constexpr int kStreamStatWarps = 3;             // statistics warps (warps 8..10); warp 11 is the producer
constexpr int kStreamThreads = (kStreamWarps + kStreamStatWarps + 1) * 32;
constexpr int kStreamZBufs = 4;                 // buffers of per-item partial sums between the two roles
constexpr int kStreamSegTab = 64;               // capacity of the per-CTA segment table
constexpr int kStreamPassRows = 16;             // hidden rows per pass (two n-tiles of 8)
constexpr int kStreamMaxH = 4096;               // 16 k-blocks of 32 columns per warp
constexpr int kStreamMaxM = 128;                // beyond this the pass count makes the path pointless
constexpr int kStreamSpin = 1 << 20;            // bound of every mbarrier wait
constexpr int kStreamSpinAfterAbort = 1 << 8;

struct StreamGeom {
    int grid;         // CTAs launched
    int kc;           // columns per slab (512, or 256 when H is not a multiple of 512)
    int kstages;      // slabs per item = H / kc
    int n_stages;     // ring depth
    int seg_max;      // most virtual groups one CTA's run can overlap
    int T;            // items per group = ceil(v / kStreamTile)
    int stage_bytes;  // 16 rows x kc columns: one slab, contiguous in the packed copy as kc / 64 blocks of [16][64]
    int tc_rows;      // rows per pass of the tensor-core kernel's partial layout
    int tc_tiles;     // 0: partials come from the streaming kernel; > 0: from the tensor-core kernel, which
                      // writes one partial per (pass, sub-tile, row) with this many sub-tiles per pass
};

// One partial per (CTA, segment, hidden row of the pass).
struct StreamPartials {
    float* pmax;      // [grid][seg_max][kStreamPassRows]
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
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}


__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// D += A(16x16, bf16, row) * B(16x8, bf16, col), fp32 accumulate.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct StreamShared {
    unsigned char* ring;      // n_stages * stage_bytes
    float* zpart;             // [kStreamZBufs][kStreamWarps][kStreamTile][kStreamPassRows]
    uint64_t* full;           // [n_stages] completion of the copy into a slot
    uint64_t* empty;          // [n_stages] all MMA warps have finished reading the slot
    uint64_t* zfull;          // [kStreamZBufs] all MMA warps have written the buffer
    uint64_t* zfree;          // [kStreamZBufs] all statistics warps have read the buffer
    int* segtab;              // [kStreamSegTab] union_list entries of this CTA's run
    volatile int* abort_flag;
    volatile int* issued;     // slabs the producer has issued so far
    int lo, hi, j_first;      // this CTA's run of items and its first virtual group
};

// Fold the 16 logits of one item into a warp's running statistics of one hidden row.  Lane i < rows holds
// the logit of tile row i.  Softmax part: every lane keeps an online (max, sum-exp) over the values it has
// seen, combined across lanes once per segment.  Top-k part: the sorted list lives one entry per lane
// (entry i in lane i < k_tokens); a value that can beat the current k-th entry is inserted by shifting the
// tail of the list one lane up, so the common case (no candidate) costs one ballot.
__device__ __forceinline__ void fold_item(float zv, const int32_t* __restrict__ tokens, bool have, int k_tokens,
                                          int lane, float& lane_max, float& lane_sum, float& lv, int& lid,
                                          float& kth, int& kth_id) {
    if (have) {
        const float nmax = fmaxf(lane_max, zv);
        lane_sum = lane_sum * __expf(lane_max - nmax) + __expf(zv - nmax);   // exp(-inf) = 0 the first time
        lane_max = nmax;
    }
    unsigned cand = __ballot_sync(0xffffffffu, have && (kth_id == kNoToken || zv >= kth));
    if (cand == 0) return;
    const int tok = ((cand >> lane) & 1u) ? __ldg(tokens + lane) : kNoToken;
    while (cand) {
        const int src = __ffs(cand) - 1;
        cand &= cand - 1;
        const float v = __shfl_sync(0xffffffffu, zv, src);
        const int id = __shfl_sync(0xffffffffu, tok, src);
        const int pos = __popc(__ballot_sync(0xffffffffu, better(lv, lid, v, id)));   // entries that stay ahead
        const float up_v = __shfl_up_sync(0xffffffffu, lv, 1);
        const int up_id = __shfl_up_sync(0xffffffffu, lid, 1);
        if (pos < k_tokens) {
            if (lane == pos) { lv = v; lid = id; }
            else if (lane > pos && lane < k_tokens) { lv = up_v; lid = up_id; }
        }
    }
    kth = __shfl_sync(0xffffffffu, lv, k_tokens - 1);
    kth_id = __shfl_sync(0xffffffffu, lid, k_tokens - 1);
}

// MMA side of one segment: items [lo, hi) of the run, all inside virtual group j = (group n, pass) with R
// hidden rows.  NT n-tiles of 8 hidden rows.  A slab (16 vocab rows x kc columns) belongs to ONE warp: slab ks
// of every item to warp ks % 8, which multiplies it with its own kc columns of the hidden rows (held in
// registers) and frees the slot by itself, so the warps never wait for each other on the ring; their partial
// sums meet in the item's z-buffer.  KBW = 2: kc = 512, one slab per warp and item; KBW = 1: kc = 256, up to two.
template <int NT, int KBW>
__device__ __forceinline__ void stream_segment_mma(const CallView& c, const StreamGeom& g, const StreamShared& sh,
                                                   int n, int pass, int R, int lo, int hi, int& it) {
    constexpr int KBS = 8 * KBW;          // 32-column blocks per slab
    constexpr int SL = 2 / KBW;           // slabs of an item this warp can own
    const int cw = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gq = lane >> 2, tq = lane & 3;
    const int off = c.group_offset[n] + pass * kStreamPassRows;

    // B operands: hidden row (nt*8 + gq), the lane's 8 columns of every 32-column block of this warp's slabs
    uint4 breg[NT][16];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int rr = nt * 8 + gq;
        const bool valid = rr < R;
        const uint16_t* hp = c.hidden + (size_t)(valid ? CORAL_IDX(c.bucket_row[CORAL_IDX(off + rr, c.cap_pairs, c.state)], c.M, c.state) : 0) * c.H;
#pragma unroll
        for (int sl = 0; sl < SL; ++sl)
#pragma unroll
            for (int i = 0; i < KBS; ++i) {
                const int ks = cw + kStreamWarps * sl;
                uint4 hv = make_uint4(0, 0, 0, 0);
                if (valid && ks < g.kstages) hv = __ldg(reinterpret_cast<const uint4*>(hp + ks * g.kc + i * 32 + tq * 8));
                breg[nt][sl * KBS + i] = hv;
            }
    }
    const uint32_t ring = smem_u32(sh.ring);

    for (int item = lo; item < hi; ++item, ++it) {
        float acc[NT][2][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) { acc[nt][0][e] = 0.f; acc[nt][1][e] = 0.f; }
#pragma unroll
        for (int sl = 0; sl < SL; ++sl) {
            const int ks = cw + kStreamWarps * sl;
            if (ks < g.kstages) {
                const int idx = it * g.kstages + ks;            // position of the slab in the CTA's stream
                const int stage = idx % g.n_stages;
                // A warp may run several items ahead of the slowest one, i.e. more than one turn of the ring:
                // the parity wait below is only meaningful once the slot's barrier has entered the phase of this
                // very slab, which the producer announces after issuing its copy.
                {
                    const int limit = *sh.abort_flag ? kStreamSpinAfterAbort : kStreamSpin;
                    int i = 0;
                    while (*sh.issued <= idx && ++i < limit) {}
                    if (*sh.issued <= idx) { *sh.abort_flag = 1; set_status(c.state, -5); }
                    __threadfence_block();
                }
                mbar_wait(smem_u32(&sh.full[stage]), (uint32_t)(idx / g.n_stages) & 1u, sh.abort_flag, c.state);
                const uint32_t sp = ring + (uint32_t)stage * g.stage_bytes;
#pragma unroll
                for (int i = 0; i < KBS; ++i) {
                    const uint32_t cs = (uint32_t)(i * 32 + tq * 8);            // column inside the slab
                    const uint32_t at = sp + (cs >> 6) * 2048u + (uint32_t)gq * 128u + (cs & 63u) * 2u;
                    const uint4 wg = lds128(at);
                    const uint4 wh = lds128(at + 1024u);                        // row gq + 8
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint4 b = breg[nt][sl * KBS + i];
                        mma_bf16_16816(acc[nt][0], wg.x, wh.x, wg.y, wh.y, b.x, b.y);
                        mma_bf16_16816(acc[nt][1], wg.z, wh.z, wg.w, wh.w, b.z, b.w);
                    }
                }
                // The slot is refilled by a bulk copy (async proxy) as soon as it is released, and this warp has just
                // read it with ordinary shared-memory loads (generic proxy): order the two before letting go.
                // (Without this fence the first item after a change of segment, where the producer is already
                // waiting for this very slot, was occasionally computed from a half-overwritten slab.)
                __syncwarp();
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                if (lane == 0) mbar_arrive(smem_u32(&sh.empty[stage]));
            }
        }
        // this warp's partial sums over its columns: rows gq, gq+8; hidden rows nt*8 + 2*tq, +1
        const int zb = it % kStreamZBufs;
        mbar_wait(smem_u32(&sh.zfree[zb]), ((uint32_t)(it / kStreamZBufs) & 1u) ^ 1u, sh.abort_flag, c.state);
        float* zp = sh.zpart + ((size_t)(zb * kStreamWarps + cw) * kStreamTile) * kStreamPassRows;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            *reinterpret_cast<float2*>(zp + gq * kStreamPassRows + nt * 8 + 2 * tq) =
                make_float2(acc[nt][0][0] + acc[nt][1][0], acc[nt][0][1] + acc[nt][1][1]);
            *reinterpret_cast<float2*>(zp + (gq + 8) * kStreamPassRows + nt * 8 + 2 * tq) =
                make_float2(acc[nt][0][2] + acc[nt][1][2], acc[nt][0][3] + acc[nt][1][3]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh.zfull[zb]));
    }
}

// Statistics side of one segment.  Warp sw (0..2) owns hidden rows sw, sw+3, sw+6, ... of the pass.
__device__ __forceinline__ void stream_segment_stats(const CallView& c, const StreamGeom& g, const StreamShared& sh,
                                                     const StreamPartials& pp, float* __restrict__ logits_tap, int n,
                                                     int pass, int R, int j, int lo, int hi, int seg, int& it) {
    constexpr int kOwn = (kStreamPassRows + kStreamStatWarps - 1) / kStreamStatWarps;
    const int sw = (threadIdx.x >> 5) - kStreamWarps, lane = threadIdx.x & 31;
    const int off = c.group_offset[n] + pass * kStreamPassRows;
    float run_max[kOwn], run_sum[kOwn], lv[kOwn], kth[kOwn];
    int lid[kOwn], kth_id[kOwn], my_m[kOwn], my_slot[kOwn];
#pragma unroll
    for (int u = 0; u < kOwn; ++u) {
        run_max[u] = kNegInf; run_sum[u] = 0.f; lv[u] = kNegInf; lid[u] = kNoToken;
        kth[u] = kNegInf; kth_id[u] = kNoToken;
        const int r = sw + kStreamStatWarps * u;
        my_m[u] = r < R ? CORAL_IDX(c.bucket_row[CORAL_IDX(off + r, c.cap_pairs, c.state)], c.M, c.state) : 0;
        my_slot[u] = r < R ? CORAL_IDX(c.bucket_slot[CORAL_IDX(off + r, c.cap_pairs, c.state)], c.k_groups, c.state) : 0;
    }
    for (int item = lo; item < hi; ++item, ++it) {
        const int row0 = (item - j * g.T) * kStreamTile;
        const int rows = min(kStreamTile, c.v - row0);
        const bool have = lane < rows;
        const int32_t* tokens = c.group_tokens + CORAL_IDX((size_t)n * c.v + row0, c.V, c.state);
        const int zb = it % kStreamZBufs;
        mbar_wait(smem_u32(&sh.zfull[zb]), (uint32_t)(it / kStreamZBufs) & 1u, sh.abort_flag, c.state);
        float zv[kOwn];
#pragma unroll
        for (int u = 0; u < kOwn; ++u) {
            const int r = sw + kStreamStatWarps * u;
            zv[u] = kNegInf;
            if (r < R && have) {
                const float* zr = sh.zpart + ((size_t)(zb * kStreamWarps) * kStreamTile + lane) * kStreamPassRows + r;
                float z = 0.f;
#pragma unroll
                for (int w = 0; w < kStreamWarps; ++w) z += zr[(size_t)w * kStreamTile * kStreamPassRows];
                zv[u] = z;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh.zfree[zb]));      // the buffer is in registers now
#pragma unroll
        for (int u = 0; u < kOwn; ++u) {
            const int r = sw + kStreamStatWarps * u;
            if (r < R) {
                if (logits_tap && have)
                    logits_tap[((size_t)my_m[u] * c.k_groups + my_slot[u]) * c.v + row0 + lane] = zv[u];
                fold_item(zv[u], tokens, have, c.k_tokens, lane, run_max[u], run_sum[u], lv[u], lid[u], kth[u], kth_id[u]);
            }
        }
    }
#pragma unroll
    for (int u = 0; u < kOwn; ++u) {
        const int r = sw + kStreamStatWarps * u;
        if (r < R) {
            const size_t p = ((size_t)blockIdx.x * g.seg_max + seg) * kStreamPassRows + r;
            const bool p_ok = CORAL_IDX_OK(p, c.cap_part_stream, c.state);
            const float mx = warp_max(run_max[u]);                       // combine the lanes' online softmax states
            const float sm = warp_sum(run_sum[u] * __expf(run_max[u] - mx));
            if (p_ok && lane == 0) { pp.pmax[p] = mx; pp.psum[p] = sm; }
            if (p_ok && lane < c.k_tokens) { pp.pval[p * c.k_tokens + lane] = lv[u]; pp.pid[p * c.k_tokens + lane] = lid[u]; }
        }
    }
}

// grid = g.grid CTAs of kStreamThreads threads; dynamic shared memory laid out as StreamShared.
template <int KBW>
__global__ void __launch_bounds__(kStreamThreads, 1) head_stream_kernel(CallView c, StreamGeom g, StreamPartials pp,
                                                                        float* __restrict__ logits_tap) {
    extern __shared__ __align__(128) unsigned char stream_smem_raw[];
    unsigned char* smem_raw = stream_smem_raw;
    StreamShared sh;
    sh.ring = smem_raw;
    size_t o = (size_t)g.n_stages * g.stage_bytes;
    sh.zpart = reinterpret_cast<float*>(smem_raw + o);
    o += sizeof(float) * kStreamZBufs * kStreamWarps * kStreamTile * kStreamPassRows;
    sh.full = reinterpret_cast<uint64_t*>(smem_raw + o);
    o += sizeof(uint64_t) * g.n_stages;
    sh.zfull = reinterpret_cast<uint64_t*>(smem_raw + o);
    o += sizeof(uint64_t) * kStreamZBufs;
    sh.zfree = reinterpret_cast<uint64_t*>(smem_raw + o);
    o += sizeof(uint64_t) * kStreamZBufs;
    sh.empty = reinterpret_cast<uint64_t*>(smem_raw + o);
    o += sizeof(uint64_t) * g.n_stages;
    sh.segtab = reinterpret_cast<int*>(smem_raw + o);
    o += sizeof(int) * kStreamSegTab;
    sh.abort_flag = reinterpret_cast<volatile int*>(smem_raw + o);
    sh.issued = sh.abort_flag + 1;

    pdl_wait();                   // the router stage's outputs are complete from here on
    pdl_launch_dependents();      // the merge kernel may start reading the router's outputs
    if (call_is_poisoned(c.state)) return;                   // the router stage reported a problem: index with nothing
    if (c.adaptive && c.state->path_choice != 1) return;     // the router chose the tensor-core kernel for this call
    const int n_items = c.state->n_virtual * g.T;
    const int per = (n_items + g.grid - 1) / g.grid;
    sh.lo = min(n_items, (int)blockIdx.x * per);
    sh.hi = min(n_items, sh.lo + per);
    if (sh.lo >= sh.hi) return;
    sh.j_first = sh.lo / g.T;
    const int n_segs = min((sh.hi - 1) / g.T - sh.j_first + 1, kStreamSegTab);

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.n_stages; ++s) {
            mbar_init(smem_u32(&sh.full[s]), 1);
            mbar_init(smem_u32(&sh.empty[s]), 1);           // a slab is read, and its slot freed, by one warp
        }
        for (int b = 0; b < kStreamZBufs; ++b) {
            mbar_init(smem_u32(&sh.zfull[b]), kStreamWarps);
            mbar_init(smem_u32(&sh.zfree[b]), kStreamStatWarps);
        }
        *sh.abort_flag = 0;
        *sh.issued = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x < n_segs) sh.segtab[threadIdx.x] = c.union_list[sh.j_first + threadIdx.x];
    __syncthreads();

    const int cw = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (cw == kStreamWarps + kStreamStatWarps) {
        // producer: one contiguous copy per slab; a slab's valid rows are a prefix of its 16 rows
        if (lane != 0) return;
        int stage = 0, n_issued = 0;
        uint32_t phase = 0;
        uint64_t pol_keep = 0;
        if (c.hot_groups > 0) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
        for (int pos = sh.lo; pos < sh.hi;) {
            const int j = pos / g.T;
            const int seg_hi = min(sh.hi, (j + 1) * g.T);
            const int n = sh.segtab[min(j - sh.j_first, kStreamSegTab - 1)] & 0xffff;
            int t = pos - j * g.T;
            const uint16_t* src = c.packed + (((size_t)(n / c.pack_div) * g.T + t) * g.kstages) * (size_t)(kStreamTile * g.kc);
#ifdef CORAL_CHECK_BOUNDS
            {   // the whole run of slabs copied for this segment must lie inside the packed copy
                const long long first16 = (src - c.packed) / 8, n16 = (long long)(seg_hi - pos) * g.kstages * (g.stage_bytes / 16);
                if (!CORAL_IDX_OK(n, c.N, c.state) || !CORAL_IDX_OK(first16 + n16 - 1, c.cap_packed, c.state)) src = c.packed;
            }
#endif
            for (int item = pos; item < seg_hi; ++item, ++t) {
                const uint32_t bytes = (uint32_t)g.stage_bytes;    // rows past the group's size are zero padding
                for (int ks = 0; ks < g.kstages; ++ks) {
                    mbar_wait(smem_u32(&sh.empty[stage]), phase ^ 1u, sh.abort_flag, c.state);
                    const uint32_t bar = smem_u32(&sh.full[stage]);
                    mbar_expect_tx(bar, bytes);
                    if (n < c.hot_groups)      // a hot group: ask L2 to keep its lines when others have to go
                        bulk_g2s_hint(smem_u32(sh.ring + (size_t)stage * g.stage_bytes), src, bytes, bar, pol_keep);
                    else
                        bulk_g2s(smem_u32(sh.ring + (size_t)stage * g.stage_bytes), src, bytes, bar);
                    __threadfence_block();
                    *sh.issued = ++n_issued;      // the slot's barrier is now in the phase of this slab
                    src += (size_t)kStreamTile * g.kc;
                    if (++stage == g.n_stages) { stage = 0; phase ^= 1u; }
                }
            }
            pos = seg_hi;
        }
        return;
    }
    const bool mma_role = cw < kStreamWarps;

    // both roles walk the run segment by segment (one virtual group each)
    int it = 0;
    for (int pos = sh.lo; pos < sh.hi;) {
        const int j = pos / g.T;
        const int seg = min(j - sh.j_first, kStreamSegTab - 1);
        const int seg_hi = min(sh.hi, (j + 1) * g.T);
        const int entry = sh.segtab[seg];
        const int n = CORAL_IDX(entry & 0xffff, c.N, c.state), pass = entry >> 16;
        const int R = max(1, min(c.group_count[n] - pass * kStreamPassRows, kStreamPassRows));
        if (!mma_role)
            stream_segment_stats(c, g, sh, pp, logits_tap, n, pass, R, j, pos, seg_hi, seg, it);
        else if (R <= 8)
            stream_segment_mma<1, KBW>(c, g, sh, n, pass, R, pos, seg_hi, it);
        else
            stream_segment_mma<2, KBW>(c, g, sh, n, pass, R, pos, seg_hi, it);
        pos = seg_hi;
    }
}

// Merge for the streaming and tensor-core paths: block per row.  The pieces of row m, slot s are the partials
// that the CTAs overlapping that slot's (group, pass) wrote for the row's position in the pass.  Every piece
// holds a sorted top-k list, so two lower bounds of the row's k-th value are at hand: the largest of the
// pieces' k-th entries, and the k-th largest of the pieces' first entries.  Only candidates at or above the
// better bound are kept, and those few are ranked by counting.
// Output modes: joint (log-softmax over all active logits of the row) adds -LSE_row to every logit;
// factorised (CORAL Eq. 8, p(x) = p_router(n) p_group(x)) adds log p_router(n) - LSE_group(n), a per-slot
// offset, where p_router is the softmax of the row's N gate scores (Eq. 7).  Adding a per-slot constant
// keeps every piece's list sorted, so both modes share the selection code.
// Partial mode (vocab sharding over several GPUs): the row's record of 2 + 2 k_tokens words - max, sum of
// exp(z - max), the k_tokens best raw logits (descending), their token ids - over the groups this GPU
// computed, written to `out_logprobs` (as a [M][2 + 2 k_tokens] word array); slots whose group belongs to
// another GPU have descriptor -1 and no pieces.  merge_partials_kernel combines the GPUs' records.
constexpr int kMergeJoint = 0, kMergeFactorised = 1, kMergePartial = 2, kMergeFactorisedRenorm = 3;
constexpr int kMergeStreamThreads = 256;
constexpr int kMergeMaxPieces = 2048;         // >= grid + 2 * k_groups for every supported shape
constexpr int kMergeRankMax = 256;            // survivors ranked by counting; more fall back to k rounds
__global__ void __launch_bounds__(kMergeStreamThreads) merge_stream_kernel(CallView c, StreamGeom g_in, StreamPartials pp_in,
                                                                           StreamGeom g_tc, StreamPartials pp_tc,
                                                                           float* __restrict__ cand_val_scratch,
                                                                           int32_t* __restrict__ cand_id_scratch,
                                                                           int cand_cap, int smem_cands, int p_cap, int mode,
                                                                           int32_t* __restrict__ out_ids,
                                                                           float* __restrict__ out_logprobs,
                                                                           float* __restrict__ lse_tap) {
    extern __shared__ __align__(16) unsigned char msm[];
    // adaptive call: the partials are those of the kernel the router chose (complete by the time this grid runs:
    // it is launched behind the tensor-core kernel, which does not release its dependents early)
    const bool took_tc = c.adaptive && c.state->path_choice == 2;
    const StreamGeom g = took_tc ? g_tc : g_in;
    const StreamPartials pp = took_tc ? pp_tc : pp_in;
    const int m = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kMergeStreamThreads / 32;
    const bool renorm = mode == kMergeFactorisedRenorm;      // p_router over the row's selected groups only
    const bool factorised = mode == kMergeFactorised || renorm, partial = mode == kMergePartial;
    float* rec = partial ? out_logprobs + (size_t)m * (2 + 2 * c.k_tokens) : nullptr;
    __shared__ float s_f[kWarps], s_t[kWarps];
    __shared__ float s_lse, s_glse, s_thr2;
    __shared__ int s_n, s_nlive;
    __shared__ int s_first[kMaxGroups], s_base[kMaxGroups + 1], s_rpos[kMaxGroups], s_j[kMaxGroups];
    __shared__ float s_off[kMaxGroups];           // per slot: what is added to a logit to give the emitted log-prob
    // dynamic shared memory: candidates (smem_cands values + ids), then per-piece arrays of capacity p_cap
    float* s_pm = reinterpret_cast<float*>(msm + (size_t)smem_cands * 8);
    float* s_ps = s_pm + p_cap;
    float* s_last = s_ps + p_cap;
    float* s_head = s_last + p_cap;
    int* s_piece = reinterpret_cast<int*>(s_head + p_cap);
    int* s_live = s_piece + p_cap;                // pieces that can hold a candidate
    unsigned char* s_pslot = reinterpret_cast<unsigned char*>(s_live + p_cap);

    // The router's outputs were complete before the streaming kernel let this grid start.
    if (call_is_poisoned(c.state)) return;        // the descriptors may be inconsistent: emit nothing (the status says why)
    const int n_items = c.state->n_virtual * g.T;
    const int per = max(1, (n_items + g.grid - 1) / g.grid);
    for (int s = threadIdx.x; s < c.k_groups; s += kMergeStreamThreads) {
        const int desc = c.slot_desc[(size_t)m * c.k_groups + s];
        const int j = desc < 0 ? 0 : desc >> 8;
        const int fb = g.tc_tiles > 0 ? j * g.tc_tiles : (j * g.T) / per;
        const int lb = g.tc_tiles > 0 ? fb + g.tc_tiles - 1 : ((j + 1) * g.T - 1) / per;
        s_first[s] = fb;
        s_base[s] = desc < 0 ? 0 : lb - fb + 1;       // piece count, turned into an exclusive prefix below
        s_j[s] = j;
        s_rpos[s] = desc & 255;
        s_off[s] = factorised ? c.gate[(size_t)m * c.N + c.sel[(size_t)m * c.k_groups + s]] : 0.f;
    }
    if (threadIdx.x == 0) { s_n = 0; s_nlive = 0; s_thr2 = kNegInf; }
    if (factorised) {                 // log-sum-exp of the row's N gate scores (kMergeStreamThreads >= N), or of
                                      // the k_groups selected ones in the renormalised variant
        const bool mine = renorm ? threadIdx.x < c.k_groups : threadIdx.x < c.N;
        const float gv = !mine ? kNegInf
                         : c.gate[(size_t)m * c.N + (renorm ? c.sel[(size_t)m * c.k_groups + threadIdx.x] : (int)threadIdx.x)];
        const float wm = warp_max(gv);
        if (lane == 0) s_f[warp] = wm;
        __syncthreads();
        float gm = s_f[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) gm = fmaxf(gm, s_f[w]);
        const float ws = warp_sum(mine ? expf(gv - gm) : 0.f);
        if (lane == 0) s_t[warp] = ws;
        __syncthreads();
        if (threadIdx.x == 0) {
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) tot += s_t[w];
            s_glse = gm + logf(tot);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int s = 0; s < c.k_groups; ++s) { const int cnt = s_base[s]; s_base[s] = run; run += cnt; }
        s_base[c.k_groups] = run;
    }
    __syncthreads();
    const int P = min(s_base[c.k_groups], p_cap);
    if (partial) {                 // defaults; a row none of whose groups is computed here keeps them
        if (threadIdx.x < c.k_tokens) {
            rec[2 + threadIdx.x] = kNegInf;
            reinterpret_cast<int32_t*>(rec)[2 + c.k_tokens + threadIdx.x] = kNoToken;
        }
        if (P == 0) {
            if (threadIdx.x == 0) { rec[0] = kNegInf; rec[1] = 0.f; }
            return;
        }
    }
    for (int q = threadIdx.x; q < P; q += kMergeStreamThreads) {
        int s = 0;
        while (s + 1 < c.k_groups && s_base[s + 1] <= q) ++s;
        const int b = s_first[s] + (q - s_base[s]);
        s_pslot[q] = (unsigned char)s;
        if (g.tc_tiles > 0) {
            s_piece[q] = b * g.tc_rows + s_rpos[s];       // (pass * tiles + sub-tile) * rows per pass + row
        } else {
            const int seg = s_j[s] - (b * per) / g.T;
            s_piece[q] = (int)(((size_t)b * g.seg_max + seg) * kStreamPassRows + s_rpos[s]);
        }
    }
    __syncthreads();

    pdl_wait();                   // partials of the streaming kernel are complete from here on

    // pass 1 over the pieces (all loads of a thread's pieces issued together)
    float mx = kNegInf;
    for (int q = threadIdx.x; q < P; q += kMergeStreamThreads) {
#ifdef CORAL_CHECK_BOUNDS
        if (!index_ok(s_piece[q], took_tc || g.tc_tiles > 0 ? c.cap_part_tc : c.cap_part_stream, c.state)) s_piece[q] = 0;
#endif
        const size_t p = (size_t)s_piece[q];
        const float a = pp.pmax[p], b = pp.psum[p];
        float l = pp.pval[p * c.k_tokens + c.k_tokens - 1], h = pp.pval[p * c.k_tokens];
        if (a == kNegInf) { l = kNegInf; h = kNegInf; }      // empty piece: its candidate list was not written
        s_pm[q] = a; s_ps[q] = b; s_last[q] = l; s_head[q] = h;
        mx = fmaxf(mx, a);
    }
    mx = warp_max(mx);
    if (lane == 0) s_f[warp] = mx;
    __syncthreads();
    mx = s_f[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) mx = fmaxf(mx, s_f[w]);
    float sum = 0.f;
    for (int q = threadIdx.x; q < P; q += kMergeStreamThreads) sum += s_ps[q] * expf(s_pm[q] - mx);
    sum = warp_sum(sum);
    if (lane == 0) s_t[warp] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot += s_t[w];
        s_lse = mx + logf(tot);
        if (lse_tap) lse_tap[m] = s_lse;
        if (partial) { rec[0] = mx; rec[1] = tot; }
    }
    __syncthreads();
    // per-slot offsets
    for (int s = threadIdx.x; s < c.k_groups; s += kMergeStreamThreads) {
        if (factorised) {
            float sm = kNegInf;
            for (int q = s_base[s]; q < min(s_base[s + 1], P); ++q) sm = fmaxf(sm, s_pm[q]);
            float ss = 0.f;
            for (int q = s_base[s]; q < min(s_base[s + 1], P); ++q) ss += s_ps[q] * expf(s_pm[q] - sm);
            s_off[s] = (s_off[s] - s_glse) - (sm + logf(ss));
        } else {
            s_off[s] = partial ? 0.f : -s_lse;
        }
    }
    __syncthreads();
    // thresholds on the emitted values
    float thr = kNegInf;
    for (int q = threadIdx.x; q < P; q += kMergeStreamThreads) {
        const float off = s_off[s_pslot[q]];
        thr = fmaxf(thr, s_last[q] + off);
        s_head[q] += off;
    }
    thr = warp_max(thr);
    if (lane == 0) s_f[warp] = thr;
    __syncthreads();
    thr = s_f[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) thr = fmaxf(thr, s_f[w]);
    // k-th largest first entry: the piece whose head is beaten by exactly k_tokens - 1 others (index breaks ties)
    for (int q = threadIdx.x; q < P; q += kMergeStreamThreads) {
        const float hq = s_head[q];
        int rank = 0;
        for (int i = 0; i < P; ++i) rank += better(s_head[i], i, hq, q) ? 1 : 0;
        if (rank == c.k_tokens - 1) s_thr2 = hq;
    }
    __syncthreads();
    thr = fmaxf(thr, s_thr2);

    // pass 2: keep the candidates at or above the threshold (order of arrival does not matter: the
    // ranking below is by the total order (value desc, token id asc)).  Only pieces whose first entry reaches
    // the threshold can hold one; they are listed first, then all their entries are fetched at once.
    const int C = P * c.k_tokens;
    const int cap = (C <= smem_cands) ? smem_cands : cand_cap;
    float* cv = (C <= smem_cands) ? reinterpret_cast<float*>(msm) : cand_val_scratch + (size_t)m * cand_cap;
    int32_t* ci = (C <= smem_cands) ? reinterpret_cast<int32_t*>(msm + sizeof(float) * smem_cands)
                                    : cand_id_scratch + (size_t)m * cand_cap;
    for (int q = threadIdx.x; q < P; q += kMergeStreamThreads)
        if (s_pm[q] != kNegInf && s_head[q] >= thr) s_live[atomicAdd(&s_nlive, 1)] = q;
    __syncthreads();
    const int n_entries = s_nlive * c.k_tokens;
    for (int e0 = threadIdx.x; e0 < n_entries; e0 += 4 * kMergeStreamThreads) {
        float v[4];
        int id[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int e = e0 + u * kMergeStreamThreads;
            v[u] = kNegInf;
            id[u] = kNoToken;
            if (e < n_entries) {
                const int q = s_live[e / c.k_tokens], l = e - (e / c.k_tokens) * c.k_tokens;
                const size_t p = (size_t)s_piece[q];
                v[u] = pp.pval[p * c.k_tokens + l] + s_off[s_pslot[q]];
                id[u] = pp.pid[p * c.k_tokens + l];
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (id[u] != kNoToken && v[u] >= thr) {
                const int at = atomicAdd(&s_n, 1);
                if (at < cap) { cv[at] = v[u]; ci[at] = id[u]; }
            }
        }
    }
    __syncthreads();
    const int S = min(s_n, cap);

    if (S <= kMergeRankMax) {
        // rank by counting: survivor i goes to output position (number of survivors that beat it)
        if (threadIdx.x < S) {
            const float v = cv[threadIdx.x];
            const int id = ci[threadIdx.x];
            int rank = 0;
            for (int i = 0; i < S; ++i) rank += better(cv[i], ci[i], v, id) ? 1 : 0;
            if (rank < c.k_tokens) {
                if (partial) {
                    rec[2 + rank] = v;
                    reinterpret_cast<int32_t*>(rec)[2 + c.k_tokens + rank] = id;
                } else {
                    out_ids[(size_t)m * c.k_tokens + rank] = id;
                    out_logprobs[(size_t)m * c.k_tokens + rank] = v;
                }
            }
        }
        return;
    }
    // many survivors (short or tied lists): k rounds of "best strictly after the last pick"
    __shared__ int s_i[kWarps];
    float last_v = __builtin_huge_valf();
    int last_id = -1;
    for (int k = 0; k < c.k_tokens; ++k) {
        float bv = kNegInf;
        int bk = kNoToken;
        for (int i = threadIdx.x; i < S; i += kMergeStreamThreads) {
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
            if (partial) {
                rec[2 + k] = bv;
                reinterpret_cast<int32_t*>(rec)[2 + c.k_tokens + k] = bk;
            } else {
                out_ids[(size_t)m * c.k_tokens + k] = bk;
                out_logprobs[(size_t)m * c.k_tokens + k] = bv;
            }
        }
        last_v = bv;
        last_id = bk;
    }
}

// Combines the records that `world` GPUs wrote in partial mode (records[r][m] = record of row m from rank r,
// 2 + 2 k_tokens words each): joint log-sum-exp over all ranks' active logits and the k_tokens best tokens
// of the row, emitted like the single-GPU merge (log-probabilities, descending, equal -> lower token id).
// grid M, block kMergePartialsThreads >= world * k_tokens.
constexpr int kMergePartialsThreads = 256;
__global__ void __launch_bounds__(kMergePartialsThreads)
    merge_partials_kernel(const float* __restrict__ records, int world, int M, int k_tokens,
                          int32_t* __restrict__ out_ids, float* __restrict__ out_logprobs) {
    __shared__ float s_v[kMergePartialsThreads];
    __shared__ int s_id[kMergePartialsThreads];
    __shared__ float s_lse;
    const int m = blockIdx.x;
    const int W = 2 + 2 * k_tokens;
    const int C = world * k_tokens;
    if (threadIdx.x == 0) {
        float mx = kNegInf;
        for (int r = 0; r < world; ++r) mx = fmaxf(mx, records[((size_t)r * M + m) * W]);
        float tot = 0.f;
        for (int r = 0; r < world; ++r) {
            const float* rec = records + ((size_t)r * M + m) * W;
            if (rec[0] != kNegInf) tot += rec[1] * expf(rec[0] - mx);
        }
        s_lse = mx + logf(tot);
    }
    if (threadIdx.x < C) {
        const int r = threadIdx.x / k_tokens, i = threadIdx.x - r * k_tokens;
        const float* rec = records + ((size_t)r * M + m) * W;
        s_v[threadIdx.x] = rec[2 + i];
        s_id[threadIdx.x] = reinterpret_cast<const int32_t*>(rec)[2 + k_tokens + i];
    }
    __syncthreads();
    if (threadIdx.x < C) {
        const float v = s_v[threadIdx.x];
        const int id = s_id[threadIdx.x];
        int rank = 0;
        for (int i = 0; i < C; ++i) rank += better(s_v[i], s_id[i], v, id) ? 1 : 0;
        if (rank < k_tokens) {
            out_ids[(size_t)m * k_tokens + rank] = id;
            out_logprobs[(size_t)m * k_tokens + rank] = v - s_lse;
        }
    }
}

}  // namespace coral
