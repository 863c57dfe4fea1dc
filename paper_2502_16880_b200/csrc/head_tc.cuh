// Routed grouped GEMM for many query rows on the 5th-generation tensor cores, computed by CTA pairs.
//
// For every (group, pass) entry of the union list the rows that selected the group (up to 256 per pass,
// gathered beforehand, see tc_gather_kernel) are multiplied with the group's vocab rows:
//   D[vocab row, hidden row] = sum_k W[vocab row, k] * hg[hidden row, k]
// One tcgen05.mma of the pair (cta_group::2, kind::f16, bf16 x bf16 -> fp32) has 256 vocab rows on its M axis
// - a sub-tile of 128 rows from each CTA - and the entry's hidden rows, rounded up to a multiple of 16, on its
// N axis.  The hidden rows are the shared operand: each CTA fetches only half of them and the instruction
// reads both halves, so per 64 columns a CTA takes in 16 KiB of weights per accumulator and n/2 x 128 bytes of
// hidden rows (with 120 rows and two accumulators: 40 KiB for 128 x 256 x 64 multiply-adds against 48 KiB when
// every CTA fetches all rows itself), and a group selected by up to 256 rows is streamed once.
//
// A unit is a pair of sub-tiles (sub-tile 2u of a group for rank 0, 2u + 1 for rank 1).  A batch is two units
// of one entry (two accumulators per CTA sharing the read of the hidden rows) when the entry has at most 128
// padded rows, else one unit with one accumulator of up to 256 columns; either way it fills half of the
// tensor memory, so the epilogue of one batch runs under the MMAs of the next.
//
// Epilogue.  A tensor-memory lane holds one vocab row and a column one hidden row, and a warp reads only its
// own quarter of the lanes; the per-row statistics need one thread per hidden row.  The four warps of an
// accumulator therefore exchange 32 x 32 blocks through shared memory: in step s warp q reads columns
// 32 ((q + s) mod 4) .. + 31 of its lanes and hands them to warp (q + s) mod 4, which owns those hidden rows
// and folds the block's 32 logits per row into its running (max, sum-exp, top-k), carried in registers over
// the sub-tiles the warp sees of an entry; logits never travel to HBM.  (CORAL Section 3.3: logits only for
// the activated groups; Appendix B: the union of the rows' groups is what gets read.)
//
// Warp roles: warp 0 = producer (TMA tiled loads of the weights, one bulk copy of the hidden rows), warp 1 =
// MMA issuer in the CTA of rank 0 and, in rank 1, the relay that tells rank 0 when a stage has landed;
// warps 2..9 = epilogue, four per accumulator (with one wide accumulator: four per half of its columns).
// Work split: the units of all entries form one list; pair p owns a contiguous run of it.
#pragma once
#include "tc_prims.cuh"

namespace coral {

constexpr int kTcPassRows = 256;                    // hidden rows per pass over a group's weights (the MMA's largest N)
constexpr int kTcStages = 4;
constexpr int kTcStageBytes = 40 * 1024;            // two weight tiles + up to 8 KiB of hidden rows, or one + up to 16 KiB
constexpr int kTcXchgBytes = 2 * 4 * 32 * 32 * 4;   // [accumulator][owner warp][32 vocab rows][32 hidden rows] fp32
constexpr size_t kTcSmemBytes = 1024 + (size_t)kTcStages * kTcStageBytes + kTcXchgBytes + 256;

struct TcGeom {
    int pairs;        // CTA pairs launched
    int tiles;        // sub-tiles per group = ceil(v / 128)
    int units;        // units per group = ceil(tiles / 2)
    int ksteps;       // ceil(H / 64) = 64-column blocks of the packed layout
    int hg_rows;      // rows of one column block of the gathered hidden matrix
};

struct TcPartials {
    float* pmax;      // [entry][tiles][kTcPassRows]
    float* psum;
    float* pval;      // [...][k_tokens]
    int32_t* pid;
};

// First row, in the gathered matrix, of the entry whose first bucket position is `first` and whose index in
// the union list is j: entries are packed in bucket order, each starting on a multiple of 16 rows (the step
// from one entry to the next is at least its row count rounded up to 16).
__host__ __device__ __forceinline__ int tc_entry_row(int first, int j) { return ((first + 15) & ~15) + 16 * j; }

// Gathers the hidden rows of every entry into the operand layout
//   hg[column block kb][row][64 columns]     (row = tc_entry_row(...) + position in the entry)
// with the 16-byte chunks of every 128-byte row permuted the way the 128-byte shared-memory swizzle wants
// them (chunk c of row r at position c ^ (r & 7)), so that a plain contiguous bulk copy of n/2 rows lands in
// shared memory as a K-major operand tile.  One thread block per (row, slot) pair in bucket order; columns
// past H are written as zero; rows between an entry's size and its padded size keep whatever they held
// (their accumulator columns are never read).
__global__ void __launch_bounds__(128) tc_gather_kernel(CallView c, uint16_t* __restrict__ hg, int hg_rows) {
    const int p = blockIdx.x;
    pdl_wait();                                              // launched over the tail of the router stage
    pdl_launch_dependents();
    if (call_is_poisoned(c.state)) return;                   // the router stage reported a problem: index with nothing
    if (c.adaptive && c.state->path_choice != 2) return;     // the router chose the streaming kernel for this call
    if (p >= c.group_offset[c.N]) return;          // fewer pairs than M * k_groups when the vocab is sharded
    const int m = c.bucket_row[p];
    const int n = c.sel[(size_t)m * c.k_groups + c.bucket_slot[p]];
    const int rg = p - c.group_offset[n];
    const int pass = rg / kTcPassRows;
    const int row = tc_entry_row(c.group_offset[n] + pass * kTcPassRows, c.union_rank[n] + pass) + rg % kTcPassRows;
    const uint4* src = reinterpret_cast<const uint4*>(c.hidden + (size_t)m * c.H);
    uint4* dst = reinterpret_cast<uint4*>(hg);
    const int chunks = c.H >> 3;
    for (int ch = threadIdx.x; ch < c.KB * 8; ch += 128)
        dst[((size_t)(ch >> 3) * hg_rows + row) * 8 + ((ch & 7) ^ (row & 7))] =
            ch < chunks ? __ldg(src + ch) : make_uint4(0, 0, 0, 0);
}

// Sorted insertion into a thread-private top-KT list (value desc, row index asc).
template <int KT>
__device__ __forceinline__ void tc_insert(float (&lv)[KT], int (&li)[KT], float v, int idx) {
#pragma unroll
    for (int j = 0; j < KT; ++j) {
        if (better(v, idx, lv[j], li[j])) {
            const float tv = lv[j];
            const int ti = li[j];
            lv[j] = v; li[j] = idx;
            v = tv; idx = ti;
        }
    }
}

// Running statistics of one hidden row over the sub-tiles one epilogue thread sees of an entry.
template <int KT>
struct TcRowState {
    float lv[KT];
    int li[KT];
    float mx, sum;
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int j = 0; j < KT; ++j) { lv[j] = kNegInf; li[j] = kNoToken; }
        mx = kNegInf;
        sum = 0.f;
    }
};

// Folds the logits of 32 vocab rows [base, base + 32) of the group (nv of them real) into the running
// statistics of one hidden row.  The values sit in a shared-memory block, element k at xb[k * 32 + (lane ^ k)].
template <int KT>
__device__ __forceinline__ void tc_fold_block(const CallView& c, TcRowState<KT>& st, const float* xb, int lane, int base,
                                              int nv, float* __restrict__ tap_row) {
    constexpr float kLog2e = 1.4426950408889634f;
    float z[32];
#pragma unroll
    for (int k = 0; k < 32; ++k) z[k] = xb[k * 32 + (lane ^ k)];
    float cm = kNegInf;
#pragma unroll
    for (int k = 0; k < 32; ++k) cm = fmaxf(cm, k < nv ? z[k] : kNegInf);
    const float nm = fmaxf(st.mx, cm);
    float add = 0.f;
#pragma unroll
    for (int k = 0; k < 32; ++k) add += k < nv ? exp2f((z[k] - nm) * kLog2e) : 0.f;
    st.sum = st.sum * exp2f((st.mx - nm) * kLog2e) + add;   // exp2(-inf) = 0 on the first block
    st.mx = nm;
    if (tap_row) {
#pragma unroll
        for (int k = 0; k < 32; ++k)
            if (k < nv) tap_row[base + k] = z[k];
    }
    // candidates for the top-k list: a bit per element that reaches the current k-th entry; the few that do are
    // fetched again by index from the block
    if (cm >= st.lv[KT - 1]) {
        unsigned cand = 0;
#pragma unroll
        for (int k = 0; k < 32; ++k) cand |= (k < nv && z[k] >= st.lv[KT - 1]) ? (1u << k) : 0u;   // ties are settled by the insertion
        while (cand) {
            const int k = __ffs(cand) - 1;
            cand &= cand - 1;
            const float zk = xb[k * 32 + (lane ^ k)];
            if (zk >= st.lv[KT - 1]) tc_insert<KT>(st.lv, st.li, zk, base + k);
        }
    }
}

// Writes the thread's running partial as piece `pidx` (token ids through the group's row -> token table).
template <int KT>
__device__ __forceinline__ void tc_flush_row(const CallView& c, const TcPartials& pp, const TcRowState<KT>& st, int n,
                                             size_t pidx) {
    pp.pmax[pidx] = st.mx;
    pp.psum[pidx] = st.sum;
#pragma unroll
    for (int j = 0; j < KT; ++j) {
        if (j < c.k_tokens) {
            pp.pval[pidx * c.k_tokens + j] = st.lv[j];
            pp.pid[pidx * c.k_tokens + j] =
                st.li[j] == kNoToken ? kNoToken : __ldg(c.group_tokens + (size_t)n * c.v + st.li[j]);
        }
    }
}

// One batch of a pair's run: its entry, first unit, rows, and whether it holds two units.
struct TcBatch {
    int j, u, n, R, npad, nunits, hrow, first;
    bool read_again;
};
__device__ __forceinline__ TcBatch tc_batch_at(const CallView& c, const TcGeom& g, int pos, int hi) {
    TcBatch b;
    b.j = pos / g.units;
    b.u = pos - b.j * g.units;
    const int entry = c.union_list[b.j];
    b.n = entry & 0xffff;
    const int pass = entry >> 16;
    const int left = c.group_count[b.n] - pass * kTcPassRows;
    b.R = max(1, min(left, kTcPassRows));
    b.read_again = left > kTcPassRows;                         // a later pass streams the group's weights again
    b.npad = (b.R + 15) & ~15;
    b.nunits = (b.npad <= kTcSub && b.u + 1 < g.units && pos + 1 < hi) ? 2 : 1;
    b.first = c.group_offset[b.n] + pass * kTcPassRows;         // first bucket position of the entry
    b.hrow = tc_entry_row(b.first, b.j);
    return b;
}

// The four warps of accumulator `quad` meet (hardware barriers 1 and 2; barrier 0 is the block's own).
__device__ __forceinline__ void quad_sync(int quad) {
    __syncwarp();
    if (quad == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
    else asm volatile("bar.sync 2, 128;" ::: "memory");
}

// Epilogue warps' loop over the pair's run [lo, hi).  `tmem_empty_at` is the (cluster) address of rank 0's
// "accumulators drained" barriers.
template <int KT>
__device__ __forceinline__ void tc_epilogue(const CallView& c, const TcGeom& g, const TcPartials& pp,
                                            float* __restrict__ logits_tap, uint32_t tmem_base, uint64_t* tmem_full,
                                            uint32_t tmem_empty_at, bool leader, volatile int* abort_flag, float* xchg,
                                            int lo, int hi, int rank) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q = warp & 3;                                // lane quarter this warp may read = block it owns
    const int quad = (warp - 2) >> 2;                      // accumulator 0 or 1 of the batch
    float* xq = xchg + quad * (4 * 1024);
    TcRowState<KT> st;
    st.reset();
    long long pending = -1;                                // piece of the last sub-tile folded into `st`
    int pending_j = -1, pending_n = 0;
    bool pending_valid = false;
    int batch = 0;
    for (int pos = lo; pos < hi; ++batch) {
        const TcBatch b = tc_batch_at(c, g, pos, hi);
        const int buf = batch & 1;
        tc_wait(smem_u32(&tmem_full[buf]), ((uint32_t)batch >> 1) & 1u, abort_flag, c.state);
        tc_fence_after();
        if (pending >= 0 && pending_j != b.j) {            // the entry is behind us: its running partial goes out
            if (pending_valid) tc_flush_row<KT>(c, pp, st, pending_n, (size_t)pending);
            st.reset();
            pending = -1;
        }
        const bool wide = b.npad > kTcSub;
        const int t = 2 * (b.u + (wide ? 0 : quad)) + rank;                   // this quad's sub-tile
        const bool tile_ok = (wide || quad < b.nunits) && t < g.tiles;
        const int hbase = wide ? quad * kTcSub : 0;                            // hidden row of the quad's first column
        const int ncols = tile_ok ? min(kTcSub, b.npad - hbase) : 0;           // columns this quad handles
        if (ncols > 0) {
            const int hrow = hbase + q * 32 + lane;                            // the hidden row this thread owns
            const bool row_valid = hrow < b.R;
            const size_t pidx = ((size_t)b.j * g.tiles + t) * kTcPassRows + hrow;
            if (pending >= 0 && pending_valid) {                               // not the entry's last piece after all
                pp.pmax[pending] = kNegInf;
                pp.psum[pending] = 0.f;
            }
            float* tap_row = nullptr;
            if (logits_tap && row_valid)
                tap_row = logits_tap + ((size_t)c.bucket_row[b.first + hrow] * c.k_groups + c.bucket_slot[b.first + hrow]) * c.v;
            const uint32_t acc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 2 * kTcSub + quad * kTcSub);
            const bool own = q * 32 < ncols;
#pragma unroll 1
            for (int s = 0; s < 4; ++s) {
                const int cch = (q + s) & 3;
                if (cch * 32 < ncols) {
                    float z[32];
                    tc_ld32(acc + (uint32_t)(cch * 32), z);
                    float* xw = xq + cch * 1024 + lane * 32;
#pragma unroll
                    for (int i = 0; i < 32; ++i) xw[i ^ lane] = z[i];
                }
                quad_sync(quad);
                if (own && row_valid) {
                    const int w = (q - s) & 3;                                 // the warp that wrote the block
                    const int base = t * kTcSub + w * 32;
                    const int nv = min(32, c.v - base);
                    if (nv > 0) tc_fold_block<KT>(c, st, xq + q * 1024, lane, base, nv, tap_row);
                }
                quad_sync(quad);
            }
            pending = (long long)pidx;
            pending_j = b.j;
            pending_n = b.n;
            pending_valid = row_valid;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
            if (leader) mbar_arrive(tmem_empty_at + (uint32_t)buf * 8u);
            else mbar_arrive_cluster(tmem_empty_at + (uint32_t)buf * 8u);
        }
        pos += b.nunits;
    }
    if (pending >= 0 && pending_valid) tc_flush_row<KT>(c, pp, st, pending_n, (size_t)pending);
}

// grid = 2 * g.pairs CTAs of kTcThreads threads in clusters of two; dynamic shared memory: 1 KiB alignment
// slack + kTcStages stages + the epilogue's exchange blocks + barriers.
__global__ void __launch_bounds__(kTcThreads, 1)
    head_tc_kernel(CallView c, TcGeom g, TcPartials pp, const __grid_constant__ CUtensorMap map_w,
                   const uint16_t* __restrict__ hg, float* __restrict__ logits_tap) {
    extern __shared__ unsigned char tc_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    float* xchg = reinterpret_cast<float*>(smem + kTcStages * kTcStageBytes);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kTcStages * kTcStageBytes + kTcXchgBytes);
    uint64_t* empty = full + kTcStages;
    uint64_t* peer_full = empty + kTcStages;      // rank 0: the other CTA's copy of the stage has landed
    uint64_t* tmem_full = peer_full + kTcStages;  // [2]
    uint64_t* tmem_empty = tmem_full + 2;         // [2] rank 0: both CTAs' epilogue warps have drained the buffer
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_ctarank();
    const bool leader = rank == 0;

    // The kernel may be launched while its predecessors (gather, router) still run: everything up to the
    // dependency wait touches only the pair's shared and tensor memory.
    if (threadIdx.x == 0) {
        for (int s = 0; s < kTcStages; ++s) {
            mbar_init(smem_u32(&full[s]), 1);
            mbar_init(smem_u32(&empty[s]), 1);
            mbar_init(smem_u32(&peer_full[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&tmem_full[s]), 1);
            mbar_init(smem_u32(&tmem_empty[s]), 2 * kTcEpilogueWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        // every CTA allocates all of its own tensor memory, so the accumulators have the same address in both
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTcTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();                                      // both CTAs' barriers exist before anyone arrives on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();                                              // gathered rows and router outputs are complete from here on
    // (no early release of the merge kernel: it reads this kernel's partials right after its own metadata)
    // nothing to do: the router chose the streaming kernel for this call, or the router stage reported a problem
    const bool skip = (c.adaptive && c.state->path_choice != 2) || call_is_poisoned(c.state);

    // this pair's run of units
    const int n_units = skip ? 0 : c.state->n_virtual * g.units;
    const int per = (n_units + g.pairs - 1) / g.pairs;
    const int lo = min(n_units, (int)(blockIdx.x >> 1) * per);
    const int hi = min(n_units, lo + per);

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            const uint64_t pol_first = l2_policy_evict_first(), pol_normal = l2_policy_evict_normal(),
                           pol_last = l2_policy_evict_last();
            for (int pos = lo; pos < hi;) {
                const TcBatch b = tc_batch_at(c, g, pos, hi);
                const bool wide = b.npad > kTcSub;
                const int t0 = 2 * b.u + rank, t1 = 2 * (b.u + 1) + rank;       // this CTA's sub-tiles
                const bool w0 = t0 < g.tiles, w1 = b.nunits == 2 && t1 < g.tiles;
                const uint32_t hbytes = (uint32_t)(b.npad >> 1) * 128u;         // this CTA's half of the hidden rows
                const uint32_t hoff = wide ? kTcTileBytes : 2 * kTcTileBytes;
                const uint32_t bytes = hbytes + (w0 ? kTcTileBytes : 0) + (w1 ? kTcTileBytes : 0);
                const uint64_t pol_w = b.read_again ? pol_normal : pol_first;
                const uint16_t* hsrc = hg + ((size_t)b.hrow + (size_t)rank * (b.npad >> 1)) * kTcK;
                for (int ks = 0; ks < g.ksteps; ++ks) {
                    tc_wait(smem_u32(&empty[stage]), phase ^ 1u, abort_flag, c.state);
                    const uint32_t bar = smem_u32(&full[stage]);
                    const uint32_t sb = smem_u32(smem + (size_t)stage * kTcStageBytes);
                    mbar_expect_tx(bar, bytes);
                    if (w0) tma_load_5d(sb, &map_w, 0, 0, ks, t0 * 8, b.n / c.pack_div, bar, pol_w);
                    if (w1) tma_load_5d(sb + kTcTileBytes, &map_w, 0, 0, ks, t1 * 8, b.n / c.pack_div, bar, pol_w);
                    bulk_g2s_hint(sb + hoff, hsrc + (size_t)ks * g.hg_rows * kTcK, hbytes, bar, pol_last);
                    if (++stage == kTcStages) { stage = 0; phase ^= 1u; }
                }
                pos += b.nunits;
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            int stage = 0, batch = 0;
            uint32_t phase = 0;
            for (int pos = lo; pos < hi; ++batch) {
                const TcBatch b = tc_batch_at(c, g, pos, hi);
                const int buf = batch & 1;
                const bool wide = b.npad > kTcSub;
                const uint32_t hoff = wide ? kTcTileBytes : 2 * kTcTileBytes;
                const uint32_t idesc = tc_idesc(256, b.npad);
                tc_wait_cluster(smem_u32(&tmem_empty[buf]), (((uint32_t)batch >> 1) & 1u) ^ 1u, abort_flag, c.state);   // drained
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(buf * 2 * kTcSub);
                for (int ks = 0; ks < g.ksteps; ++ks) {
                    tc_wait(smem_u32(&full[stage]), phase, abort_flag, c.state);
                    tc_wait_cluster(smem_u32(&peer_full[stage]), phase, abort_flag, c.state);
                    tc_fence_after();
                    const uint32_t sb = smem_u32(smem + (size_t)stage * kTcStageBytes);
#pragma unroll
                    for (int kk = 0; kk < kTcK / 16; ++kk) {
                        const uint64_t bdesc = tc_smem_desc(sb + hoff + kk * 32);
                        for (int a = 0; a < b.nunits; ++a) {
                            const uint64_t adesc = tc_smem_desc(sb + a * kTcTileBytes + kk * 32);
                            tc_mma_pair(acc + (uint32_t)(a * kTcSub), adesc, bdesc, idesc, (ks | kk) ? 1u : 0u);
                        }
                    }
                    tc_commit_pair(smem_u32(&empty[stage]));  // the stage is free in both CTAs once these MMAs have read it
                    if (++stage == kTcStages) { stage = 0; phase ^= 1u; }
                }
                tc_commit_pair(smem_u32(&tmem_full[buf]));    // accumulators complete, in both CTAs
                pos += b.nunits;
            }
        } else if (lane == 0) {
            // rank 1: pass the news that a stage of this CTA has landed on to the MMA issuer in rank 0
            const uint32_t peer_at = cluster_map_shared(smem_u32(peer_full), 0);
            int stage = 0;
            uint32_t phase = 0;
            for (int pos = lo; pos < hi;) {
                const TcBatch b = tc_batch_at(c, g, pos, hi);
                for (int ks = 0; ks < g.ksteps; ++ks) {
                    tc_wait(smem_u32(&full[stage]), phase, abort_flag, c.state);
                    mbar_arrive_cluster(peer_at + (uint32_t)stage * 8u);
                    if (++stage == kTcStages) { stage = 0; phase ^= 1u; }
                }
                pos += b.nunits;
            }
        }
    } else {
        // epilogue: the four warps of an accumulator exchange blocks so that every thread owns one hidden row
        const uint32_t tmem_empty_at = leader ? smem_u32(tmem_empty) : cluster_map_shared(smem_u32(tmem_empty), 0);
        if (c.k_tokens <= 10)
            tc_epilogue<10>(c, g, pp, logits_tap, tmem_base, tmem_full, tmem_empty_at, leader, abort_flag, xchg, lo, hi, rank);
        else
            tc_epilogue<32>(c, g, pp, logits_tap, tmem_base, tmem_full, tmem_empty_at, leader, abort_flag, xchg, lo, hi, rank);
    }
    tc_fence_before();
    cluster_sync_all();          // nothing of the other CTA is still on its way to this CTA's barriers or tensor memory
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols) : "memory");
    }
}

}  // namespace coral
