// Routed grouped GEMM for many query rows on the 5th-generation tensor cores.
//
// For every (group, pass) of the union list the rows that selected the group (gathered beforehand into
// blocks of 128 rows x 64 columns, one contiguous 16 KiB block per pass and column block) are multiplied
// with the group's vocab rows:
//   D[hidden row, vocab row] = sum_k hg[row, k] * W[vocab row, k]
// tcgen05.mma (kind::f16, bf16 x bf16 -> fp32) with M = 128 hidden rows (one pass) and N = 128 vocab rows per
// sub-tile.  A batch is two accumulators: two sub-tiles sharing one read of the hidden rows (one at the end
// of a pass or of the CTA's run).  Operands arrive through TMA tiled loads (128-byte swizzle) in a 4-stage ring; accumulators live in tensor memory, double-buffered
// (2 x 2 x 128 columns), so the epilogue of one batch runs under the MMAs of the next.  The epilogue reads
// each thread's hidden row straight from tensor memory and folds the logits into (max, sum-exp, top-k), one
// partial per (pass, sub-tile, row), so logits never travel to HBM.  (CORAL Section 3.3: logits only for the activated groups; Appendix B: the
// union of the rows' groups is what gets read.)
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and tensor-memory owner, warps 2..9 = epilogue
// (warp w reads the 32 tensor-memory lanes of quarter w % 4; warps 2..5 take the batch's first accumulator,
// warps 6..9 the second).
// Work split: all sub-tiles of all passes form one list; CTA b owns a contiguous run of it.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "head_stream.cuh"   // mbarrier helpers

namespace coral {

constexpr int kTcEpilogueWarps = 8;
constexpr int kTcEpilogueThreads = kTcEpilogueWarps * 32;
constexpr int kTcThreads = (2 + kTcEpilogueWarps) * 32;
constexpr int kTcSub = 128;          // vocab rows per sub-tile (MMA N)
constexpr int kTcBlockRows = 128;    // hidden rows per accumulator block (MMA M)
constexpr int kTcPassRows = 128;     // hidden rows per pass over a group's weights: one accumulator block, so
                                     // that two weight sub-tiles share every read of the hidden rows (a group
                                     // with more rows is read again; the re-read mostly hits L2)
constexpr int kTcK = 64;             // columns per stage (one 128-byte swizzle atom of bf16)
constexpr int kTcStages = 4;
constexpr int kTcTileBytes = kTcBlockRows * kTcK * 2;   // 16 KiB: one 128 x 64 bf16 operand tile
constexpr int kTcStageBytes = 3 * kTcTileBytes;         // (A, B0, B1)
constexpr int kTcTmemCols = 512;
constexpr int kTcSpin = 1 << 22;

struct TcGeom {
    int grid;
    int tiles;        // sub-tiles per group = ceil(v / 128)
    int ksteps;       // ceil(H / 64) = 64-column blocks of the packed layout
};

struct TcPartials {
    float* pmax;      // [pass][tiles][kTcPassRows]
    float* psum;
    float* pval;      // [...][k_tokens]
    int32_t* pid;
};

__device__ __forceinline__ void tc_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, DeviceState* st) {
    const int limit = *abort_flag ? 64 : kTcSpin;
    for (int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return;
    *abort_flag = 1;
    set_status(st, -5);
}

// L2 eviction policies for the tiled loads: the weights of a group are streamed once per pass (evict first,
// unless a later pass reads them again), the gathered hidden rows are re-read for every pair of sub-tiles
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
// Instruction descriptor: D = f32, A = B = bf16, both K-major, N = 128, M = 128.
constexpr uint32_t kTcIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTcSub >> 3) << 17) |
                              ((uint32_t)(kTcBlockRows >> 4) << 24);

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

// Gathers the hidden rows of every (group, pass) into the blocked operand layout
//   hg[pass entry j][column block kb][row r of the pass, 128][64 columns]
// so that the 128 x 64 operand tile of a pass is one contiguous 16 KiB block.  One thread block per
// (row, slot) pair in bucket order; columns past H are written as zero; rows past the pass's size keep
// whatever they held (their accumulator lanes are never read).
__global__ void __launch_bounds__(128) tc_gather_kernel(CallView c, uint16_t* __restrict__ hg) {
    const int p = blockIdx.x;
    pdl_wait();                                              // launched over the tail of the router stage
    pdl_launch_dependents();
    if (call_is_poisoned(c.state)) return;                   // the router stage reported a problem: index with nothing
    if (c.adaptive && c.state->path_choice != 2) return;     // the router chose the streaming kernel for this call
    if (p >= c.group_offset[c.N]) return;          // fewer pairs than M * k_groups when the vocab is sharded
    const int m = c.bucket_row[p];
    const int n = c.sel[(size_t)m * c.k_groups + c.bucket_slot[p]];
    const int rg = p - c.group_offset[n];
    const int j = c.union_rank[n] + rg / kTcPassRows;
    const int r = rg % kTcPassRows;
    const uint4* src = reinterpret_cast<const uint4*>(c.hidden + (size_t)m * c.H);
    uint4* dst = reinterpret_cast<uint4*>(hg) + ((size_t)j * c.KB * kTcPassRows + r) * 8;
    const int chunks = c.H >> 3;
    for (int ch = threadIdx.x; ch < c.KB * 8; ch += 128)
        dst[(size_t)(ch >> 3) * kTcPassRows * 8 + (ch & 7)] = ch < chunks ? __ldg(src + ch) : make_uint4(0, 0, 0, 0);
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

// Running statistics of one hidden row over the sub-tiles one epilogue thread sees of a pass: the thread
// keeps (max, sum-exp, top-k) in registers from sub-tile to sub-tile and writes one full partial at the
// last of them; the other sub-tiles get an "empty" marker (max = -inf, sum = 0), which the merge skips.
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

// Epilogue of one 128 x 128 accumulator for one thread (= one hidden row): fold the 128 logits of vocab rows
// [base, base + valid) of the group into the running (max, sum-exp, top-k).
template <int KT>
__device__ __forceinline__ void tc_fold_row(const CallView& c, TcRowState<KT>& st, float* __restrict__ logits_tap,
                                            uint32_t tmem_acc_row, int base, bool row_valid, int tap_m, int tap_slot,
                                            float* zs) {
    constexpr float kLog2e = 1.4426950408889634f;
    const int valid = min(kTcSub, c.v - base);
#pragma unroll 1
    for (int ch = 0; ch < 4; ++ch) {
        float z[32];
        tc_ld32(tmem_acc_row + (uint32_t)(ch * 32), z);
        const int nv = min(32, valid - ch * 32);
        if (!row_valid || nv <= 0) continue;
        float cm = kNegInf;
#pragma unroll
        for (int i = 0; i < 32; ++i) cm = fmaxf(cm, i < nv ? z[i] : kNegInf);
        const float nm = fmaxf(st.mx, cm);
        float add = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) add += i < nv ? exp2f((z[i] - nm) * kLog2e) : 0.f;
        st.sum = st.sum * exp2f((st.mx - nm) * kLog2e) + add;   // exp2(-inf) = 0 on the first chunk
        st.mx = nm;
        if (logits_tap) {
            float* dst = logits_tap + ((size_t)tap_m * c.k_groups + tap_slot) * c.v + base + ch * 32;
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < nv) dst[i] = z[i];
        }
        // candidates for the top-k list: a bit per element that reaches the current k-th entry; the few that do
        // are fetched by index from a shared-memory copy of the chunk (element i of thread t at zs[i * T + t])
        if (cm >= st.lv[KT - 1]) {
            unsigned cand = 0;
#pragma unroll
            for (int i = 0; i < 32; ++i)
                cand |= (i < nv && z[i] >= st.lv[KT - 1]) ? (1u << i) : 0u;   // ties are settled by the insertion
#pragma unroll
            for (int i = 0; i < 32; ++i) zs[i * kTcEpilogueThreads] = z[i];
            while (cand) {
                const int i = __ffs(cand) - 1;
                cand &= cand - 1;
                const float zi = zs[i * kTcEpilogueThreads];
                if (zi >= st.lv[KT - 1]) tc_insert<KT>(st.lv, st.li, zi, base + ch * 32 + i);
            }
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

// One batch of the run: the pass it belongs to, its first sub-tile, and whether it holds two sub-tiles.
struct TcBatch {
    int j, t, n, pass, R, nsub, hrow;
};
__device__ __forceinline__ TcBatch tc_batch_at(const CallView& c, const TcGeom& g, int pos, int hi) {
    TcBatch b;
    b.j = pos / g.tiles;
    b.t = pos - b.j * g.tiles;
    const int entry = c.union_list[b.j];
    b.n = entry & 0xffff;
    b.pass = entry >> 16;
    b.R = min(c.group_count[b.n] - b.pass * kTcPassRows, kTcPassRows);
    b.nsub = (b.t + 1 < g.tiles && pos + 1 < hi) ? 2 : 1;
    b.hrow = c.group_offset[b.n] + b.pass * kTcPassRows;      // first bucket position of the pass
    return b;
}

// Epilogue warps' loop over the CTA's run [lo, hi).  Of the sub-tiles of a pass inside the run, the warps of
// accumulator `which` see every second one; they write their running partial at the last one they see.
template <int KT>
__device__ __forceinline__ void tc_epilogue(const CallView& c, const TcGeom& g, const TcPartials& pp,
                                            float* __restrict__ logits_tap, uint32_t tmem_base, uint64_t* tmem_full,
                                            uint64_t* tmem_empty, volatile int* abort_flag, float* zstash, int lo, int hi) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int quarter = warp & 3;
    const int which = (warp - 2) >> 2;                    // accumulator 0 or 1 of the batch
    const int row_in_block = quarter * 32 + lane;
    float* zs = zstash + (threadIdx.x - 64);
    TcRowState<KT> st;
    st.reset();
    int batch = 0;
    for (int pos = lo; pos < hi; ++batch) {
        const TcBatch b = tc_batch_at(c, g, pos, hi);
        const int buf = batch & 1;
        tc_wait(smem_u32(&tmem_full[buf]), ((uint32_t)batch >> 1) & 1u, abort_flag, c.state);
        tc_fence_after();
        if (which < b.nsub) {
            const int sub = which;
            const int r = row_in_block;
            const bool row_valid = r < b.R;
            const int tap_m = row_valid && logits_tap ? c.bucket_row[b.hrow + r] : 0;
            const int tap_slot = row_valid && logits_tap ? c.bucket_slot[b.hrow + r] : 0;
            const size_t pidx = ((size_t)b.j * g.tiles + b.t + sub) * kTcPassRows + r;
            const uint32_t acc_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((buf * 2 + which) * kTcSub);
            tc_fold_row<KT>(c, st, logits_tap, acc_row, (b.t + sub) * kTcSub, row_valid, tap_m, tap_slot, zs);
            // is this the last sub-tile of the pass that these warps see in this run?
            const int npos = pos + b.nsub;
            bool last = npos >= hi || npos / g.tiles != b.j;
            if (!last && which == 1) {
                const int nt = npos - b.j * g.tiles;
                last = nt + 1 >= g.tiles || npos + 1 >= hi;       // the next batch is a single sub-tile
            }
            if (row_valid) {
                if (last) {
                    tc_flush_row<KT>(c, pp, st, b.n, pidx);
                } else {
                    pp.pmax[pidx] = kNegInf;
                    pp.psum[pidx] = 0.f;
                }
            }
            if (last) st.reset();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&tmem_empty[buf]));
        pos += b.nsub;
    }
}

// grid = g.grid CTAs of kTcThreads threads; dynamic shared memory: 1 KiB alignment slack + kTcStages stages + barriers.
__global__ void __launch_bounds__(kTcThreads, 1)
    head_tc_kernel(CallView c, TcGeom g, TcPartials pp, const __grid_constant__ CUtensorMap map_w,
                   const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_h64,
                   const __grid_constant__ CUtensorMap map_h32, float* __restrict__ logits_tap) {
    extern __shared__ unsigned char tc_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    float* zstash = reinterpret_cast<float*>(smem + kTcStages * kTcStageBytes);          // [32][epilogue threads]
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kTcStages * kTcStageBytes + 32 * kTcEpilogueThreads * 4);
    uint64_t* empty = full + kTcStages;
    uint64_t* tmem_full = empty + kTcStages;      // [2]
    uint64_t* tmem_empty = tmem_full + 2;         // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // The kernel may be launched while its predecessors (gather, router) still run: everything up to the
    // dependency wait touches only this CTA's shared and tensor memory.
    if (threadIdx.x == 0) {
        for (int s = 0; s < kTcStages; ++s) {
            mbar_init(smem_u32(&full[s]), 1);
            mbar_init(smem_u32(&empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&tmem_full[s]), 1);
            mbar_init(smem_u32(&tmem_empty[s]), kTcEpilogueWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTcTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();                                              // gathered rows and router outputs are complete from here on
    // (no early release of the merge kernel: it reads this kernel's partials right after its own metadata)
    // nothing to do: the router chose the streaming kernel for this call, or the router stage reported a problem
    const bool skip = (c.adaptive && c.state->path_choice != 2) || call_is_poisoned(c.state);

    // this CTA's run of sub-tiles
    const int n_tiles = skip ? 0 : c.state->n_virtual * g.tiles;
    const int per = (n_tiles + g.grid - 1) / g.grid;
    const int lo = min(n_tiles, (int)blockIdx.x * per);
    const int hi = min(n_tiles, lo + per);

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            const uint64_t pol_first = l2_policy_evict_first(), pol_normal = l2_policy_evict_normal(),
                           pol_last = l2_policy_evict_last();
            for (int pos = lo; pos < hi;) {
                const TcBatch b = tc_batch_at(c, g, pos, hi);
                // a pass with few rows fetches only the first 64 or 32 rows of its block of hidden rows; the MMA
                // still spans 128 rows, whose remaining accumulator lanes hold leftovers nobody reads
                const CUtensorMap* mh = b.R <= 32 ? &map_h32 : b.R <= 64 ? &map_h64 : &map_h;
                const uint32_t hbytes = b.R <= 32 ? kTcTileBytes / 4 : b.R <= 64 ? kTcTileBytes / 2 : kTcTileBytes;
                const uint32_t bytes = hbytes + (uint32_t)b.nsub * kTcTileBytes;
                const bool read_again = c.group_count[b.n] > (b.pass + 1) * kTcPassRows;   // a later pass follows
                const uint64_t pol_w = read_again ? pol_normal : pol_first;
                for (int ks = 0; ks < g.ksteps; ++ks) {
                    tc_wait(smem_u32(&empty[stage]), phase ^ 1u, abort_flag, c.state);
                    const uint32_t bar = smem_u32(&full[stage]);
                    const uint32_t sb = smem_u32(smem + (size_t)stage * kTcStageBytes);
                    mbar_expect_tx(bar, bytes);
                    // tile 0 of a stage is the pass's block of hidden rows, tiles 1 and 2 the weight sub-tiles
                    tma_load_2d(sb, mh, 0, (b.j * g.ksteps + ks) * kTcPassRows, bar, pol_last);
                    for (int sub = 0; sub < b.nsub; ++sub)
                        tma_load_5d(sb + (1 + sub) * kTcTileBytes, &map_w, 0, 0, ks, (b.t + sub) * 8, b.n / c.pack_div, bar, pol_w);
                    if (++stage == kTcStages) { stage = 0; phase ^= 1u; }
                }
                pos += b.nsub;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int stage = 0, batch = 0;
            uint32_t phase = 0;
            for (int pos = lo; pos < hi; ++batch) {
                const TcBatch b = tc_batch_at(c, g, pos, hi);
                const int buf = batch & 1;
                tc_wait(smem_u32(&tmem_empty[buf]), (((uint32_t)batch >> 1) & 1u) ^ 1u, abort_flag, c.state);   // drained
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(buf * 2 * kTcSub);
                for (int ks = 0; ks < g.ksteps; ++ks) {
                    tc_wait(smem_u32(&full[stage]), phase, abort_flag, c.state);
                    tc_fence_after();
                    const uint32_t sb = smem_u32(smem + (size_t)stage * kTcStageBytes);
#pragma unroll
                    for (int kk = 0; kk < kTcK / 16; ++kk) {
                        const uint64_t adesc = tc_smem_desc(sb + kk * 32);
                        for (int sub = 0; sub < b.nsub; ++sub) {
                            const uint64_t bdesc = tc_smem_desc(sb + (1 + sub) * kTcTileBytes + kk * 32);
                            tc_mma(acc + (uint32_t)(sub * kTcSub), adesc, bdesc, (ks | kk) ? 1u : 0u);
                        }
                    }
                    tc_commit(smem_u32(&empty[stage]));       // the stage is free once these MMAs have read it
                    if (++stage == kTcStages) { stage = 0; phase ^= 1u; }
                }
                tc_commit(smem_u32(&tmem_full[buf]));         // accumulators complete
                pos += b.nsub;
            }
        }
    } else {
        // epilogue: thread <-> tensor-memory lane = hidden row; the two warps of a lane quarter take one
        // accumulator of the batch each
        if (c.k_tokens <= 10)
            tc_epilogue<10>(c, g, pp, logits_tap, tmem_base, tmem_full, tmem_empty, abort_flag, zstash, lo, hi);
        else
            tc_epilogue<32>(c, g, pp, logits_tap, tmem_base, tmem_full, tmem_empty, abort_flag, zstash, lo, hi);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols) : "memory");
    }
}

}  // namespace coral
