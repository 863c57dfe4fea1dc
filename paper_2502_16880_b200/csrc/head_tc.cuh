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
// accumulator therefore exchange blocks through shared memory: in step s warp q reads columns
// 32 ((q + s) mod 4) .. + 31 of its lanes and hands them, 16 vocab rows at a time (16 KiB of shared memory
// for both accumulators), to warp (q + s) mod 4, which owns those hidden rows and folds the block's 16 logits
// per row into its running (max, sum-exp, top-k), carried in registers over the sub-tiles the warp sees of an
// entry; logits never travel to HBM.  (CORAL Section 3.3: logits only for
// the activated groups; Appendix B: the union of the rows' groups is what gets read.)
//
// Warp roles: warps 0 and 11 = producers, a 64-column step each in turn (TMA tiled loads of the weights, bulk
// copies of the hidden rows; one thread issues a step's copies in some 150 ns); warps 1 and
// 10 = MMA issuers in the CTA of rank 0, one per accumulator of the batch (issuing an MMA costs its thread
// some 50 ns, which for eight MMAs per 64 columns would be the pair's critical path); warp 1 of rank 1 is the
// relay that tells rank 0 when a slot of the operand ring has landed; warps 2..9 = epilogue, four per accumulator (with one wide
// accumulator: four per half of its columns).
// Work split: the units of all entries form one list; pair p owns a contiguous run of it, cut so that the
// runs cost the same (tc_unit_cost: a unit of a wide entry, which is a batch by itself, counts as 1.6 narrow ones).
#pragma once
#include "tc_prims.cuh"

namespace coral {

constexpr int kTcHeadThreads = kTcThreads + 64;     // warp 10 issues the MMAs of a batch's second accumulator, warp 11 is the second producer
// The operand ring is cut into slots of the size the current batch needs per 64 columns, so that the bytes in
// flight - what hides the memory latency - stay the same whatever the batch: two weight tiles + up to 8 KiB of
// hidden rows (40 KiB, five slots), one + up to 8 KiB (24 KiB, eight slots), one + up to 16 KiB (32 KiB, six).
// When the kind of batch changes the producer lets the ring run empty first.
constexpr int kTcRingBytes = 200 * 1024;
constexpr int kTcMaxSlots = 8;
struct TcRing {
    int slots;            // slots of the current geometry
    uint32_t bytes;       // their size
    uint32_t hoff;        // offset of the hidden rows inside a slot (the weight tiles come first)
};
__device__ __forceinline__ TcRing tc_ring_for(bool wide, int nunits) {
    if (wide) return TcRing{6, 32 * 1024, (uint32_t)kTcTileBytes};
    if (nunits == 2) return TcRing{5, 40 * 1024, 2u * kTcTileBytes};
    return TcRing{8, 24 * 1024, (uint32_t)kTcTileBytes};
}
// A role's place in the ring: the slot it uses next and, per slot, the parity of the slot's next use (the
// barriers keep their history across changes of geometry; only the slot counter starts over).
struct TcRingPos {
    int slot = 0, kind = -1;
    uint32_t parity = 0;
    // true when the geometry changed (the caller then starts at slot 0 of the new one)
    __device__ __forceinline__ bool enter(const TcRing& r) {
        if (r.slots == kind) return false;
        kind = r.slots;       // the three geometries differ in their slot count
        slot = 0;
        return true;
    }
    __device__ __forceinline__ uint32_t par() const { return (parity >> slot) & 1u; }
    __device__ __forceinline__ void advance(const TcRing& r) {
        parity ^= 1u << slot;
        if (++slot == r.slots) slot = 0;
    }
};
constexpr int kTcXchgBytes = 2 * 4 * 16 * 32 * 4;   // [accumulator][owner warp][16 vocab rows][32 hidden rows] fp32
constexpr size_t kTcSmemBytes = 1024 + (size_t)kTcRingBytes + kTcXchgBytes + 256 + 4096;   // + the run split's cost cache

struct TcGeom {
    int pairs;        // CTA pairs launched
    int tiles;        // sub-tiles per group = ceil(v / 128)
    int units;        // units per group = ceil(tiles / 2)
    int ksteps;       // ceil(H / 64) = 64-column blocks of the packed layout
    int hg_rows;      // rows of one column block of the gathered hidden matrix
    int strided;      // 1: the pairs take the batches of the call in turn (see tc_split_runs)
};

struct TcPartials {
    float* pmax;      // [entry][tiles][kTcPassRows]
    float* psum;
    float* pval;      // [...][k_tokens]
    int32_t* pid;
};

// Gathers the hidden rows of every entry into the operand layout
//   hg[column block kb][row][64 columns]     (row = tc_entry_row(...) + position in the entry)
// with the 16-byte chunks of every 128-byte row permuted the way the 128-byte shared-memory swizzle wants
// them (chunk c of row r at position c ^ (r & 7)), so that a plain contiguous bulk copy of n/2 rows lands in
// shared memory as a K-major operand tile.  A block copies kGatherPairs (row, slot) pairs in bucket order, 64
// threads each; where a pair's row comes from and goes to was written by the router stage (bucket_row,
// bucket_dst), so one round of loads finds it.  Columns past H are written as zero; rows between an entry's
// size and its padded size keep whatever they held (their accumulator columns are never read).
constexpr int kGatherPairs = 4;
__global__ void __launch_bounds__(64 * kGatherPairs) tc_gather_kernel(CallView c, uint16_t* __restrict__ hg, int hg_rows) {
    const int p = blockIdx.x * kGatherPairs + (threadIdx.x >> 6), t = threadIdx.x & 63;
    pdl_wait();                                              // launched over the tail of the router stage
    pdl_launch_dependents();
    if (call_is_poisoned(c.state)) return;                   // the router stage reported a problem: index with nothing
    if (c.adaptive && c.state->path_choice != 2) return;     // the router chose the streaming kernel for this call
    if (p >= c.group_offset[c.N]) return;          // fewer pairs than M * k_groups when the vocab is sharded
    const int m = CORAL_IDX(c.bucket_row[p], c.M, c.state);
    const int row = c.bucket_dst[p];
    if (!CORAL_IDX_OK(row, hg_rows, c.state)) return;
    const uint4* src = reinterpret_cast<const uint4*>(c.hidden + (size_t)m * c.H);
    uint4* dst = reinterpret_cast<uint4*>(hg);
    const int chunks = c.H >> 3;
    for (int ch0 = 0; ch0 < c.KB * 8; ch0 += 64 * 4) {      // four loads in flight per thread
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int ch = ch0 + u * 64 + t;
            v[u] = ch < chunks ? __ldg(src + ch) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int ch = ch0 + u * 64 + t;
            if (ch < c.KB * 8) dst[((size_t)(ch >> 3) * hg_rows + row) * 8 + ((ch & 7) ^ (row & 7))] = v[u];
        }
    }
}

// Insertion into a thread-private top-KT list kept sorted (value desc, row index asc).  The new entry's
// position is the number of entries that stay ahead of it - KT independent comparisons - and every slot then
// picks its new content by itself, so the instruction stream has no chain as long as the list.
template <int KT>
__device__ __forceinline__ void tc_insert(float (&lv)[KT], int (&li)[KT], float v, int idx) {
    int p0 = 0, p1 = 0;
#pragma unroll
    for (int j = 0; j < KT; j += 2) {
        p0 += better(lv[j], li[j], v, idx) ? 1 : 0;
        if (j + 1 < KT) p1 += better(lv[j + 1], li[j + 1], v, idx) ? 1 : 0;
    }
    const int p = p0 + p1;
#pragma unroll
    for (int j = KT - 1; j >= 1; --j) {                       // descending: slot j - 1 is still the old one
        const bool shift = j > p, here = j == p;
        lv[j] = shift ? lv[j - 1] : (here ? v : lv[j]);
        li[j] = shift ? li[j - 1] : (here ? idx : li[j]);
    }
    if (p == 0) { lv[0] = v; li[0] = idx; }
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

__device__ __forceinline__ float tc_ex2(float x) {            // 2^x for x <= 0; tiny results flush to zero
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Folds the logits of kTcHalf vocab rows [base, base + 16) of the group (nv of them real) into the running
// statistics of one hidden row.  The values sit in a shared-memory block, element k at xb[k * 32 + (lane ^ (k + kofs))].
// Four independent chains for the maximum, the sum and the candidate mask keep the one thread busy.
constexpr int kTcHalf = 16;
template <int KT>
__device__ __forceinline__ void tc_fold_block(TcRowState<KT>& st, const float* xb, int lane, int kofs, int base, int nv,
                                              float* __restrict__ tap_row) {
    constexpr float kLog2e = 1.4426950408889634f;
    float z[kTcHalf];
#pragma unroll
    for (int k = 0; k < kTcHalf; ++k) z[k] = xb[k * 32 + (lane ^ (k + kofs))];
    if (nv < kTcHalf) {                                       // ragged end of the group: rows past it do not count
#pragma unroll
        for (int k = 0; k < kTcHalf; ++k) z[k] = k < nv ? z[k] : kNegInf;
    }
    float m[4] = {z[0], z[1], z[2], z[3]};
#pragma unroll
    for (int k = 4; k < kTcHalf; ++k) m[k & 3] = fmaxf(m[k & 3], z[k]);
    const float cm = fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3]));
    const float nm = fmaxf(st.mx, cm);
    const float nb = -nm * kLog2e;
    float a[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int k = 0; k < kTcHalf; ++k) a[k & 3] += tc_ex2(fmaf(z[k], kLog2e, nb));   // 2^-inf = 0 for the rows past the end
    st.sum = st.sum * tc_ex2((st.mx - nm) * kLog2e) + ((a[0] + a[1]) + (a[2] + a[3]));   // 2^-inf = 0 on the first block
    st.mx = nm;
    if (tap_row) {
#pragma unroll
        for (int k = 0; k < kTcHalf; ++k)
            if (k < nv) tap_row[base + k] = z[k];
    }
    // candidates for the top-k list: a bit per element that reaches the current k-th entry (ties are settled by
    // the insertion); the few that do are fetched again by index from the block
    const float thr = st.lv[KT - 1];
    if (cm >= thr) {
        unsigned cb[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int k = 0; k < kTcHalf; ++k) cb[k & 3] |= (k < nv && z[k] >= thr) ? (1u << k) : 0u;
        unsigned cand = (cb[0] | cb[1]) | (cb[2] | cb[3]);
        while (cand) {
            const int k = __ffs(cand) - 1;
            cand &= cand - 1;
            const float zk = xb[k * 32 + (lane ^ (k + kofs))];
            if (zk >= st.lv[KT - 1]) tc_insert<KT>(st.lv, st.li, zk, base + k);
        }
    }
}

// Writes the thread's running partial as piece `pidx` (token ids through the group's row -> token table).
template <int KT>
__device__ __forceinline__ void tc_flush_row(const CallView& c, const TcPartials& pp, const TcRowState<KT>& st, int n,
                                             size_t pidx) {
    if (!CORAL_IDX_OK(pidx, c.cap_part_tc, c.state)) return;
    pp.pmax[pidx] = st.mx;
    pp.psum[pidx] = st.sum;
#pragma unroll
    for (int j = 0; j < KT; ++j) {
        if (j < c.k_tokens) {
            pp.pval[pidx * c.k_tokens + j] = st.lv[j];
            pp.pid[pidx * c.k_tokens + j] =
                st.li[j] == kNoToken ? kNoToken : __ldg(c.group_tokens + CORAL_IDX((size_t)n * c.v + st.li[j], c.V, c.state));
        }
    }
}

// Relative time of one unit of an entry with `rows` rows.  A narrow entry's units go two to a batch and a batch
// streams at what an SM can take in (its weight tiles plus its share of the hidden rows, in 128-byte units per
// 64 columns); a wide entry's unit is a batch of its own, whose pace the MMA issue and the slot hand-over set
// rather than the bytes: about 0.8 of a narrow batch of two (the weight that gave the shortest whole step at
// 960 and 1440 rows on the Llama3-8B shape; between 0.75 and 0.9 it matters by 1-2 %).
__device__ __forceinline__ int tc_unit_cost(int rows) {
    const int npad = (max(1, min(rows, kTcPassRows)) + 15) & ~15;
    return npad > kTcSub ? kTcSub + 96 + (npad >> 2) : kTcSub + (npad >> 2);
}
constexpr int kTcCostNarrowMax = kTcSub + (kTcSub >> 2);      // the largest cost of a narrow entry's unit
__device__ __forceinline__ bool tc_cost_is_wide(int cost) { return cost > kTcCostNarrowMax; }

// Walks a pair's run batch by batch.  A batch is two units of one entry of at most 128 padded rows ("narrow"),
// else one unit.  A run is either a number of consecutive units of the unit list (entry by entry, unit by unit;
// its batches are cut from the run's first unit on), or every stride-th batch of the call's batch list (the
// entries' batches in order, a narrow entry's being its units 0-1, 2-3, ...), found through the entries' cached
// costs.
struct TcWalk {
    int j, u;             // entry (index in the union list) and unit inside it
    int left;             // consecutive: units of the run still to do, this batch included; strided: batches
    int strided, stride;  // strided run: distance between its batches in the batch list
    int b, bbase;         // strided run: this batch's index in the list, index of entry j's first batch
    int n_entries;
    const int* cost;      // the entries' unit costs (shared memory), which tell narrow from wide
    int n, R, npad, first, hrow;
    bool wide, read_again;
    __device__ __forceinline__ void load(const CallView& c) {
        const int entry = c.union_list[CORAL_IDX(j, c.union_cap, c.state)];
        n = CORAL_IDX(entry & 0xffff, c.N, c.state);
        const int pass = entry >> 16;
        const int rows = c.group_count[n] - pass * kTcPassRows;
        R = max(1, min(rows, kTcPassRows));
        read_again = rows > kTcPassRows;                      // a later pass streams the group's weights again
        npad = (R + 15) & ~15;
        wide = npad > kTcSub;
        first = c.group_offset[n] + pass * kTcPassRows;        // first bucket position of the entry
        hrow = tc_entry_row(first, j);
        if (!CORAL_IDX_OK(hrow + npad - 1, c.cap_hg_rows, c.state)) hrow = 0;     // (checked build) read rows that exist
        if (!CORAL_IDX_OK(first + R - 1, c.cap_pairs, c.state)) first = 0;
    }
    __device__ __forceinline__ int batches_of(int e, const TcGeom& g) const {
        return tc_cost_is_wide(cost[e]) ? g.units : (g.units + 1) >> 1;
    }
    // strided run: the entry and unit of batch b (entries are only ever passed forwards)
    __device__ __forceinline__ void seek(const TcGeom& g) {
        while (j + 1 < n_entries && b >= bbase + batches_of(j, g)) { bbase += batches_of(j, g); ++j; }
        u = (b - bbase) * (tc_cost_is_wide(cost[j]) ? 1 : 2);
    }
    __device__ __forceinline__ void start(const CallView& c, const TcGeom& g, const int* run, const int* cost_cache) {
        left = run[2]; strided = run[3]; n_entries = run[4];
        cost = cost_cache;
        if (!strided) {
            j = run[0]; u = run[1];
        } else {
            b = run[0]; stride = run[1]; j = 0; bbase = 0;
            if (left > 0) seek(g);
        }
        if (left > 0) load(c);
    }
    __device__ __forceinline__ int nunits(const TcGeom& g) const {
        return wide ? 1 : strided ? min(2, g.units - u) : min(2, min(g.units - u, left));
    }
    __device__ __forceinline__ void next(const CallView& c, const TcGeom& g) {
        if (strided) {
            if (--left > 0) { b += stride; seek(g); load(c); }
            return;
        }
        const int nu = nunits(g);
        u += nu;
        left -= nu;
        if (u == g.units) { ++j; u = 0; if (left > 0) load(c); }
    }
};

// Gives every pair its run (one warp).
// Consecutive (out[3] = 0): the unit list is cut into g.pairs runs of (almost) equal cost.  out[0], out[1]: entry
// and unit where the pair's run starts; out[2]: its number of units.  Run p holds the units whose cost prefix
// (tc_unit_cost), taken at the unit's middle, lies in [p, p + 1) * total / pairs.
// Strided (out[3] = 1, when g.strided and the costs fit the cache): pair p takes batches p, p + pairs, ... of
// the call's batch list; out[0] = p, out[1] = pairs, out[2] = its number of batches.  The pairs then work on
// the same few entries at the same time, so an entry's gathered hidden rows, which every one of its batches
// reads in full, and the weights of a group that a second pass reads again are found in L2 by all but the first
// reader; with consecutive runs each pair sweeps its own entry's rows (2 MB at 256 rows and H = 4096) once per
// unit, and from some 70 MB of gathered rows on those sweeps push each other out of L2 (Llama3-8B shape, 1920
// rows: 2.11 GB from HBM for 1.05 GB of weights).
// out[4]: entries of the call.
// (The entries' costs are read from global memory once - two dependent loads each, all of a lane's in flight together -
// and kept in `cost_cache` for the second pass; beyond kTcCostCache entries the second pass reads them again.)
constexpr int kTcCostCache = 1024;
__device__ __forceinline__ void tc_split_runs(const CallView& c, const TcGeom& g, int n_entries, int pair, int* out,
                                              int* cost_cache) {
    const int lane = threadIdx.x & 31;
    long long total = 0;
    int batches = 0;
#pragma unroll 4
    for (int j0 = 0; j0 < n_entries; j0 += 32) {
        const int j = j0 + lane;
        if (j < n_entries) {
            const int entry = c.union_list[j];
            const int w = tc_unit_cost(c.group_count[entry & 0xffff] - (entry >> 16) * kTcPassRows);
            if (j < kTcCostCache) cost_cache[j] = w;
            total += (long long)g.units * w;
            batches += tc_cost_is_wide(w) ? g.units : (g.units + 1) >> 1;
        }
    }
    __syncwarp();
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        total += __shfl_xor_sync(0xffffffffu, total, o);
        batches += __shfl_xor_sync(0xffffffffu, batches, o);
    }
    if (g.strided && n_entries <= kTcCostCache) {
        if (lane == 0) {
            out[0] = pair;
            out[1] = g.pairs;
            out[2] = pair < batches ? (batches - pair + g.pairs - 1) / g.pairs : 0;
            out[3] = 1;
            out[4] = n_entries;
        }
        return;
    }
    const long long t_lo = pair * total / g.pairs, t_hi = (pair + 1) * total / g.pairs;
    // global index (entry * units + unit) of the first unit whose middle reaches t_lo, and t_hi
    const int n_units = n_entries * g.units;
    int lo = n_units, hi = n_units;
    long long before = 0;
    for (int j0 = 0; j0 < n_entries; j0 += 32) {
        const int j = j0 + lane;
        int w = 0;
        if (j < n_entries) {
            if (j < kTcCostCache) {
                w = cost_cache[j];
            } else {
                const int entry = c.union_list[j];
                w = tc_unit_cost(c.group_count[entry & 0xffff] - (entry >> 16) * kTcPassRows);
            }
        }
        const long long cost = (long long)w * g.units;
        long long incl = cost;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const long long start = before + incl - cost;           // cost prefix of the entry's first unit
        if (w > 0) {
            // unit u's middle is at start + w * u + w / 2; the first u whose middle is >= t
            const long long a_lo = 2 * (t_lo - start) - w, a_hi = 2 * (t_hi - start) - w;
            long long u_lo = a_lo <= 0 ? 0 : (a_lo + 2 * w - 1) / (2 * w);
            long long u_hi = a_hi <= 0 ? 0 : (a_hi + 2 * w - 1) / (2 * w);
            // A narrow entry with many rows is cut between its batches of two: there a batch of one unit takes about
            // as long as a batch of two (measured at 112-128 rows: 293 against 300 us whole step), while with fewer
            // rows per entry it is cheap and the finer cut balances better (60 rows: 241 against 249 us; 96 rows:
            // 258 against 263 us).
            if (w <= kTcSub + (kTcSub >> 2) && w >= kTcSub + (112 >> 2)) {
                u_lo = (u_lo + 1) & ~1ll;
                u_hi = (u_hi + 1) & ~1ll;
            }
            if (u_lo < g.units) lo = min(lo, j * g.units + (int)u_lo);
            if (u_hi < g.units) hi = min(hi, j * g.units + (int)u_hi);
        }
        before += __shfl_sync(0xffffffffu, incl, 31);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = min(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (pair == g.pairs - 1) hi = n_units;
    if (lane == 0) {
        out[0] = lo / g.units;
        out[1] = lo - (lo / g.units) * g.units;
        out[2] = max(0, hi - lo);
        out[3] = 0;
        out[4] = n_entries;
    }
}

// The four warps of accumulator `quad` meet (hardware barriers 1 and 2; barrier 0 is the block's own).
__device__ __forceinline__ void quad_sync(int quad) {
    __syncwarp();
    if (quad == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
    else asm volatile("bar.sync 2, 128;" ::: "memory");
}

// Epilogue warps' loop over the pair's run.  `tmem_empty_at` is the (cluster) address of rank 0's
// "accumulators drained" barriers.
template <int KT>
__device__ __forceinline__ void tc_epilogue(const CallView& c, const TcGeom& g, const TcPartials& pp,
                                            float* __restrict__ logits_tap, uint32_t tmem_base, uint64_t* tmem_full,
                                            uint32_t tmem_empty_at, bool leader, volatile int* abort_flag, float* xchg,
                                            const int* run, const int* cost_cache, int rank) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q = warp & 3;                                // lane quarter this warp may read = block it owns
    const int quad = (warp - 2) >> 2;                      // accumulator 0 or 1 of the batch
    float* xq = xchg + quad * (4 * kTcHalf * 32);
    TcRowState<KT> st;
    st.reset();
    long long pending = -1;                                // piece of the last sub-tile folded into `st`
    int pending_j = -1, pending_n = 0;
    bool pending_valid = false;
    TcWalk w;
    w.start(c, g, run, cost_cache);
    for (int batch = 0; w.left > 0; ++batch) {
        const int buf = batch & 1;
        tc_wait(smem_u32(&tmem_full[buf]), ((uint32_t)batch >> 1) & 1u, abort_flag, c.state);
        tc_fence_after();
        if (pending >= 0 && pending_j != w.j) {            // the entry is behind us: its running partial goes out
            if (pending_valid) tc_flush_row<KT>(c, pp, st, pending_n, (size_t)pending);
            st.reset();
            pending = -1;
        }
        const int t = 2 * (w.u + (w.wide ? 0 : quad)) + rank;                  // this quad's sub-tile
        const bool tile_ok = (w.wide || quad < w.nunits(g)) && t < g.tiles;
        const int hbase = w.wide ? quad * kTcSub : 0;                          // hidden row of the quad's first column
        const int ncols = tile_ok ? min(kTcSub, w.npad - hbase) : 0;           // columns this quad handles
        if (ncols > 0) {
            const int hrow = hbase + q * 32 + lane;                            // the hidden row this thread owns
            const bool row_valid = hrow < w.R;
            const size_t pidx = ((size_t)w.j * g.tiles + t) * kTcPassRows + hrow;
            if (pending >= 0 && pending_valid && CORAL_IDX_OK(pending, c.cap_part_tc, c.state)) {   // not the entry's last piece after all
                pp.pmax[pending] = kNegInf;
                pp.psum[pending] = 0.f;
            }
            float* tap_row = nullptr;
            if (logits_tap && row_valid)
                tap_row = logits_tap + ((size_t)c.bucket_row[w.first + hrow] * c.k_groups + c.bucket_slot[w.first + hrow]) * c.v;
            const uint32_t acc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 2 * kTcSub + quad * kTcSub);
            const bool own = q * 32 < ncols;
            const int half = lane >> 4;
#pragma unroll 1
            for (int s = 0; s < 4; ++s) {
                const int cch = (q + s) & 3;
                const bool give = cch * 32 < ncols;
                float z[32];
                if (give) tc_ld32(acc + (uint32_t)(cch * 32), z);
                const int wsrc = (q - s) & 3;                                  // the warp that writes this warp's block
#pragma unroll 1
                for (int hf = 0; hf < 2; ++hf) {
                    // lanes of vocab rows 16 hf .. 16 hf + 15 of the quarter hand their 32 columns over
                    if (give && half == hf) {
                        float* xw = xq + cch * (kTcHalf * 32) + (lane & 15) * 32;
#pragma unroll
                        for (int i = 0; i < 32; ++i) xw[i ^ lane] = z[i];
                    }
                    quad_sync(quad);
                    if (own && row_valid) {
                        const int base = t * kTcSub + wsrc * 32 + hf * kTcHalf;
                        const int nv = min(kTcHalf, c.v - base);
                        if (nv > 0) tc_fold_block<KT>(st, xq + q * (kTcHalf * 32), lane, hf * kTcHalf, base, nv, tap_row);
                    }
                    quad_sync(quad);
                }
            }
            pending = (long long)pidx;
            pending_j = w.j;
            pending_n = w.n;
            pending_valid = row_valid;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
            if (leader) mbar_arrive(tmem_empty_at + (uint32_t)buf * 8u);
            else mbar_arrive_cluster(tmem_empty_at + (uint32_t)buf * 8u);
        }
        w.next(c, g);
    }
    if (pending >= 0 && pending_valid) tc_flush_row<KT>(c, pp, st, pending_n, (size_t)pending);
}

// grid = 2 * g.pairs CTAs of kTcHeadThreads threads in clusters of two; dynamic shared memory: 1 KiB alignment
// slack + the operand ring + the epilogue's exchange blocks + barriers.
__global__ void __launch_bounds__(kTcHeadThreads, 1)
    head_tc_kernel(CallView c, TcGeom g, TcPartials pp, const __grid_constant__ CUtensorMap map_w,
                   const uint16_t* __restrict__ hg, float* __restrict__ logits_tap) {
    extern __shared__ unsigned char tc_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    float* xchg = reinterpret_cast<float*>(smem + kTcRingBytes);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kTcRingBytes + kTcXchgBytes);
    uint64_t* empty = full + kTcMaxSlots;
    uint64_t* tmem_full = empty + kTcMaxSlots;    // [2]
    uint64_t* tmem_empty = tmem_full + 2;         // [2] rank 0: both CTAs' epilogue warps have drained the buffer
    uint64_t* recut = tmem_empty + 2;             // the first producer has let the ring run empty for a new geometry
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(recut + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* cost_cache = reinterpret_cast<int*>(smem + kTcRingBytes + kTcXchgBytes + 256);      // [kTcCostCache]
    int* run = const_cast<int*>(abort_flag) + 1;  // [5] the pair's run, see tc_split_runs
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_ctarank();
    const bool leader = rank == 0;
    if (c.adaptive) {
        // the router decides between this kernel and the streaming one: when it is the other, leave before any
        // set-up (every thread of both CTAs takes the same way out)
        pdl_wait();
        if (c.state->path_choice != 2) return;
    }

    // The kernel may be launched while its predecessors (gather, router) still run: everything up to the
    // dependency wait touches only the pair's shared and tensor memory.
    if (threadIdx.x == 0) {
        for (int s = 0; s < kTcMaxSlots; ++s) {
            // rank 0's "stage has landed" also counts an arrival from rank 1, sent once its own copies are in
            mbar_init(smem_u32(&full[s]), leader ? 2 : 1);
            mbar_init(smem_u32(&empty[s]), 2);                  // both issuers' MMAs on the stage have completed
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&tmem_full[s]), 2);
            mbar_init(smem_u32(&tmem_empty[s]), 2 * kTcEpilogueWarps);
        }
        mbar_init(smem_u32(recut), 2);
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
    if (warp == 0) tc_split_runs(c, g, skip ? 0 : c.state->n_virtual, (int)(blockIdx.x >> 1), run, cost_cache);
    __syncthreads();

    if (warp == 0 || warp == 11) {
        if (lane == 0) {
            // two producers, one column step each in turn: a thread issues the copies of a step in some 150 ns,
            // which alone would set the pace of the batches with one unit
            const uint32_t mine = warp == 0 ? 0u : 1u;
            uint32_t step = 0, recuts = 0;
            TcRingPos rp;
            const uint64_t pol_first = l2_policy_evict_first(), pol_normal = l2_policy_evict_normal(),
                           pol_last = l2_policy_evict_last();
            TcWalk w;
            w.start(c, g, run, cost_cache);
            while (w.left > 0) {
                const int u = w.u, nu = w.nunits(g);
                const int t0 = 2 * u + rank, t1 = 2 * (u + 1) + rank;           // this CTA's sub-tiles
                const bool w0 = t0 < g.tiles, w1 = nu == 2 && t1 < g.tiles;
                // this CTA's half of the entry's hidden rows (the first half in rank 0)
                const uint32_t hbytes = (uint32_t)(w.npad >> 1) * 128u;
                const TcRing ring = tc_ring_for(w.wide, nu);
                if (rp.enter(ring)) {
                    // another slot size from here on: every copy issued so far, by either producer, must have been
                    // consumed first.  The first producer sees to that, then the two meet.  Its own last step is at
                    // most one use of its slot ahead of the barrier, the other producer's last step may be two
                    // (a parity wait cannot tell that from none): after one round over the slots everything but that
                    // step has been consumed, the second round waits for it too.
                    if (mine == 0) {
                        for (int round = 0; round < 2; ++round)
                            for (int s = 0; s < kTcMaxSlots; ++s)
                                tc_wait(smem_u32(&empty[s]), ((rp.parity >> s) & 1u) ^ 1u, abort_flag, c.state);
                    }
                    mbar_arrive(smem_u32(recut));
                    tc_wait(smem_u32(recut), recuts & 1u, abort_flag, c.state);
                    ++recuts;
                }
                const uint32_t bytes = hbytes + (w0 ? kTcTileBytes : 0) + (w1 ? kTcTileBytes : 0);
                const uint64_t pol_w = w.read_again ? pol_normal : pol_first;
                const uint16_t* hsrc = hg + ((size_t)w.hrow + (size_t)rank * (w.npad >> 1)) * kTcK;
                const int gidx = w.n / c.pack_div;
                for (int ks = 0; ks < g.ksteps; ++ks, ++step) {
                    if ((step & 1u) != mine) { rp.advance(ring); continue; }
                    tc_wait(smem_u32(&empty[rp.slot]), rp.par() ^ 1u, abort_flag, c.state);
                    const uint32_t bar = smem_u32(&full[rp.slot]);
                    const uint32_t sb = smem_u32(smem) + (uint32_t)rp.slot * ring.bytes;
                    mbar_expect_tx(bar, bytes);
                    if (w0) tma_load_5d(sb, &map_w, 0, 0, ks, t0 * 8, gidx, bar, pol_w);
                    if (w1) tma_load_5d(sb + kTcTileBytes, &map_w, 0, 0, ks, t1 * 8, gidx, bar, pol_w);
                    bulk_g2s_hint(sb + ring.hoff, hsrc + (size_t)ks * g.hg_rows * kTcK, hbytes, bar, pol_last);
                    rp.advance(ring);
                }
                w.next(c, g);
            }
        }
    } else if (warp == 1 || warp == 10) {
        if (lane == 0 && leader) {
            // issuer `a` owns accumulator a of a batch of two units; a batch of one unit - a wide entry's, with up
            // to 256 columns in one MMA, or a run's odd unit - is the first issuer's (splitting a wide entry's columns
            // between the two changed nothing: 442 against 441 us at 1920 rows).  Both issuers commit on
            // every slot and every batch (a commit with nothing pending arrives at once), so the barriers always
            // count two arrivals
            const int a = warp == 1 ? 0 : 1;
            TcRingPos rp;
            const uint32_t ring_lo = tc_smem_desc_lo(smem_u32(smem));
            TcWalk w;
            w.start(c, g, run, cost_cache);
            for (int batch = 0; w.left > 0; ++batch) {
                const int buf = batch & 1;
                const TcRing ring = tc_ring_for(w.wide, w.nunits(g));
                rp.enter(ring);
                const uint32_t aoff_lo = w.wide ? 0u : (uint32_t)a * (kTcTileBytes >> 4);
                const uint32_t boff_lo = ring.hoff >> 4;
                const uint32_t idesc = tc_idesc(256, w.npad);
                const bool mine = a < w.nunits(g);            // (a wide entry's one unit: the first issuer's)
                tc_wait(smem_u32(&tmem_empty[buf]), (((uint32_t)batch >> 1) & 1u) ^ 1u, abort_flag, c.state);   // drained
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(buf * 2 * kTcSub + a * kTcSub);
                for (int ks = 0; ks < g.ksteps; ++ks) {
                    // (an issuer with nothing to do in this batch waits all the same: its commits must not get
                    // ahead of the stage they speak for)
                    tc_wait(smem_u32(&full[rp.slot]), rp.par(), abort_flag, c.state);   // this CTA's copies and the other's
                    if (mine) {
                        tc_fence_after();
                        const uint32_t s_lo = ring_lo + (uint32_t)rp.slot * (ring.bytes >> 4);
                        const uint32_t a_lo = s_lo + aoff_lo, b_lo = s_lo + boff_lo;
#pragma unroll
                        for (int kk = 0; kk < kTcK / 16; ++kk)               // 32 bytes (two 16-byte units) per 16 columns
                            tc_mma_pair(acc, a_lo + 2 * kk, b_lo + 2 * kk, idesc, kk ? 1u : (ks ? 1u : 0u));
                    }
                    tc_commit_pair(smem_u32(&empty[rp.slot]));  // the slot is free in both CTAs once both issuers' MMAs have read it
                    rp.advance(ring);
                }
                tc_commit_pair(smem_u32(&tmem_full[buf]));    // accumulators complete, in both CTAs
                w.next(c, g);
            }
        } else if (lane == 0 && warp == 1) {
            // rank 1: pass the news that a stage of this CTA has landed on to the MMA issuer in rank 0
            const uint32_t peer_at = cluster_map_shared(smem_u32(full), 0);
            TcRingPos rp;
            TcWalk w;
            w.start(c, g, run, cost_cache);
            while (w.left > 0) {
                const TcRing ring = tc_ring_for(w.wide, w.nunits(g));
                rp.enter(ring);
                for (int ks = 0; ks < g.ksteps; ++ks) {
                    tc_wait(smem_u32(&full[rp.slot]), rp.par(), abort_flag, c.state);
                    mbar_arrive_cluster(peer_at + (uint32_t)rp.slot * 8u);      // counts on rank 0's barrier of the slot
                    rp.advance(ring);
                }
                w.next(c, g);
            }
        }
    } else {
        // epilogue: the four warps of an accumulator exchange blocks so that every thread owns one hidden row
        const uint32_t tmem_empty_at = leader ? smem_u32(tmem_empty) : cluster_map_shared(smem_u32(tmem_empty), 0);
        if (c.k_tokens <= 10)
            tc_epilogue<10>(c, g, pp, logits_tap, tmem_base, tmem_full, tmem_empty_at, leader, abort_flag, xchg, run, cost_cache, rank);
        else
            tc_epilogue<32>(c, g, pp, logits_tap, tmem_base, tmem_full, tmem_empty_at, leader, abort_flag, xchg, run, cost_cache, rank);
    }
    tc_fence_before();
    cluster_sync_all();          // nothing of the other CTA is still on its way to this CTA's barriers or tensor memory
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols) : "memory");
    }
}

}  // namespace coral
