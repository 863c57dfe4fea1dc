// Cross-Step Representation Alignment objective (CORAL Section 3.1, Eq. 2): InfoNCE over cosine similarities,
//   loss_i = LSE_j( q^_i . k^_j / tau ) - mean_s ( q^_i . k^_{i + s n} / tau ),   loss = mean_i loss_i,
// n query features, m = views * n key features, q^ and k^ the features divided by their norms.
//
// Three steps: (1) csra_normalise_kernel divides every feature by its norm (float64) and stores it as bf16 in
// blocks of 128 rows x 64 columns (one contiguous 16 KiB operand tile per block); (2) csra_sim_kernel is a
// dense n x m x D contraction on the 5th-generation tensor cores built from the pieces of head_tc_kernel (TMA
// tiled loads into a ring of stages, tcgen05.mma with M = 128 query rows x N = 128 key rows per accumulator,
// 2 x 2 accumulators per batch in tensor memory) whose epilogue
// folds the scaled similarities into a running (max, sum-exp) per query row and picks out the positives, so
// the n x m similarity matrix never reaches HBM; (3) csra_finalize_kernel combines the partials per row and
// csra_mean_kernel averages the rows in a fixed order.
#pragma once
#include "head_tc.cuh"

namespace coral {

constexpr int kCsraMaxViews = 8;

struct CsraGeom {
    int n, m, views, D;
    int RB, KT;        // query row blocks, key tiles (of 128 rows)
    int ksteps;        // 64-column blocks = ceil(D / 64)
    int grid;
    float inv_tau;
};

// One block per feature row: x / ||x||, rounded to bf16, into the blocked layout
// out[row block][column block][128 rows][64 columns]; columns past D are zero, and the blocks past the last row
// write zero rows, so that every operand tile is defined.  The rounding to bf16 decides which of two
// neighbouring operand values the contraction sees, so it is taken from a float64 value (norm and scaling in
// float64): whoever repeats it in float64 lands on the same side of the rounding boundary.
// x * inv rounded to bf16 (nearest, ties to even) as if from the exact product, in float32 arithmetic: inv is
// given as hi + lo (two floats, from a float64), p = fl(x * hi), and err = (x * hi - p) + x * lo is the rest,
// far below half a unit in the last place of p.  A float32 is either exactly half-way between two bf16 values
// (then the sign of err decides, and only err = 0 is a true tie) or at least one float32 spacing away from
// the half-way point, further than err can move it.
__device__ __forceinline__ uint32_t csra_scale_round_bf16(float x, float hi, float lo) {
    const float p = x * hi;
    const float err = fmaf(x, hi, -p) + x * lo;
    const uint32_t u = __float_as_uint(p);
    const uint32_t low = u & 0xFFFFu;
    uint32_t r = u >> 16;
    if (low == 0x8000u) {                                   // exactly half-way: p's magnitude grows with err's sign
        const bool away = (err > 0.f) != (p < 0.f);         // the exact value lies beyond the half-way point
        if (err != 0.f ? away : (r & 1u)) ++r;
    } else if (low > 0x8000u) {
        ++r;
    }
    return r;
}

__global__ void __launch_bounds__(128) csra_normalise_kernel(const uint16_t* __restrict__ x, int rows, int D, int KB,
                                                             uint16_t* __restrict__ out) {
    __shared__ double s_part[4];
    const int row = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = D >> 3;                                   // 8 columns = one 128-bit word
    const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)(row < rows ? row : 0) * D);
    double ss = 0.0;
    if (row < rows)
        for (int ch = threadIdx.x; ch < chunks; ch += 128) {
            const uint4 w = __ldg(src + ch);
            const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = bf16_lo(u[i]), hi = bf16_hi(u[i]);
                ss += (double)(lo * lo);                    // squares of bf16 values are exact in float32
                ss += (double)(hi * hi);
            }
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) s_part[warp] = ss;
    __syncthreads();
    ss = (s_part[0] + s_part[1]) + (s_part[2] + s_part[3]);
    // x * (1 / norm) instead of x / norm: the two differ by about one unit in the last place of a float64,
    // 13 orders of magnitude below the spacing of bf16 values, so they round to the same bf16
    const double inv = ss > 0.0 ? 1.0 / sqrt(ss) : 0.0;
    const float inv_hi = (float)inv, inv_lo = (float)(inv - (double)inv_hi);
    uint4* dst = reinterpret_cast<uint4*>(out + ((size_t)(row >> 7) * KB * 128 + (row & 127)) * 64);
    for (int ch = threadIdx.x; ch < KB * 8; ch += 128) {
        uint4 r = make_uint4(0, 0, 0, 0);
        if (row < rows && ch < chunks) {
            const uint4 w = __ldg(src + ch);
            const uint32_t u[4] = {w.x, w.y, w.z, w.w};
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                o[i] = csra_scale_round_bf16(bf16_lo(u[i]), inv_hi, inv_lo) |
                       (csra_scale_round_bf16(bf16_hi(u[i]), inv_hi, inv_lo) << 16);
            r = make_uint4(o[0], o[1], o[2], o[3]);
        }
        dst[(size_t)(ch >> 3) * 128 * 8 + (ch & 7)] = r;          // block kb = ch / 8, 16 bytes at column (ch % 8) * 8
    }
}

struct CsraRowState {
    float mx, sum;
    __device__ __forceinline__ void reset() { mx = kNegInf; sum = 0.f; }
};

// Epilogue of one 128 x 128 accumulator for one thread (= one query row): scale by 1 / tau, fold the
// similarities to key rows [base, base + 128) into the running (max, sum-exp), store the positives.
__device__ __forceinline__ void csra_fold_row(const CsraGeom& g, CsraRowState& st, uint32_t tmem_acc_row, int row,
                                              int base, bool row_valid, float* __restrict__ out_pos,
                                              float* __restrict__ logits_tap) {
    constexpr float kLog2e = 1.4426950408889634f;
    const int valid = min(kTcSub, g.m - base);
#pragma unroll 1
    for (int ch = 0; ch < 4; ++ch) {
        float z[32];
        tc_ld32(tmem_acc_row + (uint32_t)(ch * 32), z);
        const int nv = min(32, valid - ch * 32);
        if (!row_valid || nv <= 0) continue;
#pragma unroll
        for (int i = 0; i < 32; ++i) z[i] *= g.inv_tau;
        float cm = kNegInf;
#pragma unroll
        for (int i = 0; i < 32; ++i) cm = fmaxf(cm, i < nv ? z[i] : kNegInf);
        const float nm = fmaxf(st.mx, cm);
        float add = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) add += i < nv ? exp2f((z[i] - nm) * kLog2e) : 0.f;
        st.sum = st.sum * exp2f((st.mx - nm) * kLog2e) + add;
        st.mx = nm;
        if (logits_tap) {
            float* dst = logits_tap + (size_t)row * g.m + base + ch * 32;
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < nv) dst[i] = z[i];
        }
        // positives of this row: key row + s * n, s = 0 .. views - 1
        for (int s = 0; s < g.views; ++s) {
            const int col = row + s * g.n - base - ch * 32;
            if (col >= 0 && col < nv) {
                float v = 0.f;
#pragma unroll
                for (int i = 0; i < 32; ++i) v = i == col ? z[i] : v;
                out_pos[(size_t)row * g.views + s] = v;
            }
        }
    }
}

// The contraction.  A batch is a 256 x 256 block of the similarity matrix: two query row blocks x two key
// tiles, four 128 x 128 accumulators that fill the 512 columns of tensor memory, so every operand tile that
// enters shared memory is used twice (128 flop per byte taken in, against 85 for a 128 x 256 block; what an
// SM can take in - about 66 GB/s - is what bounds this kernel design).  Three stages of 64 KiB (A0, A1, B0,
// B1).  There is no second set of accumulators, so the epilogue of a batch is not hidden behind the next
// batch's MMAs; it is short here (one exp per similarity, no top-k).
// grid = g.grid CTAs of kTcThreads threads; the list of (row block pair, key tile pair) positions is cut into
// contiguous runs, one per CTA.  Partials pmax / psum: [row block * KT + key tile][128 rows]; an epilogue
// thread carries its row's running (max, sum-exp) over the batches of the run that belong to its row block
// and writes it at the first key tile of the last of them; the other slots get an empty marker
// (max = -inf, sum = 0).  Warps 2..5 read row block 0 of the pair, warps 6..9 row block 1.
constexpr int kCsraStages = 3;
constexpr int kCsraStageBytes = 4 * kTcTileBytes;
constexpr size_t kCsraSmemBytes = 1024 + (size_t)kCsraStages * kCsraStageBytes + 256;

__global__ void __launch_bounds__(kTcThreads, 1)
    csra_sim_kernel(CsraGeom g, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    float* __restrict__ pmax, float* __restrict__ psum, float* __restrict__ out_pos,
                    float* __restrict__ logits_tap, DeviceState* state) {
    extern __shared__ unsigned char tc_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kCsraStages * kCsraStageBytes);
    uint64_t* empty = full + kCsraStages;
    uint64_t* tmem_full = empty + kCsraStages;    // [1]
    uint64_t* tmem_empty = tmem_full + 1;         // [1]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kCsraStages; ++s) {
            mbar_init(smem_u32(&full[s]), 1);
            mbar_init(smem_u32(&empty[s]), 1);
        }
        mbar_init(smem_u32(tmem_full), 1);
        mbar_init(smem_u32(tmem_empty), kTcEpilogueWarps);
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

    const int RB2 = (g.RB + 1) >> 1, KT2 = (g.KT + 1) >> 1;
    const int n_pos = RB2 * KT2;
    const int per = (n_pos + g.grid - 1) / g.grid;
    const int lo = min(n_pos, (int)blockIdx.x * per);
    const int hi = min(n_pos, lo + per);

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            const uint64_t pol_normal = l2_policy_evict_normal();
            for (int pos = lo; pos < hi; ++pos) {
                const int rb2 = pos / KT2, kt2 = pos - rb2 * KT2;
                for (int ks = 0; ks < g.ksteps; ++ks) {
                    tc_wait(smem_u32(&empty[stage]), phase ^ 1u, abort_flag, state);
                    const uint32_t bar = smem_u32(&full[stage]);
                    const uint32_t sb = smem_u32(smem + (size_t)stage * kCsraStageBytes);
                    mbar_expect_tx(bar, (uint32_t)kCsraStageBytes);
                    // blocks past the last row block / key tile lie outside the tensor: the copy fills zeros
                    for (int mb = 0; mb < 2; ++mb)
                        tma_load_2d(sb + mb * kTcTileBytes, &map_q, 0, ((rb2 * 2 + mb) * g.ksteps + ks) * 128, bar, pol_normal);
                    for (int sub = 0; sub < 2; ++sub)
                        tma_load_2d(sb + (2 + sub) * kTcTileBytes, &map_k, 0, ((kt2 * 2 + sub) * g.ksteps + ks) * 128, bar,
                                    pol_normal);
                    if (++stage == kCsraStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int stage = 0, batch = 0;
            uint32_t phase = 0;
            for (int pos = lo; pos < hi; ++pos, ++batch) {
                tc_wait(smem_u32(tmem_empty), ((uint32_t)batch & 1u) ^ 1u, abort_flag, state);   // epilogue has drained
                tc_fence_after();
                for (int ks = 0; ks < g.ksteps; ++ks) {
                    tc_wait(smem_u32(&full[stage]), phase, abort_flag, state);
                    tc_fence_after();
                    const uint32_t sb = smem_u32(smem + (size_t)stage * kCsraStageBytes);
#pragma unroll
                    for (int kk = 0; kk < kTcK / 16; ++kk) {
#pragma unroll
                        for (int mb = 0; mb < 2; ++mb) {
                            const uint64_t adesc = tc_smem_desc(sb + mb * kTcTileBytes + kk * 32);
#pragma unroll
                            for (int sub = 0; sub < 2; ++sub) {
                                const uint64_t bdesc = tc_smem_desc(sb + (2 + sub) * kTcTileBytes + kk * 32);
                                tc_mma(tmem_base + (uint32_t)((mb * 2 + sub) * kTcSub), adesc, bdesc, (ks | kk) ? 1u : 0u);
                            }
                        }
                    }
                    tc_commit(smem_u32(&empty[stage]));
                    if (++stage == kCsraStages) { stage = 0; phase ^= 1u; }
                }
                tc_commit(smem_u32(tmem_full));
            }
        }
    } else {
        const int quarter = warp & 3;
        const int mb = (warp - 2) >> 2;                       // row block of the pair this warp reads
        const int row_in_block = quarter * 32 + lane;
        CsraRowState st;
        st.reset();
        int batch = 0;
        for (int pos = lo; pos < hi; ++pos, ++batch) {
            const int rb2 = pos / KT2, kt2 = pos - rb2 * KT2;
            const int rb = rb2 * 2 + mb;
            tc_wait(smem_u32(tmem_full), (uint32_t)batch & 1u, abort_flag, state);
            tc_fence_after();
            const int row = rb * 128 + row_in_block;
            const bool row_valid = row < g.n;
            for (int sub = 0; sub < 2; ++sub) {
                const int kt = kt2 * 2 + sub;
                if (kt >= g.KT) continue;                      // warp-uniform
                const uint32_t acc_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((mb * 2 + sub) * kTcSub);
                csra_fold_row(g, st, acc_row, row, kt * kTcSub, row_valid, out_pos, logits_tap);
            }
            const bool last = pos + 1 >= hi || (pos + 1) / KT2 != rb2;
            if (row_valid) {
                const size_t p0 = ((size_t)rb * g.KT + kt2 * 2) * 128 + row_in_block;
                pmax[p0] = last ? st.mx : kNegInf;
                psum[p0] = last ? st.sum : 0.f;
                if (kt2 * 2 + 1 < g.KT) { pmax[p0 + 128] = kNegInf; psum[p0 + 128] = 0.f; }
            }
            if (last) st.reset();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(tmem_empty));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols) : "memory");
    }
}

// One thread per query row: log-sum-exp over the row's KT partials, minus the mean of its positives.
__global__ void __launch_bounds__(256) csra_finalize_kernel(CsraGeom g, const float* __restrict__ pmax,
                                                            const float* __restrict__ psum,
                                                            const float* __restrict__ pos,
                                                            float* __restrict__ out_row_loss) {
    const int row = blockIdx.x * 256 + threadIdx.x;
    if (row >= g.n) return;
    const size_t p0 = (size_t)(row >> 7) * g.KT * 128 + (row & 127);
    float mx = kNegInf;
    for (int t = 0; t < g.KT; ++t) mx = fmaxf(mx, pmax[p0 + (size_t)t * 128]);
    float sum = 0.f;
    for (int t = 0; t < g.KT; ++t) {
        const float a = pmax[p0 + (size_t)t * 128];
        if (a != kNegInf) sum += psum[p0 + (size_t)t * 128] * expf(a - mx);
    }
    float pm = 0.f;
    for (int s = 0; s < g.views; ++s) pm += pos[(size_t)row * g.views + s];
    out_row_loss[row] = mx + logf(sum) - pm / (float)g.views;
}

// Mean of the n row losses by one block, in a fixed order (bitwise reproducible).
__global__ void __launch_bounds__(1024) csra_mean_kernel(const float* __restrict__ row_loss, int n, float* __restrict__ out) {
    __shared__ float s_part[32];
    float acc = 0.f;
    for (int i = threadIdx.x; i < n; i += 1024) acc += row_loss[i];
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x < 32) {
        float v = s_part[threadIdx.x];
        v = warp_sum(v);
        if (threadIdx.x == 0) out[0] = v / (float)n;
    }
}

}  // namespace coral
