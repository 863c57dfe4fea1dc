// Gathered GEMV for few query rows: every touched group's vocab rows are read
// once with 128-bit loads, each row dotted (fp32 FMA) with the hidden rows that
// selected the group, and the tile's logits reduced on chip to a partial
// (max, sum-exp, top-k) per (row, tile).  (CORAL Section 3.3: logits only for
// the activated groups; softmax over them; Appendix B: top candidates per row.)
#pragma once
#include "common.cuh"

namespace coral {

constexpr int kSimtThreads = 256;
constexpr int kSimtWarps = kSimtThreads / 32;
constexpr int kSimtRowBlock = 8;     // hidden rows processed per pass over a weight tile

// Partial statistics of one hidden row over the logits z[0..rows) of a tile, by one warp.
// z lives in shared memory; tokens[j] is the global id of tile row j (ascending in j).
__device__ __forceinline__ void tile_partials(const CallView& c, const float* z, int rows,
                                              const int32_t* __restrict__ tokens, size_t pidx, int lane) {
    constexpr int kPer = kTileRows / 32;
    float val[kPer];
    float mx = kNegInf;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int j = lane + 32 * i;
        val[i] = (j < rows) ? z[j] : kNegInf;
        mx = fmaxf(mx, val[i]);
    }
    mx = warp_max(mx);
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < kPer; ++i)
        if (lane + 32 * i < rows) sum += __expf(val[i] - mx);
    sum = warp_sum(sum);
    if (lane == 0) {
        c.part_max[pidx] = mx;
        c.part_sum[pidx] = sum;
    }
    // k_tokens rounds of warp arg-best; the tile-local index orders equal values
    // (ascending token id inside a group).
    for (int k = 0; k < c.k_tokens; ++k) {
        float bv = kNegInf;
        int bj = kNoToken;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int j = lane + 32 * i;
            if (j < rows && better(val[i], j, bv, bj)) { bv = val[i]; bj = j; }
        }
        warp_argbest(bv, bj);
        if (bj != kNoToken) {
#pragma unroll
            for (int i = 0; i < kPer; ++i)
                if (lane + 32 * i == bj) val[i] = kNegInf;
        }
        if (lane == 0) {
            const bool ok = bj != kNoToken && bv > kNegInf;
            c.part_val[pidx * c.k_tokens + k] = ok ? bv : kNegInf;
            c.part_id[pidx * c.k_tokens + k] = ok ? __ldg(tokens + bj) : kNoToken;
        }
    }
}

template <int R>
__device__ __forceinline__ void simt_tile_dots(const CallView& c, int n, int row0, const uint16_t* hs, float* zs,
                                               int rows, int H, int warp, int lane) {
    const int chunks = H >> 3;
    const uint4* __restrict__ wbase = reinterpret_cast<const uint4*>(c.packed);
    for (int j = warp; j < rows; j += kSimtWarps) {
        float acc[R];
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r] = 0.f;
#pragma unroll 4
        for (int ch = lane; ch < chunks; ch += 32) {
            const uint4 w = __ldg(wbase + packed_chunk_offset(n / c.pack_div, row0 + j, ch, c.KB, c.T16));
#pragma unroll
            for (int r = 0; r < R; ++r)
                acc[r] = dot8(w, *reinterpret_cast<const uint4*>(hs + (size_t)r * H + ch * 8), acc[r]);
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float s = warp_sum(acc[r]);
            if (lane == 0) zs[r * kTileRows + j] = s;
        }
    }
}

// grid (T, N): one block per (vocab tile, group); blocks of untouched groups exit.
// dynamic shared memory: kSimtRowBlock * H bf16 (hidden rows) + kSimtRowBlock * kTileRows floats.
__global__ void __launch_bounds__(kSimtThreads) head_simt_kernel(CallView c, float* __restrict__ logits_tap) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint16_t* hs = reinterpret_cast<uint16_t*>(smem_raw);
    float* zs = reinterpret_cast<float*>(smem_raw + (size_t)kSimtRowBlock * c.H * sizeof(uint16_t));
    const int n = blockIdx.y, t = blockIdx.x;
    if (call_is_poisoned(c.state)) return;        // the router stage reported a problem: index with nothing
    const int cnt = c.group_count[n];
    if (cnt == 0) return;
    const int off = c.group_offset[n];
    const int row0 = t * kTileRows;
    const int rows = min(kTileRows, c.v - row0);
    const int32_t* __restrict__ tokens = c.group_tokens + (size_t)n * c.v + row0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = c.H >> 3;

    for (int c0 = 0; c0 < cnt; c0 += kSimtRowBlock) {
        const int rb = min(kSimtRowBlock, cnt - c0);
        for (int i = threadIdx.x; i < rb * chunks; i += kSimtThreads) {
            const int r = i / chunks, ch = i - r * chunks;
            const int m = c.bucket_row[off + c0 + r];
            reinterpret_cast<uint4*>(hs)[(size_t)r * chunks + ch] =
                __ldg(reinterpret_cast<const uint4*>(c.hidden + (size_t)m * c.H) + ch);
        }
        __syncthreads();
        switch (rb) {
            case 1: simt_tile_dots<1>(c, n, row0, hs, zs, rows, c.H, warp, lane); break;
            case 2: simt_tile_dots<2>(c, n, row0, hs, zs, rows, c.H, warp, lane); break;
            case 3: simt_tile_dots<3>(c, n, row0, hs, zs, rows, c.H, warp, lane); break;
            case 4: simt_tile_dots<4>(c, n, row0, hs, zs, rows, c.H, warp, lane); break;
            case 5: simt_tile_dots<5>(c, n, row0, hs, zs, rows, c.H, warp, lane); break;
            case 6: simt_tile_dots<6>(c, n, row0, hs, zs, rows, c.H, warp, lane); break;
            case 7: simt_tile_dots<7>(c, n, row0, hs, zs, rows, c.H, warp, lane); break;
            default: simt_tile_dots<8>(c, n, row0, hs, zs, rows, c.H, warp, lane); break;
        }
        __syncthreads();
        for (int r = warp; r < rb; r += kSimtWarps) {
            const int m = c.bucket_row[off + c0 + r];
            const int slot = c.bucket_slot[off + c0 + r];
            const size_t pidx = ((size_t)m * c.k_groups + slot) * c.T + t;
            if (logits_tap) {
                float* dst = logits_tap + ((size_t)m * c.k_groups + slot) * c.v + row0;
                for (int j = lane; j < rows; j += 32) dst[j] = zs[r * kTileRows + j];
            }
            tile_partials(c, zs + r * kTileRows, rows, tokens, pidx, lane);
        }
        __syncthreads();
    }
}

}  // namespace coral
