// Shared device helpers for the grouped LM-head kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace coral {

constexpr int kTileRows = 128;        // vocab rows per work tile
constexpr int kMaxKTokens = 32;       // CORAL_MAX_K_TOKENS
constexpr int kMaxGroups = 256;       // CORAL_MAX_GROUPS
constexpr float kNegInf = -__builtin_huge_valf();
constexpr int kNoToken = 0x7fffffff;
constexpr int kTcPassRows = 256;      // tensor-core path: hidden rows per pass over a group's weights (the MMA's largest N)

// Tensor-core path: first row, in the gathered hidden matrix, of the union-list entry whose first bucket position is
// `first` and whose index in the union list is j: entries are packed in bucket order, each starting on a multiple of
// 16 rows (the step from one entry to the next is at least its row count rounded up to 16).
__host__ __device__ __forceinline__ int tc_entry_row(int first, int j) { return ((first + 15) & ~15) + 16 * j; }

// Device-resident per-handle state written by the kernels.
struct DeviceState {
    int status;        // 0 or a CORAL_ERR_* code (first error wins)
    int n_union;       // groups touched by the last call
    int ticket;        // arrival counter of the fused router kernel; zero between calls
    int n_virtual;     // (group, pass) entries of the union list; equals n_union when no group needs a second pass
    int path_choice;   // adaptive calls: 1 = streaming kernel, 2 = tensor-core kernel, chosen by the router from the row counts
};

// Per-call view of the workspace handed to the kernels.
struct CallView {
    int M, H, V, N, v, T;          // T = tiles per group = ceil(v / kTileRows)
    int k_groups, k_tokens;
    int union_cap;                 // capacity of union_list
    int pass_rows;                 // rows of a group handled per pass over its weights (0: one pass for any count)
    int adaptive;                  // 1: the router picks pass_rows (streaming) or pass_rows_tc (tensor cores) and records it
    int pass_rows_tc, union_cap_tc;   // the tensor-core alternative of an adaptive call
    int hot_groups;                // groups below this index are loaded with an evict-last L2 hint (kept across calls)
    int pack_div;                  // the packed copy holds group n at index n / pack_div (1, or shard_world when only this rank's groups are stored)
    int shard_rank, shard_world;   // vocab sharding: this call computes only the groups n with n % shard_world == shard_rank
    const uint16_t* packed;        // blocked copy of W_vocab, see packed_chunk_offset
    int KB, T16;                   // packed layout: 64-column blocks per row, 16-row items per group
    const uint16_t* w_gate;        // [N][H] bf16
    const int32_t* group_tokens;   // [N][v] global token id of packed row
    const uint16_t* hidden;        // [M][H] bf16
    const float* router_in;        // [M][H] fp32 router input act(W1 h) + h (Eq. 7), or null: the gate reads `hidden`
    float* gate;                   // [M][N]
    int32_t* sel;                  // [M][k_groups]
    int16_t* slot_of;              // [M][N] slot of group n in row m, -1 if not selected
    int32_t* group_count;          // [N]
    int32_t* group_offset;         // [N+1]
    int32_t* bucket_row;           // [M*k_groups] rows that selected a group, ascending per group
    int32_t* bucket_slot;          // [M*k_groups] the slot the group has in that row
    int32_t* bucket_dst;           // [M*k_groups] tensor-core calls: the pair's row in the gathered hidden matrix
    int32_t* slot_desc;            // [M][k_groups] (index in union_list of the slot's (group, pass)) << 8 | row's position in the pass
    int32_t* union_list;           // [n_virtual] group | pass << 16, ascending (group, pass)
    int32_t* union_rank;           // [N] index of (group n, pass 0) in union_list, -1 if untouched
    float* part_max;               // [M][k_groups][T]
    float* part_sum;               // [M][k_groups][T]
    float* part_val;               // [M][k_groups][T][k_tokens]
    int32_t* part_id;              // [M][k_groups][T][k_tokens]
    DeviceState* state;
    // capacities of the arrays above, for the range-checked build (CORAL_CHECK_BOUNDS)
    int cap_pairs;                 // entries of bucket_row / bucket_slot / slot_desc / sel
    int cap_hg_rows;               // rows of one column block of the tensor-core path's gathered hidden matrix
    long long cap_part_stream;     // partial records of the streaming path
    long long cap_part_tc;         // partial records of the tensor-core path
    long long cap_packed;          // 16-byte units of the packed copy
};

// Packed layout of the LM head: [group][item of 16 vocab rows, ascending token id][block of 64 columns]
// [16 rows][64 columns] bf16.  A 16-row item is contiguous (so a slab of 512 columns of an item is one
// contiguous 16 KiB bulk copy) and every 16 x 64 block is a contiguous 2 KiB piece (so a 128-row x 64-column
// operand tile is eight such pieces, fetched by one tiled TMA load).  Rows past the group's size and
// columns past H are zero.
// Returns the offset, in 16-byte units, of chunk `ch` (8 columns) of row `j` of group `n`.
__host__ __device__ __forceinline__ size_t packed_chunk_offset(int n, int j, int ch, int KB, int T16) {
    const int item = j >> 4, r = j & 15;
    const int kb = ch >> 3, cc = ch & 7;
    return ((((size_t)n * T16 + item) * KB + kb) * 16 + r) * 8 + cc;
}

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// fp32 dot product of 8 bf16 pairs held in two 128-bit words.
__device__ __forceinline__ float dot8(const uint4& a, const uint4& b, float acc) {
    acc = fmaf(bf16_lo(a.x), bf16_lo(b.x), acc);
    acc = fmaf(bf16_hi(a.x), bf16_hi(b.x), acc);
    acc = fmaf(bf16_lo(a.y), bf16_lo(b.y), acc);
    acc = fmaf(bf16_hi(a.y), bf16_hi(b.y), acc);
    acc = fmaf(bf16_lo(a.z), bf16_lo(b.z), acc);
    acc = fmaf(bf16_hi(a.z), bf16_hi(b.z), acc);
    acc = fmaf(bf16_lo(a.w), bf16_lo(b.w), acc);
    acc = fmaf(bf16_hi(a.w), bf16_hi(b.w), acc);
    return acc;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

// Order used everywhere: larger value first, equal values -> smaller key first.
__device__ __forceinline__ bool better(float va, int ka, float vb, int kb) {
    return va > vb || (va == vb && ka < kb);
}

// All lanes receive the best (value, key) pair of the warp.
__device__ __forceinline__ void warp_argbest(float& v, int& k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, v, o);
        int ok = __shfl_xor_sync(0xffffffffu, k, o);
        if (better(ov, ok, v, k)) { v = ov; k = ok; }
    }
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialisation attribute may start
// while its predecessor in the stream still runs; pdl_wait() blocks until the predecessor has completed
// and its writes are visible (no-op without the attribute).  pdl_launch_dependents() lets the successor start.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void set_status(DeviceState* st, int code) { atomicCAS(&st->status, 0, code); }

// Range-checked build (-DCORAL_CHECK_BOUNDS; the stand-in for a memory checker): every index the kernels
// compute from the router's output - bucket positions, slot descriptors, union-list entries, piece indices,
// token-table reads, offsets into the packed copy and the gathered rows - is compared with the capacity of
// what it indexes.  A violation sets CORAL_ERR_BOUNDS in the status word; a read then takes element 0
// instead and a write is skipped, so nothing traps and nothing outside the buffers is touched.  In the
// normal build the macros cost nothing.
#ifdef CORAL_CHECK_BOUNDS
__device__ __forceinline__ bool index_ok(long long i, long long n, DeviceState* st) {
    if (i >= 0 && i < n) return true;
    set_status(st, -6);
    return false;
}
#define CORAL_IDX(i, n, st) (::coral::index_ok((long long)(i), (long long)(n), (st)) ? (i) : 0)
#define CORAL_IDX_OK(i, n, st) ::coral::index_ok((long long)(i), (long long)(n), (st))
#else
#define CORAL_IDX(i, n, st) (i)
#define CORAL_IDX_OK(i, n, st) true
#endif

// The status word is sticky until the host reads it.  A call whose router stage reported a problem (forced
// groups out of range or repeated: the bucket arrays are then inconsistent) must not be followed by kernels
// that index with those arrays; every kernel after the router stage checks this first and does nothing.
__device__ __forceinline__ bool call_is_poisoned(const DeviceState* st) {
    return *reinterpret_cast<const volatile int*>(&st->status) != 0;
}

// Vocab sharding over several GPUs: group n belongs to the GPU with rank n % world.
__device__ __forceinline__ bool group_is_local(const CallView& c, int n) {
    return c.shard_world <= 1 || n % c.shard_world == c.shard_rank;
}

}  // namespace coral
