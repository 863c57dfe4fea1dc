// C ABI of the grouped LM-head draft step: handle management, argument checks,
// workspace layout and kernel launches.  See include/coral_lmhead.h.
#include "coral_lmhead.h"

#include <cuda_runtime.h>

#include <new>
#include <vector>

#include "common.cuh"
#include "head_simt.cuh"
#include "head_stream.cuh"
#include "head_tc.cuh"
#include "copy_probe.cuh"
#include "tc_probe.cuh"
#include "csra.cuh"
#include "merge.cuh"
#include "route.cuh"
#include "tree.cuh"

using namespace coral;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Offsets of the workspace sections (bytes from the workspace base).
struct Layout {
    size_t w_gate, group_tokens, state, gate, sel, slot_of, group_count, group_offset, bucket_row, bucket_slot, bucket_dst,
        slot_desc, union_list, union_rank, part_max, part_sum, part_val, part_id, sp_max, sp_sum, sp_val, sp_id,
        cand_val, cand_id, route_mid, route_part, tc_hg, tc_max, tc_sum, tc_val, tc_id, stage_hidden, stage_ids, stage_logprobs, total;
    size_t packed_bytes, cand_cap, cand_rows;
    int v, T;
    int KB, T16;                 // packed layout (see packed_chunk_offset)
    size_t route_bands;
    int packed_groups;           // groups stored in the packed copy (all, or this rank's)
    int tc_tiles, tc_vcap;       // tensor-core path: sub-tiles per group, capacity in (group, pass) entries
    size_t tc_rows;              // (row, slot) pairs the path is provisioned for (0: not provisioned)
    int tc_hg_rows;              // rows of one column block of the gathered hidden matrix
};

bool config_ok(const coral_lmhead_config* c) {
    if (!c || c->struct_size != sizeof(coral_lmhead_config)) return false;
    if (c->H < 8 || c->H % 8 != 0 || c->V < 1 || c->n_groups < 1 || c->n_groups > CORAL_MAX_GROUPS) return false;
    if (c->V % c->n_groups != 0) return false;
    if (c->max_M < 1 || c->max_k_groups < 1 || c->max_k_groups > c->n_groups) return false;
    if (c->max_k_tokens < 1 || c->max_k_tokens > CORAL_MAX_K_TOKENS) return false;
    const int world = (int)(c->flags & 0xff), rank = (int)((c->flags >> 8) & 0xff);
    if (c->flags >> 16) return false;
    if (world == 0 ? rank != 0 : (rank >= world || world > c->n_groups)) return false;
    return true;
}
inline int cfg_world(const coral_lmhead_config& c) { return (c.flags & 0xff) > 1 ? (int)(c.flags & 0xff) : 1; }
inline int cfg_rank(const coral_lmhead_config& c) { return (int)((c.flags >> 8) & 0xff); }

// Geometry of the streaming path.  The workspace layout must not depend on the device (sizes are
// queried before a device is chosen), so it is sized for any grid in [kStreamGridMin, kStreamGridCap];
// the launch geometry is fixed at create from the device's SM count and shared-memory limit.
constexpr int kStreamGridMin = 64, kStreamGridCap = 160;
constexpr int kStreamMaxPasses = kStreamMaxM / kStreamPassRows;

// Most (group, pass) entries a CTA's run of ceil(n_virtual * T / grid) items can overlap.
int stream_seg_max(int n_groups, int grid) {
    const long n_virtual_max = (long)n_groups * kStreamMaxPasses;
    return (int)((n_virtual_max + grid - 1) / grid) + 1;
}

StreamGeom make_stream_geom(const coral_lmhead_config& c, int sms, int smem_optin) {
    StreamGeom g{};
    const int v = c.V / c.n_groups;
    g.grid = sms < kStreamGridCap ? sms : kStreamGridCap;
    g.T = (v + kStreamTile - 1) / kStreamTile;
    g.kc = (c.H % 512 == 0) ? 512 : 256;
    g.kstages = c.H / g.kc;
    g.stage_bytes = kStreamTile * g.kc * 2;
    const long fixed = (long)sizeof(float) * kStreamZBufs * kStreamWarps * kStreamTile * kStreamPassRows + 1024;
    long ns = ((long)smem_optin - fixed) / g.stage_bytes;
    g.n_stages = (int)(ns > 12 ? 12 : ns);
    g.seg_max = stream_seg_max(c.n_groups, g.grid);
    return g;
}

size_t stream_smem_bytes(const StreamGeom& g) {
    return (size_t)g.n_stages * g.stage_bytes +
           sizeof(float) * kStreamZBufs * kStreamWarps * kStreamTile * kStreamPassRows +
           sizeof(uint64_t) * 2 * g.n_stages + sizeof(uint64_t) * 2 * kStreamZBufs +
           sizeof(int) * kStreamSegTab + 16;
}

constexpr int kTcMinRows = 96;          // above this many rows the tensor-core path is the faster one (measured, iid rows)
constexpr int kTcMinRowsPerGroup = 10;  // ... and from this many rows per group on average (the streaming path reads a
                                        // group once per 16 rows; measured on the three paper shapes: within 10 % either
                                        // way at 7.5-8, 1.15x-2x faster from 12 on)
constexpr int kTcProvisionRows = 32;    // handles for more rows get the tensor-core workspace (adaptive calls use it from 33 rows)
constexpr int kMergeSmemCands = 4096;   // candidates the streaming merge keeps in shared memory

Layout make_layout(const coral_lmhead_config& c) {
    Layout L{};
    L.v = c.V / c.n_groups;
    L.T = (L.v + kTileRows - 1) / kTileRows;
    L.T16 = (L.v + 15) / 16;
    L.KB = (c.H + 63) / 64;
    const size_t M = c.max_M, N = c.n_groups, H = c.H, kg = c.max_k_groups, kt = c.max_k_tokens, T = L.T;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
    L.w_gate = take(N * H * 2);
    L.group_tokens = take((size_t)c.V * 4);
    L.state = take(sizeof(DeviceState));
    L.route_bands = (M + 7) / 8 > (size_t)kRouteMidBands ? (M + 7) / 8 : (size_t)kRouteMidBands;
    L.route_mid = take((L.route_bands + 5 * N) * 4);      // band tickets, 4 mask words and one counter per group
    L.route_part = take(L.route_bands * kRouteMidSplitMax * ((N + 15) / 16) * 128 * 4);   // partial score tiles when H is split
    L.gate = take(M * N * 4);
    L.sel = take(M * kg * 4);
    L.slot_of = take(M * N * 2);
    L.group_count = take(N * 4);
    L.group_offset = take((N + 1) * 4);
    L.bucket_row = take(M * kg * 4);
    L.bucket_slot = take(M * kg * 4);
    L.bucket_dst = take(M * kg * 4);
    L.slot_desc = take(M * kg * 4);
    L.union_list = take(N * kStreamMaxPasses * 4);
    L.union_rank = take(N * 4);
    const size_t sp = (size_t)kStreamGridCap * stream_seg_max(c.n_groups, kStreamGridMin) * kStreamPassRows;
    L.sp_max = take(sp * 4);
    L.sp_sum = take(sp * 4);
    L.sp_val = take(sp * kt * 4);
    L.sp_id = take(sp * kt * 4);
    // candidate scratch of the merge: what does not fit its shared memory.  The streaming path has at most
    // grid + 2 k_groups pieces per row and at most kStreamMaxM rows; the tensor-core path one piece per (slot,
    // sub-tile), which only outgrows shared memory when very many groups are active (dense-equivalent calls)
    size_t cand_rows = M < (size_t)kStreamMaxM ? M : (size_t)kStreamMaxM;
    L.cand_cap = ((size_t)kStreamGridCap + 2 * kg) * kt;
    const size_t tc_cands = M > (size_t)kTcProvisionRows ? kg * (size_t)((L.v + kTcSub - 1) / kTcSub) * kt : 0;
    if (tc_cands > (size_t)kMergeSmemCands) {
        cand_rows = M;
        if (tc_cands > L.cand_cap) L.cand_cap = tc_cands;
    }
    L.cand_rows = cand_rows;
    L.cand_val = take(cand_rows * L.cand_cap * 4);
    L.cand_id = take(cand_rows * L.cand_cap * 4);
    L.part_max = take(M * kg * T * 4);
    L.part_sum = take(M * kg * T * 4);
    L.part_val = take(M * kg * T * kt * 4);
    L.part_id = take(M * kg * T * kt * 4);
    // tensor-core path (only provisioned when calls can exceed the streaming path's row limit)
    L.tc_tiles = (L.v + kTcSub - 1) / kTcSub;
    L.tc_rows = M > (size_t)kTcProvisionRows ? M * kg : 0;
    L.tc_vcap = L.tc_rows ? (int)(N + (M * kg + kTcPassRows - 1) / kTcPassRows) : 0;
    const size_t tcp = (size_t)L.tc_vcap * L.tc_tiles * kTcPassRows;
    L.tc_hg_rows = L.tc_rows ? (int)((L.tc_rows + 15) / 16 * 16 + 16 * (size_t)L.tc_vcap) : 0;   // see tc_entry_row
    L.tc_hg = take((size_t)L.KB * L.tc_hg_rows * kTcK * 2);              // [column block][row][64]
    L.tc_max = take(tcp * 4);
    L.tc_sum = take(tcp * 4);
    L.tc_val = take(tcp * kt * 4);
    L.tc_id = take(tcp * kt * 4);
    L.stage_hidden = take(M * H * 2);
    L.stage_ids = take(M * kt * 4);
    L.stage_logprobs = take(M * kt * 4);
    L.total = o;
    L.packed_groups = (c.n_groups - cfg_rank(c) + cfg_world(c) - 1) / cfg_world(c);   // groups n = rank, rank + world, ...
    L.packed_bytes = (size_t)L.packed_groups * L.T16 * L.KB * 16 * 64 * 2;
    return L;
}

// Row i of group n of the packed copy = W_vocab[group_tokens[n][i]], in the blocked layout; one block per row.
__global__ void pack_rows_kernel(const uint16_t* __restrict__ W, const int32_t* __restrict__ group_tokens,
                                 uint16_t* __restrict__ packed, int H, int v, int KB, int T16, int rank, int world) {
    const int row = blockIdx.x;
    const int ng = row / v, j = row - ng * v;
    if (ng % world != rank) return;               // another rank's group: not stored here
    const int n = ng / world;
    const uint4* src = reinterpret_cast<const uint4*>(W + (size_t)group_tokens[row] * H);
    uint4* dst = reinterpret_cast<uint4*>(packed);
    for (int ch = threadIdx.x; ch < (H >> 3); ch += blockDim.x)
        dst[packed_chunk_offset(n, j, ch, KB, T16)] = __ldg(src + ch);
}

}  // namespace

struct coral_lmhead_s {
    coral_lmhead_config cfg;
    Layout L;
    unsigned char* packed;
    unsigned char* ws;
    bool own_packed, own_ws;
    int forced_path;
    int simt_smem;
    StreamGeom sg;
    int stream_smem;     // 0 if the streaming path is not available for this shape/device
    bool tc_ok;          // tensor-core path available (maps encoded)
    int out_mode;        // CORAL_OUTPUT_*
    int shard_rank, shard_world;   // vocab sharding (coral_lmhead_set_group_shard); world 1 = off
    int hot_groups;                // leading groups whose weights are loaded with an evict-last L2 hint (0 = off)
    bool l2_limit_changed;         // this handle raised the context's persisting-L2 limit ...
    size_t l2_limit_before;        // ... from this value (restored when the hot groups are released)
    uint16_t* w1;        // [H][H] bf16 first router layer (Eq. 7), library-owned, or null
    float* router_u;     // [max_M][H] fp32 act(W1 h) + h, library-owned
    CUtensorMap map_w;   // the packed weights as a 5-d tensor, read in 128-row x 64-column boxes
    int tc_pairs;        // CTA pairs the tensor-core kernel is launched with
    int sms;
    cudaEvent_t ev_head0, ev_head1;   // around the weight-streaming kernel when kernel timing is on
    cudaEvent_t ev_begin, ev_end;     // before the router stage / after the merge
    bool timing;
    // facts about the last draft call
    int last_path, last_M, last_kg, last_kt, last_launches;
    // coral_lmhead_draft_host: the host output buffers seen last and their device aliases (null: not pinned)
    const void* host_seen[2] = {nullptr, nullptr};
    void* host_alias[2] = {nullptr, nullptr};
};

namespace {

CallView make_view(const coral_lmhead_s* h, const void* hidden, int M, int kg, int kt) {
    CallView c{};
    const Layout& L = h->L;
    unsigned char* ws = h->ws;
    c.M = M; c.H = h->cfg.H; c.V = h->cfg.V; c.N = h->cfg.n_groups; c.v = L.v; c.T = L.T;
    c.k_groups = kg; c.k_tokens = kt;
    c.packed = reinterpret_cast<const uint16_t*>(h->packed);
    c.KB = L.KB; c.T16 = L.T16;
    c.w_gate = reinterpret_cast<const uint16_t*>(ws + L.w_gate);
    c.group_tokens = reinterpret_cast<const int32_t*>(ws + L.group_tokens);
    c.hidden = reinterpret_cast<const uint16_t*>(hidden);
    c.router_in = h->w1 ? h->router_u : nullptr;
    c.gate = reinterpret_cast<float*>(ws + L.gate);
    c.sel = reinterpret_cast<int32_t*>(ws + L.sel);
    c.slot_of = reinterpret_cast<int16_t*>(ws + L.slot_of);
    c.group_count = reinterpret_cast<int32_t*>(ws + L.group_count);
    c.group_offset = reinterpret_cast<int32_t*>(ws + L.group_offset);
    c.bucket_row = reinterpret_cast<int32_t*>(ws + L.bucket_row);
    c.bucket_slot = reinterpret_cast<int32_t*>(ws + L.bucket_slot);
    c.bucket_dst = reinterpret_cast<int32_t*>(ws + L.bucket_dst);
    c.slot_desc = reinterpret_cast<int32_t*>(ws + L.slot_desc);
    c.union_list = reinterpret_cast<int32_t*>(ws + L.union_list);
    c.union_rank = reinterpret_cast<int32_t*>(ws + L.union_rank);
    c.union_cap = h->cfg.n_groups * kStreamMaxPasses;
    c.hot_groups = h->hot_groups;
    c.pack_div = cfg_world(h->cfg);
    c.shard_rank = h->shard_rank;
    c.shard_world = h->shard_world;
    c.part_max = reinterpret_cast<float*>(ws + L.part_max);
    c.part_sum = reinterpret_cast<float*>(ws + L.part_sum);
    c.part_val = reinterpret_cast<float*>(ws + L.part_val);
    c.part_id = reinterpret_cast<int32_t*>(ws + L.part_id);
    c.state = reinterpret_cast<DeviceState*>(ws + L.state);
    c.cap_pairs = (int)((size_t)h->cfg.max_M * h->cfg.max_k_groups);
    c.cap_hg_rows = L.tc_hg_rows;
    c.cap_part_stream = (long long)kStreamGridCap * stream_seg_max(h->cfg.n_groups, kStreamGridMin) * kStreamPassRows;
    c.cap_part_tc = (long long)L.tc_vcap * L.tc_tiles * kTcPassRows;
    c.cap_packed = (long long)(L.packed_bytes / 16);
    return c;
}

// Launch with the programmatic-serialisation attribute: the kernel may begin while the previous kernel of
// the stream is still running and synchronises with it through pdl_wait().
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// The same for a kernel that runs as clusters of two CTAs.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_pairs(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Clusters of two CTAs of the tensor-core kernel that the device can hold at once (0 on failure).
int tc_max_pairs(int sms) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(sms / 2 * 2);
    cfg.blockDim = dim3(kTcHeadThreads);
    cfg.dynamicSmemBytes = kTcSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, head_tc_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n < sms / 2 ? n : sms / 2;
}

// cuTensorMapEncodeTiled, looked up through the runtime so that the library does not link against libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
        return nullptr;
    return reinterpret_cast<EncodeTiledFn>(fn);
}

// Tensor map of the tensor-core path: the packed weights as a 5-d tensor (column in block, row in item,
// 64-column block, item, group) read in boxes of 64 columns x 128 rows (8 items = eight contiguous 2 KiB
// pieces) that land in shared memory with the 128-byte swizzle.
bool make_tc_maps(coral_lmhead_s* h) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const Layout& L = h->L;
    const cuuint64_t wdim[5] = {64, 16, (cuuint64_t)L.KB, (cuuint64_t)L.T16, (cuuint64_t)L.packed_groups};
    const cuuint64_t wstr[4] = {128, 2048, (cuuint64_t)L.KB * 2048, (cuuint64_t)L.T16 * L.KB * 2048};
    const cuuint32_t wbox[5] = {(cuuint32_t)kTcK, 16, 1, 8, 1};
    const cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    return enc(&h->map_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, h->packed, wdim, wstr, wbox, ones,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Dynamic shared memory of merge_stream_kernel for p_cap pieces and c_cap in-smem candidates.
inline size_t merge_smem_bytes(int p_cap, int c_cap) { return (size_t)c_cap * 8 + (size_t)p_cap * 25 + 16; }

bool stream_ok(const coral_lmhead_s* h, int M) { return h->stream_smem > 0 && M <= kStreamMaxM; }

// CORAL_PATH_STREAM: streaming kernel (M <= 128, H a multiple of 256, <= 4096); CORAL_PATH_SIMT_PLAIN: any shape.  Returns 0 if the
// forced path cannot run this call.
// The gathered hidden rows of a call (one copy per row and selected group).  Above this many bytes the pair kernel's
// consecutive runs no longer find them in L2 (126 MB, shared with the weight stream) and the pairs take the
// batches in turn instead.
constexpr size_t kTcStridedHgBytes = (size_t)96 << 20;
int tc_strided(const coral_lmhead_s* h, int M, int kg) {
    return (size_t)M * kg * h->cfg.H * 2 > kTcStridedHgBytes ? 1 : 0;
}

bool tc_usable(const coral_lmhead_s* h, int M, int kg) {
    const size_t cands = (size_t)kg * h->L.tc_tiles * h->cfg.max_k_tokens;
    return h->tc_ok && (size_t)M * kg <= h->L.tc_rows && kg * h->L.tc_tiles <= kMergeMaxPieces &&
           (cands <= (size_t)kMergeSmemCands || (cands <= h->L.cand_cap && (size_t)M <= h->L.cand_rows));
}

int choose_path(const coral_lmhead_s* h, int M, int kg) {
    if (h->forced_path == CORAL_PATH_STREAM) return stream_ok(h, M) ? CORAL_PATH_STREAM : 0;
    if (h->forced_path == CORAL_PATH_TCGEN05) return tc_usable(h, M, kg) ? CORAL_PATH_TCGEN05 : 0;
    if (h->forced_path != CORAL_PATH_AUTO && h->forced_path != CORAL_PATH_ADAPTIVE) return h->forced_path;
    if ((M > kTcMinRows || (long long)M * kg >= (long long)kTcMinRowsPerGroup * h->cfg.n_groups) && tc_usable(h, M, kg))
        return CORAL_PATH_TCGEN05;
    if (stream_ok(h, M)) return CORAL_PATH_STREAM;
    return tc_usable(h, M, kg) ? CORAL_PATH_TCGEN05 : CORAL_PATH_SIMT_PLAIN;
}

}  // namespace

extern "C" {

int coral_lmhead_version(void) { return CORAL_LMHEAD_ABI_VERSION; }

const char* coral_lmhead_error_string(int code) {
    switch (code) {
        case CORAL_OK: return "ok";
        case CORAL_ERR_INVALID: return "invalid argument";
        case CORAL_ERR_GROUPING: return "group_map does not split the vocabulary into equal groups";
        case CORAL_ERR_CUDA: return "CUDA runtime error";
        case CORAL_ERR_NOMEM: return "out of memory";
        case CORAL_ERR_TIMEOUT: return "device-side wait timed out";
        case CORAL_ERR_BOUNDS: return "device-side index check failed";
        case CORAL_ERR_NONFINITE: return "a router score was NaN";
        case CORAL_ERR_TOO_LARGE: return "size exceeds a built-in limit (fixed scratch of the no-allocation entry point, tree step)";
        default: return "unknown status";
    }
}

int coral_lmhead_query_sizes(const coral_lmhead_config* cfg, size_t* packed_bytes, size_t* workspace_bytes) {
    if (!config_ok(cfg) || !packed_bytes || !workspace_bytes) return CORAL_ERR_INVALID;
    const Layout L = make_layout(*cfg);
    *packed_bytes = L.packed_bytes;
    *workspace_bytes = L.total;
    return CORAL_OK;
}

int coral_lmhead_create(coral_lmhead_handle* out, const coral_lmhead_config* cfg, const void* W_vocab_dev,
                        const int32_t* group_map_host, const void* W_gate_dev, void* packed_buf_dev,
                        void* workspace_dev, void* stream) {
    if (!out) return CORAL_ERR_INVALID;
    *out = nullptr;
    if (!config_ok(cfg) || !W_vocab_dev || !group_map_host || !W_gate_dev) return CORAL_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(W_vocab_dev) & 15) || (reinterpret_cast<uintptr_t>(W_gate_dev) & 15) ||
        (reinterpret_cast<uintptr_t>(packed_buf_dev) & (kAlign - 1)) ||
        (reinterpret_cast<uintptr_t>(workspace_dev) & (kAlign - 1)))
        return CORAL_ERR_INVALID;
    const int N = cfg->n_groups, V = cfg->V, v = V / N;

    // token -> group must be in range and split V into N equal groups (Section 3.3)
    std::vector<int32_t> group_tokens;
    std::vector<int32_t> fill;
    try {
        group_tokens.resize((size_t)V);
        fill.assign((size_t)N, 0);
    } catch (const std::bad_alloc&) {
        return CORAL_ERR_NOMEM;
    }
    for (int x = 0; x < V; ++x) {
        const int g = group_map_host[x];
        if (g < 0 || g >= N) return CORAL_ERR_INVALID;
        if (fill[g] >= v) return CORAL_ERR_GROUPING;
        group_tokens[(size_t)g * v + fill[g]++] = x;   // ascending token id inside a group
    }
    for (int n = 0; n < N; ++n)
        if (fill[n] != v) return CORAL_ERR_GROUPING;

    coral_lmhead_s* h = new (std::nothrow) coral_lmhead_s();
    if (!h) return CORAL_ERR_NOMEM;
    h->cfg = *cfg;
    h->L = make_layout(*cfg);
    h->forced_path = CORAL_PATH_AUTO;
    h->shard_rank = cfg_rank(*cfg);
    h->shard_world = cfg_world(*cfg);
    h->hot_groups = 0;
    h->packed = static_cast<unsigned char*>(packed_buf_dev);
    h->ws = static_cast<unsigned char*>(workspace_dev);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = CORAL_OK;
    do {
        if (!h->packed) {
            if (cudaMalloc(&h->packed, h->L.packed_bytes) != cudaSuccess) { h->packed = nullptr; rc = CORAL_ERR_NOMEM; break; }
            h->own_packed = true;
        }
        if (!h->ws) {
            if (cudaMalloc(&h->ws, h->L.total) != cudaSuccess) { h->ws = nullptr; rc = CORAL_ERR_NOMEM; break; }
            h->own_ws = true;
        }
        h->simt_smem = kSimtRowBlock * cfg->H * 2 + kSimtRowBlock * kTileRows * 4;
        // The attribute is per kernel, not per handle: always raise it to the device's opt-in limit.
        int dev = 0, smem_optin = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
            rc = CORAL_ERR_CUDA; break;
        }
        if (h->simt_smem > smem_optin) { rc = CORAL_ERR_INVALID; break; }
        if (cudaFuncSetAttribute(head_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) !=
            cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
        h->sms = sms;
        h->tc_ok = false;
        if (h->L.tc_rows > 0 && h->L.tc_vcap <= cfg->n_groups * kStreamMaxPasses && cfg->H >= kTcK && cfg->H % 8 == 0 && (int)kTcSmemBytes <= smem_optin &&
            cudaFuncSetAttribute(head_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes) == cudaSuccess) {
            h->tc_pairs = tc_max_pairs(sms);
            h->tc_ok = h->tc_pairs > 0 && make_tc_maps(h);
        }
        h->sg = make_stream_geom(*cfg, sms, smem_optin);
        h->stream_smem = 0;
        if (cfg->H <= kStreamMaxH && cfg->H % 256 == 0 && sms >= kStreamGridMin && h->sg.n_stages >= 2) {
            h->stream_smem = (int)stream_smem_bytes(h->sg);
            if (cudaFuncSetAttribute(head_stream_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) !=
                    cudaSuccess ||
                cudaFuncSetAttribute(head_stream_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) !=
                    cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
            if (cudaFuncSetAttribute(merge_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)merge_smem_bytes(kMergeMaxPieces, kMergeSmemCands)) != cudaSuccess) {
                rc = CORAL_ERR_CUDA; break;
            }
        }
        if (cudaMemcpyAsync(h->ws + h->L.group_tokens, group_tokens.data(), (size_t)V * 4, cudaMemcpyHostToDevice, st) !=
            cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
        if (cudaMemcpyAsync(h->ws + h->L.w_gate, W_gate_dev, (size_t)N * cfg->H * 2, cudaMemcpyDeviceToDevice, st) !=
            cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
        if (cudaMemsetAsync(h->ws + h->L.state, 0, sizeof(DeviceState), st) != cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
        if (cudaMemsetAsync(h->ws + h->L.route_mid, 0, (h->L.route_bands + 5 * (size_t)cfg->n_groups) * 4, st) != cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
        if (cudaMemsetAsync(h->packed, 0, h->L.packed_bytes, st) != cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
        pack_rows_kernel<<<V, 128, 0, st>>>(static_cast<const uint16_t*>(W_vocab_dev),
                                            reinterpret_cast<const int32_t*>(h->ws + h->L.group_tokens),
                                            reinterpret_cast<uint16_t*>(h->packed), cfg->H, v, h->L.KB, h->L.T16,
                                            cfg_rank(*cfg), cfg_world(*cfg));
        if (cudaGetLastError() != cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
        if (cudaStreamSynchronize(st) != cudaSuccess) { rc = CORAL_ERR_CUDA; break; }
    } while (0);
    if (rc != CORAL_OK) {
        coral_lmhead_destroy(h);
        return rc;
    }
    *out = h;
    return CORAL_OK;
}

static int release_hot_groups(coral_lmhead_handle h);

int coral_lmhead_destroy(coral_lmhead_handle h) {
    if (!h) return CORAL_OK;
    release_hot_groups(h);
    if (h->own_packed && h->packed) cudaFree(h->packed);
    if (h->own_ws && h->ws) cudaFree(h->ws);
    if (h->w1) cudaFree(h->w1);
    if (h->router_u) cudaFree(h->router_u);
    if (h->ev_head0) cudaEventDestroy(h->ev_head0);
    if (h->ev_head1) cudaEventDestroy(h->ev_head1);
    if (h->ev_begin) cudaEventDestroy(h->ev_begin);
    if (h->ev_end) cudaEventDestroy(h->ev_end);
    delete h;
    return CORAL_OK;
}

int coral_lmhead_set_path(coral_lmhead_handle h, int path) {
    if (!h || path < CORAL_PATH_AUTO || path > CORAL_PATH_ADAPTIVE) return CORAL_ERR_INVALID;
    h->forced_path = path;
    return CORAL_OK;
}

// The draft step.  partial_dev != null: vocab-sharded call, the merge writes per-row records there instead of
// out_ids / out_logprobs (which may then be null).
static int draft_impl(coral_lmhead_handle h, const void* hidden_dev, int M, int k_groups, int k_tokens,
                      const int32_t* forced_groups_dev, int32_t* out_groups_dev, float* out_gate_dev,
                      float* out_logits_dev, float* out_lse_dev, int32_t* out_ids_dev, float* out_logprobs_dev,
                      float* partial_dev, void* stream) {
    if (!h || !hidden_dev) return CORAL_ERR_INVALID;
    if (!partial_dev && (!out_ids_dev || !out_logprobs_dev)) return CORAL_ERR_INVALID;
    if (!partial_dev && h->shard_world > 1) return CORAL_ERR_INVALID;   // a shard alone cannot normalise a row
    if (reinterpret_cast<uintptr_t>(hidden_dev) & 15) return CORAL_ERR_INVALID;
    const coral_lmhead_config& cfg = h->cfg;
    if (M < 1 || M > cfg.max_M) return CORAL_ERR_INVALID;
    if (k_groups < 1 || k_groups > cfg.max_k_groups) return CORAL_ERR_INVALID;
    if (k_tokens < 1 || k_tokens > cfg.max_k_tokens || (long long)k_tokens > (long long)k_groups * h->L.v)
        return CORAL_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CallView c = make_view(h, hidden_dev, M, k_groups, k_tokens);
    int path = choose_path(h, M, k_groups);
    if (path == 0) return CORAL_ERR_INVALID;   // the forced path does not support this call
    if (h->out_mode != CORAL_OUTPUT_JOINT && path == CORAL_PATH_SIMT_PLAIN) return CORAL_ERR_INVALID;
    if (partial_dev && (path == CORAL_PATH_SIMT_PLAIN || h->out_mode != CORAL_OUTPUT_JOINT)) return CORAL_ERR_INVALID;
    const int merge_mode = partial_dev ? kMergePartial
                           : h->out_mode == CORAL_OUTPUT_FACTORISED ? kMergeFactorised
                           : h->out_mode == CORAL_OUTPUT_FACTORISED_RENORM ? kMergeFactorisedRenorm : kMergeJoint;
    float* merge_out = partial_dev ? partial_dev : out_logprobs_dev;
    // adaptive: both fast paths can take the call and the band-ticket router (which makes the choice) runs it
    const bool adaptive = h->forced_path == CORAL_PATH_ADAPTIVE && !h->w1 && M > kRouteFusedMaxM && M <= kRouteMidMaxM &&
                          M * cfg.n_groups <= kRouteMidMaxCells && cfg.H % 32 == 0 && stream_ok(h, M) &&
                          tc_usable(h, M, k_groups);
    if (adaptive) path = CORAL_PATH_STREAM;      // the launch sequence below starts from the streaming one
    c.pass_rows = path == CORAL_PATH_STREAM ? kStreamPassRows : path == CORAL_PATH_TCGEN05 ? kTcPassRows : 0;
    if (path == CORAL_PATH_TCGEN05) c.union_cap = h->L.tc_vcap;
    c.adaptive = adaptive ? 1 : 0;
    c.pass_rows_tc = kTcPassRows;
    c.union_cap_tc = h->L.tc_vcap;
    int launches = 0;
    unsigned* rt_bands = reinterpret_cast<unsigned*>(h->ws + h->L.route_mid);
    unsigned* rt_masks = rt_bands + h->L.route_bands;
    int* rt_counts = reinterpret_cast<int*>(rt_masks + 4 * (size_t)cfg.n_groups);

    if (h->timing) cudaEventRecord(h->ev_begin, st);
    if (h->w1) {
        if (cfg.H % 32 == 0)
            router_hidden_mma_kernel<<<(cfg.H + 15) / 16, 256, 0, st>>>(c, h->w1, h->router_u);
        else
            router_hidden_kernel<<<dim3((cfg.H + kGateTile - 1) / kGateTile, (M + kGateTile - 1) / kGateTile), 256, 0, st>>>(
                c, h->w1, h->router_u);
        ++launches;
    }
    if (h->w1 && M <= kRouteFusedMaxM) {
        // scores, selection and bucketing in one launch, reading the fp32 router input
        launch_pdl(route_fused_kernel, dim3(c.N), dim3(kRouteThreads), (size_t)0, st, c, forced_groups_dev, out_groups_dev,
                   out_gate_dev);
        ++launches;
    } else if (h->w1) {
        launch_pdl(gate_f32_kernel, dim3(c.N, (M + kGateRows - 1) / kGateRows), dim3(kGateThreads), (size_t)0, st, c,
                   out_gate_dev);
        ++launches;
        select_kernel<<<(M + kSelectWarps - 1) / kSelectWarps, kSelectWarps * 32, 0, st>>>(c, forced_groups_dev,
                                                                                          out_groups_dev);
        ++launches;
        count_groups_kernel<<<(M * k_groups + kSelectWarps * 32 - 1) / (kSelectWarps * 32), kSelectWarps * 32, 0, st>>>(c);
        ++launches;
        bucket_group_kernel<<<c.N, 256, 0, st>>>(c, nullptr);
        ++launches;
    } else if (M <= kRouteFusedMaxM) {
        route_fused_kernel<<<c.N, kRouteThreads, 0, st>>>(c, forced_groups_dev, out_groups_dev, out_gate_dev);
        ++launches;
    } else if (M <= kRouteMidMaxM && M * c.N <= kRouteMidMaxCells && cfg.H % 32 == 0) {
        // few tiles: split H over up to four blocks per tile, so that the GPU is filled and every block's loads
        // are in flight at once
        const int tiles = ((c.N + 15) / 16) * ((M + 7) / 8);
        const int split = tiles >= 128 ? 1 : tiles >= 64 ? 2 : kRouteMidSplitMax;
        route_mid_kernel<<<dim3((c.N + 15) / 16, (M + 7) / 8, split), 256, 0, st>>>(
            c, forced_groups_dev, out_groups_dev, out_gate_dev, rt_bands, rt_masks, rt_counts, 1,
            reinterpret_cast<float*>(h->ws + h->L.route_part));
        ++launches;
    } else if (cfg.H % 32 == 0) {
        // (up to some 300 tiles two blocks per tile still pay: 27 -> 23 us at 256 rows; beyond, the tiles fill the GPU by themselves)
        const int tiles = ((c.N + 15) / 16) * ((M + 7) / 8);
        route_mid_kernel<<<dim3((c.N + 15) / 16, (M + 7) / 8, tiles < 300 ? 2 : 1), 256, 0, st>>>(
            c, forced_groups_dev, out_groups_dev, out_gate_dev, rt_bands, rt_masks, rt_counts, 0,
            reinterpret_cast<float*>(h->ws + h->L.route_part));
        ++launches;
        launch_pdl(bucket_group_kernel, dim3(c.N), dim3(256), (size_t)0, st, c, rt_counts);
        ++launches;
    } else {
        gate_tile_kernel<<<dim3((c.N + kGateTile - 1) / kGateTile, (M + kGateTile - 1) / kGateTile), 256, 0, st>>>(
                c, out_gate_dev);
        ++launches;
        select_kernel<<<(M + kSelectWarps - 1) / kSelectWarps, kSelectWarps * 32, 0, st>>>(c, forced_groups_dev,
                                                                                          out_groups_dev);
        ++launches;
        count_groups_kernel<<<(M * k_groups + kSelectWarps * 32 - 1) / (kSelectWarps * 32), kSelectWarps * 32, 0, st>>>(c);
        ++launches;
        bucket_group_kernel<<<c.N, 256, 0, st>>>(c, nullptr);
        ++launches;
    }
    if (h->timing) cudaEventRecord(h->ev_head0, st);
    if (path == CORAL_PATH_STREAM) {
        const Layout& L = h->L;
        StreamPartials pp{reinterpret_cast<float*>(h->ws + L.sp_max), reinterpret_cast<float*>(h->ws + L.sp_sum),
                          reinterpret_cast<float*>(h->ws + L.sp_val), reinterpret_cast<int32_t*>(h->ws + L.sp_id)};
        StreamPartials tpp{reinterpret_cast<float*>(h->ws + L.tc_max), reinterpret_cast<float*>(h->ws + L.tc_sum),
                           reinterpret_cast<float*>(h->ws + L.tc_val), reinterpret_cast<int32_t*>(h->ws + L.tc_id)};
        StreamGeom mg = h->sg;                   // geometry of the tensor-core partials, as the merge reads them
        mg.tc_tiles = L.tc_tiles;
        mg.tc_rows = kTcPassRows;
        mg.T = L.tc_tiles;
        if (adaptive) {
            // both head kernels are launched; each reads the router's choice first and the one not chosen returns
            TcGeom tg{h->tc_pairs, L.tc_tiles, (L.tc_tiles + 1) / 2, L.KB, L.tc_hg_rows, tc_strided(h, M, k_groups)};
            TcPartials tp{tpp.pmax, tpp.psum, tpp.pval, tpp.pid};
            launch_pdl(tc_gather_kernel, dim3((M * k_groups + kGatherPairs - 1) / kGatherPairs), dim3(64 * kGatherPairs), (size_t)0, st, c,
                       reinterpret_cast<uint16_t*>(h->ws + L.tc_hg), L.tc_hg_rows);
            ++launches;
            launch_pdl_pairs(head_tc_kernel, dim3(2 * tg.pairs), dim3(kTcHeadThreads), kTcSmemBytes, st, c, tg, tp, h->map_w,
                             reinterpret_cast<const uint16_t*>(h->ws + L.tc_hg), out_logits_dev);
            ++launches;
        }
        launch_pdl(h->sg.kc == 512 ? head_stream_kernel<2> : head_stream_kernel<1>, dim3(h->sg.grid),
                   dim3(kStreamThreads), (size_t)h->stream_smem, st, c, h->sg, pp, out_logits_dev);
        ++launches;
        if (h->timing) cudaEventRecord(h->ev_head1, st);
        {
            int p_cap = h->sg.grid + 2 * k_groups;
            int c_cap = p_cap * k_tokens < kMergeSmemCands ? p_cap * k_tokens : kMergeSmemCands;
            if (adaptive) {
                p_cap = p_cap > k_groups * L.tc_tiles ? p_cap : k_groups * L.tc_tiles;
                c_cap = c_cap > k_groups * L.tc_tiles * k_tokens ? c_cap : k_groups * L.tc_tiles * k_tokens;
            }
            launch_pdl(merge_stream_kernel, dim3(M), dim3(kMergeStreamThreads), merge_smem_bytes(p_cap, c_cap), st, c,
                       h->sg, pp, mg, tpp, reinterpret_cast<float*>(h->ws + L.cand_val),
                       reinterpret_cast<int32_t*>(h->ws + L.cand_id), (int)L.cand_cap, c_cap, p_cap, merge_mode,
                       out_ids_dev, merge_out, out_lse_dev);
        }
        ++launches;
    } else if (path == CORAL_PATH_TCGEN05) {
        const Layout& L = h->L;
        TcGeom tg{h->tc_pairs, L.tc_tiles, (L.tc_tiles + 1) / 2, L.KB, L.tc_hg_rows, tc_strided(h, M, k_groups)};
        TcPartials tp{reinterpret_cast<float*>(h->ws + L.tc_max), reinterpret_cast<float*>(h->ws + L.tc_sum),
                      reinterpret_cast<float*>(h->ws + L.tc_val), reinterpret_cast<int32_t*>(h->ws + L.tc_id)};
        launch_pdl(tc_gather_kernel, dim3((M * k_groups + kGatherPairs - 1) / kGatherPairs), dim3(64 * kGatherPairs), (size_t)0, st, c,
                   reinterpret_cast<uint16_t*>(h->ws + L.tc_hg), L.tc_hg_rows);
        ++launches;
        launch_pdl_pairs(head_tc_kernel, dim3(2 * tg.pairs), dim3(kTcHeadThreads), kTcSmemBytes, st, c, tg, tp, h->map_w,
                         reinterpret_cast<const uint16_t*>(h->ws + L.tc_hg), out_logits_dev);
        ++launches;
        if (h->timing) cudaEventRecord(h->ev_head1, st);
        StreamGeom mg = h->sg;
        mg.tc_tiles = L.tc_tiles;
        mg.tc_rows = kTcPassRows;
        mg.T = L.tc_tiles;
        StreamPartials pp{tp.pmax, tp.psum, tp.pval, tp.pid};
        {
            const int p_cap = k_groups * L.tc_tiles;
            const int c_cap = p_cap * k_tokens < kMergeSmemCands ? p_cap * k_tokens : kMergeSmemCands;   // more: global scratch
            launch_pdl(merge_stream_kernel, dim3(M), dim3(kMergeStreamThreads), merge_smem_bytes(p_cap, c_cap), st, c, mg,
                       pp, mg, pp, reinterpret_cast<float*>(h->ws + L.cand_val), reinterpret_cast<int32_t*>(h->ws + L.cand_id),
                       (int)L.cand_cap, c_cap, p_cap, merge_mode, out_ids_dev, merge_out, out_lse_dev);
        }
        ++launches;
    } else {
        head_simt_kernel<<<dim3(c.T, c.N), kSimtThreads, h->simt_smem, st>>>(c, out_logits_dev);
        ++launches;
        if (h->timing) cudaEventRecord(h->ev_head1, st);
        merge_kernel<<<M, kMergeThreads, 0, st>>>(c, out_ids_dev, out_logprobs_dev, out_lse_dev);
        ++launches;
    }
    if (h->timing) cudaEventRecord(h->ev_end, st);
    if (cudaGetLastError() != cudaSuccess) return CORAL_ERR_CUDA;

    h->last_path = adaptive ? CORAL_PATH_ADAPTIVE : path; h->last_M = M; h->last_kg = k_groups; h->last_kt = k_tokens; h->last_launches = launches;
    return CORAL_OK;
}

int coral_lmhead_draft_ex(coral_lmhead_handle h, const void* hidden_dev, int M, int k_groups, int k_tokens,
                          const int32_t* forced_groups_dev, int32_t* out_groups_dev, float* out_gate_dev,
                          float* out_logits_dev, float* out_lse_dev, int32_t* out_ids_dev, float* out_logprobs_dev,
                          void* stream) {
    return draft_impl(h, hidden_dev, M, k_groups, k_tokens, forced_groups_dev, out_groups_dev, out_gate_dev,
                      out_logits_dev, out_lse_dev, out_ids_dev, out_logprobs_dev, nullptr, stream);
}

int coral_lmhead_set_group_shard(coral_lmhead_handle h, int rank, int world) {
    if (!h || world < 1 || rank < 0 || rank >= world || world > h->cfg.n_groups) return CORAL_ERR_INVALID;
    if (cfg_world(h->cfg) > 1 && (rank != cfg_rank(h->cfg) || world != cfg_world(h->cfg)))
        return CORAL_ERR_INVALID;                 // the handle stores one shard only
    h->shard_rank = rank;
    h->shard_world = world;
    return CORAL_OK;
}

int coral_lmhead_draft_partial(coral_lmhead_handle h, const void* hidden_dev, int M, int k_groups, int k_tokens,
                               void* out_records_dev, void* stream) {
    if (!out_records_dev) return CORAL_ERR_INVALID;
    return draft_impl(h, hidden_dev, M, k_groups, k_tokens, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                      nullptr, static_cast<float*>(out_records_dev), stream);
}

int coral_lmhead_merge_partials(const void* records_dev, int world, int M, int k_tokens, int32_t* out_ids_dev,
                                float* out_logprobs_dev, void* stream) {
    if (!records_dev || !out_ids_dev || !out_logprobs_dev) return CORAL_ERR_INVALID;
    if (world < 1 || M < 1 || k_tokens < 1 || k_tokens > CORAL_MAX_K_TOKENS) return CORAL_ERR_INVALID;
    if (world * k_tokens > kMergePartialsThreads) return CORAL_ERR_TOO_LARGE;
    merge_partials_kernel<<<M, kMergePartialsThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const float*>(records_dev), world, M, k_tokens, out_ids_dev, out_logprobs_dev);
    return cudaGetLastError() == cudaSuccess ? CORAL_OK : CORAL_ERR_CUDA;
}

int coral_lmhead_draft(coral_lmhead_handle h, const void* hidden_dev, int M, int k_groups, int k_tokens,
                       int32_t* out_ids_dev, float* out_logprobs_dev, void* stream) {
    return coral_lmhead_draft_ex(h, hidden_dev, M, k_groups, k_tokens, nullptr, nullptr, nullptr, nullptr, nullptr,
                                 out_ids_dev, out_logprobs_dev, stream);
}

// The address through which kernels may write a buffer of pinned (page-locked, mapped) host memory, or null for any
// other kind of memory.  The answer for the buffer seen last is remembered: callers reuse their buffers, and
// the query costs about a microsecond.
static void* pinned_alias(coral_lmhead_handle h, int which, const void* host) {
    if (h->host_seen[which] == host) return h->host_alias[which];
    cudaPointerAttributes attr{};
    void* alias = nullptr;
    if (cudaPointerGetAttributes(&attr, host) == cudaSuccess) {
        if (attr.type == cudaMemoryTypeHost) alias = attr.devicePointer;
    } else {
        cudaGetLastError();              // unregistered memory is not an error of this call
    }
    h->host_seen[which] = host;
    h->host_alias[which] = alias;
    return alias;
}

int coral_lmhead_draft_host(coral_lmhead_handle h, const void* hidden_host, int M, int k_groups, int k_tokens,
                            int32_t* out_ids_host, float* out_logprobs_host, void* stream) {
    if (!h || !hidden_host || !out_ids_host || !out_logprobs_host) return CORAL_ERR_INVALID;
    if (M < 1 || M > h->cfg.max_M || k_tokens < 1 || k_tokens > h->cfg.max_k_tokens) return CORAL_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* ws = h->ws;
    void* d_hidden = ws + h->L.stage_hidden;
    // Pinned output buffers are written by the merge itself (a few hundred bytes over the host link); the two
    // copies back, and what it costs to queue them behind the kernels, fall away.  Other memory is staged.
    int32_t* ids_alias = static_cast<int32_t*>(pinned_alias(h, 0, out_ids_host));
    float* lp_alias = static_cast<float*>(pinned_alias(h, 1, out_logprobs_host));
    int32_t* d_ids = ids_alias ? ids_alias : reinterpret_cast<int32_t*>(ws + h->L.stage_ids);
    float* d_lp = lp_alias ? lp_alias : reinterpret_cast<float*>(ws + h->L.stage_logprobs);
    if (cudaMemcpyAsync(d_hidden, hidden_host, (size_t)M * h->cfg.H * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return CORAL_ERR_CUDA;
    const int rc = coral_lmhead_draft(h, d_hidden, M, k_groups, k_tokens, d_ids, d_lp, stream);
    if (rc != CORAL_OK) return rc;
    if (!ids_alias &&
        cudaMemcpyAsync(out_ids_host, d_ids, (size_t)M * k_tokens * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return CORAL_ERR_CUDA;
    if (!lp_alias &&
        cudaMemcpyAsync(out_logprobs_host, d_lp, (size_t)M * k_tokens * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return CORAL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return CORAL_ERR_CUDA;
    return CORAL_OK;
}

int coral_tree_expand(const float* parent_scores_dev, const int32_t* cand_ids_dev, const float* cand_logprobs_dev,
                      int n_seq, int nodes, int k_tokens, int K, int32_t* out_parent_dev, int32_t* out_token_dev,
                      float* out_score_dev, void* stream) {
    if (!parent_scores_dev || !out_parent_dev || !out_token_dev || !out_score_dev) return CORAL_ERR_INVALID;
    if (n_seq < 1 || nodes < 1 || k_tokens < 1) return CORAL_ERR_INVALID;
    if ((long long)nodes * k_tokens > kTreeMaxCand) return CORAL_ERR_TOO_LARGE;
    if (K < 1 || K > kTreeMaxK || K > nodes * k_tokens) return CORAL_ERR_INVALID;
    if (!cand_logprobs_dev && k_tokens != 1) return CORAL_ERR_INVALID;
    tree_expand_kernel<<<n_seq, kTreeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        parent_scores_dev, cand_ids_dev, cand_logprobs_dev, nodes, k_tokens, K, out_parent_dev, out_token_dev,
        out_score_dev);
    return cudaGetLastError() == cudaSuccess ? CORAL_OK : CORAL_ERR_CUDA;
}

// The L2 set-aside is a limit of the process's CUDA context, shared with every other handle and with whatever
// else the process runs.  The handle only ever raises it, remembers what it found, and puts that back when its
// hot groups are switched off or the handle is destroyed.
static int release_hot_groups(coral_lmhead_handle h) {
    if (h->hot_groups == 0) return CORAL_OK;
    h->hot_groups = 0;
    if (!h->l2_limit_changed) return CORAL_OK;
    h->l2_limit_changed = false;
    if (cudaCtxResetPersistingL2Cache() != cudaSuccess) return CORAL_ERR_CUDA;
    return cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, h->l2_limit_before) == cudaSuccess ? CORAL_OK : CORAL_ERR_CUDA;
}

int coral_lmhead_set_hot_groups(coral_lmhead_handle h, int n_hot) {
    if (!h || n_hot < 0 || n_hot > h->cfg.n_groups) return CORAL_ERR_INVALID;
    if (n_hot == 0) return release_hot_groups(h);
    // evict-last lines only outlive other traffic inside the part of L2 that is set aside for them
    int dev = 0, max_persist = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, dev) != cudaSuccess)
        return CORAL_ERR_CUDA;
    if (max_persist <= 0) return CORAL_ERR_INVALID;                     // the device has no such set-aside
    const size_t want = (size_t)n_hot * h->L.T16 * h->L.KB * 2048;      // packed bytes of the hot groups
    const size_t carve = want < (size_t)max_persist ? want : (size_t)max_persist;
    size_t now = 0;
    if (cudaDeviceGetLimit(&now, cudaLimitPersistingL2CacheSize) != cudaSuccess) return CORAL_ERR_CUDA;
    if (carve > now) {                                                  // never shrink what somebody else set
        if (!h->l2_limit_changed) h->l2_limit_before = now;
        if (cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, carve) != cudaSuccess) return CORAL_ERR_CUDA;
        h->l2_limit_changed = true;
    }
    h->hot_groups = n_hot;
    return CORAL_OK;
}

int coral_lmhead_copy_floor(coral_lmhead_handle h, long long bytes, int in_flight, int repeats, void* stream) {
    if (!h || bytes < kCopyChunk || (size_t)bytes > h->L.packed_bytes) return CORAL_ERR_INVALID;
    if (in_flight == 0) in_flight = kCopyStages;
    if (in_flight < 1 || in_flight > kCopyMaxStages || repeats < 1 || repeats > 64) return CORAL_ERR_INVALID;
    if (cudaFuncSetAttribute(copy_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kCopyMaxStages * kCopyChunk) != cudaSuccess) return CORAL_ERR_CUDA;
    copy_probe_kernel<<<h->sms, 32, in_flight * kCopyChunk, static_cast<cudaStream_t>(stream)>>>(
        h->packed, bytes / kCopyChunk, in_flight, repeats, reinterpret_cast<DeviceState*>(h->ws + h->L.state),
        reinterpret_cast<unsigned*>(h->ws + h->L.cand_val));
    return cudaGetLastError() == cudaSuccess ? CORAL_OK : CORAL_ERR_CUDA;
}

int coral_lmhead_tc_issue_probe(coral_lmhead_handle h, int n, int per_commit, int issuers, int rounds,
                                unsigned long long* out_ns_dev, void* stream) {
    if (!h || !out_ns_dev || !h->tc_ok) return CORAL_ERR_INVALID;
    if (n < 16 || n > 256 || n % 16 || per_commit < 1 || per_commit > 16 || issuers < 1 || issuers > 2 || rounds < 1 ||
        rounds > (1 << 16))
        return CORAL_ERR_INVALID;
    const size_t smem = 1024 + kTcProbeOperandBytes + 256;
    if (cudaFuncSetAttribute(tc_issue_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return CORAL_ERR_CUDA;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * h->tc_pairs);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tc_issue_probe_kernel, n, per_commit, rounds, issuers, out_ns_dev,
                              reinterpret_cast<DeviceState*>(h->ws + h->L.state)) == cudaSuccess ? CORAL_OK : CORAL_ERR_CUDA;
}

// ---- CSRA objective (Eq. 2) -------------------------------------------------------------------------------
namespace {
struct CsraLayout {
    size_t state, qn, kn, pmax, psum, pos, row_loss, total;
    int RB, KT, KB;
};
CsraLayout csra_layout(int n, int views, int D) {
    CsraLayout L{};
    L.RB = (n + 127) / 128;
    L.KT = (int)(((long long)n * views + 127) / 128);
    L.KB = (D + 63) / 64;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
    L.state = take(sizeof(DeviceState));
    L.qn = take((size_t)L.RB * L.KB * 128 * 64 * 2);
    L.kn = take((size_t)L.KT * L.KB * 128 * 64 * 2);
    L.pmax = take((size_t)L.RB * L.KT * 128 * 4);
    L.psum = take((size_t)L.RB * L.KT * 128 * 4);
    L.pos = take((size_t)n * views * 4);
    L.row_loss = take((size_t)n * 4);
    L.total = o;
    return L;
}
bool csra_args_ok(int n, int views, int D) {
    return n >= 1 && views >= 1 && views <= kCsraMaxViews && D >= 8 && D % 8 == 0 && (long long)n * views <= (1 << 24) &&
           D <= (1 << 16);
}
}  // namespace

int coral_csra_workspace_bytes(int n, int views, int D, size_t* bytes) {
    if (!bytes || !csra_args_ok(n, views, D)) return CORAL_ERR_INVALID;
    *bytes = csra_layout(n, views, D).total;
    return CORAL_OK;
}

int coral_csra_infonce(const void* Q_dev, const void* K_dev, int n, int views, int D, float tau, void* workspace_dev,
                       float* out_row_loss_dev, float* out_loss_dev, float* out_logits_dev, void* stream) {
    if (!Q_dev || !K_dev || !workspace_dev || !out_loss_dev || !csra_args_ok(n, views, D) || !(tau > 0.f))
        return CORAL_ERR_INVALID;
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 255) return CORAL_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const CsraLayout L = csra_layout(n, views, D);
    unsigned char* ws = static_cast<unsigned char*>(workspace_dev);
    int dev = 0, sms = 0, smem_optin = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
        return CORAL_ERR_CUDA;
    if ((int)kCsraSmemBytes > smem_optin) return CORAL_ERR_INVALID;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return CORAL_ERR_CUDA;
    CUtensorMap map_q, map_k;
    {
        const cuuint64_t qdim[2] = {(cuuint64_t)kTcK, (cuuint64_t)L.RB * L.KB * 128};
        const cuuint64_t kdim[2] = {(cuuint64_t)kTcK, (cuuint64_t)L.KT * L.KB * 128};
        const cuuint64_t str[1] = {(cuuint64_t)kTcK * 2};
        const cuuint32_t box[2] = {(cuuint32_t)kTcK, 128};
        const cuuint32_t ones[2] = {1, 1};
        if (enc(&map_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ws + L.qn, qdim, str, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) !=
                CUDA_SUCCESS ||
            enc(&map_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ws + L.kn, kdim, str, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) !=
                CUDA_SUCCESS)
            return CORAL_ERR_CUDA;
    }
    if (cudaFuncSetAttribute(csra_sim_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCsraSmemBytes) != cudaSuccess)
        return CORAL_ERR_CUDA;
    if (cudaMemsetAsync(ws + L.state, 0, sizeof(DeviceState), st) != cudaSuccess) return CORAL_ERR_CUDA;
    CsraGeom g{};
    g.n = n; g.views = views; g.m = n * views; g.D = D;
    g.RB = L.RB; g.KT = L.KT; g.ksteps = L.KB; g.grid = sms; g.inv_tau = 1.0f / tau;
    uint16_t* qn = reinterpret_cast<uint16_t*>(ws + L.qn);
    uint16_t* kn = reinterpret_cast<uint16_t*>(ws + L.kn);
    float* row_loss = out_row_loss_dev ? out_row_loss_dev : reinterpret_cast<float*>(ws + L.row_loss);
    csra_normalise_kernel<<<L.RB * 128, 128, 0, st>>>(static_cast<const uint16_t*>(Q_dev), n, D, L.KB, qn);
    csra_normalise_kernel<<<L.KT * 128, 128, 0, st>>>(static_cast<const uint16_t*>(K_dev), g.m, D, L.KB, kn);
    csra_sim_kernel<<<g.grid, kTcThreads, kCsraSmemBytes, st>>>(
        g, map_q, map_k, reinterpret_cast<float*>(ws + L.pmax), reinterpret_cast<float*>(ws + L.psum),
        reinterpret_cast<float*>(ws + L.pos), out_logits_dev, reinterpret_cast<DeviceState*>(ws + L.state));
    csra_finalize_kernel<<<(n + 255) / 256, 256, 0, st>>>(g, reinterpret_cast<const float*>(ws + L.pmax),
                                                          reinterpret_cast<const float*>(ws + L.psum),
                                                          reinterpret_cast<const float*>(ws + L.pos), row_loss);
    csra_mean_kernel<<<1, 1024, 0, st>>>(row_loss, n, out_loss_dev);
    return cudaGetLastError() == cudaSuccess ? CORAL_OK : CORAL_ERR_CUDA;
}

int coral_csra_status(void* workspace_dev, void* stream) {
    if (!workspace_dev) return CORAL_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceState s{};
    if (cudaMemcpyAsync(&s, workspace_dev, sizeof s, cudaMemcpyDeviceToHost, st) != cudaSuccess) return CORAL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return CORAL_ERR_CUDA;
    return s.status;
}

int coral_lmhead_selftest_wait_expiry(coral_lmhead_handle h, void* stream) {
    if (!h) return CORAL_ERR_INVALID;
    wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(reinterpret_cast<DeviceState*>(h->ws + h->L.state));
    return cudaGetLastError() == cudaSuccess ? CORAL_OK : CORAL_ERR_CUDA;
}

int coral_lmhead_set_output_mode(coral_lmhead_handle h, int mode) {
    if (!h || mode < CORAL_OUTPUT_JOINT || mode > CORAL_OUTPUT_FACTORISED_RENORM) return CORAL_ERR_INVALID;
    h->out_mode = mode;
    return CORAL_OK;
}

int coral_lmhead_set_router_mlp(coral_lmhead_handle h, const void* W1_dev, void* stream) {
    if (!h) return CORAL_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!W1_dev) {                       // back to the single-matrix gate
        if (cudaStreamSynchronize(st) != cudaSuccess) return CORAL_ERR_CUDA;
        if (h->w1) cudaFree(h->w1);
        if (h->router_u) cudaFree(h->router_u);
        h->w1 = nullptr;
        h->router_u = nullptr;
        return CORAL_OK;
    }
    if (reinterpret_cast<uintptr_t>(W1_dev) & 15) return CORAL_ERR_INVALID;
    const size_t H = h->cfg.H;
    if (!h->w1 && cudaMalloc(&h->w1, H * H * 2) != cudaSuccess) { h->w1 = nullptr; return CORAL_ERR_NOMEM; }
    if (!h->router_u && cudaMalloc(&h->router_u, (size_t)h->cfg.max_M * H * 4) != cudaSuccess) {
        h->router_u = nullptr;
        return CORAL_ERR_NOMEM;
    }
    if (cudaMemcpyAsync(h->w1, W1_dev, H * H * 2, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return CORAL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return CORAL_ERR_CUDA;
    return CORAL_OK;
}

int coral_lmhead_set_kernel_timing(coral_lmhead_handle h, int on) {
    if (!h) return CORAL_ERR_INVALID;
    if (on && !h->ev_head0) {
        if (cudaEventCreate(&h->ev_head0) != cudaSuccess || cudaEventCreate(&h->ev_head1) != cudaSuccess ||
            cudaEventCreate(&h->ev_begin) != cudaSuccess || cudaEventCreate(&h->ev_end) != cudaSuccess)
            return CORAL_ERR_CUDA;
    }
    h->timing = on != 0;
    return CORAL_OK;
}

int coral_lmhead_head_kernel_ms(coral_lmhead_handle h, float* ms) {
    if (!h || !ms || !h->ev_head0) return CORAL_ERR_INVALID;
    if (cudaEventSynchronize(h->ev_head1) != cudaSuccess) return CORAL_ERR_CUDA;
    if (cudaEventElapsedTime(ms, h->ev_head0, h->ev_head1) != cudaSuccess) return CORAL_ERR_CUDA;
    return CORAL_OK;
}

int coral_lmhead_stage_ms(coral_lmhead_handle h, float* route_ms, float* head_ms, float* merge_ms) {
    if (!h || !route_ms || !head_ms || !merge_ms || !h->ev_head0) return CORAL_ERR_INVALID;
    if (cudaEventSynchronize(h->ev_end) != cudaSuccess) return CORAL_ERR_CUDA;
    if (cudaEventElapsedTime(route_ms, h->ev_begin, h->ev_head0) != cudaSuccess ||
        cudaEventElapsedTime(head_ms, h->ev_head0, h->ev_head1) != cudaSuccess ||
        cudaEventElapsedTime(merge_ms, h->ev_head1, h->ev_end) != cudaSuccess)
        return CORAL_ERR_CUDA;
    return CORAL_OK;
}

int coral_lmhead_status(coral_lmhead_handle h, void* stream) {
    if (!h) return CORAL_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceState s{};
    DeviceState* d = reinterpret_cast<DeviceState*>(h->ws + h->L.state);
    if (cudaMemcpyAsync(&s, d, sizeof s, cudaMemcpyDeviceToHost, st) != cudaSuccess) return CORAL_ERR_CUDA;
    if (cudaMemsetAsync(&d->status, 0, sizeof(int), st) != cudaSuccess) return CORAL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return CORAL_ERR_CUDA;
    return s.status;
}

int coral_lmhead_last_stats(coral_lmhead_handle h, coral_lmhead_stats* out, void* stream) {
    if (!h || !out) return CORAL_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceState s{};
    if (cudaMemcpyAsync(&s, h->ws + h->L.state, sizeof s, cudaMemcpyDeviceToHost, st) != cudaSuccess) return CORAL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return CORAL_ERR_CUDA;
    out->path = h->last_path == CORAL_PATH_ADAPTIVE ? (s.path_choice == 2 ? CORAL_PATH_TCGEN05 : CORAL_PATH_STREAM)
                                                    : h->last_path;
    out->M = h->last_M;
    out->k_groups = h->last_kg;
    out->k_tokens = h->last_kt;
    out->groups_touched = s.n_union;
    out->kernel_launches = h->last_launches;
    out->weight_bytes = (int64_t)s.n_union * h->L.v * h->cfg.H * 2;
    out->algorithmic_bytes = out->weight_bytes + (int64_t)h->cfg.n_groups * h->cfg.H * 2 +
                             (int64_t)h->last_M * h->cfg.H * 2 + (int64_t)h->last_M * h->last_kt * 8;
    return CORAL_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Router step without any allocation (see coral_lmhead_route_static in the header).
// The gate scores, the per-row slot table and the status word that the router kernels use as
// scratch live in this file-scope device array instead of a caller- or library-allocated
// workspace.  Every GPU that loads the library holds one copy of it until the process exits.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxRows = CORAL_ROUTE_STATIC_MAX_ROWS;
constexpr size_t kStaticGateOff = 0;                                                       // float [rows][N]
constexpr size_t kStaticSelOff = kStaticGateOff + (size_t)kStaticMaxRows * kMaxGroups * 4;  // int32 [rows][k]
constexpr size_t kStaticSlotOff = kStaticSelOff + (size_t)kStaticMaxRows * kMaxGroups * 4;  // int16 [rows][N]
constexpr size_t kStaticStateOff = kStaticSlotOff + (size_t)kStaticMaxRows * kMaxGroups * 2;
constexpr size_t kStaticBytes = kStaticStateOff + 256;

static __device__ __align__(256) unsigned char g_route_scratch[kStaticBytes];

// In host code `g_route_scratch` is only a handle for the runtime, not a device address.  The
// address is looked up once per device, with that device current, and cached here.
constexpr int kMaxDevices = 64;
unsigned char* g_route_scratch_addr[kMaxDevices] = {};

int route_scratch_for_current_device(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return CORAL_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return CORAL_ERR_INVALID;
    unsigned char* p = __atomic_load_n(&g_route_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_route_scratch) != cudaSuccess || !p)
            return CORAL_ERR_CUDA;
        __atomic_store_n(&g_route_scratch_addr[dev], p, __ATOMIC_RELEASE);   // same value from any thread
    }
    *out = p;
    return CORAL_OK;
}

}  // namespace

extern "C" int coral_lmhead_route_static(const void* W_gate_dev, const void* hidden_dev, int M, int H, int n_groups,
                                         int k_groups, int32_t* out_groups_dev, float* out_gate_dev, void* stream) {
    if (!W_gate_dev || !hidden_dev || !out_groups_dev) return CORAL_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(W_gate_dev) & 15) || (reinterpret_cast<uintptr_t>(hidden_dev) & 15))
        return CORAL_ERR_INVALID;
    if (H < 8 || H % 8 != 0 || n_groups < 1 || n_groups > CORAL_MAX_GROUPS) return CORAL_ERR_INVALID;
    if (k_groups < 1 || k_groups > n_groups) return CORAL_ERR_INVALID;
    if (M < 1) return CORAL_ERR_INVALID;
    if (M > kStaticMaxRows) return CORAL_ERR_TOO_LARGE;   // the built-in scratch holds at most that many rows
    unsigned char* scratch = nullptr;
    const int rc = route_scratch_for_current_device(&scratch);
    if (rc != CORAL_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    CallView c{};
    c.M = M; c.H = H; c.N = n_groups; c.k_groups = k_groups;
    c.w_gate = static_cast<const uint16_t*>(W_gate_dev);
    c.hidden = static_cast<const uint16_t*>(hidden_dev);
    c.gate = reinterpret_cast<float*>(scratch + kStaticGateOff);
    c.sel = reinterpret_cast<int32_t*>(scratch + kStaticSelOff);
    c.slot_of = reinterpret_cast<int16_t*>(scratch + kStaticSlotOff);
    c.state = reinterpret_cast<DeviceState*>(scratch + kStaticStateOff);
    // The array keeps the previous call's contents.  The status word must start at zero; the gate,
    // selection and slot tables are fully rewritten for rows < M before anything reads them.
    if (cudaMemsetAsync(c.state, 0, sizeof(DeviceState), st) != cudaSuccess) return CORAL_ERR_CUDA;
    gate_kernel<<<dim3(c.N, (M + kGateRows - 1) / kGateRows), kGateThreads, 0, st>>>(c, out_gate_dev);
    select_kernel<<<(M + kSelectWarps - 1) / kSelectWarps, kSelectWarps * 32, 0, st>>>(c, nullptr, out_groups_dev);
    if (cudaGetLastError() != cudaSuccess) return CORAL_ERR_CUDA;
    return CORAL_OK;
}
