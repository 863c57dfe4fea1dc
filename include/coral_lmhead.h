/*
 * coral_lmhead.h - C ABI of the weight-grouped LM-head draft step (sm_100a).
 *
 * The operation is the "LM Head Router" of the CORAL paper (Section 3.3): the
 * draft model's LM head W_vocab [V x H] is divided equally into N groups of
 * v = V/N tokens; per query row a router scores the groups, only the top-n
 * groups are activated, logits are computed for the tokens of the activated
 * groups only, a softmax is taken over them, and the best k_tokens candidates
 * (Appendix B, "Tree decoding": top 10 candidates per node) are returned.
 *
 * Conventions
 *  - Every function returns an int status: CORAL_OK (0) or a negative
 *    CORAL_ERR_* code.  Nothing throws, aborts or prints.
 *  - "dev" pointers are CUDA device pointers of the current device, "host"
 *    pointers are ordinary host memory.  bf16 tensors are raw 16-bit patterns.
 *  - All matrices are row-major and densely packed.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *  - One draft call may be in flight per handle (the workspace is per handle);
 *    different handles are independent.
 */
#ifndef CORAL_LMHEAD_H_
#define CORAL_LMHEAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CORAL_LMHEAD_ABI_VERSION 1

#define CORAL_OK 0
#define CORAL_ERR_INVALID (-1)     /* bad argument (NULL, out of range, unsupported shape) */
#define CORAL_ERR_GROUPING (-2)    /* group_map does not split V into N equal groups */
#define CORAL_ERR_CUDA (-3)        /* a CUDA runtime call failed */
#define CORAL_ERR_NOMEM (-4)       /* host or device allocation failed */
#define CORAL_ERR_TIMEOUT (-5)     /* a bounded device-side wait gave up (device status word) */
#define CORAL_ERR_BOUNDS (-6)      /* a device-side index check failed (device status word) */
#define CORAL_ERR_TOO_LARGE (-7)   /* request exceeds a built-in size limit (coral_lmhead_route_static, coral_tree_expand) */
#define CORAL_ERR_NONFINITE (-8)   /* a router score was NaN (device status word) */

/* Limits of this build. */
#define CORAL_MAX_GROUPS 256       /* n_groups <= 256 */
#define CORAL_MAX_K_TOKENS 32      /* k_tokens <= 32 */
#define CORAL_ROUTE_STATIC_MAX_ROWS 64 /* M <= 64 for coral_lmhead_route_static */

/* config flags: a handle that stores (and computes) only the groups n with n % world == rank */
#define CORAL_CFG_SHARD(rank, world) ((uint32_t)(((world) & 0xff) | (((rank) & 0xff) << 8)))

/* Execution paths (coral_lmhead_set_path / coral_lmhead_stats.path). */
#define CORAL_PATH_AUTO 0          /* TCGEN05 for more than 96 rows or 10 rows per group and more on average, else STREAM, else SIMT_PLAIN */
#define CORAL_PATH_STREAM 1        /* bulk-copy weight streaming + warp MMA (fp32 accumulate); M <= 128, H % 256 == 0, H <= 4096 */
#define CORAL_PATH_TCGEN05 2       /* routed grouped GEMM by CTA pairs on tcgen05 / TMEM tiles; handle created with max_M > 32 */
#define CORAL_PATH_SIMT_PLAIN 3    /* gathered GEMV with plain 128-bit loads, any M */
#define CORAL_PATH_ADAPTIVE 4      /* 33..128 rows: the router picks STREAM or TCGEN05 on the device from the rows per group */

/* Output modes (coral_lmhead_set_output_mode). */
#define CORAL_OUTPUT_JOINT 0       /* log-softmax over all active logits of the row (default) */
#define CORAL_OUTPUT_FACTORISED 1  /* Eq. 8: log p_router(n) + log p_group(x), p_router = Softmax over all N groups */
#define CORAL_OUTPUT_FACTORISED_RENORM 2 /* Eq. 8 with p_router renormalised over the row's selected groups */

typedef struct coral_lmhead_s *coral_lmhead_handle;

typedef struct coral_lmhead_config {
    uint32_t struct_size;   /* sizeof(coral_lmhead_config), for versioning */
    int32_t H;              /* hidden size d; multiple of 8 (128-bit loads) */
    int32_t V;              /* vocabulary size; multiple of n_groups */
    int32_t n_groups;       /* N, 1..CORAL_MAX_GROUPS */
    int32_t max_M;          /* largest number of query rows per draft call */
    int32_t max_k_groups;   /* largest top-n, 1..n_groups */
    int32_t max_k_tokens;   /* largest number of candidates, 1..CORAL_MAX_K_TOKENS */
    uint32_t flags;         /* 0, or CORAL_CFG_SHARD(rank, world): store only this rank's groups (see vocab sharding) */
} coral_lmhead_config;

typedef struct coral_lmhead_stats {
    int32_t path;            /* CORAL_PATH_* taken by the last draft call */
    int32_t M, k_groups, k_tokens;
    int32_t groups_touched;  /* |U|: size of the union of selected groups over the rows */
    int32_t kernel_launches; /* kernels the last draft call enqueued */
    int64_t weight_bytes;    /* |U| * v * H * 2: LM-head bytes the step has to read */
    int64_t algorithmic_bytes; /* weight_bytes + gate N*H*2 + hidden M*H*2 + outputs M*k_tokens*8 */
} coral_lmhead_stats;

/* ABI version of the loaded library (CORAL_LMHEAD_ABI_VERSION). */
int coral_lmhead_version(void);

/*
 * Sizes of the two device buffers a handle needs, so that the caller can
 * allocate them (Section 3.3: N groups of v = V/N tokens fixes the packed
 * copy's size; the workspace holds the gate, tables and per-call partials).
 * CORAL_ERR_INVALID if cfg is NULL/inconsistent: V % n_groups != 0,
 * H % 8 != 0, a field < 1, or a limit above is exceeded.
 */
int coral_lmhead_query_sizes(const coral_lmhead_config *cfg, size_t *packed_bytes, size_t *workspace_bytes);

/*
 * Build a handle (Section 3.3: "divide the LM head equally into N groups").
 *   W_vocab_dev    [V x H] bf16, device.  Frozen LM head of the draft model.
 *   group_map_host [V] int32, host.  token -> group in [0, N); every group
 *                  must hold exactly V/N tokens, else CORAL_ERR_GROUPING.
 *   W_gate_dev     [N x H] bf16, device.  Router matrix (the W2 of Eq. 7).
 *   packed_buf_dev / workspace_dev: device buffers of at least the sizes
 *                  coral_lmhead_query_sizes reports, 256-byte aligned, owned by
 *                  the caller and alive until destroy.  Either may be NULL:
 *                  the library then allocates (cudaMalloc) and owns that one.
 * The weights are copied group-contiguously (tokens of a group in ascending
 * token id) into packed_buf; W_gate and the tables go to the workspace.  The
 * call synchronises `stream` before returning, so the inputs may be freed.
 */
int coral_lmhead_create(coral_lmhead_handle *out, const coral_lmhead_config *cfg, const void *W_vocab_dev,
                        const int32_t *group_map_host, const void *W_gate_dev, void *packed_buf_dev,
                        void *workspace_dev, void *stream);

/*
 * One draft step for M query rows (Section 3.3 and Appendix B, tree decoding):
 *   gate scores g = W_gate h per row; the k_groups best groups per row
 *   (descending score, equal scores -> lower group index); logits of the
 *   tokens of those groups (bf16 inputs, fp32 accumulation); log-softmax over
 *   the row's active logits; the k_tokens best tokens per row (descending,
 *   equal -> lower token id).
 *   hidden_dev       [M x H] bf16, device
 *   out_ids_dev      [M x k_tokens] int32, device: global token ids
 *   out_logprobs_dev [M x k_tokens] float, device: natural-log probabilities
 * Asynchronous on `stream`: no allocation, no host synchronisation.
 * CORAL_ERR_INVALID (nothing enqueued) for NULL pointers, M < 1 or > max_M,
 * k_groups outside [1, min(N, max_k_groups)], k_tokens outside
 * [1, min(max_k_tokens, k_groups * v)].  Device-side problems are reported by
 * coral_lmhead_status.
 */
int coral_lmhead_draft(coral_lmhead_handle h, const void *hidden_dev, int M, int k_groups, int k_tokens,
                       int32_t *out_ids_dev, float *out_logprobs_dev, void *stream);

/*
 * Same step with optional taps for checking each stage (all device, any may
 * be NULL):
 *   forced_groups_dev [M x k_groups] int32: use these groups (distinct, in
 *                     [0, N)) instead of the router's choice
 *   out_groups_dev    [M x k_groups] int32: selected groups in selection order
 *   out_gate_dev      [M x N] float: router scores
 *   out_logits_dev    [M x k_groups x v] float: slot s of row m holds the
 *                     logits of the tokens of group out_groups[m][s] in
 *                     ascending token id
 *   out_lse_dev       [M] float: log-sum-exp over the row's active logits
 */
int coral_lmhead_draft_ex(coral_lmhead_handle h, const void *hidden_dev, int M, int k_groups, int k_tokens,
                          const int32_t *forced_groups_dev, int32_t *out_groups_dev, float *out_gate_dev,
                          float *out_logits_dev, float *out_lse_dev, int32_t *out_ids_dev,
                          float *out_logprobs_dev, void *stream);

/*
 * The same draft step for callers that hold HOST buffers (hidden_host
 * [M x H] bf16; out_ids_host / out_logprobs_host [M x k_tokens]).  Copies the
 * rows to the device, runs coral_lmhead_draft, copies the results back and
 * synchronises `stream` before returning.  Pinned host memory makes the copy
 * in asynchronous up to that final synchronisation, and pinned output buffers
 * are written by the last kernel directly (no copies back); pageable buffers
 * work too, staged through the workspace.
 */
int coral_lmhead_draft_host(coral_lmhead_handle h, const void *hidden_host, int M, int k_groups, int k_tokens,
                            int32_t *out_ids_host, float *out_logprobs_host, void *stream);

/*
 * Vocab sharding over several GPUs (one exchange step).  Appendix B's union of groups is what a call must
 * read; with `world` GPUs, GPU `rank` reads only the groups n with n % world == rank (Section 3.3's N equal
 * groups dealt round-robin), so the weight bytes per GPU fall about `world`-fold.  Every GPU runs the router
 * on all N scores (the gate matrix is small), computes logits for its own groups among each row's top-n,
 * and coral_lmhead_draft_partial writes one record per row; the records of all GPUs are gathered (one
 * all-gather of M x (2 + 2 k_tokens) words per GPU, the caller's collective) and
 * coral_lmhead_merge_partials turns them into the same output coral_lmhead_draft gives on one GPU.
 *
 * coral_lmhead_set_group_shard: rank in [0, world), world in [1, n_groups]; world = 1 (the default) switches
 * sharding off.  While world > 1 the handle accepts only coral_lmhead_draft_partial (a shard alone cannot
 * normalise a row): the other draft calls return CORAL_ERR_INVALID.  A handle created with flags = 0 holds the
 * full packed head and can take any shard (set_group_shard reduces what is read per call, not what is stored);
 * a handle created with cfg.flags = CORAL_CFG_SHARD(rank, world) packs only its own groups (packed_bytes is
 * about 1/world of the full size; W_vocab_dev is still the full matrix, read once at create), starts with that
 * shard set and accepts no other.
 *
 * coral_lmhead_draft_partial: arguments as coral_lmhead_draft; out_records_dev is [M][2 + 2 k_tokens] 32-bit
 * words, per row: max of this GPU's active logits (float; -inf if none of the row's groups is local), sum of
 * exp(logit - max) (float), the k_tokens largest logits in descending order (float; -inf where absent), their
 * global token ids (int32; 0x7fffffff where absent).  Joint output mode only; not on the plain fallback path
 * (CORAL_ERR_INVALID).  Asynchronous on `stream`, no allocation.
 *
 * coral_lmhead_merge_partials: records_dev is [world][M][2 + 2 k_tokens] words (rank-major, as an all-gather
 * leaves them); writes out_ids_dev / out_logprobs_dev [M x k_tokens] exactly as coral_lmhead_draft defines
 * them (log-softmax over the union of all ranks' active logits, descending, equal -> lower token id).  Needs
 * no handle.  world * k_tokens <= 256, else CORAL_ERR_TOO_LARGE.
 */
int coral_lmhead_set_group_shard(coral_lmhead_handle h, int rank, int world);
int coral_lmhead_draft_partial(coral_lmhead_handle h, const void *hidden_dev, int M, int k_groups, int k_tokens,
                               void *out_records_dev, void *stream);
int coral_lmhead_merge_partials(const void *records_dev, int world, int M, int k_tokens, int32_t *out_ids_dev,
                                float *out_logprobs_dev, void *stream);

/*
 * Output mode of later draft calls.  CORAL_OUTPUT_FACTORISED emits the paper's final distribution (Section
 * 3.3, Eq. 8): p(x) = p_router(n) * p_group(x^n), where p_router is the softmax of the row's N router scores
 * (Eq. 7) and p_group the softmax inside group n, independent of the other groups; candidates are ranked by
 * that log-probability (equal -> lower token id).  The emitted log-probabilities of a row sum, over its active
 * vocabulary, to the router mass of its selected groups.  out_lse_dev keeps reporting the joint log-sum-exp.
 * CORAL_OUTPUT_FACTORISED_RENORM divides p_router by the router mass of the row's selected groups (the paper
 * does not say whether it does), so that the active vocabulary carries probability 1; the ranking is the same,
 * every log-probability of a row moves by one constant.
 * Neither is available on CORAL_PATH_SIMT_PLAIN (the draft call then returns CORAL_ERR_INVALID).
 */
int coral_lmhead_set_output_mode(coral_lmhead_handle h, int mode);

/*
 * Two-layer router of the paper's Eq. 7: scores = W2 (act(W1 h) + h), with W2 the W_gate given at create, W1
 * [H x H] bf16 (device, 16-byte aligned; copied into library-owned memory, the call synchronises `stream`) and
 * act = SiLU (the paper does not name the activation).  act(W1 h) + h is kept in fp32.  W1_dev = NULL returns
 * to the single-matrix gate.  Allocates (cudaMalloc) H*H*2 + max_M*H*4 bytes on first use.
 */
int coral_lmhead_set_router_mlp(coral_lmhead_handle h, const void *W1_dev, void *stream);

/*
 * Force an execution path (CORAL_PATH_*) for later draft calls; AUTO restores the default choice.
 * A draft call that the forced path cannot run (e.g. CORAL_PATH_STREAM with M > 128) returns
 * CORAL_ERR_INVALID.
 * CORAL_PATH_ADAPTIVE: Appendix B notes that the rows of a tree seldom spread over all groups; rows then pile
 * up on a few groups, and the streaming kernel, which reads a group once per 16 rows, reads those several
 * times.  For calls of 33..128 rows (on a handle created with max_M > 32, H a multiple of 256) the router
 * then compares, on the device, the reads the two kernels would need and records its choice; both kernels
 * are launched and the one not chosen returns at once (about 4 us per call).  Other calls behave as with
 * AUTO.  coral_lmhead_last_stats reports the kernel that ran.
 */
int coral_lmhead_set_path(coral_lmhead_handle h, int path);

/*
 * Cross-Step Representation Alignment objective (Section 3.1, Eq. 2; temperature 0.07 in Appendix A; the same
 * quantity between the features of two training steps in the appendix on step discrepancies), forward only:
 *   loss_i = LSE_j( sim(q_i, k_j) / tau ) - mean_s sim(q_i, k_{i + s n}) / tau,   loss = mean_i loss_i,
 * sim = cosine similarity.  Q_dev [n x D] bf16 row-major are the query features (the B x S output features of
 * the current step), K_dev [views * n x D] bf16 the key set, block s holding the features at positions 0..n-1
 * of another step or the targets; the positives of query i are the keys at position i of every block.  Which
 * features form the key set is the caller's choice (the paper leaves it open).  Every feature is divided by its
 * norm (sum of squares, norm and scaling in float64) and the unit vector is rounded once to bf16, the operand type
 * of the contraction: a scaled similarity can differ from Eq. 2 in real arithmetic by up to
 * (2^-7 + 2^-16) sum_d |q_d k_d| / tau (at most 0.11 at tau = 0.07; typically 1e-3 at D = 4096).  The n x m
 * contraction runs on the tensor cores with fp32 accumulation and its epilogue keeps only (max, sum-exp) per row and the positives, so the similarity matrix is not stored.
 *
 * coral_csra_workspace_bytes: size of the caller-owned scratch for (n, views, D).
 * coral_csra_infonce: workspace_dev 256-byte aligned, at least that size.  out_loss_dev [1] float;
 *   out_row_loss_dev [n] float or NULL; out_logits_dev [n x views*n] float or NULL (the scaled similarities,
 *   for checks on small cases).  n >= 1, 1 <= views <= 8, D a multiple of 8, tau > 0, else CORAL_ERR_INVALID.
 *   Asynchronous on `stream`; no allocation.
 * coral_csra_status: synchronises `stream` and returns the status word of the last call that used the
 *   workspace (0 or CORAL_ERR_TIMEOUT).
 */
int coral_csra_workspace_bytes(int n, int views, int D, size_t *bytes);
int coral_csra_infonce(const void *Q_dev, const void *K_dev, int n, int views, int D, float tau, void *workspace_dev,
                       float *out_row_loss_dev, float *out_loss_dev, float *out_logits_dev, void *stream);
int coral_csra_status(void *workspace_dev, void *stream);

/*
 * Ask L2 to keep the first n_hot groups of the packed head between calls (Appendix B: with a
 * frequency-ordered vocabulary the low-index groups hold the frequent tokens and are activated by almost every
 * row).  The streaming kernel then loads those groups' weights with an evict-last cache hint, and up to their
 * size of L2 is set aside for such lines (cudaLimitPersistingL2CacheSize: a setting of this process's CUDA
 * context that takes L2 away from everything else the process runs and ends with the process; without the
 * set-aside the hint alone changed nothing).  How much survives depends on what runs between two calls.
 * Meant for contiguous, frequency-ordered group maps; n_hot = 0 (the default) switches it off.  Applies to
 * calls on the streaming path.  Synchronises nothing, but the set-aside is PROCESS-WIDE state of the CUDA context,
 * shared with every other handle and with anything else the process runs (last writer wins): the call only ever
 * raises the limit, remembers the value it found, and puts that value back (and resets the persisting lines)
 * when the hot groups are switched off or the handle is destroyed.  Call it at set-up time, not between
 * overlapping work, and not from two handles that are meant to hold different set-asides at once.
 */
int coral_lmhead_set_hot_groups(coral_lmhead_handle h, int n_hot);

/*
 * Failure-detection self-test with no counterpart in the paper.  Every wait inside the kernels (on a ring
 * slot, a statistics buffer, a tensor-memory buffer) polls a bounded number of times and, when the bound
 * runs out, writes CORAL_ERR_TIMEOUT to the handle's status word and carries on to a normal exit.  This
 * call launches a one-warp kernel that polls the same way (with a shorter bound) on a barrier nothing
 * completes, so a caller can check that an expired wait is reported by coral_lmhead_status and leaves
 * the handle and the context usable.  Asynchronous on `stream`; nothing faults, traps or spins unbounded.
 */
int coral_lmhead_selftest_wait_expiry(coral_lmhead_handle h, void *stream);

/*
 * Bench-side measurement aid with no counterpart in the paper (not part of the draft step): streams the first
 * `bytes` of the packed head into shared memory with plain contiguous 16 KiB bulk copies (one CTA per SM,
 * `in_flight` copies outstanding each; 0 = the default of 8, at most 13) and does nothing with them; the region
 * is swept `repeats` times (1..64).  Timed by the caller with events on `stream`, from a cold L2 and with
 * repeats = 1, it gives the floor for the weight-streaming kernel of a draft call that reads as many bytes: a
 * one-shot read of a few hundred megabytes does not reach the bandwidth of a long copy.  With a region smaller
 * than L2, the time difference between two repeat counts gives the rate at which the SMs can take bytes in from
 * L2.  bytes in [16384, packed_bytes]; asynchronous, no allocation.
 */
int coral_lmhead_copy_floor(coral_lmhead_handle h, long long bytes, int in_flight, int repeats, void *stream);

/*
 * Bench-side measurement aid with no counterpart in the paper (not part of the draft step): what issuing the
 * tensor-core path's MMAs costs by itself.  Every CTA pair of the tensor-core kernel's grid runs `rounds` rounds
 * of `per_commit` (1..16) tcgen05.mma of 256 x n x 16 (n a multiple of 16 in [16, 256]; the instruction forms of
 * the tensor-core path) on zeroed shared memory followed by one tcgen05.commit, from `issuers` (1 or 2) threads;
 * nothing is loaded.  out_ns_dev[0] receives the nanoseconds the first pair's first issuer needed to issue its
 * rounds, out_ns_dev[1] until its last MMA had completed (device memory, two 64-bit words).  Needs a handle created
 * with max_M > 32 (CORAL_ERR_INVALID otherwise); asynchronous, no allocation; every wait is bounded.
 */
int coral_lmhead_tc_issue_probe(coral_lmhead_handle h, int n, int per_commit, int issuers, int rounds,
                                unsigned long long *out_ns_dev, void *stream);

/*
 * Measurement aid for the dominant kernel (the one that streams the selected
 * groups' weights; Section 3.3 names the LM head as the drafter's main cost).
 * With timing on, every draft call records a CUDA event before and after that
 * kernel on the call's stream; coral_lmhead_head_kernel_ms waits for the last
 * call's second event and returns the elapsed milliseconds between the two.
 * Timing is off by default.  CORAL_ERR_INVALID if timing was never switched on.
 */
int coral_lmhead_set_kernel_timing(coral_lmhead_handle h, int on);
int coral_lmhead_head_kernel_ms(coral_lmhead_handle h, float *ms);
/* Same aid, three spans of the last timed call: router stage, weight-streaming kernel, merge. */
int coral_lmhead_stage_ms(coral_lmhead_handle h, float *route_ms, float *head_ms, float *merge_ms);

/*
 * Synchronise `stream`, return the device status word of the handle and clear it: CORAL_OK;
 * CORAL_ERR_TIMEOUT (a bounded wait gave up); CORAL_ERR_BOUNDS (forced_groups held a group outside [0, N) or
 * the same group twice in a row); CORAL_ERR_NONFINITE (a router score was NaN, e.g. from a NaN hidden state:
 * such a score is ranked below every other score, so each row still gets k_groups distinct groups).
 * The word is sticky: the first problem stays until this call reads it, and while it is non-zero the
 * kernels after the router stage of every draft call on the handle do nothing, so that nothing ever indexes
 * with an inconsistent selection; the outputs of those calls are not written.  (The paper does not say what
 * a router should do with non-finite scores; inputs are expected to be finite.)
 */
int coral_lmhead_status(coral_lmhead_handle h, void *stream);

/*
 * Facts about the last draft call (Appendix B: in tree decoding all the groups
 * involved by any candidate are activated; groups_touched is that union).
 * Synchronises `stream` to read the union size back.
 */
int coral_lmhead_last_stats(coral_lmhead_handle h, coral_lmhead_stats *out, void *stream);

/*
 * Router step (gate scores and the k_groups best groups per row) for callers
 * that must not allocate.  The paper has no counterpart to this entry point;
 * it computes the same scores and selections as coral_lmhead_draft_ex reports
 * through out_gate_dev / out_groups_dev.
 *
 * Who needs it: code that runs where device allocation is off limits, for
 * example a serving loop whose memory pool is fixed up front and audited, a
 * plug-in that is handed a stream but no allocator, or a latency-critical
 * section where cudaMalloc's implicit device synchronisation is unacceptable.
 * Such callers cannot create a handle (that needs a workspace).  Here they pass
 * only inputs and outputs; the scratch the router kernels need lives in a fixed
 * array inside the library's device image, CORAL_ROUTE_STATIC_MAX_ROWS rows x
 * CORAL_MAX_GROUPS groups (about 160 KiB), which every GPU that loads the
 * library keeps until the process exits.  The call makes no cudaMalloc,
 * cudaFree or other allocating call.
 *
 *   W_gate_dev     [n_groups x H] bf16, device, 16-byte aligned
 *   hidden_dev     [M x H] bf16, device, 16-byte aligned
 *   out_groups_dev [M x k_groups] int32, device: groups in selection order
 *                  (descending score, equal scores -> lower index)
 *   out_gate_dev   [M x n_groups] float, device, or NULL
 * Asynchronous on `stream`.  CORAL_ERR_TOO_LARGE if M exceeds
 * CORAL_ROUTE_STATIC_MAX_ROWS; CORAL_ERR_INVALID for NULL/misaligned pointers,
 * H not a positive multiple of 8, n_groups outside [1, CORAL_MAX_GROUPS] or
 * k_groups outside [1, n_groups].
 *
 * The first call on each device looks up the array's device address (a
 * runtime query, made with that device current); make that first call before
 * starting any stream capture.  All calls on a device share the one array and
 * it keeps the previous call's contents (the call clears what has to start at
 * zero): two calls whose kernels may overlap on the GPU (different streams,
 * no ordering between them) race and give undefined results.
 */
int coral_lmhead_route_static(const void *W_gate_dev, const void *hidden_dev, int M, int H, int n_groups,
                              int k_groups, int32_t *out_groups_dev, float *out_gate_dev, void *stream);

/*
 * Tree-expansion score step on the outputs of coral_lmhead_draft (Section 2.2: multiple candidates per
 * timestep form a tree of drafts; Section 4.1: tree depth 6, 60 candidate tokens; Appendix B: top 10 candidates
 * per node).  For each of n_seq sequences with `nodes` rows:
 *   child score = parent_scores[node] + cand_logprobs[node][i]      (one fp32 addition)
 * and the K best children (descending score; equal -> lower node * k_tokens + i) are returned, sorted:
 *   out_parent [n_seq x K] node index inside the sequence, out_token [n_seq x K] = cand_ids of the child,
 *   out_score [n_seq x K].
 * With cand_logprobs_dev = NULL and k_tokens = 1 the call re-ranks the nodes themselves (e.g. the final choice
 * of the best 60 nodes); cand_ids_dev may be NULL (the flat child index is returned as token).
 * All pointers device; asynchronous on `stream`; no scratch memory.  CORAL_ERR_TOO_LARGE if nodes * k_tokens
 * exceeds 2048; CORAL_ERR_INVALID for NULL outputs, sizes < 1, K > min(256, nodes * k_tokens).
 */
int coral_tree_expand(const float *parent_scores_dev, const int32_t *cand_ids_dev, const float *cand_logprobs_dev,
                      int n_seq, int nodes, int k_tokens, int K, int32_t *out_parent_dev, int32_t *out_token_dev,
                      float *out_score_dev, void *stream);

/* Static, NUL-terminated description of a status code. */
const char *coral_lmhead_error_string(int code);

/* Free what the library allocated.  NULL is accepted. */
int coral_lmhead_destroy(coral_lmhead_handle h);

#ifdef __cplusplus
}
#endif
#endif /* CORAL_LMHEAD_H_ */
