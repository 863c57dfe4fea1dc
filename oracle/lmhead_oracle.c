/*
 * CPU oracle for the weight-grouped LM-head draft step.  TEST INFRASTRUCTURE:
 * only the tests, the smoke check and the bench's CPU-baseline leg may call
 * it.  It shares no code with the CUDA library and is never a fallback for it.
 *
 * What it computes, per query row h (paper Section 3.3, "LM Head Router"):
 *   1. router scores over the N groups.  Single-matrix gate: g = W_gate h
 *      (the reading the workload definitions fix).  With W1 given, Eq. 7's
 *      argument: g = W2 (act(W1 h) + h), W2 = W_gate, act = SiLU
 *      (the paper leaves act unnamed).
 *   2. the top-n groups by score (descending; equal scores -> lower index),
 *      the "activate only a subset of LM head parameters" step.
 *   3. logits z[x] = W_vocab[x] . h for the tokens x of the selected groups
 *      only (V split equally into N groups of v = V/N, Section 3.3).
 *   4. joint mode: log-softmax over all active logits of the row;
 *      factorised mode (Eq. 8): log p(x) = log p_router(n) + log p_group(x^n),
 *      p_router = Softmax over all N scores (Eq. 7), p_group = softmax inside
 *      group n, independent of the other groups.  The paper does not say
 *      whether p_router is renormalised over the selected groups; mode 2 is
 *      that variant: log p(x) = log (p_router(n) / sum of p_router over the
 *      selected groups) + log p_group(x^n), whose mass over the active
 *      vocabulary is 1.
 *   5. the k_tokens best tokens by log-probability (descending; equal ->
 *      lower token id): the "top 10 candidates" of Appendix B, tree decoding.
 *
 * Arithmetic: every bf16 input is widened exactly to double and all sums,
 * exps and logs are taken in double, in the order written.  No blocking, no
 * fusion, no reuse of partial results beyond what the definition states.
 * Rows of the batch are independent (Appendix B: the union of groups matters
 * for cost only).
 *
 * Pins (tests/test_oracle_pins.py): dense-head equivalence with all groups
 * active against numpy/scipy, probabilities sum to 1, brute force on toys,
 * closed forms (zero weights, one-hot hidden states), monotonicity in k,
 * relabelling invariances, the ideal-router identity for Eq. 8, the paper's
 * "1002M" byte count.  The paper prints no numeric head outputs, so value
 * parity with the paper itself is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_INVALID (-1)
#define ORACLE_ERR_GROUPING (-2)
#define ORACLE_ERR_NOMEM (-3)

static double bf16_value(uint16_t bits) {
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

typedef struct {
    double score;
    int32_t index;
} scored_t;

/* descending score, ascending index among equals */
static int by_score_desc(const void *pa, const void *pb) {
    const scored_t *a = (const scored_t *)pa, *b = (const scored_t *)pb;
    if (a->score > b->score) return -1;
    if (a->score < b->score) return 1;
    return (a->index > b->index) - (a->index < b->index);
}

static double log_sum_exp(const double *z, long n) {
    double mx = z[0];
    for (long i = 1; i < n; ++i)
        if (z[i] > mx) mx = z[i];
    double s = 0.0;
    for (long i = 0; i < n; ++i) s += exp(z[i] - mx);
    return mx + log(s);
}

int coral_oracle_threads(void);

/*
 * All arrays are host memory, row-major.  bf16 tensors are uint16 bit patterns.
 *   W_vocab   [V x H] bf16       group_map [V] int32 in [0, N)
 *   W_gate    [N x H] bf16       hidden    [M x H] bf16
 *   W1        [H x H] bf16 or NULL (NULL: g = W_gate h)
 *   forced_groups [M x k_groups] or NULL: use these groups instead of step 2
 *   gate_override [M x N] doubles or NULL: use these scores instead of step 1
 *   factorised: 0 = joint log-softmax over the active logits, 1 = Eq. 8,
 *               2 = Eq. 8 with p_router renormalised over the selected groups
 * Outputs (any may be NULL):
 *   out_gate [M x N], out_groups [M x k_groups] (selection order),
 *   out_logits [M x k_groups x v] and out_logit_tokens (same shape): slot s
 *   of row m holds the tokens of group out_groups[m][s] in ascending token id,
 *   out_lse [M] joint log-sum-exp of the active logits,
 *   out_group_lse [M x k_groups] log-sum-exp inside each selected group,
 *   out_log_router [M x N] log Softmax(g),
 *   out_ids / out_logprobs [M x k_tokens].
 */
int coral_oracle_draft(const uint16_t *W_vocab, const int32_t *group_map, const uint16_t *W_gate,
                       const uint16_t *W1, const uint16_t *hidden, int H, int V, int N, int M,
                       int k_groups, int k_tokens, const int32_t *forced_groups,
                       const double *gate_override, int factorised, double *out_gate,
                       int32_t *out_groups, double *out_logits, int32_t *out_logit_tokens,
                       double *out_lse, double *out_group_lse, double *out_log_router,
                       int32_t *out_ids, double *out_logprobs) {
    if (!W_vocab || !group_map || !W_gate || !hidden) return ORACLE_ERR_INVALID;
    if (H < 1 || V < 1 || N < 1 || M < 1 || V % N != 0) return ORACLE_ERR_INVALID;
    const int v = V / N;
    if (k_groups < 1 || k_groups > N) return ORACLE_ERR_INVALID;
    if (k_tokens < 1 || (long)k_tokens > (long)k_groups * v) return ORACLE_ERR_INVALID;
    if (factorised < 0 || factorised > 2) return ORACLE_ERR_INVALID;
    {
        long *cnt = (long *)calloc((size_t)N, sizeof(long));
        if (!cnt) return ORACLE_ERR_NOMEM;
        int bad = 0;
        for (int x = 0; x < V; ++x) {
            if (group_map[x] < 0 || group_map[x] >= N) { bad = 1; break; }
            cnt[group_map[x]]++;
        }
        for (int n = 0; n < N && !bad; ++n)
            if (cnt[n] != v) bad = 2;
        free(cnt);
        if (bad == 1) return ORACLE_ERR_INVALID;
        if (bad == 2) return ORACLE_ERR_GROUPING;
    }

    const long n_active = (long)k_groups * v;
    double *h = (double *)malloc(sizeof(double) * (size_t)H);
    double *u = (double *)malloc(sizeof(double) * (size_t)H); /* router input */
    double *g = (double *)malloc(sizeof(double) * (size_t)N);
    double *log_router = (double *)malloc(sizeof(double) * (size_t)N);
    scored_t *order = (scored_t *)malloc(sizeof(scored_t) * (size_t)N);
    int32_t *sel = (int32_t *)malloc(sizeof(int32_t) * (size_t)k_groups);
    int32_t *slot_of_group = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    double *z = (double *)malloc(sizeof(double) * (size_t)n_active);
    int32_t *tok = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_active);
    double *group_lse = (double *)malloc(sizeof(double) * (size_t)k_groups);
    double *z_sel = (double *)malloc(sizeof(double) * (size_t)k_groups);
    scored_t *cand = (scored_t *)malloc(sizeof(scored_t) * (size_t)n_active);
    int rc = ORACLE_OK;
    if (!h || !u || !g || !log_router || !order || !sel || !slot_of_group || !z || !tok ||
        !group_lse || !z_sel || !cand) {
        rc = ORACLE_ERR_NOMEM;
        goto done;
    }

    for (int m = 0; m < M; ++m) {
        for (int j = 0; j < H; ++j) h[j] = bf16_value(hidden[(size_t)m * H + j]);

        /* step 1: router scores */
        if (W1) { /* Eq. 7: u = act(W1 h) + h */
#pragma omp parallel for schedule(static)
            for (int i = 0; i < H; ++i) {
                double a = 0.0;
                for (int j = 0; j < H; ++j) a += bf16_value(W1[(size_t)i * H + j]) * h[j];
                u[i] = a / (1.0 + exp(-a)) + h[i];
            }
        } else {
            for (int j = 0; j < H; ++j) u[j] = h[j];
        }
        for (int n = 0; n < N; ++n) {
            double a = 0.0;
            for (int j = 0; j < H; ++j) a += bf16_value(W_gate[(size_t)n * H + j]) * u[j];
            g[n] = a;
        }
        if (gate_override)
            for (int n = 0; n < N; ++n) g[n] = gate_override[(size_t)m * N + n];
        {
            double l = log_sum_exp(g, N);
            for (int n = 0; n < N; ++n) log_router[n] = g[n] - l;
        }

        /* step 2: top-n groups */
        if (forced_groups) {
            for (int s = 0; s < k_groups; ++s) {
                sel[s] = forced_groups[(size_t)m * k_groups + s];
                if (sel[s] < 0 || sel[s] >= N) { rc = ORACLE_ERR_INVALID; goto done; }
                for (int t = 0; t < s; ++t)
                    if (sel[t] == sel[s]) { rc = ORACLE_ERR_INVALID; goto done; }
            }
        } else {
            for (int n = 0; n < N; ++n) { order[n].score = g[n]; order[n].index = n; }
            qsort(order, (size_t)N, sizeof(scored_t), by_score_desc);
            for (int s = 0; s < k_groups; ++s) sel[s] = order[s].index;
        }
        for (int n = 0; n < N; ++n) slot_of_group[n] = -1;
        for (int s = 0; s < k_groups; ++s) slot_of_group[sel[s]] = s;

        /* step 3: logits of the active tokens only; slot layout, ascending id */
        {
            long *fill = (long *)calloc((size_t)k_groups, sizeof(long));
            if (!fill) { rc = ORACLE_ERR_NOMEM; goto done; }
            for (int x = 0; x < V; ++x) {
                int s = slot_of_group[group_map[x]];
                if (s < 0) continue;
                tok[(long)s * v + fill[s]++] = x;
            }
            free(fill);
        }
#pragma omp parallel for schedule(static)
        for (long i = 0; i < n_active; ++i) {
            const uint16_t *w = W_vocab + (size_t)tok[i] * H;
            double a = 0.0;
            for (int j = 0; j < H; ++j) a += bf16_value(w[j]) * h[j];
            z[i] = a;
        }

        /* step 4: normalisers */
        const double lse = log_sum_exp(z, n_active);
        for (int s = 0; s < k_groups; ++s) group_lse[s] = log_sum_exp(z + (long)s * v, v);

        /* step 5: rank by log-probability */
        double log_selected_mass = 0.0;     /* log of the router mass of the selected groups (mode 2) */
        if (factorised == 2) {
            for (int s = 0; s < k_groups; ++s) z_sel[s] = log_router[sel[s]];
            log_selected_mass = log_sum_exp(z_sel, k_groups);
        }
        for (long i = 0; i < n_active; ++i) {
            int s = (int)(i / v);
            cand[i].index = tok[i];
            cand[i].score = factorised ? log_router[sel[s]] - log_selected_mass + (z[i] - group_lse[s]) : z[i] - lse;
        }
        qsort(cand, (size_t)n_active, sizeof(scored_t), by_score_desc);

        if (out_gate) memcpy(out_gate + (size_t)m * N, g, sizeof(double) * (size_t)N);
        if (out_log_router) memcpy(out_log_router + (size_t)m * N, log_router, sizeof(double) * (size_t)N);
        if (out_groups) memcpy(out_groups + (size_t)m * k_groups, sel, sizeof(int32_t) * (size_t)k_groups);
        if (out_logits) memcpy(out_logits + (size_t)m * n_active, z, sizeof(double) * (size_t)n_active);
        if (out_logit_tokens) memcpy(out_logit_tokens + (size_t)m * n_active, tok, sizeof(int32_t) * (size_t)n_active);
        if (out_lse) out_lse[m] = lse;
        if (out_group_lse) memcpy(out_group_lse + (size_t)m * k_groups, group_lse, sizeof(double) * (size_t)k_groups);
        for (int i = 0; i < k_tokens; ++i) {
            if (out_ids) out_ids[(size_t)m * k_tokens + i] = cand[i].index;
            if (out_logprobs) out_logprobs[(size_t)m * k_tokens + i] = cand[i].score;
        }
    }

done:
    free(h); free(u); free(g); free(log_router); free(order); free(sel); free(slot_of_group);
    free(z); free(tok); free(group_lse); free(z_sel); free(cand);
    return rc;
}

#ifdef _OPENMP
#include <omp.h>
int coral_oracle_threads(void) { return omp_get_max_threads(); }
#else
int coral_oracle_threads(void) { return 1; }
#endif
