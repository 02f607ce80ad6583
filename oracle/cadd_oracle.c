/*
 * CaDDTree oracle: a plain, slow, fp64 CPU implementation of one decoding round's tree build
 * and tree verification.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It exists to check the CUDA path and to be timed beside it
 * as a CPU baseline.  Nothing in the product (the package, its C-ABI library) may import, link
 * or call it, and it shares no code, header, table or constant with the CUDA path.
 *
 * What it computes, step by step, in the paper's order and notation:
 *   O1  per-position marginals q_i = softmax(l_i)                        (Eq. 1)
 *   O2  top-K tokens v_i^(k) and log-probs log q_i^(k) per position      (Algorithm 1, Require)
 *   O3  best-first expansion with the greedy throughput stopping rule    (Algorithm 1; Eq. 7,
 *       Eq. 11; Corollary 1)
 *   O4  draft-tree arrays and the ancestor ("tree attention") mask       (Section 3.3)
 *   O5  greedy verification: argmax of the target logits at every node   (Section 3.1)
 *   O6  walk along the longest accepted path, next bonus token           (Sections 3.1, 3.3)
 *   O7  target logits from hidden states and the output projection      (Section 3.1; feeds O5)
 * The convex regression of the cost tables (Eq. 12) lives in the Python wrapper, written as a
 * non-negative least-squares problem for the library's NNLS routine.
 *
 * All floating point is double.  bf16 / fp32 inputs are widened exactly.  No blocking, fusion
 * or reordering: sums run in ascending token order, the heap H of Algorithm 1 is an unordered
 * array popped by a linear scan for the maximum.
 *
 * Readings where the paper is silent (also listed in the design notes of the repository):
 *   - top-K order and membership among equal logits: (logit descending, token id ascending);
 *   - node score sigma = A - S_d, where A is the root-to-node sum of (logit - row max) and
 *     S_d the running sum of log-partitions of depths 1..d, so that equal logit sums at one
 *     depth give bit-equal scores;
 *   - pop order among equal scores: lower depth, then lower token id, then lower parent row;
 *   - n counts draft nodes only (the root / bonus token is row 0 and is not counted);
 *   - stop at the first n with theta(n+1) <= theta(n); the node cap B_max ends the loop
 *     before the next candidate is evaluated;
 *   - argmax ties go to the lowest token id; NaN orders as -Inf;
 *   - the next bonus token is the target's argmax at the last accepted node.
 *
 * Pins (tests that fix this file to something other than itself): brute-force enumeration of
 * all nodes and of all prefix-closed trees on tiny (K, L); fp64 log-softmax and stable argsort
 * from numpy/scipy; closed forms (uniform logits, K=1 chain, near-one-hot marginals);
 * the invariants the paper proves (Lemma 1, Theorem 1, Corollaries 1 and 2); numpy argmax;
 * brute-force accepted-path search; the two diagnostic margins (pop_gap, stop_gap) by hand-worked
 * rationals, by the heap contents rebuilt from the pop order, and by a constructed near-tie.
 * No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_BF16 = 0, ORC_FP32 = 1 };
enum { ORC_COST_QUADRATIC = 0, ORC_COST_TABLE = 1, ORC_COST_TABLE_INTERP = 2 };
enum { ORC_FLAG_FIXED_BUDGET = 4 };
enum { ORC_ROWS_LIVE = 0, ORC_ROWS_DENSE = 1 };
enum {
    ORC_ST_NONFINITE = 1,
    ORC_ST_FEWER_THAN_K = 2,
    ORC_ST_CAP_HIT = 4,
    ORC_ST_FRONTIER_EXHAUSTED = 8,
    ORC_ST_L_EFF_CLAMPED = 16,
    ORC_ST_COST_NONPOSITIVE = 32,
    ORC_ST_BAD_N_NODES = 64,
    ORC_ST_BAD_TABLE_IDX = 256
};

int cadd_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Threads the batch loops below may use from now on (timing aid: the same code on one core). */
void cadd_oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Exact widening of one stored logit to double. */
static double logit_at(const void *base, int dtype, int64_t idx)
{
    if (dtype == ORC_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t *)base)[idx] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[idx];
}

/*
 * O1 + O2 for one row of V logits (Eq. 1; Algorithm 1, Require).
 *   m     = max_v x_v
 *   Z     = sum_v exp(x_v - m)      (ascending v)
 *   tok[k], a[k] = x_(k) - m, lp[k] = a[k] - log Z   for the K_eff best under
 *           (x descending, v ascending); K_eff = min(K, number of finite logits).
 * NaN and infinite logits carry no mass, are never candidates and do not enter m (m is the
 * largest finite logit); NaN or +Inf raise `nonfinite`, +Inf additionally `has_pinf` (the caller
 * then returns the empty tree; the lists reported for such a row are those of its finite logits).
 */
int cadd_oracle_row_softmax_topk(const void *row, int dtype, int64_t V, int K,
                                 double *m_out, double *logZ_out,
                                 int32_t *tok, double *a, double *lp,
                                 int32_t *k_eff_out, int32_t *nonfinite, int32_t *has_pinf)
{
    double m = -INFINITY;
    int nf = 0, pinf = 0;
    for (int64_t v = 0; v < V; ++v) {
        double x = logit_at(row, dtype, v);
        if (isnan(x)) { nf = 1; continue; }
        if (isinf(x) && x > 0) { nf = 1; pinf = 1; continue; }   /* invalid input: flagged, kept out of m */
        if (x > m) m = x;
    }
    double Z = 0.0;
    int k_eff = 0;
    double *val = (double *)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
    for (int64_t v = 0; v < V; ++v) {
        double x = logit_at(row, dtype, v);
        if (isnan(x) || isinf(x)) continue;      /* no mass, never a candidate */
        Z += exp(x - m);
        /* insert into the list kept sorted by (x descending, v ascending); v only grows, so
           an equal value goes after the ones already there */
        int pos = k_eff;
        while (pos > 0 && val[pos - 1] < x) --pos;
        if (pos < K) {
            int last = (k_eff < K) ? k_eff : K - 1;
            for (int j = last; j > pos; --j) { val[j] = val[j - 1]; tok[j] = tok[j - 1]; }
            val[pos] = x;
            tok[pos] = (int32_t)v;
            if (k_eff < K) ++k_eff;
        }
    }
    double logZ = log(Z);
    for (int k = 0; k < K; ++k) {
        if (k < k_eff) { a[k] = val[k] - m; lp[k] = a[k] - logZ; }
        else { tok[k] = -1; a[k] = -INFINITY; lp[k] = -INFINITY; }
    }
    free(val);
    *m_out = m; *logZ_out = logZ; *k_eff_out = k_eff; *nonfinite = nf; *has_pinf = pinf;
    return 0;
}

typedef struct {
    int32_t parent;   /* tree row of the parent (0 = root) */
    int32_t depth;    /* d >= 1 */
    int32_t rank;     /* s_d in 1..K: index into the depth-d top-K list */
    int32_t token;    /* v_d^(rank) */
    double A;         /* root-to-node sum of (logit - row max) */
    double sigma;     /* A - S_d = log prefix probability */
} cand_t;

/* The total order of Algorithm 1's heap: higher score, then lower depth, lower token id,
   lower parent row.  Returns nonzero when x precedes y. */
static int cand_before(const cand_t *x, const cand_t *y)
{
    if (x->sigma != y->sigma) return x->sigma > y->sigma;
    if (x->depth != y->depth) return x->depth < y->depth;
    if (x->token != y->token) return x->token < y->token;
    return x->parent < y->parent;
}

/* The verification cost C_v(n; l) of one request.  QUADRATIC: a + b n + c n^2.  TABLE: one table row.
 * TABLE_INTERP (context interpolation at inference, Eq. 13): with L_j <= l < L_{j+1} and
 * alpha = (l - L_j) / (L_{j+1} - L_j),  C_v(n; l) = (1 - alpha) C_v(n; L_j) + alpha C_v(n; L_{j+1});
 * outside the profiled range the nearest table is used. */
typedef struct {
    int kind;
    const double *coef4;      /* QUADRATIC */
    const double *row0;       /* TABLE: the row; TABLE_INTERP: the row of L_j */
    const double *row1;       /* TABLE_INTERP: the row of L_{j+1} */
    double alpha;             /* TABLE_INTERP */
} cost_model_t;

static double cost_verify(const cost_model_t *cm, int n)
{
    if (cm->kind == ORC_COST_TABLE) return cm->row0[n];
    if (cm->kind == ORC_COST_TABLE_INTERP) return (1.0 - cm->alpha) * cm->row0[n] + cm->alpha * cm->row1[n];
    double x = (double)n;
    return cm->coef4[1] + cm->coef4[2] * x + cm->coef4[3] * (x * x);
}

/*
 * O1-O4 for a batch (Eq. 1; Algorithm 1; Section 3.3).  Host pointers; element strides.
 * Optional outputs may be NULL.  Rows past n*+1 are padded: token -1, parent -1, depth 0,
 * position 0, log-prob 0, empty mask row.
 * Diagnostics (oracle only): logZ[batch,L]; pop_gap[batch,R] = 1 - exp(sigma_2 - sigma_1) with
 * sigma_2 the best strictly smaller score in the heap when row j was popped (1 if none);
 * stop_gap[batch] = |theta_new - theta_prev| / theta_prev at the evaluation that stopped the
 * loop, or the smallest such margin over accepted nodes when nothing stopped it;
 * theta_curve[batch,R]: theta(n) for n = 0..n*.
 */
int cadd_oracle_build_tree(
    int batch, int L, int64_t V, int K, int B_max, int R,
    int dtype, const void *draft_logits, int64_t stride_b, int64_t stride_l,
    const int32_t *l_eff_in, const int32_t *bonus_token, const int32_t *ctx_len,
    int cost_kind, const double *cost_coef, const double *cost_table, const int32_t *table_idx,
    const double *t_draft, int n_tables, const int32_t *ctx_grid, uint32_t flags,
    int32_t *n_nodes, int32_t *token_ids, int32_t *parent_idx, int32_t *depth,
    int32_t *position_ids, double *node_logprob, double *phi_out, double *theta_out,
    uint32_t *mask_bits, uint8_t *mask_dense, int32_t *topk_token, double *topk_logprob,
    int32_t *status,
    double *logZ_out, double *pop_gap, double *stop_gap, double *theta_curve, int32_t *node_rank)
{
    if (batch < 1 || L < 1 || K < 1 || V < 1 || B_max < 0 || R < B_max + 1) return -1;
    const int W = (R + 31) / 32;
    const size_t esz = (dtype == ORC_BF16) ? 2 : 4;

#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < batch; ++b) {
        int st = 0;
        int Le = l_eff_in ? l_eff_in[b] : L;
        if (Le < 0) { Le = 0; st |= ORC_ST_L_EFF_CLAMPED; }
        if (Le > L) { Le = L; st |= ORC_ST_L_EFF_CLAMPED; }

        /* ---- O1 + O2: per-position marginals and top-K lists ---- */
        int32_t *tk_tok = (int32_t *)malloc(sizeof(int32_t) * (size_t)L * K);
        double *tk_a = (double *)malloc(sizeof(double) * (size_t)L * K);
        double *tk_lp = (double *)malloc(sizeof(double) * (size_t)L * K);
        int32_t *k_eff = (int32_t *)calloc((size_t)L + 2, sizeof(int32_t));
        double *lz = (double *)calloc((size_t)L + 1, sizeof(double));
        int any_pinf = 0;
        for (int i = 0; i < L; ++i) {
            for (int k = 0; k < K; ++k) {
                tk_tok[i * K + k] = -1; tk_a[i * K + k] = -INFINITY; tk_lp[i * K + k] = -INFINITY;
            }
            if (i >= Le) continue;
            const char *row = (const char *)draft_logits +
                              esz * (size_t)((int64_t)b * stride_b + (int64_t)i * stride_l);
            double m, logZ; int32_t ke, nf, pinf;
            cadd_oracle_row_softmax_topk(row, dtype, V, K, &m, &logZ, tk_tok + i * K,
                                         tk_a + i * K, tk_lp + i * K, &ke, &nf, &pinf);
            k_eff[i + 1] = ke;           /* k_eff[d] for depth d = i+1 */
            lz[i] = logZ;
            if (nf) st |= ORC_ST_NONFINITE;
            if (pinf) any_pinf = 1;
            if (ke < K) st |= ORC_ST_FEWER_THAN_K;
        }
        for (int i = 0; i < L; ++i) {
            if (logZ_out) logZ_out[(size_t)b * L + i] = (i < Le) ? lz[i] : 0.0;
            for (int k = 0; k < K; ++k) {
                if (topk_token) topk_token[((size_t)b * L + i) * K + k] = tk_tok[i * K + k];
                if (topk_logprob) topk_logprob[((size_t)b * L + i) * K + k] = tk_lp[i * K + k];
            }
        }

        /* ---- O3: Algorithm 1 ---- */
        cost_model_t cm = { cost_kind, NULL, NULL, NULL, 0.0 };
        int bad_table = 0;
        if (cost_kind == ORC_COST_QUADRATIC) cm.coef4 = cost_coef + (size_t)b * 4;
        else if (cost_kind == ORC_COST_TABLE) {
            /* a table index outside [0, n_tables) names no cost model: flagged, empty tree */
            int ti = table_idx[b];
            if (ti < 0 || ti >= n_tables) { st |= ORC_ST_BAD_TABLE_IDX; bad_table = 1; ti = 0; }
            cm.row0 = cost_table + (size_t)ti * (B_max + 1);
        } else {                                   /* Eq. 13: the two profiled context lengths around l */
            const int l = ctx_len ? ctx_len[b] : 0;
            int jlo = 0;
            while (jlo + 1 < n_tables && ctx_grid[jlo + 1] <= l) ++jlo;      /* largest j with L_j <= l (or 0) */
            int jhi = (jlo + 1 < n_tables) ? jlo + 1 : jlo;
            if (l <= ctx_grid[0]) { jlo = jhi = 0; }
            cm.row0 = cost_table + (size_t)jlo * (B_max + 1);
            cm.row1 = cost_table + (size_t)jhi * (B_max + 1);
            cm.alpha = (jhi == jlo) ? 0.0
                                    : ((double)l - (double)ctx_grid[jlo]) / ((double)ctx_grid[jhi] - (double)ctx_grid[jlo]);
        }
        const double C_d = (cost_kind == ORC_COST_QUADRATIC) ? cm.coef4[0] : t_draft[b];

        cand_t *node = (cand_t *)calloc((size_t)R + 1, sizeof(cand_t));   /* rows 1..n */
        cand_t *H = (cand_t *)malloc(sizeof(cand_t) * ((size_t)B_max + 2));
        double *S = (double *)calloc((size_t)L + 1, sizeof(double));      /* S_d = sum_{i<=d} logZ_i */
        for (int d = 1; d <= Le; ++d) S[d] = S[d - 1] + lz[d - 1];
        int hn = 0, n = 0;
        double Phi = 0.0, theta_prev = 0.0;
        double min_margin = INFINITY, stop_margin = -1.0;
        double den0 = C_d + cost_verify(&cm, 0);
        int ok = !bad_table;
        if (ok && !(den0 > 0.0)) { st |= ORC_ST_COST_NONPOSITIVE; ok = 0; }
        else theta_prev = 1.0 / den0;
        if (any_pinf) ok = 0;
        if (theta_curve) theta_curve[(size_t)b * R] = theta_prev;
        if (ok && Le >= 1 && k_eff[1] >= 1) {
            cand_t c = { 0, 1, 1, tk_tok[0], 0.0 + tk_a[0], 0.0 };
            c.sigma = c.A - S[1];
            H[hn++] = c;
        }
        int stopped_by_rule = 0;
        while (ok && hn > 0 && n < B_max) {
            int best = 0;
            for (int i = 1; i < hn; ++i) if (cand_before(&H[i], &H[best])) best = i;
            cand_t s = H[best];
            double runner = -INFINITY;
            for (int i = 0; i < hn; ++i)
                if (H[i].sigma < s.sigma && H[i].sigma > runner) runner = H[i].sigma;
            double delta = exp(s.sigma);
            double den = C_d + cost_verify(&cm, n + 1);
            if (!(den > 0.0)) { st |= ORC_ST_COST_NONPOSITIVE; stopped_by_rule = 1; break; }
            double theta_new = (1.0 + Phi + delta) / den;
            double margin = fabs(theta_new - theta_prev) / theta_prev;
            if (!(flags & ORC_FLAG_FIXED_BUDGET) && theta_new <= theta_prev) {
                stop_margin = margin; stopped_by_rule = 1; break;
            }
            if (margin < min_margin) min_margin = margin;
            H[best] = H[--hn];
            n += 1;
            node[n] = s;
            Phi += delta;
            theta_prev = theta_new;
            if (pop_gap) pop_gap[(size_t)b * R + n] = (runner == -INFINITY) ? 1.0 : 1.0 - exp(runner - s.sigma);
            if (theta_curve) theta_curve[(size_t)b * R + n] = theta_new;
            if (s.rank + 1 <= k_eff[s.depth]) {                 /* next sibling */
                cand_t c = s;
                c.rank = s.rank + 1;
                c.token = tk_tok[(s.depth - 1) * K + (c.rank - 1)];
                double A_parent = (s.parent == 0) ? 0.0 : node[s.parent].A;
                c.A = A_parent + tk_a[(s.depth - 1) * K + (c.rank - 1)];
                c.sigma = c.A - S[s.depth];
                H[hn++] = c;
            }
            if (s.depth < Le && k_eff[s.depth + 1] >= 1) {      /* first child */
                cand_t c;
                c.parent = n; c.depth = s.depth + 1; c.rank = 1;
                c.token = tk_tok[s.depth * K + 0];
                c.A = s.A + tk_a[s.depth * K + 0];
                c.sigma = c.A - S[c.depth];
                H[hn++] = c;
            }
        }
        if (ok && !stopped_by_rule) {
            if (hn == 0) st |= ORC_ST_FRONTIER_EXHAUSTED;
            else st |= ORC_ST_CAP_HIT;
        }
        if (stop_gap) stop_gap[b] = (stop_margin >= 0.0) ? stop_margin : min_margin;

        /* ---- O4: tree arrays and ancestor mask ---- */
        n_nodes[b] = n;
        if (phi_out) phi_out[b] = Phi;
        if (theta_out) theta_out[b] = theta_prev;
        for (int j = 0; j < R; ++j) {
            size_t o = (size_t)b * R + j;
            int32_t t = -1, p = -1, d = 0, pos = 0, rk = 0; double lpj = 0.0;
            if (j == 0) { t = bonus_token ? bonus_token[b] : -1; pos = ctx_len ? ctx_len[b] : 0; }
            else if (j <= n) {
                t = node[j].token; p = node[j].parent; d = node[j].depth; rk = node[j].rank;
                pos = (ctx_len ? ctx_len[b] : 0) + d; lpj = node[j].sigma;
            }
            if (token_ids) token_ids[o] = t;
            if (parent_idx) parent_idx[o] = p;
            if (depth) depth[o] = d;
            if (position_ids) position_ids[o] = pos;
            if (node_logprob) node_logprob[o] = lpj;
            if (node_rank) node_rank[o] = rk;
            if (pop_gap && (j == 0 || j > n)) pop_gap[o] = 1.0;
            if (theta_curve && j > n) theta_curve[o] = 0.0;
            if (mask_bits) memset(mask_bits + o * W, 0, sizeof(uint32_t) * (size_t)W);
            if (mask_dense) memset(mask_dense + o * R, 0, (size_t)R);
            if (j <= n) {                       /* self and every ancestor up to the root */
                int cur = j;
                for (;;) {
                    if (mask_bits) mask_bits[o * W + (cur >> 5)] |= (uint32_t)1 << (cur & 31);
                    if (mask_dense) mask_dense[o * R + cur] = 1;
                    if (cur == 0) break;
                    cur = node[cur].parent;
                }
            }
        }
        if (status) status[b] = st;
        free(tk_tok); free(tk_a); free(tk_lp); free(k_eff); free(lz); free(node); free(H); free(S);
    }
    return 0;
}

/* O5 for one row: argmax_v y_v, ties to the lowest v, NaN ordered as -Inf (Section 3.1). */
int32_t cadd_oracle_row_argmax(const void *row, int dtype, int64_t V)
{
    double best = -INFINITY;
    int64_t arg = 0;
    for (int64_t v = 0; v < V; ++v) {
        double y = logit_at(row, dtype, v);
        if (isnan(y)) continue;
        if (y > best) { best = y; arg = v; }
    }
    return (int32_t)arg;
}

/*
 * O5 + O6 for a batch (Sections 3.1 and 3.3): per-node argmax of the target logits, then the
 * walk from the root that follows, at each node, the child whose token equals that node's
 * argmax, until no child matches.  next_bonus is the argmax at the last accepted node.
 * rows_mode LIVE reads rows 0..n_nodes[b] (others get node_argmax -1); DENSE reads all R rows.
 */
int cadd_oracle_verify_tree(
    int batch, int64_t V, int R, int L, int dtype,
    const void *target_logits, int64_t stride_b, int64_t stride_row, int rows_mode,
    const int32_t *n_nodes, const int32_t *token_ids, const int32_t *parent_idx,
    int32_t *node_argmax, int32_t *accepted_len, int32_t *accepted_nodes, int32_t *next_bonus,
    int32_t *status)
{
    if (batch < 1 || V < 1 || R < 1 || L < 1) return -1;
    const size_t esz = (dtype == ORC_BF16) ? 2 : 4;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < batch; ++b) {
        int st = 0;
        int n = n_nodes[b];
        if (n < 0) { n = 0; st |= ORC_ST_BAD_N_NODES; }
        if (n > R - 1) { n = R - 1; st |= ORC_ST_BAD_N_NODES; }
        for (int j = 0; j < R; ++j) {
            size_t o = (size_t)b * R + j;
            if (j <= n || rows_mode == ORC_ROWS_DENSE) {
                const char *row = (const char *)target_logits +
                                  esz * (size_t)((int64_t)b * stride_b + (int64_t)j * stride_row);
                node_argmax[o] = cadd_oracle_row_argmax(row, dtype, V);
            } else node_argmax[o] = -1;
        }
        int cur = 0, alpha = 0;
        for (int i = 0; i < L; ++i) accepted_nodes[(size_t)b * L + i] = -1;
        for (;;) {
            int32_t g = node_argmax[(size_t)b * R + cur];
            int child = -1;
            for (int c = 1; c <= n; ++c)
                if (parent_idx[(size_t)b * R + c] == cur && token_ids[(size_t)b * R + c] == g) { child = c; break; }
            if (child < 0 || alpha >= L) break;
            accepted_nodes[(size_t)b * L + alpha] = child;
            alpha += 1;
            cur = child;
        }
        accepted_len[b] = alpha;
        next_bonus[b] = node_argmax[(size_t)b * R + cur];
        if (status) status[b] = st;
    }
    return 0;
}

/*
 * Target logits from the target's last hidden states and its output-projection weight (Section 3.1:
 * the target's prediction at tree node j is argmax_v of  y_{j,v} = sum_k h_{j,k} W_{v,k}):
 *   out[r*V + v] = sum_{k < hidden} h[r*stride_row + k] * w[v*stride_w + k]      (ascending k, fp64)
 * h and w are bf16, widened exactly; a product of two bf16 values is exact in double.
 */
int cadd_oracle_head_logits(int64_t rows, int64_t V, int hidden,
                            const void *h, int64_t stride_row, const void *w, int64_t stride_w,
                            double *out)
{
    if (rows < 1 || V < 1 || hidden < 1) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t v = 0; v < V; ++v) {
            double acc = 0.0;
            for (int k = 0; k < hidden; ++k)
                acc += logit_at(h, ORC_BF16, r * stride_row + k) * logit_at(w, ORC_BF16, v * stride_w + k);
            out[r * V + v] = acc;
        }
    }
    return 0;
}
