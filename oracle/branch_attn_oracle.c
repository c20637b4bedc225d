/*
 * CPU oracle for draft branch attention -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 restatement of what the method computes, used by the
 * tests, the smoke check and the benchmark's CPU-baseline leg.  The product
 * (the CUDA library) never links, imports or calls anything in this file, and
 * this file shares no code, table or helper with it.
 *
 * What is computed (paper Section 3.2, "Branch Attention under Context
 * Parallelism"):
 *   - every branch query attends to two key sets: the causal prefix of its
 *     packed main sequence up to its anchor, and the keys of its own branch
 *     under a branch-local mask (EAGLE-3 chain, DFlash block, or a tree);
 *   - a main query attends causally inside its own packed sequence;
 *   - O = softmax(scale * q.k over the visible set) V and the natural-log
 *     log-sum-exp l of the scaled scores;
 *   - partial results over disjoint key sets are combined with the paper's
 *     Eq. (lse-merge):  l = log(e^la + e^lb),  O = e^(la-l) Oa + e^(lb-l) Ob;
 *   - the backward pass of the same attention ("accumulates gradients
 *     locally" over key chunks, Section 3.2): dQ, dK, dV for the loss
 *     sum_r <dO_r, O_r>.
 *
 * There is no tiling, no bitmask, no prefix shortcut: visibility is a
 * predicate evaluated for every (query row, key row) pair, the score row of a
 * query is materialised over ALL keys with -inf where the predicate says no,
 * and each gradient is its defining sum.
 *
 * Parity pins (tests/test_oracle_*.py): hand-written visibility matrices,
 * closed forms (zero queries, index-coded values), a library causal attention
 * for the no-branch case, Eq. (lse-merge) over arbitrary key partitions,
 * shift invariances, central finite differences for every gradient, and GQA
 * versus explicitly repeated K/V heads.  The paper prints no numeric worked
 * example of O / l / gradients, so agreement with the paper's own numbers is
 * "parity unpinned"; the definition itself is pinned as listed.
 *
 * Row numbering: query rows and key rows are both "main rows [0, N) then
 * branch tokens [N, N + M)", branch tokens stored branch-major.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define KIND_CHAIN 0
#define KIND_BLOCK 1
#define KIND_TREE 2
#define PART_MAIN 1
#define PART_BRANCH 2

typedef struct {
    int64_t n_main;                /* N */
    int64_t n_branch;              /* M */
    int64_t num_seqs;              /* B */
    int64_t num_branches;          /* A */
    const int32_t *cu_seqlens;     /* [B+1] */
    const int32_t *anchor_idx;     /* [A] global packed main index */
    const int32_t *branch_offsets; /* [A+1] */
    const int32_t *parent;         /* [M] branch-local parent, -1 root (tree only) */
    int32_t kind;
    int32_t h_q, h_kv, d;
    double scale;
    /* key-set restriction (partial mode); full = parts 3, [0, N) */
    int32_t parts;
    int64_t kv_begin, kv_end;
} oracle_problem;

/* Which packed sequence holds main index i (scan of cu_seqlens). */
static int64_t seq_of(const oracle_problem *p, int64_t i)
{
    for (int64_t s = 0; s < p->num_seqs; ++s)
        if (i >= p->cu_seqlens[s] && i < p->cu_seqlens[s + 1])
            return s;
    return -1;
}

/* Which branch holds branch token t (scan of branch_offsets). */
static int64_t branch_of(const oracle_problem *p, int64_t t)
{
    for (int64_t b = 0; b < p->num_branches; ++b)
        if (t >= p->branch_offsets[b] && t < p->branch_offsets[b + 1])
            return b;
    return -1;
}

/* Branch-local mask: may token i of a branch see token u of the same branch? */
static int local_visible(const oracle_problem *p, int64_t branch_start, int64_t i, int64_t u)
{
    if (p->kind == KIND_CHAIN)
        return u <= i;
    if (p->kind == KIND_BLOCK)
        return 1;
    /* tree: u is i itself or one of its ancestors */
    for (int64_t a = i; a >= 0; a = p->parent[branch_start + a])
        if (a == u)
            return 1;
    return 0;
}

/*
 * The visibility predicate.  `q_seq`, `q_branch` describe the query row and
 * are looked up once per row by the callers (scans above); `key_seq` and
 * `key_branch` are per-key lookup tables filled by the same scans.
 */
typedef struct {
    int is_branch;
    int64_t seq;      /* sequence of the main query / of the anchor */
    int64_t last;     /* last visible main index: own index or the anchor */
    int64_t branch;   /* branch id (branch queries) */
    int64_t local;    /* index inside the branch */
} query_info;

static query_info describe_query(const oracle_problem *p, int64_t r)
{
    query_info qi;
    memset(&qi, 0, sizeof qi);
    if (r < p->n_main) {
        qi.is_branch = 0;
        qi.seq = seq_of(p, r);
        qi.last = r;
        qi.branch = -1;
    } else {
        int64_t t = r - p->n_main;
        qi.is_branch = 1;
        qi.branch = branch_of(p, t);
        qi.local = t - p->branch_offsets[qi.branch];
        qi.last = p->anchor_idx[qi.branch];
        qi.seq = seq_of(p, qi.last);
    }
    return qi;
}

static int visible(const oracle_problem *p, const query_info *qi, int64_t x,
                   const int64_t *key_seq, const int64_t *key_branch)
{
    if (x < p->n_main) {
        /* main key: causal prefix inside the query's (anchor's) sequence */
        if (!(p->parts & PART_MAIN))
            return 0;
        if (x < p->kv_begin || x >= p->kv_end)
            return 0;
        return key_seq[x] == qi->seq && x <= qi->last;
    }
    /* branch key: only for a branch query of the same branch */
    if (!qi->is_branch || !(p->parts & PART_BRANCH))
        return 0;
    int64_t u = x - p->n_main;
    if (key_branch[u] != qi->branch)
        return 0;
    int64_t start = p->branch_offsets[qi->branch];
    return local_visible(p, start, qi->local, u - start);
}

static void fill_key_tables(const oracle_problem *p, int64_t *key_seq, int64_t *key_branch)
{
    for (int64_t s = 0; s < p->num_seqs; ++s)
        for (int64_t i = p->cu_seqlens[s]; i < p->cu_seqlens[s + 1]; ++i)
            key_seq[i] = s;
    for (int64_t b = 0; b < p->num_branches; ++b)
        for (int64_t t = p->branch_offsets[b]; t < p->branch_offsets[b + 1]; ++t)
            key_branch[t] = b;
}

static double dot(const double *a, const double *b, int d)
{
    double s = 0.0;
    for (int c = 0; c < d; ++c)
        s += a[c] * b[c];
    return s;
}

/* Dense boolean visibility matrix [n_rows x (N+M)] for the listed query rows. */
int oracle_visibility(const oracle_problem *p, int64_t n_rows, const int64_t *rows, uint8_t *out)
{
    int64_t nk = p->n_main + p->n_branch;
    int64_t *key_seq = malloc(sizeof(int64_t) * (size_t)(p->n_main + 1));
    int64_t *key_branch = malloc(sizeof(int64_t) * (size_t)(p->n_branch + 1));
    if (!key_seq || !key_branch)
        return -1;
    fill_key_tables(p, key_seq, key_branch);
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t ri = 0; ri < n_rows; ++ri) {
        query_info qi = describe_query(p, rows[ri]);
        for (int64_t x = 0; x < nk; ++x)
            out[ri * nk + x] = (uint8_t)visible(p, &qi, x, key_seq, key_branch);
    }
    free(key_seq);
    free(key_branch);
    return 0;
}

/*
 * Forward for the listed query rows.
 *   q   [n_rows, h_q, d]   query vectors of those rows
 *   k,v [N+M, h_kv, d]
 *   o   [n_rows, h_q, d],  lse [n_rows, h_q]
 * A row whose visible set is empty (possible only with a key-set restriction)
 * gets lse = -inf and O = 0.
 */
int oracle_forward(const oracle_problem *p, int64_t n_rows, const int64_t *rows,
                   const double *q, const double *k, const double *v,
                   double *o, double *lse)
{
    const int64_t nk = p->n_main + p->n_branch;
    const int d = p->d, hq = p->h_q, hkv = p->h_kv, grp = hq / hkv;
    int64_t *key_seq = malloc(sizeof(int64_t) * (size_t)(p->n_main + 1));
    int64_t *key_branch = malloc(sizeof(int64_t) * (size_t)(p->n_branch + 1));
    if (!key_seq || !key_branch)
        return -1;
    fill_key_tables(p, key_seq, key_branch);
    int fail = 0;
#pragma omp parallel
    {
        uint8_t *vis = malloc((size_t)nk + 1);
        double *score = malloc(sizeof(double) * (size_t)(nk + 1));
        int64_t *idx = malloc(sizeof(int64_t) * (size_t)(nk + 1));
        if (!vis || !score || !idx) {
#pragma omp atomic write
            fail = 1;
        } else {
#pragma omp for schedule(dynamic, 4)
            for (int64_t ri = 0; ri < n_rows; ++ri) {
                query_info qi = describe_query(p, rows[ri]);
                /* predicate for every key; the score row starts fully masked */
                int64_t n_vis = 0;
                for (int64_t x = 0; x < nk; ++x) {
                    vis[x] = (uint8_t)visible(p, &qi, x, key_seq, key_branch);
                    score[x] = -INFINITY;
                    if (vis[x])
                        idx[n_vis++] = x;
                }
                for (int h = 0; h < hq; ++h) {
                    const int g = h / grp;
                    const double *qv = q + ((size_t)ri * hq + h) * d;
                    double *ov = o + ((size_t)ri * hq + h) * d;
                    /* scores where visible (all other entries stay -inf) */
                    double mx = -INFINITY;
                    for (int64_t j = 0; j < n_vis; ++j) {
                        const int64_t x = idx[j];
                        score[x] = p->scale * dot(qv, k + ((size_t)x * hkv + g) * d, d);
                        if (score[x] > mx)
                            mx = score[x];
                    }
                    for (int c = 0; c < d; ++c)
                        ov[c] = 0.0;
                    if (mx == -INFINITY) {
                        lse[(size_t)ri * hq + h] = -INFINITY;
                        continue;
                    }
                    /* exp(-inf) = 0: masked entries add nothing, so the sums
                       below run over the visible entries only */
                    double sum = 0.0;
                    for (int64_t j = 0; j < n_vis; ++j)
                        sum += exp(score[idx[j]] - mx);
                    const double l = mx + log(sum);
                    lse[(size_t)ri * hq + h] = l;
                    for (int64_t j = 0; j < n_vis; ++j) {
                        const int64_t x = idx[j];
                        const double pr = exp(score[x] - l);
                        const double *vv = v + ((size_t)x * hkv + g) * d;
                        for (int c = 0; c < d; ++c)
                            ov[c] += pr * vv[c];
                    }
                }
            }
        }
        free(vis);
        free(score);
        free(idx);
    }
    free(key_seq);
    free(key_branch);
    return fail ? -1 : 0;
}

/* Eq. (lse-merge), max-subtracted; both inputs empty (-inf) gives (0, -inf). */
int oracle_lse_merge(int64_t rows_heads, int d,
                     const double *o_a, const double *lse_a,
                     const double *o_b, const double *lse_b,
                     double *o_out, double *lse_out)
{
    for (int64_t i = 0; i < rows_heads; ++i) {
        const double la = lse_a[i], lb = lse_b[i];
        const double m = la > lb ? la : lb;
        if (m == -INFINITY) {
            lse_out[i] = -INFINITY;
            for (int c = 0; c < d; ++c)
                o_out[(size_t)i * d + c] = 0.0;
            continue;
        }
        const double l = m + log(exp(la - m) + exp(lb - m));
        const double wa = exp(la - l), wb = exp(lb - l);
        lse_out[i] = l;
        for (int c = 0; c < d; ++c)
            o_out[(size_t)i * d + c] = wa * o_a[(size_t)i * d + c] + wb * o_b[(size_t)i * d + c];
    }
    return 0;
}

/*
 * Backward for the loss  sum over the listed rows of <dO_r, O_r>.
 *   lse   [n_rows, h_q]  log-sum-exp over the row's COMPLETE visible set
 *   delta [n_rows, h_q]  <dO_r, O_r> with the COMPLETE output
 * (the caller gets both from oracle_forward with parts = 3 and the full key
 * range).  The key-set restriction in `p` selects which keys' terms are summed:
 * every gradient is additive over disjoint key chunks.
 *   dq [n_rows, h_q, d];  dk, dv [N+M, h_kv, d] (overwritten)
 * With p = exp(s - lse):  dP = <dO, v>,  dS = p (dP - delta),
 *   dQ_r = scale sum_x dS_rx k_x,  dK_x = scale sum_r dS_rx q_r,  dV_x = sum_r p_rx dO_r,
 * the K/V sums running over all listed rows and all query heads of the kv head.
 */
int oracle_backward(const oracle_problem *p, int64_t n_rows, const int64_t *rows,
                    const double *q, const double *k, const double *v,
                    const double *d_o, const double *lse, const double *delta,
                    double *dq, double *dk, double *dv)
{
    const int64_t nk = p->n_main + p->n_branch;
    const int d = p->d, hq = p->h_q, hkv = p->h_kv, grp = hq / hkv;
    int64_t *key_seq = malloc(sizeof(int64_t) * (size_t)(p->n_main + 1));
    int64_t *key_branch = malloc(sizeof(int64_t) * (size_t)(p->n_branch + 1));
    query_info *qis = malloc(sizeof(query_info) * (size_t)(n_rows + 1));
    if (!key_seq || !key_branch || !qis)
        return -1;
    fill_key_tables(p, key_seq, key_branch);
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t ri = 0; ri < n_rows; ++ri)
        qis[ri] = describe_query(p, rows[ri]);

    /* dQ: one query row at a time */
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t ri = 0; ri < n_rows; ++ri) {
        for (int h = 0; h < hq; ++h) {
            double *g_out = dq + ((size_t)ri * hq + h) * d;
            for (int c = 0; c < d; ++c)
                g_out[c] = 0.0;
        }
        for (int64_t x = 0; x < nk; ++x) {
            if (!visible(p, &qis[ri], x, key_seq, key_branch))
                continue;
            for (int h = 0; h < hq; ++h) {
                const int g = h / grp;
                const size_t rh = (size_t)ri * hq + h;
                const double *kv_ = k + ((size_t)x * hkv + g) * d;
                const double *vv = v + ((size_t)x * hkv + g) * d;
                const double s = p->scale * dot(q + rh * d, kv_, d);
                const double pr = exp(s - lse[rh]);
                const double dp = dot(d_o + rh * d, vv, d);
                const double ds = pr * (dp - delta[rh]);
                double *g_out = dq + rh * d;
                for (int c = 0; c < d; ++c)
                    g_out[c] += p->scale * ds * kv_[c];
            }
        }
    }

    /* dK, dV: one key row at a time */
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t x = 0; x < nk; ++x) {
        for (int g = 0; g < hkv; ++g) {
            double *gk = dk + ((size_t)x * hkv + g) * d;
            double *gv = dv + ((size_t)x * hkv + g) * d;
            for (int c = 0; c < d; ++c) {
                gk[c] = 0.0;
                gv[c] = 0.0;
            }
        }
        for (int64_t ri = 0; ri < n_rows; ++ri) {
            if (!visible(p, &qis[ri], x, key_seq, key_branch))
                continue;
            for (int h = 0; h < hq; ++h) {
                const int g = h / grp;
                const size_t rh = (size_t)ri * hq + h;
                const double *kv_ = k + ((size_t)x * hkv + g) * d;
                const double *vv = v + ((size_t)x * hkv + g) * d;
                const double *qv = q + rh * d;
                const double *gov = d_o + rh * d;
                const double s = p->scale * dot(qv, kv_, d);
                const double pr = exp(s - lse[rh]);
                const double dp = dot(gov, vv, d);
                const double ds = pr * (dp - delta[rh]);
                double *gk = dk + ((size_t)x * hkv + g) * d;
                double *gv = dv + ((size_t)x * hkv + g) * d;
                for (int c = 0; c < d; ++c) {
                    gk[c] += p->scale * ds * qv[c];
                    gv[c] += pr * gov[c];
                }
            }
        }
    }
    free(key_seq);
    free(key_branch);
    free(qis);
    return 0;
}
