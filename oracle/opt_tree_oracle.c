/*
 * OPT-Tree CPU oracle — TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, single-threaded fp64 implementation of the paper's draft-tree
 * construction (Algorithm 1, Eq. 2, Eq. 3), tree packing / attention mask
 * (Algorithm 2, second line) and greedy verification (Preliminaries, greedy
 * sampling paragraph; Algorithm 2, Verify).  It follows the algorithm's steps in
 * the paper's order, with no blocking, fusion or reordering.  It shares no code,
 * header, table or helper with the CUDA library and must never be called from it;
 * only tests, the smoke check and the benchmark's cpu_baseline leg use it.
 *
 * Pinned by tests that do not use this file's own formulas: NumPy fp64 softmax /
 * sort on the same bytes, closed forms on constant and one-hot rows, exhaustive
 * search over all parent-closed node subsets on tiny vocabularies, a hand-computed
 * example of Eq. 2 / Eq. 3, Theorem 1, Theorem 2, the closure proof, and a
 * path-enumeration definition of the greedy acceptance length.  The two outputs that the
 * parity tests use to tell a near-tie from an error, min_gap and stop_margin, are pinned by
 * the same hand example (every boundary worked out by hand), by constructed ties and gaps,
 * and by a NumPy replay of the selections on small random tables.
 * Not pinned ("parity unpinned"): the value E(A) = 2.07 of the paper's Figure 2 and the
 * mean acceptance lengths of Tables 1-3, which need the missing figure / real models.
 *
 * Readings of points the paper leaves open (each is also applied by the CUDA library,
 * written independently):
 *   - the root has path value 1 in products and is never a node of the output (the
 *     paper gives it +infinity, meaning "always kept", and does not count it);
 *   - a node expands into at most k children (the k highest draft probabilities), ranked
 *     (logit descending, token id ascending);
 *   - a layer keeps the min(n, #candidates) candidates ranked (path value descending,
 *     candidate index ascending), candidate index = frontier slot * k + sibling rank, and
 *     stores them in candidate-index order;
 *   - E_sub(T, n) is the sum of the n largest path values in T (all of T if |T| < n),
 *     ranked (path value descending, depth ascending, candidate index ascending);
 *   - the loop test of Algorithm 1 is evaluated after each layer exists: growth stops when
 *     depth >= min(max_depth, n) or when not (E_sub - E > delta); the last drafted layer
 *     stays in T;
 *   - packed node order: depth ascending, then parent's packed index ascending, then
 *     sibling rank ascending;
 *   - argmax ties in a target row go to the lowest token id;
 *   - acceptance length A = matched draft nodes + 1 (the bonus token).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Model abstraction: "next-token logits after this path".                   */
/* path[0..depth-1] are the draft tokens from the root's child down to the   */
/* node being expanded; depth 0 means the root itself.                       */
/* key() returns an id such that equal ids imply equal logits (for the       */
/* optional memo), or -1 for "do not memoise".                               */
/* ------------------------------------------------------------------------- */
typedef void (*ot_logits_fn)(void *user, int32_t root_token, const int32_t *path, int32_t depth, double *logits);
typedef int64_t (*ot_key_fn)(void *user, int32_t root_token, const int32_t *path, int32_t depth);

typedef struct {
    ot_logits_fn logits;
    ot_key_fn key;      /* may be NULL */
    void *user;
} ot_model;

/* Table model: bf16 table [H][V]; the node with token t at depth d reads row (t*31+d) mod H. */
typedef struct {
    const uint16_t *table;
    int32_t H, V;
} ot_table_model;

static double bf16_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static int64_t table_row(const ot_table_model *tm, int32_t root_token, const int32_t *path, int32_t depth)
{
    int64_t t = depth == 0 ? root_token : path[depth - 1];
    return (t * 31 + depth) % tm->H;
}

void ot_table_logits(void *user, int32_t root_token, const int32_t *path, int32_t depth, double *logits)
{
    const ot_table_model *tm = (const ot_table_model *)user;
    const uint16_t *row = tm->table + table_row(tm, root_token, path, depth) * (int64_t)tm->V;
    for (int32_t v = 0; v < tm->V; ++v) logits[v] = bf16_to_double(row[v]);
}

int64_t ot_table_key(void *user, int32_t root_token, const int32_t *path, int32_t depth)
{
    return table_row((const ot_table_model *)user, root_token, path, depth);
}

/* ------------------------------------------------------------------------- */
/* Row step: softmax normaliser and the k most probable tokens.              */
/* Children rule (Section 3, sentence after Eq. 2): a node's children are    */
/* the k tokens of highest draft probability.                                */
/* ------------------------------------------------------------------------- */
typedef struct { double logit; int32_t token; } ot_lt;

static int cmp_logit_desc_token_asc(const void *a, const void *b)
{
    const ot_lt *x = (const ot_lt *)a, *y = (const ot_lt *)b;
    if (x->logit > y->logit) return -1;
    if (x->logit < y->logit) return 1;
    return (x->token > y->token) - (x->token < y->token);
}

/* logits[V] -> kk = min(k, V) tokens and probabilities; returns kk.
 * m_out / S_out: row maximum and sum_v exp(l_v - m). */
int32_t ot_row_softmax_topk(const double *logits, int32_t V, int32_t k,
                            int32_t *tok_out, double *p_out, double *m_out, double *S_out)
{
    double m = logits[0];
    for (int32_t v = 1; v < V; ++v) if (logits[v] > m) m = logits[v];
    double S = 0.0;
    for (int32_t v = 0; v < V; ++v) S += exp(logits[v] - m);
    /* k best (logit descending, token id ascending) by insertion into a sorted list of k. */
    int32_t kk = k < V ? k : V;
    ot_lt *best = (ot_lt *)malloc((size_t)kk * sizeof *best);
    int32_t nb = 0;
    for (int32_t v = 0; v < V; ++v) {
        ot_lt e = { logits[v], v };
        if (nb == kk && cmp_logit_desc_token_asc(&e, &best[nb - 1]) >= 0) continue;
        int32_t pos = nb < kk ? nb++ : kk - 1;
        while (pos > 0 && cmp_logit_desc_token_asc(&e, &best[pos - 1]) < 0) { best[pos] = best[pos - 1]; --pos; }
        best[pos] = e;
    }
    for (int32_t j = 0; j < kk; ++j) {
        tok_out[j] = best[j].token;
        p_out[j] = exp(best[j].logit - m) / S;
    }
    free(best);
    if (m_out) *m_out = m;
    if (S_out) *S_out = S;
    return kk;
}

/* Optional memo of row results keyed by ot_key_fn (parity runs only; the timed
 * oracle runs without it). Open addressing, fixed capacity. */
typedef struct {
    int64_t cap, k;
    int64_t *keys;     /* -1 = empty */
    int32_t *kk;
    int32_t *tok;      /* [cap][k] */
    double *p;         /* [cap][k] */
} ot_memo;

ot_memo *ot_memo_create(int64_t cap, int32_t k)
{
    ot_memo *mm = (ot_memo *)calloc(1, sizeof *mm);
    mm->cap = cap; mm->k = k;
    mm->keys = (int64_t *)malloc((size_t)cap * sizeof(int64_t));
    for (int64_t i = 0; i < cap; ++i) mm->keys[i] = -1;
    mm->kk = (int32_t *)calloc((size_t)cap, sizeof(int32_t));
    mm->tok = (int32_t *)calloc((size_t)(cap * k), sizeof(int32_t));
    mm->p = (double *)calloc((size_t)(cap * k), sizeof(double));
    return mm;
}

void ot_memo_destroy(ot_memo *mm)
{
    if (!mm) return;
    free(mm->keys); free(mm->kk); free(mm->tok); free(mm->p); free(mm);
}

static int64_t memo_slot(const ot_memo *mm, int64_t key)
{
    int64_t i = (int64_t)(((uint64_t)key * 0x9E3779B97F4A7C15ull) % (uint64_t)mm->cap);
    for (int64_t probe = 0; probe < mm->cap; ++probe) {
        if (mm->keys[i] == key || mm->keys[i] == -1) return i;
        i = (i + 1) % mm->cap;
    }
    return -1;
}

static int32_t expand_node(const ot_model *model, ot_memo *memo, int32_t V, int32_t k,
                           int32_t root_token, const int32_t *path, int32_t depth,
                           double *scratch, int32_t *tok_out, double *p_out)
{
    int64_t key = (memo && model->key) ? model->key(model->user, root_token, path, depth) : -1;
    int64_t slot = key >= 0 ? memo_slot(memo, key) : -1;
    if (slot >= 0 && memo->keys[slot] == key) {
        int32_t kk = memo->kk[slot];
        memcpy(tok_out, memo->tok + slot * memo->k, (size_t)kk * sizeof(int32_t));
        memcpy(p_out, memo->p + slot * memo->k, (size_t)kk * sizeof(double));
        return kk;
    }
    model->logits(model->user, root_token, path, depth, scratch);
    int32_t kk = ot_row_softmax_topk(scratch, V, k, tok_out, p_out, NULL, NULL);
    if (slot >= 0) {
        memo->keys[slot] = key;
        memo->kk[slot] = kk;
        memcpy(memo->tok + slot * memo->k, tok_out, (size_t)kk * sizeof(int32_t));
        memcpy(memo->p + slot * memo->k, p_out, (size_t)kk * sizeof(double));
    }
    return kk;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1: construct an OPT-Tree.                                       */
/* ------------------------------------------------------------------------- */
typedef struct {
    int32_t token;
    int32_t parent;     /* index into T, -1 = child of the root */
    int32_t depth;      /* 1-based */
    int32_t rank;       /* sibling rank among the parent's children */
    int64_t cidx;       /* candidate index within its layer */
    double phat;        /* Eq. 2 */
} ot_node;

typedef struct { double phat; int32_t depth; int64_t cidx; int32_t id; } ot_rank;

static int cmp_phat_desc_cidx_asc(const void *a, const void *b)
{
    const ot_node *x = (const ot_node *)a, *y = (const ot_node *)b;
    if (x->phat > y->phat) return -1;
    if (x->phat < y->phat) return 1;
    return (x->cidx > y->cidx) - (x->cidx < y->cidx);
}

static int cmp_cidx_asc(const void *a, const void *b)
{
    const ot_node *x = (const ot_node *)a, *y = (const ot_node *)b;
    return (x->cidx > y->cidx) - (x->cidx < y->cidx);
}

static int cmp_rank_phat_depth_cidx(const void *a, const void *b)
{
    const ot_rank *x = (const ot_rank *)a, *y = (const ot_rank *)b;
    if (x->phat > y->phat) return -1;
    if (x->phat < y->phat) return 1;
    if (x->depth != y->depth) return x->depth < y->depth ? -1 : 1;
    return (x->cidx > y->cidx) - (x->cidx < y->cidx);
}

typedef struct { int32_t depth, pcanon, rank, id; } ot_canon;

static int cmp_canon(const void *a, const void *b)
{
    const ot_canon *x = (const ot_canon *)a, *y = (const ot_canon *)b;
    if (x->depth != y->depth) return x->depth < y->depth ? -1 : 1;
    if (x->pcanon != y->pcanon) return x->pcanon < y->pcanon ? -1 : 1;
    return (x->rank > y->rank) - (x->rank < y->rank);
}

static double rel_gap(double kept, double dropped)
{
    /* relative distance between the last kept and the first dropped value.  Path values are never
     * negative and dropped <= kept, so kept == 0 means both are zero: an exact tie, gap 0. */
    double d = kept - dropped;
    if (kept <= 0.0) return 0.0;
    return d / kept;
}

/*
 * Builds one tree.
 *   force_depth > 0: ignore the threshold test and draft exactly that many layers
 *                    (still capped by min(max_depth, n)); used by the harness to take
 *                    "the other decision" when |gain - delta| is within rounding.
 * Outputs (arrays sized n unless noted; unused tail slots: token -1, parent -1, depth 0, phat 0):
 *   token, parent, depth, phat   packed tree
 *   n_sel, depth_reached         nodes kept; layers drafted
 *   expected_len                 E(A) = sum of kept path values (Eq. 3)
 *   esub_trace[max_depth]        E_sub(T, n) after each drafted layer (0 beyond depth_reached)
 *   min_gap                      smallest relative gap between a kept and a dropped value at
 *                                any layer selection or E_sub / final selection boundary
 *   stop_margin                  smallest |gain - delta| over the threshold tests evaluated
 * Returns 0, or -1 on bad arguments.
 */
/* prune != 0: the variant that drafts, of every new layer, only the nodes that are among the n
 * largest of T at that moment.  By Theorem 1 a node's descendants have smaller path values than the
 * node, so the descendants of a node outside the n largest can never be among the n largest later:
 * T_opt, E_sub after every layer and the loop test come out the same, with fewer draft rows read
 * (rows_read counts them).  Once no node of the newest layer is among the n largest, further layers
 * change nothing; the loop then only replays its test, as the full version would. */
static int build_impl(const ot_model *model, ot_memo *memo, int32_t root_token,
             int32_t V, int32_t n, int32_t k, int32_t max_depth, double delta, int32_t force_depth,
             int32_t *token, int32_t *parent, int32_t *depth, double *phat,
             int32_t *n_sel, int32_t *depth_reached, double *expected_len,
             double *esub_trace, double *min_gap, double *stop_margin, int32_t prune, int64_t *rows_read)
{
    if (V < 1 || n < 1 || k < 1 || max_depth < 1) return -1;
    int32_t D = max_depth < n ? max_depth : n;       /* Algorithm 1 loop: depth of tree < n */
    int32_t kk_max = k < V ? k : V;
    ot_node *T = (ot_node *)malloc((size_t)D * n * sizeof *T);
    int32_t nT = 0;
    ot_node *cands = (ot_node *)malloc((size_t)n * kk_max * sizeof *cands);
    ot_rank *R = (ot_rank *)malloc((size_t)D * n * sizeof *R);
    double *scratch = (double *)malloc((size_t)V * sizeof(double));
    int32_t *ctok = (int32_t *)malloc((size_t)kk_max * sizeof(int32_t));
    double *cp = (double *)malloc((size_t)kk_max * sizeof(double));
    int32_t *path = (int32_t *)malloc((size_t)(D + 1) * sizeof(int32_t));

    double E = 0.0, Esub = 0.0, gapmin = INFINITY, margin = INFINITY;
    int32_t *front = (int32_t *)malloc((size_t)n * sizeof(int32_t));   /* nodes of T to draft from; -1 = the root */
    int32_t nfront = 1;
    front[0] = -1;
    int32_t d = 0, nR = 0;
    int64_t rows = 0;
    for (int32_t i = 0; i < max_depth; ++i) esub_trace[i] = 0.0;

    for (;;) {
        d += 1;
        /* Draft step: next-token distribution of every node to draft from. */
        int32_t ncand = 0;
        rows += nfront;
        for (int32_t s = 0; s < nfront; ++s) {
            int32_t f = front[s];
            double fphat = 1.0;                       /* root: factor 1 */
            int32_t fdepth = 0;
            if (f >= 0) {
                fphat = T[f].phat;
                fdepth = T[f].depth;
                for (int32_t a = f, i = fdepth - 1; a >= 0; a = T[a].parent, --i) path[i] = T[a].token;
            }
            int32_t kk = expand_node(model, memo, V, k, root_token, path, fdepth, scratch, ctok, cp);
            for (int32_t j = 0; j < kk; ++j) {
                ot_node *c = &cands[ncand++];
                c->token = ctok[j];
                c->parent = f;
                c->depth = d;
                c->rank = j;
                c->cidx = (int64_t)s * k + j;
                c->phat = fphat * cp[j];              /* Eq. 2 */
            }
        }
        /* Next layer: the n candidates of largest path value. */
        qsort(cands, (size_t)ncand, sizeof *cands, cmp_phat_desc_cidx_asc);
        int32_t nl = ncand < n ? ncand : n;
        if (ncand > nl) {
            double g = rel_gap(cands[nl - 1].phat, cands[nl].phat);
            if (g < gapmin) gapmin = g;
        }
        qsort(cands, (size_t)nl, sizeof *cands, cmp_cidx_asc);
        int32_t layer_begin = nT;
        for (int32_t i = 0; i < nl; ++i) T[nT++] = cands[i];

        /* E_sub(T, n): the n largest path values of T (closure proof after Algorithm 1). */
        for (int32_t i = 0; i < nT; ++i) {
            R[i].phat = T[i].phat; R[i].depth = T[i].depth; R[i].cidx = T[i].cidx; R[i].id = i;
        }
        qsort(R, (size_t)nT, sizeof *R, cmp_rank_phat_depth_cidx);
        nR = nT < n ? nT : n;
        Esub = 0.0;
        for (int32_t i = 0; i < nR; ++i) Esub += R[i].phat;
        if (nT > nR) {
            double g = rel_gap(R[nR - 1].phat, R[nR].phat);
            if (g < gapmin) gapmin = g;
        }
        esub_trace[d - 1] = Esub;

        /* Who is drafted from next: the whole new layer, or (prune) its members among the n largest. */
        nfront = 0;
        for (int32_t i = layer_begin; i < nT; ++i) {
            int32_t in_top = 0;
            if (prune) {
                for (int32_t q = 0; q < nR; ++q) if (R[q].id == i) { in_top = 1; break; }
            }
            if (!prune || in_top) front[nfront++] = i;
        }

        /* Loop test of Algorithm 1. */
        if (d >= D) break;
        if (force_depth > 0) {
            if (d >= force_depth) break;
        } else {
            double gain = Esub - E;
            double mg = fabs(gain - delta);
            if (mg < margin) margin = mg;
            if (!(gain > delta)) break;
        }
        E = Esub;
    }

    /* T_opt: the n nodes of largest path value (last line of Algorithm 1) = R[0..nR). */
    ot_canon *C = (ot_canon *)malloc((size_t)(nR > 0 ? nR : 1) * sizeof *C);
    int32_t *canon_of = (int32_t *)malloc((size_t)nT * sizeof(int32_t));
    for (int32_t i = 0; i < nT; ++i) canon_of[i] = -2;       /* -2 = not selected */
    for (int32_t i = 0; i < nR; ++i) canon_of[R[i].id] = -3; /* -3 = selected, index pending */
    int32_t done = 0;
    for (int32_t dd = 1; dd <= d; ++dd) {
        int32_t m0 = done, cnt = 0;
        for (int32_t i = 0; i < nT; ++i) {
            if (canon_of[i] != -3 || T[i].depth != dd) continue;
            ot_canon *c = &C[m0 + cnt++];
            c->depth = dd;
            c->pcanon = T[i].parent < 0 ? -1 : canon_of[T[i].parent];
            c->rank = T[i].rank;
            c->id = i;
        }
        qsort(C + m0, (size_t)cnt, sizeof *C, cmp_canon);
        for (int32_t i = 0; i < cnt; ++i) canon_of[C[m0 + i].id] = m0 + i;
        done += cnt;
    }
    double EA = 0.0;
    for (int32_t i = 0; i < n; ++i) { token[i] = -1; parent[i] = -1; depth[i] = 0; phat[i] = 0.0; }
    for (int32_t i = 0; i < nR; ++i) {
        const ot_node *nd = &T[C[i].id];
        token[i] = nd->token;
        parent[i] = nd->parent < 0 ? -1 : canon_of[nd->parent];
        depth[i] = nd->depth;
        phat[i] = nd->phat;
    }
    for (int32_t i = 0; i < nR; ++i) EA += R[i].phat;        /* Eq. 3, summed in value order like E_sub */
    *n_sel = nR;
    *depth_reached = d;
    *expected_len = EA;
    if (min_gap) *min_gap = gapmin;
    if (stop_margin) *stop_margin = margin;
    if (rows_read) *rows_read = rows;

    free(C); free(canon_of); free(T); free(cands); free(R); free(scratch); free(ctok); free(cp); free(path); free(front);
    return 0;
}

int ot_build(const ot_model *model, ot_memo *memo, int32_t root_token,
             int32_t V, int32_t n, int32_t k, int32_t max_depth, double delta, int32_t force_depth,
             int32_t *token, int32_t *parent, int32_t *depth, double *phat,
             int32_t *n_sel, int32_t *depth_reached, double *expected_len,
             double *esub_trace, double *min_gap, double *stop_margin)
{
    return build_impl(model, memo, root_token, V, n, k, max_depth, delta, force_depth, token, parent, depth, phat,
                      n_sel, depth_reached, expected_len, esub_trace, min_gap, stop_margin, 0, NULL);
}

/* The pruned variant over the table model for a batch (tree outputs and the number of draft rows
 * each sequence read; with prune == 0 the full version, for comparison of the row counts). */
int ot_table_build_rows(const uint16_t *draft, int32_t H, int32_t V, const int32_t *root_token, int32_t batch,
                        int32_t n, int32_t k, int32_t max_depth, double delta, int32_t prune,
                        int32_t *token, int32_t *parent, int32_t *depth, double *phat,
                        int32_t *n_sel, int32_t *depth_reached, double *expected_len, double *esub_trace,
                        int64_t *rows_read)
{
    ot_table_model dm = { draft, H, V };
    ot_model dmodel = { ot_table_logits, ot_table_key, &dm };
    for (int32_t b = 0; b < batch; ++b) {
        int rc = build_impl(&dmodel, NULL, root_token[b], V, n, k, max_depth, delta, 0,
                            token + (size_t)b * n, parent + (size_t)b * n, depth + (size_t)b * n, phat + (size_t)b * n,
                            n_sel + b, depth_reached + b, expected_len + b, esub_trace + (size_t)b * max_depth,
                            NULL, NULL, prune, rows_read + b);
        if (rc) return rc;
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Tree attention mask and position ids (Algorithm 2, second line: the mask  */
/* of T_opt; Figure 1: nodes of a layer share the position index).           */
/* Row i has bit j set iff node j is i or an ancestor of i; W = ceil(n/64)   */
/* words per row, bit j in word j/64 at position j%64.                       */
/* ------------------------------------------------------------------------- */
void ot_mask(const int32_t *parent, const int32_t *depth, int32_t n_sel, int32_t n, int32_t base_pos,
             uint64_t *mask, int32_t *position_ids)
{
    int32_t W = (n + 63) / 64;
    memset(mask, 0, (size_t)n * W * sizeof(uint64_t));
    for (int32_t i = 0; i < n; ++i) position_ids[i] = 0;
    for (int32_t i = 0; i < n_sel; ++i) {
        if (parent[i] >= 0)
            for (int32_t w = 0; w < W; ++w) mask[(size_t)i * W + w] = mask[(size_t)parent[i] * W + w];
        mask[(size_t)i * W + i / 64] |= (uint64_t)1 << (i % 64);
        position_ids[i] = base_pos + depth[i];
    }
}

/* ------------------------------------------------------------------------- */
/* Bookkeeping around the target forward of Algorithm 2 (the step after the  */
/* hot path).  The paper says only that the tree attention mask is computed  */
/* and that both models keep key and value caches (Section 3, after          */
/* Algorithm 2); the formats below are this build's reading:                 */
/*  - the target sees n+1 tokens per step: position 0 is the root (the last  */
/*    accepted token), position i+1 is packed node i;                        */
/*  - dense mask [n+1][n+1]: entry (r, c) is 1 iff token r may attend to     */
/*    token c inside the step: c == r, or r is a kept node and c is the root */
/*    or one of r's ancestors.  Unused positions attend to themselves only;  */
/*  - after Verify the keys and values of the root and of the A-1 matched    */
/*    nodes stay in the cache, in path order: gather[0] = 0, gather[j] =     */
/*    1 + accept_nodes[j-1]; the rest of gather is -1; A entries are kept    */
/*    (the A-th accepted token is the next step's root and has no entry yet).*/
/* ------------------------------------------------------------------------- */
void ot_dense_mask(const int32_t *parent, int32_t n_sel, int32_t n, uint8_t *dense)
{
    const int32_t S = n + 1;
    memset(dense, 0, (size_t)S * S);
    for (int32_t r = 0; r < S; ++r) dense[(size_t)r * S + r] = 1;
    for (int32_t i = 0; i < n_sel; ++i) {
        dense[(size_t)(i + 1) * S + 0] = 1;
        for (int32_t a = parent[i]; a >= 0; a = parent[a]) dense[(size_t)(i + 1) * S + (a + 1)] = 1;
    }
}

int32_t ot_kv_keep(const int32_t *accept_nodes, int32_t accept_len, int32_t max_depth, int32_t *gather)
{
    for (int32_t j = 0; j <= max_depth; ++j) gather[j] = -1;
    gather[0] = 0;
    for (int32_t j = 1; j < accept_len; ++j) gather[j] = 1 + accept_nodes[j - 1];
    return accept_len;
}

/* ------------------------------------------------------------------------- */
/* Greedy verification: the target's most probable next token after the root */
/* and after every tree node; accept the longest root branch that follows    */
/* them, plus the next token after the last hit.                             */
/* ------------------------------------------------------------------------- */
static int32_t argmax_lowest(const double *x, int32_t V)
{
    int32_t best = 0;
    for (int32_t v = 1; v < V; ++v) if (x[v] > x[best]) best = v;
    return best;
}

/*
 * accept_tokens[max_depth+1], accept_nodes[max_depth] (tail filled with -1).
 * Returns the acceptance length A >= 1.
 */
int32_t ot_verify(const ot_model *target, int32_t root_token, int32_t V, int32_t n_sel, int32_t max_depth,
                  const int32_t *token, const int32_t *parent, const int32_t *depth,
                  int32_t *accept_tokens, int32_t *accept_nodes, int32_t *next_root)
{
    double *scratch = (double *)malloc((size_t)V * sizeof(double));
    int32_t *path = (int32_t *)malloc((size_t)(max_depth + 1) * sizeof(int32_t));
    for (int32_t i = 0; i <= max_depth; ++i) accept_tokens[i] = -1;
    for (int32_t i = 0; i < max_depth; ++i) accept_nodes[i] = -1;
    int32_t cur = -1, A = 0, curdepth = 0;
    for (;;) {
        if (cur >= 0)
            for (int32_t a = cur, i = curdepth - 1; a >= 0; a = parent[a], --i) path[i] = token[a];
        target->logits(target->user, root_token, path, curdepth, scratch);
        int32_t y = argmax_lowest(scratch, V);
        accept_tokens[A++] = y;
        int32_t hit = -1;
        for (int32_t i = 0; i < n_sel; ++i)
            if (parent[i] == cur && token[i] == y) { hit = i; break; }
        if (hit < 0) break;
        accept_nodes[A - 1] = hit;
        cur = hit;
        curdepth = depth[hit];
    }
    *next_root = accept_tokens[A - 1];
    free(scratch); free(path);
    return A;
}

/* ------------------------------------------------------------------------- */
/* Verification with sampling (temperature > 0).  The paper evaluates it      */
/* (the table with temperature 1) but says only that the acceptable tokens   */
/* change; the rule here is this build's reading: at every visited position  */
/* the next token is SAMPLED from the target's distribution at temperature   */
/* tau, softmax(x / tau), and accepted as the walk's next token; the walk    */
/* goes on while the current node has a child that carries the sampled       */
/* token.  The emitted tokens are then exactly a sample of the target model, */
/* and A = matched nodes + 1 as in the greedy walk.                          */
/* Randomness: one uniform per (sequence, step position), from the counter-  */
/* based generator Philox4x32-10 (Salmon et al., "Parallel random numbers:   */
/* as easy as 1, 2, 3", 2011): key = the 64-bit seed, counter = (position,   */
/* sequence, decoding step low, decoding step high); position 0 is the root, */
/* position i+1 packed node i.  u = (53 top bits of the first two outputs) * */
/* 2^-53.  Sampling is by inverse CDF in token order: with e_v = exp((x_v -  */
/* max x) / tau) and S their sum in token order, the token is the first v    */
/* whose running sum exceeds u * S (the last token with e_v > 0 if rounding  */
/* leaves none).                                                             */
/* ------------------------------------------------------------------------- */
static void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4])
{
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

void ot_philox4x32_10(const uint32_t *ctr, const uint32_t *key, uint32_t *out) { philox4x32_10(ctr, key, out); }

double ot_uniform(uint64_t seed, uint64_t step, int32_t sequence, int32_t position)
{
    uint32_t ctr[4] = { (uint32_t)position, (uint32_t)sequence, (uint32_t)step, (uint32_t)(step >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) }, o[4];
    philox4x32_10(ctr, key, o);
    uint64_t bits = (((uint64_t)o[1] << 32) | o[0]) >> 11;
    return (double)bits * (1.0 / 9007199254740992.0);
}

/* One sample; margin (if given) = distance of u*S from the nearer of the two running sums that
 * bracket the chosen token, relative to S: a summation in another order may choose a neighbour
 * only if this is at rounding level. */
int32_t ot_sample_token(const double *x, int32_t V, double tau, double u, double *margin)
{
    double m = -INFINITY, S = 0.0;
    for (int32_t v = 0; v < V; ++v) if (x[v] > m) m = x[v];
    for (int32_t v = 0; v < V; ++v) S += exp((x[v] - m) / tau);
    const double t = u * S;
    double run = 0.0, before = 0.0;
    int32_t last = 0, y = -1;
    for (int32_t v = 0; v < V; ++v) {
        double e = exp((x[v] - m) / tau);
        if (e > 0.0) last = v;
        before = run;
        run += e;
        if (run > t) { y = v; break; }
    }
    if (y < 0) { y = last; before = run; }
    if (margin) {
        double a = fabs(t - before), b = fabs(run - t);
        *margin = (a < b ? a : b) / S;
    }
    return y;
}

int32_t ot_verify_sampled(const ot_model *target, int32_t root_token, int32_t V, int32_t n_sel, int32_t max_depth,
                          const int32_t *token, const int32_t *parent, const int32_t *depth,
                          double tau, uint64_t seed, uint64_t step, int32_t sequence,
                          int32_t *accept_tokens, int32_t *accept_nodes, int32_t *next_root, double *min_margin)
{
    double *scratch = (double *)malloc((size_t)V * sizeof(double));
    int32_t *path = (int32_t *)malloc((size_t)(max_depth + 1) * sizeof(int32_t));
    for (int32_t i = 0; i <= max_depth; ++i) accept_tokens[i] = -1;
    for (int32_t i = 0; i < max_depth; ++i) accept_nodes[i] = -1;
    int32_t cur = -1, A = 0, curdepth = 0;
    double mm = INFINITY;
    for (;;) {
        if (cur >= 0)
            for (int32_t a = cur, i = curdepth - 1; a >= 0; a = parent[a], --i) path[i] = token[a];
        target->logits(target->user, root_token, path, curdepth, scratch);
        double mg;
        int32_t y = ot_sample_token(scratch, V, tau, ot_uniform(seed, step, sequence, cur + 1), &mg);
        if (mg < mm) mm = mg;
        accept_tokens[A++] = y;
        int32_t hit = -1;
        for (int32_t i = 0; i < n_sel; ++i)
            if (parent[i] == cur && token[i] == y) { hit = i; break; }
        if (hit < 0) break;
        accept_nodes[A - 1] = hit;
        cur = hit;
        curdepth = depth[hit];
    }
    *next_root = accept_tokens[A - 1];
    if (min_margin) *min_margin = mm;
    free(scratch); free(path);
    return A;
}

/* Sampled verification of a batch on the table model. */
int ot_table_verify_sampled(const uint16_t *target, int32_t H, int32_t V, const int32_t *root_token, int32_t batch,
                            int32_t n, int32_t max_depth, const int32_t *token, const int32_t *parent, const int32_t *depth,
                            const int32_t *n_sel, double tau, uint64_t seed, uint64_t step,
                            int32_t *accept_len, int32_t *accept_tokens, int32_t *accept_nodes, int32_t *next_root,
                            double *min_margin)
{
    ot_table_model tm = { target, H, V };
    ot_model tmodel = { ot_table_logits, ot_table_key, &tm };
    for (int32_t b = 0; b < batch; ++b)
        accept_len[b] = ot_verify_sampled(&tmodel, root_token[b], V, n_sel[b], max_depth,
                                          token + (size_t)b * n, parent + (size_t)b * n, depth + (size_t)b * n,
                                          tau, seed, step, b,
                                          accept_tokens + (size_t)b * (max_depth + 1), accept_nodes + (size_t)b * max_depth,
                                          next_root + b, min_margin ? min_margin + b : NULL);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Batch driver over the table model (what the harness times and compares).  */
/* One decoding step for `batch` independent sequences, single thread.       */
/* All per-sequence outputs are [batch][...] contiguous.                     */
/* ------------------------------------------------------------------------- */
int ot_table_step(const uint16_t *draft, const uint16_t *target, int32_t H, int32_t V,
                  const int32_t *root_token, const int32_t *base_pos, int32_t batch,
                  int32_t n, int32_t k, int32_t max_depth, double delta,
                  const int32_t *force_depth /* [batch] or NULL */, ot_memo *memo,
                  int32_t *token, int32_t *parent, int32_t *depth, double *phat,
                  int32_t *n_sel, int32_t *depth_reached, double *expected_len, double *esub_trace,
                  double *min_gap, double *stop_margin,
                  uint64_t *mask, int32_t *position_ids,
                  int32_t *accept_len, int32_t *accept_tokens, int32_t *accept_nodes, int32_t *next_root)
{
    ot_table_model dm = { draft, H, V }, tm = { target, H, V };
    ot_model dmodel = { ot_table_logits, ot_table_key, &dm };
    ot_model tmodel = { ot_table_logits, ot_table_key, &tm };
    int32_t W = (n + 63) / 64;
    for (int32_t b = 0; b < batch; ++b) {
        int rc = ot_build(&dmodel, memo, root_token[b], V, n, k, max_depth, delta,
                          force_depth ? force_depth[b] : 0,
                          token + (size_t)b * n, parent + (size_t)b * n, depth + (size_t)b * n, phat + (size_t)b * n,
                          n_sel + b, depth_reached + b, expected_len + b, esub_trace + (size_t)b * max_depth,
                          min_gap ? min_gap + b : NULL, stop_margin ? stop_margin + b : NULL);
        if (rc) return rc;
        if (mask)
            ot_mask(parent + (size_t)b * n, depth + (size_t)b * n, n_sel[b], n, base_pos ? base_pos[b] : 0,
                    mask + (size_t)b * n * W, position_ids + (size_t)b * n);
        if (target && accept_len)
            accept_len[b] = ot_verify(&tmodel, root_token[b], V, n_sel[b], max_depth,
                                      token + (size_t)b * n, parent + (size_t)b * n, depth + (size_t)b * n,
                                      accept_tokens + (size_t)b * (max_depth + 1),
                                      accept_nodes + (size_t)b * max_depth, next_root + b);
    }
    return 0;
}

/* Build / verify through arbitrary callbacks (used by tests with explicit per-node distributions). */
int ot_build_cb(ot_logits_fn fn, void *user, int32_t root_token,
                int32_t V, int32_t n, int32_t k, int32_t max_depth, double delta, int32_t force_depth,
                int32_t *token, int32_t *parent, int32_t *depth, double *phat,
                int32_t *n_sel, int32_t *depth_reached, double *expected_len,
                double *esub_trace, double *min_gap, double *stop_margin)
{
    ot_model model = { fn, NULL, user };
    return ot_build(&model, NULL, root_token, V, n, k, max_depth, delta, force_depth,
                    token, parent, depth, phat, n_sel, depth_reached, expected_len, esub_trace, min_gap, stop_margin);
}

int32_t ot_verify_cb(ot_logits_fn fn, void *user, int32_t root_token, int32_t V, int32_t n_sel, int32_t max_depth,
                     const int32_t *token, const int32_t *parent, const int32_t *depth,
                     int32_t *accept_tokens, int32_t *accept_nodes, int32_t *next_root)
{
    ot_model model = { fn, NULL, user };
    return ot_verify(&model, root_token, V, n_sel, max_depth, token, parent, depth,
                     accept_tokens, accept_nodes, next_root);
}

/* Row step on a bf16 row (for per-row parity of the fused softmax + top-k kernel). */
int32_t ot_row_softmax_topk_bf16(const uint16_t *row, int32_t V, int32_t k,
                                 int32_t *tok_out, double *p_out, double *m_out, double *S_out)
{
    double *x = (double *)malloc((size_t)V * sizeof(double));
    for (int32_t v = 0; v < V; ++v) x[v] = bf16_to_double(row[v]);
    int32_t kk = ot_row_softmax_topk(x, V, k, tok_out, p_out, m_out, S_out);
    free(x);
    return kk;
}

/* Target-row argmax on a bf16 row (lowest token id on ties). */
int32_t ot_row_argmax_bf16(const uint16_t *row, int32_t V)
{
    int32_t best = 0;
    double bv = bf16_to_double(row[0]);
    for (int32_t v = 1; v < V; ++v) {
        double x = bf16_to_double(row[v]);
        if (x > bv) { bv = x; best = v; }
    }
    return best;
}
