/*
 * CPU oracle for the verification step of Graph-structured Speculative Decoding.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA
 * library is checked against; it shares no code with the CUDA path, and nothing in the
 * product may call it.  Only the tests, the smoke check and the benchmark's CPU-baseline
 * leg use it.
 *
 * What it computes
 *  - Attention (tree attention, Sec. 4.1: a flattened draft token attends only to its
 *    ancestors; the committed context sits in the KV cache, Sec. 4.2; all hypotheses are
 *    scored in one pass, Sec. 3 and Sec. 4.1).  For every sequence b, draft node n and
 *    query head h the visible keys are the first seq_lens[b] rows of the cache plus the
 *    draft nodes whose bit is set in ancestor_mask[b][n]; the output row is the
 *    max-subtracted softmax of scale * <q, k_j> over those keys applied to the matching
 *    value rows.  Everything is evaluated in double precision from the exact values of
 *    the bf16 inputs.  An empty key set gives a row of zeros.
 *  - Acceptance (deterministic verification, Sec. 3: a drafted token is kept only if the
 *    target model would emit it; a rejection discards the rest of that hypothesis and
 *    the target model supplies the next token; the longest hypothesis from the root is
 *    adopted, Sec. 4.1 and Sec. 1).  a[n] is the lowest index holding the row maximum
 *    of logits[b][n][:].  Every root-to-node path of the DAG is enumerated by a
 *    depth-first walk over child lists (no dynamic programming, no memo); a path
 *    v0=0,v1..vm is accepted iff tok[v_i] == a[v_{i-1}] on each of its edges.  The
 *    longest accepted path wins; among equally long ones the path whose node sequence,
 *    read from its last node backwards, is lexicographically smallest.  Output:
 *    tok[v1..vm] followed by a[vm], so accepted_len = m + 1.
 *  - Non-deterministic acceptance (Sec. 3: accept with probability min(1, p/q); Sec. 6.4: on
 *    the token graph), with the random numbers as inputs: the same walk with the step
 *    p -> v accepted iff u_accept[v] * q_v < softmax(logits[p])[tok v], and the regenerated
 *    token drawn by inverting the cumulative distribution of the residual max(0, P - Q) at the
 *    end node when a drafted continuation was rejected there, of P itself otherwise.
 *  - The KV-cache commit of the accepted path and the ancestor-mask closure (see there).
 *  - One growth step of the draft token graph: top-k children, probability and sibling
 *    pruning (Sec. 4.2), tau-redundant nodes and their merge edges (Sec. 5.2, 5.3).
 *
 * Readings where the paper is silent are listed in the repository's design notes
 * (scale default 1/sqrt(D), q-head h uses kv-head h / G, mask bits honoured literally,
 * node 0 is the root whose token is not re-emitted, NaN logits never win the argmax).
 *
 * Every function here is pinned by tests that do not re-use it: closed forms (uniform
 * softmax, two-key sigmoid), library attention on chain / tree / full-mask special
 * cases, numpy argmax, hand-built DAGs with hand-derived answers, and invariants.
 * Three choices are readings of a silent paper, not facts the pins can settle; for these the
 * parity is unpinned: a node merged from several branches attends to the union of its
 * ancestors (the paper un-merges the graph before verification, Sec. 5.4); the target
 * model's own next token is counted in accepted_len; in the non-deterministic rule every step
 * of the graph is tested against the target distribution of its parent, and several rejected
 * siblings share the single residual max(0, P - Q) of their parent.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t B, N, Hq, Hkv, D, Lmax;
    double scale; /* <= 0 means 1/sqrt(D) */
} gsd_oracle_attn_dims;

static double bf16_to_double(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16; /* bf16 is the top half of an IEEE float */
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int gsd_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One output row out_row[0..D) for (b, n, h).  scratch holds Lmax + N doubles. */
void gsd_oracle_attn_row(const gsd_oracle_attn_dims *dm, const uint16_t *q,
                         const uint16_t *k_cache, const uint16_t *v_cache,
                         const uint16_t *draft_k, const uint16_t *draft_v,
                         const uint32_t *ancestor_mask, const int32_t *seq_lens,
                         int b, int n, int h, double *out_row, double *scratch)
{
    const int N = dm->N, Hq = dm->Hq, Hkv = dm->Hkv, D = dm->D, Lmax = dm->Lmax;
    const int G = Hq / Hkv;
    const int c = h / G; /* kv head serving query head h */
    const int W = (N + 31) / 32;
    const double scale = dm->scale > 0 ? dm->scale : 1.0 / sqrt((double)D);
    const int L = seq_lens[b];
    const uint16_t *qrow = q + (((size_t)b * N + n) * Hq + h) * D;
    const uint32_t *mrow = ancestor_mask + ((size_t)b * N + n) * W;
    double *s = scratch;
    int nk = 0;
    double smax = -INFINITY;

    /* scores of the visible keys, prefix first then draft nodes */
    for (int j = 0; j < L; ++j) {
        const uint16_t *krow = k_cache + (((size_t)b * Lmax + j) * Hkv + c) * D;
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += bf16_to_double(qrow[d]) * bf16_to_double(krow[d]);
        s[nk] = scale * dot;
        if (s[nk] > smax) smax = s[nk];
        ++nk;
    }
    for (int j = 0; j < N; ++j) {
        if (!((mrow[j / 32] >> (j % 32)) & 1u)) continue;
        const uint16_t *krow = draft_k + (((size_t)b * N + j) * Hkv + c) * D;
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += bf16_to_double(qrow[d]) * bf16_to_double(krow[d]);
        s[nk] = scale * dot;
        if (s[nk] > smax) smax = s[nk];
        ++nk;
    }
    for (int d = 0; d < D; ++d) out_row[d] = 0.0;
    if (nk == 0) return;

    double denom = 0.0;
    for (int i = 0; i < nk; ++i) {
        s[i] = exp(s[i] - smax);
        denom += s[i];
    }
    int i = 0;
    for (int j = 0; j < L; ++j, ++i) {
        const uint16_t *vrow = v_cache + (((size_t)b * Lmax + j) * Hkv + c) * D;
        const double p = s[i] / denom;
        for (int d = 0; d < D; ++d) out_row[d] += p * bf16_to_double(vrow[d]);
    }
    for (int j = 0; j < N; ++j) {
        if (!((mrow[j / 32] >> (j % 32)) & 1u)) continue;
        const uint16_t *vrow = draft_v + (((size_t)b * N + j) * Hkv + c) * D;
        const double p = s[i] / denom;
        for (int d = 0; d < D; ++d) out_row[d] += p * bf16_to_double(vrow[d]);
        ++i;
    }
}

/* All rows: out[B,N,Hq,D] in double.  Rows are independent; they are handed to the host
 * threads as they are, nothing else is reorganised. */
int gsd_oracle_attn(const gsd_oracle_attn_dims *dm, const uint16_t *q, const uint16_t *k_cache,
                    const uint16_t *v_cache, const uint16_t *draft_k, const uint16_t *draft_v,
                    const uint32_t *ancestor_mask, const int32_t *seq_lens, double *out)
{
    const long rows = (long)dm->B * dm->N * dm->Hq;
    int failed = 0;
#pragma omp parallel
    {
        double *scratch = (double *)malloc(sizeof(double) * (size_t)(dm->Lmax + dm->N + 1));
        if (!scratch) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 16)
        for (long r = 0; r < rows; ++r) {
            if (!scratch) continue;
            const int h = (int)(r % dm->Hq);
            const int n = (int)((r / dm->Hq) % dm->N);
            const int b = (int)(r / ((long)dm->Hq * dm->N));
            gsd_oracle_attn_row(dm, q, k_cache, v_cache, draft_k, draft_v, ancestor_mask,
                                seq_lens, b, n, h, out + (size_t)r * dm->D, scratch);
        }
        free(scratch);
    }
    return failed ? -1 : 0;
}

/* A listed subset of rows: rows[3*i..3*i+2] = (b, n, h); out[i*D..]. */
int gsd_oracle_attn_rows(const gsd_oracle_attn_dims *dm, const uint16_t *q,
                         const uint16_t *k_cache, const uint16_t *v_cache,
                         const uint16_t *draft_k, const uint16_t *draft_v,
                         const uint32_t *ancestor_mask, const int32_t *seq_lens,
                         const int32_t *rows, long nrows, double *out)
{
    int failed = 0;
#pragma omp parallel
    {
        double *scratch = (double *)malloc(sizeof(double) * (size_t)(dm->Lmax + dm->N + 1));
        if (!scratch) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (long i = 0; i < nrows; ++i) {
            if (!scratch) continue;
            gsd_oracle_attn_row(dm, q, k_cache, v_cache, draft_k, draft_v, ancestor_mask,
                                seq_lens, rows[3 * i], rows[3 * i + 1], rows[3 * i + 2],
                                out + (size_t)i * dm->D, scratch);
        }
        free(scratch);
    }
    return failed ? -1 : 0;
}

/* Lowest index holding the largest non-NaN value; 0 when every entry is NaN.
 * A later entry replaces the current best only when strictly greater. */
int32_t gsd_oracle_argmax_row(const float *row, int32_t V)
{
    int32_t best = -1;
    for (int32_t i = 0; i < V; ++i) {
        if (row[i] != row[i]) continue; /* NaN never wins */
        if (best < 0 || row[i] > row[best]) best = i;
    }
    return best < 0 ? 0 : best;
}

void gsd_oracle_argmax(const float *logits, long rows, int32_t V, int32_t *out)
{
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) out[r] = gsd_oracle_argmax_row(logits + (size_t)r * V, V);
}

/* ---- brute-force path enumeration for one sequence ---- */
typedef struct {
    int N;
    const int32_t *tok;   /* [N] */
    const int32_t *amax;  /* [N] */
    const unsigned char *edge_ok; /* NULL, or [N*N]: edge_ok[p*N + v] = the step p -> v is accepted */
    const int *child_ptr; /* [N+1] */
    const int *child_idx;
    int *stack;           /* current path, stack[0] = 0 */
    int *best;            /* best accepted path so far */
    int best_edges;       /* its edge count, -1 if none yet */
    long visited;         /* number of root-to-node paths enumerated */
    long visit_cap;       /* > 0: beyond this many paths, stop extending rejected paths */
    int pruned;           /* set when the cap changed the walk */
} walk_t;

static int path_is_accepted(const walk_t *w, int len)
{
    for (int i = 1; i < len; ++i) {
        if (w->edge_ok) {
            if (!w->edge_ok[(size_t)w->stack[i - 1] * w->N + w->stack[i]]) return 0;
        } else if (w->tok[w->stack[i]] != w->amax[w->stack[i - 1]]) {
            return 0;
        }
    }
    return 1;
}

/* 1 if the candidate (w->stack, same length as w->best) comes first when both are read
 * from the last node backwards */
static int reversed_less(const walk_t *w, int len)
{
    for (int i = len - 1; i >= 0; --i) {
        if (w->stack[i] < w->best[i]) return 1;
        if (w->stack[i] > w->best[i]) return 0;
    }
    return 0;
}

static void walk(walk_t *w, int len)
{
    const int v = w->stack[len - 1];
    const int ok = path_is_accepted(w, len);
    w->visited++;
    if (ok) {
        const int edges = len - 1;
        if (edges > w->best_edges || (edges == w->best_edges && reversed_less(w, len))) {
            memcpy(w->best, w->stack, sizeof(int) * (size_t)len);
            w->best_edges = edges;
        }
    } else if (w->visit_cap > 0 && w->visited > w->visit_cap) {
        /* an extension of a rejected path is rejected too: once over the cap, skip them */
        w->pruned = 1;
        return;
    }
    for (int e = w->child_ptr[v]; e < w->child_ptr[v + 1]; ++e) {
        w->stack[len] = w->child_idx[e];
        walk(w, len + 1);
    }
}

/*
 * logits [B,N,V] f32; draft_tokens [B,N]; parent_ptr [B,N+1]; parent_idx [B,Ecap];
 * accepted_tokens [B,Tcap] (padded with -1); accepted_len [B]; accepted_nodes [B,Tcap]
 * (may be NULL; the chosen path's node ids v0..vm, padded with -1); paths_visited [B] (may be
 * NULL).  visit_cap <= 0 enumerates everything.  Returns 0, or -1 on malformed input
 * (a parent index not below its child, Tcap too small) or allocation failure.
 */
int gsd_oracle_accept(const float *logits, const int32_t *draft_tokens, const int32_t *parent_ptr,
                      const int32_t *parent_idx, int32_t B, int32_t N, int32_t V, int32_t Ecap,
                      int32_t Tcap, int32_t *accepted_tokens, int32_t *accepted_len,
                      int32_t *accepted_nodes, int64_t *paths_visited, int64_t visit_cap)
{
    int rc = 0;
    for (int b = 0; b < B; ++b) {
        const int32_t *tok = draft_tokens + (size_t)b * N;
        const int32_t *pp = parent_ptr + (size_t)b * (N + 1);
        const int32_t *pi = parent_idx + (size_t)b * Ecap;
        int32_t *amax = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
        int *cptr = (int *)calloc((size_t)N + 2, sizeof(int));
        int *cidx = (int *)malloc(sizeof(int) * (size_t)(pp[N] > 0 ? pp[N] : 1));
        int *fill = (int *)calloc((size_t)N + 1, sizeof(int));
        int *stack = (int *)malloc(sizeof(int) * (size_t)(N + 1));
        int *best = (int *)malloc(sizeof(int) * (size_t)(N + 1));
        if (!amax || !cptr || !cidx || !fill || !stack || !best) rc = -1;

        if (rc == 0) {
            gsd_oracle_argmax(logits + (size_t)b * N * V, N, V, amax);
            /* child lists (children ascending) from the parent lists */
            for (int v = 0; v < N && rc == 0; ++v)
                for (int e = pp[v]; e < pp[v + 1]; ++e) {
                    if (pi[e] < 0 || pi[e] >= v) { rc = -1; break; }
                    cptr[pi[e] + 1]++;
                }
        }
        if (rc == 0) {
            for (int v = 0; v < N; ++v) cptr[v + 1] += cptr[v];
            for (int v = 0; v < N; ++v)
                for (int e = pp[v]; e < pp[v + 1]; ++e) {
                    const int p = pi[e];
                    cidx[cptr[p] + fill[p]++] = v;
                }
            walk_t w;
            w.N = N; w.tok = tok; w.amax = amax; w.edge_ok = NULL; w.child_ptr = cptr; w.child_idx = cidx;
            w.stack = stack; w.best = best; w.best_edges = -1; w.visited = 0;
            w.visit_cap = visit_cap; w.pruned = 0;
            stack[0] = 0;
            walk(&w, 1); /* the one-node path (root alone) is always accepted */
            const int m = w.best_edges;
            if (m + 1 > Tcap) rc = -1;
            if (rc == 0) {
                for (int i = 0; i < Tcap; ++i) {
                    accepted_tokens[(size_t)b * Tcap + i] = -1;
                    if (accepted_nodes) accepted_nodes[(size_t)b * Tcap + i] = -1;
                }
                for (int i = 1; i <= m; ++i) accepted_tokens[(size_t)b * Tcap + i - 1] = tok[best[i]];
                accepted_tokens[(size_t)b * Tcap + m] = amax[best[m]];
                accepted_len[b] = m + 1;
                if (accepted_nodes)
                    for (int i = 0; i <= m; ++i) accepted_nodes[(size_t)b * Tcap + i] = best[i];
                if (paths_visited) paths_visited[b] = w.pruned ? -w.visited : w.visited;
            }
        }
        free(amax); free(cptr); free(cidx); free(fill); free(stack); free(best);
        if (rc != 0) return rc;
    }
    return 0;
}

/*
 * Non-deterministic verification (Sec. 3: the i-th drafted token is accepted with probability
 * min(1, p/q), the first rejection discards the rest of the hypothesis and the target model
 * regenerates that token, so that the accepted tokens follow the target model's distribution;
 * Sec. 6.4 runs it on the token graph).  Readings taken here: the random numbers are inputs;
 * the test is applied per step p -> v of the graph with
 * p = softmax(logits[parent])[token of v] and q = draft_q[v]:
 *     accepted(p -> v)  iff  u_accept[v] * q_v < p          (u < min(1, p/q) for q > 0)
 * the accepted hypothesis is the longest root path whose steps are all accepted (ties as in
 * gsd_oracle_accept).  The regenerated token follows the sampling scheme that Sec. 3 cites:
 * with P = softmax(logits[end node]) and Q = softmax(draft_logits[end node]) (the distribution
 * the end node's children were drafted from),
 *   - if the end node has at least one child in the graph (its drafted continuations were all
 *     rejected) it is drawn from the residual  r_j = max(0, P_j - Q_j) / sum_i max(0, P_i - Q_i);
 *   - if the end node has no child (nothing was rejected there), or draft_logits is NULL, or the
 *     residual has no mass (sum_i max(0, P_i - Q_i) <= 1e-6: the two distributions agree to
 *     single-precision rounding, and a rejection then has probability <= 1e-6), it is drawn from
 *     P itself.
 * Several rejected siblings share the one residual P - Q (the paper gives no rule for them).
 * The draw inverts the cumulative distribution in index order: the smallest t with
 * sum_{j<=t} w_j > u_sample[b] * sum_j w_j  (the last t with w_t > 0 if rounding leaves none),
 * w = P or max(0, P - Q).  All arithmetic in double.  logits (and draft_logits) must be finite
 * or -inf with at least one finite entry per row.
 *
 * logits [B,N,V]; draft_logits [B,N,V] or NULL; draft_q, u_accept [B,N]; u_sample [B]; the rest
 * as gsd_oracle_accept.  Returns 0, or -1 on malformed input or allocation failure.
 */
static void softmax_stats(const float *x, int V, double *m_out, double *s_out)
{
    double m = -INFINITY, s = 0.0;
    for (int j = 0; j < V; ++j) if ((double)x[j] > m) m = (double)x[j];
    for (int j = 0; j < V; ++j) s += exp((double)x[j] - m);
    *m_out = m; *s_out = s;
}

int gsd_oracle_accept_sampled(const float *logits, const int32_t *draft_tokens,
                              const int32_t *parent_ptr, const int32_t *parent_idx,
                              const float *draft_logits, const float *draft_q,
                              const float *u_accept, const float *u_sample,
                              int32_t B, int32_t N, int32_t V, int32_t Ecap, int32_t Tcap,
                              int32_t *accepted_tokens, int32_t *accepted_len, int32_t *accepted_nodes)
{
    int rc = 0;
    for (int b = 0; b < B; ++b) {
        const int32_t *tok = draft_tokens + (size_t)b * N;
        const int32_t *pp = parent_ptr + (size_t)b * (N + 1);
        const int32_t *pi = parent_idx + (size_t)b * Ecap;
        const float *lg = logits + (size_t)b * N * V;
        double *mx = (double *)malloc(sizeof(double) * (size_t)N);
        double *sm = (double *)malloc(sizeof(double) * (size_t)N);
        unsigned char *ok = (unsigned char *)calloc((size_t)N * N, 1);
        int *cptr = (int *)calloc((size_t)N + 2, sizeof(int));
        int *cidx = (int *)malloc(sizeof(int) * (size_t)(pp[N] > 0 ? pp[N] : 1));
        int *fill = (int *)calloc((size_t)N + 1, sizeof(int));
        int *stack = (int *)malloc(sizeof(int) * (size_t)(N + 1));
        int *best = (int *)malloc(sizeof(int) * (size_t)(N + 1));
        double *wgt = (double *)malloc(sizeof(double) * (size_t)V);
        double *res = (double *)malloc(sizeof(double) * (size_t)V);
        if (!mx || !sm || !ok || !cptr || !cidx || !fill || !stack || !best || !wgt || !res) rc = -1;
        if (rc == 0) {
#pragma omp parallel for schedule(static)
            for (int v = 0; v < N; ++v) softmax_stats(lg + (size_t)v * V, V, &mx[v], &sm[v]);
            for (int v = 0; v < N && rc == 0; ++v)
                for (int e = pp[v]; e < pp[v + 1]; ++e) {
                    const int p = pi[e];
                    if (p < 0 || p >= v || tok[v] < 0 || tok[v] >= V) { rc = -1; break; }
                    const double prob = exp((double)lg[(size_t)p * V + tok[v]] - mx[p]) / sm[p];
                    ok[(size_t)p * N + v] = ((double)u_accept[(size_t)b * N + v] * (double)draft_q[(size_t)b * N + v] < prob);
                    cptr[p + 1]++;
                }
        }
        if (rc == 0) {
            for (int v = 0; v < N; ++v) cptr[v + 1] += cptr[v];
            for (int v = 0; v < N; ++v)
                for (int e = pp[v]; e < pp[v + 1]; ++e) cidx[cptr[pi[e]] + fill[pi[e]]++] = v;
            walk_t w;
            w.N = N; w.tok = tok; w.amax = NULL; w.edge_ok = ok; w.child_ptr = cptr; w.child_idx = cidx;
            w.stack = stack; w.best = best; w.best_edges = -1; w.visited = 0;
            w.visit_cap = 0; w.pruned = 0;
            stack[0] = 0;
            walk(&w, 1);
            const int m = w.best_edges;
            if (m + 1 > Tcap) rc = -1;
            if (rc == 0) {
                /* the regenerated token: weights w over the vocabulary at the end node, then the
                 * inverse of their cumulative distribution */
                const int end = best[m];
                const float *x = lg + (size_t)end * V;
                const int rejected_children = cptr[end + 1] - cptr[end];
                double total = 0.0;
                for (int j = 0; j < V; ++j) wgt[j] = exp((double)x[j] - mx[end]) / sm[end];
                if (draft_logits && rejected_children > 0) {
                    const float *y = draft_logits + ((size_t)b * N + end) * V;
                    double mq, sq, mass = 0.0;
                    softmax_stats(y, V, &mq, &sq);
                    for (int j = 0; j < V; ++j) {
                        const double r = wgt[j] - exp((double)y[j] - mq) / sq;
                        res[j] = r > 0.0 ? r : 0.0;
                        mass += res[j];
                    }
                    if (mass > 1e-6) memcpy(wgt, res, sizeof(double) * (size_t)V);
                }
                for (int j = 0; j < V; ++j) total += wgt[j];
                const double target = (double)u_sample[b] * total;
                double cum = 0.0;
                int pick = -1, last_pos = -1;
                for (int j = 0; j < V; ++j) {
                    if (wgt[j] > 0.0) last_pos = j;
                    cum += wgt[j];
                    if (cum > target) { pick = j; break; }
                }
                if (pick < 0) pick = last_pos;
                for (int i = 0; i < Tcap; ++i) {
                    accepted_tokens[(size_t)b * Tcap + i] = -1;
                    if (accepted_nodes) accepted_nodes[(size_t)b * Tcap + i] = -1;
                }
                for (int i = 1; i <= m; ++i) accepted_tokens[(size_t)b * Tcap + i - 1] = tok[best[i]];
                accepted_tokens[(size_t)b * Tcap + m] = pick;
                accepted_len[b] = m + 1;
                if (accepted_nodes)
                    for (int i = 0; i <= m; ++i) accepted_nodes[(size_t)b * Tcap + i] = best[i];
            }
        }
        free(mx); free(sm); free(ok); free(cptr); free(cidx); free(fill); free(stack); free(best);
        free(wgt); free(res);
        if (rc != 0) return rc;
    }
    return 0;
}

/*
 * One growth step of the draft token graph (Sec. 4 token tree with out-degree k; Sec. 4.2
 * probability pruning and sibling pruning; Sec. 5.2 tau-redundant nodes; Sec. 5.3 merging).
 * For sequence b the frontier nodes frontier[b][0..frontier_len[b]) are expanded in order; for
 * a frontier node p with draft distribution P = softmax(logits[b][fi]) (double):
 *   - its k children are the k most probable tokens (ties to the lowest token id), created in
 *     that order as nodes n, n+1, ... with tokens[c] = token, tree_parent[c] = p, prob[c] = its
 *     probability q, merge_to[c] = -1;
 *   - a child is marked a leaf if q < theta_prob (probability pruning) or q < theta_sib * q_max
 *     with q_max the largest of the k sibling probabilities (sibling pruning);
 *   - a child is tau-redundant if the tau tokens ending at it along its tree path (itself and
 *     tau - 1 tree ancestors; paths shorter than tau do not count) equal the tau tokens ending at
 *     an earlier node (lower id, of this or an earlier step); it is then marked a leaf and
 *     merge_to[c] is the lowest such id (the first occurrence).
 * Creation stops when the node capacity Ncap is reached (return value bit 0).  The new
 * frontier is the list of new nodes that are not leaves, in id order.
 *
 * logits [B,F,V] f32; frontier [B,F]; frontier_len [B]; tokens, tree_parent, merge_to [B,Ncap]
 * i32, leaf [B,Ncap] u8, prob [B,Ncap] f32, num_nodes [B] (all in/out); new_frontier [B,F*k],
 * new_frontier_len [B].  Returns 0, 1 if some sequence ran out of capacity, -1 on malformed input.
 */
static int same_gram(const int32_t *tok, const int32_t *par, int a, int b, int tau)
{
    for (int i = 0; i < tau; ++i) {
        if (a < 0 || b < 0) return 0;          /* a path shorter than tau */
        if (tok[a] != tok[b]) return 0;
        a = par[a];
        b = par[b];
    }
    return 1;
}

int gsd_oracle_draft_expand(const float *logits, const int32_t *frontier, const int32_t *frontier_len,
                            int32_t *tokens, int32_t *tree_parent, int32_t *merge_to, uint8_t *leaf,
                            float *prob, int32_t *num_nodes, int32_t *new_frontier,
                            int32_t *new_frontier_len, int32_t B, int32_t F, int32_t V, int32_t Ncap,
                            int32_t k, int32_t tau, double theta_prob, double theta_sib)
{
    int rc = 0;
    if (k < 1 || k > V || tau < 1 || F < 0) return -1;
    double *P = (double *)malloc(sizeof(double) * (size_t)V);
    unsigned char *taken = (unsigned char *)malloc((size_t)V);
    if (!P || !taken) { free(P); free(taken); return -1; }
    for (int b = 0; b < B; ++b) {
        int32_t *tok = tokens + (size_t)b * Ncap, *par = tree_parent + (size_t)b * Ncap;
        int32_t *mt = merge_to + (size_t)b * Ncap;
        uint8_t *lf = leaf + (size_t)b * Ncap;
        float *pr = prob + (size_t)b * Ncap;
        const int first_new = num_nodes[b];
        int n = first_new;
        if (frontier_len[b] < 0 || frontier_len[b] > F || n < 1 || n > Ncap) { rc = -1; break; }
        for (int fi = 0; fi < frontier_len[b]; ++fi) {
            const int p = frontier[(size_t)b * F + fi];
            if (p < 0 || p >= first_new) { rc = -1; break; }
            const float *x = logits + ((size_t)b * F + fi) * V;
            double mx = -INFINITY, sum = 0.0;
            for (int j = 0; j < V; ++j) if ((double)x[j] > mx) mx = (double)x[j];
            for (int j = 0; j < V; ++j) { P[j] = exp((double)x[j] - mx); sum += P[j]; }
            for (int j = 0; j < V; ++j) { P[j] /= sum; taken[j] = 0; }
            double qmax = 0.0;
            for (int i = 0; i < k; ++i) {
                int best = -1;                 /* most probable token not taken yet, ties to the lowest id */
                for (int j = 0; j < V; ++j)
                    if (!taken[j] && (best < 0 || P[j] > P[best])) best = j;
                taken[best] = 1;
                if (i == 0) qmax = P[best];
                if (n >= Ncap) { rc |= 1; continue; }
                const int c = n++;
                tok[c] = best; par[c] = p; mt[c] = -1; pr[c] = (float)P[best];
                lf[c] = (P[best] < theta_prob) || (P[best] < theta_sib * qmax);
            }
        }
        if (rc < 0) break;
        int nf = 0;
        for (int c = first_new; c < n; ++c) {
            for (int e = 0; e < c; ++e)
                if (same_gram(tok, par, c, e, tau)) { lf[c] = 1; mt[c] = e; break; }
            if (!lf[c]) new_frontier[(size_t)b * F * k + nf++] = c;
        }
        new_frontier_len[b] = nf;
        num_nodes[b] = n;
    }
    free(P); free(taken);
    return rc;
}

/*
 * KV-cache commit of the accepted path (the cache update that follows verification; the paper
 * counts it under "Others" in its time breakdown, Sec. 7.1 / Table 3, and names KV caching in
 * Sec. 4.2).  The accepted path v0=0, v1..vm of sequence b (accepted_nodes[b][0..len), len =
 * accepted_len[b] = m + 1) becomes part of the committed context: the draft K/V rows of those
 * nodes are appended to the cache at positions seq_lens[b] .. seq_lens[b] + len - 1 and
 * seq_lens[b] grows by len.  Rows that would fall past Lmax are dropped and the length is
 * clamped (returns the number of sequences that overflowed).  Everything else is untouched.
 *
 * k_cache/v_cache [B,Lmax,Hkv,D] (in/out), draft_k/draft_v [B,N,Hkv,D], accepted_nodes [B,Tcap],
 * accepted_len [B], seq_lens [B] (in/out); elements are 2-byte bf16 patterns, copied as they are.
 */
int gsd_oracle_commit_kv(uint16_t *k_cache, uint16_t *v_cache, const uint16_t *draft_k,
                         const uint16_t *draft_v, const int32_t *accepted_nodes,
                         const int32_t *accepted_len, int32_t *seq_lens, int32_t B, int32_t N,
                         int32_t Hkv, int32_t D, int32_t Lmax, int32_t Tcap)
{
    int overflowed = 0;
    const size_t row = (size_t)Hkv * D;
    for (int b = 0; b < B; ++b) {
        const int len = accepted_len[b];
        int pos = seq_lens[b];
        for (int i = 0; i < len && i < Tcap; ++i) {
            const int node = accepted_nodes[(size_t)b * Tcap + i];
            if (node < 0 || node >= N) continue;
            if (pos >= Lmax) { overflowed++; break; }
            memcpy(k_cache + ((size_t)b * Lmax + pos) * row, draft_k + ((size_t)b * N + node) * row, row * 2);
            memcpy(v_cache + ((size_t)b * Lmax + pos) * row, draft_v + ((size_t)b * N + node) * row, row * 2);
            ++pos;
        }
        seq_lens[b] = pos;
    }
    return overflowed;
}

/*
 * Ancestor bitmask of a draft DAG from its parent lists (what "each token may only attend to
 * its ancestor nodes" of tree attention, Sec. 4.1, means for the merged token graph of
 * Sec. 5.3: a node sees itself and every node from which it can be reached).  For each node
 * the ancestors are collected by an explicit upward search over the parent lists with a
 * visited array (no reuse of other rows).  mask [B,N,W] uint32, W = ceil(N/32); bit j of row n
 * (word j / 32, bit j % 32) set iff j == n or j is an ancestor of n.  Parent indices outside
 * [0, n) are ignored.  Returns -1 on allocation failure.
 */
int gsd_oracle_build_mask(const int32_t *parent_ptr, const int32_t *parent_idx, int32_t B, int32_t N,
                          int32_t Ecap, uint32_t *mask)
{
    const int W = (N + 31) / 32;
    unsigned char *seen = (unsigned char *)malloc((size_t)N);
    int *todo = (int *)malloc(sizeof(int) * (size_t)N);
    if (!seen || !todo) { free(seen); free(todo); return -1; }
    for (int b = 0; b < B; ++b) {
        const int32_t *pp = parent_ptr + (size_t)b * (N + 1);
        const int32_t *pi = parent_idx + (size_t)b * Ecap;
        for (int n = 0; n < N; ++n) {
            uint32_t *row = mask + ((size_t)b * N + n) * W;
            memset(row, 0, sizeof(uint32_t) * (size_t)W);
            memset(seen, 0, (size_t)N);
            int top = 0;
            seen[n] = 1;
            todo[top++] = n;
            while (top > 0) {
                const int v = todo[--top];
                row[v / 32] |= 1u << (v % 32);
                for (int e = pp[v]; e < pp[v + 1]; ++e) {
                    const int p = pi[e];
                    if (p < 0 || p >= v || seen[p]) continue;
                    seen[p] = 1;
                    todo[top++] = p;
                }
            }
        }
    }
    free(seen);
    free(todo);
    return 0;
}

/*
 * Unmerging the token graph into a tree (Sec. 5.4, Fig. 4: before verification the graph is
 * reverted to a tree; the successors of every redundant node are replicated from the node it was
 * merged into, and the tree is then verified as in tree-structured decoding).  In terms of the
 * verification DAG (parent lists; a node merged into f has f's children as its own) this is the
 * unfolding of the DAG from the root: one tree node per root path.  Readings: tree nodes are
 * numbered level by level, inside a level by (tree index of the parent, then id of the copied DAG
 * node), so a parent always precedes its children; a repeating pattern makes the unfolding
 * endless, so it is cut at max_depth edges from the root; when Ucap nodes have been created
 * the rest is dropped (return value 1).
 *
 * draft_tokens [B,N]; parent_ptr [B,N+1]; parent_idx [B,Ecap] (parents below their child);
 * tree_tokens, tree_parent (tree index of the parent, -1 for the root), tree_source (the DAG
 * node a tree node copies) [B,Ucap], unused entries -1; tree_count [B].
 * Returns 0, 1 if some sequence ran out of capacity, -1 on malformed input.
 */
int gsd_oracle_unmerge_tree(const int32_t *draft_tokens, const int32_t *parent_ptr,
                            const int32_t *parent_idx, int32_t B, int32_t N, int32_t Ecap,
                            int32_t Ucap, int32_t max_depth, int32_t *tree_tokens,
                            int32_t *tree_parent, int32_t *tree_source, int32_t *tree_count)
{
    int rc = 0;
    if (N < 1 || Ucap < 1 || max_depth < 0) return -1;
    int *depth = (int *)malloc(sizeof(int) * (size_t)Ucap);
    if (!depth) return -1;
    for (int b = 0; b < B; ++b) {
        const int32_t *tok = draft_tokens + (size_t)b * N;
        const int32_t *pp = parent_ptr + (size_t)b * (N + 1);
        const int32_t *pi = parent_idx + (size_t)b * Ecap;
        int32_t *tt = tree_tokens + (size_t)b * Ucap, *tp = tree_parent + (size_t)b * Ucap;
        int32_t *ts = tree_source + (size_t)b * Ucap;
        for (int u = 0; u < Ucap; ++u) tt[u] = tp[u] = ts[u] = -1;
        for (int v = 0; v < N; ++v)
            for (int e = pp[v]; e < pp[v + 1]; ++e)
                if (pi[e] < 0 || pi[e] >= v) { free(depth); return -1; }
        int count = 1;
        tt[0] = tok[0]; tp[0] = -1; ts[0] = 0; depth[0] = 0;
        /* tree nodes are expanded in the order they were created (a queue): level order */
        for (int u = 0; u < count; ++u) {
            if (depth[u] >= max_depth) continue;
            for (int v = 0; v < N; ++v) {          /* children of the copied node, ascending id */
                int is_child = 0;
                for (int e = pp[v]; e < pp[v + 1]; ++e) is_child |= (pi[e] == ts[u]);
                if (!is_child) continue;
                if (count >= Ucap) { rc = 1; continue; }
                tt[count] = tok[v]; tp[count] = u; ts[count] = v; depth[count] = depth[u] + 1;
                ++count;
            }
        }
        tree_count[b] = count;
    }
    free(depth);
    return rc;
}
