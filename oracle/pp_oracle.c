/*
 * CPU oracle for the min-bottleneck partition-and-placement problem.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * CUDA library must compute.  It shares no code, header, table or helper with the
 * CUDA path and must never be linked into or called from it; only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may use it.
 *
 * Problem (paper, Section 1 and Section 3.2): a chain of L layers is cut into
 * m >= 1 contiguous, non-empty segments; segment j runs on its own edge node n_j
 * (Section 1: no two segments share a node, so the n_j are pairwise different);
 * a segment fits when the memory of its layers is within the node's capacity (the
 * omega(P) vs kappa predicate of the partition-graph definition, read as <=).
 * The tensor that crosses cut j is the output of the last layer of segment j, and
 * its latency is
 *      gamma_j = data / bandwidth = bits[e_j] / bw[n_j][n_{j+1}]        (Eq. 3)
 * The bottleneck latency of a plan is
 *      beta = max_j gamma_j                                             (Eq. 2)
 * and beta = +0.0 for a plan with a single segment (no inter-node transfer).
 * The exact optimum is  beta* = min over all plans of beta.
 *
 * Arithmetic: every gamma is one IEEE-754 binary64 division of the integer bit
 * count by the integer kbps (both converted exactly), so beta is in milliseconds.
 * A link with 0 kbps is unusable: gamma = +inf and a plan that uses it is no plan.
 * min and max only select values, they never create new ones.
 *
 * Canonical optimum: among all plans with beta == beta*, the one with the
 * lexicographically smallest key
 *      (m, mask, n_m, e_{m-1}, n_{m-1}, e_{m-2}, n_{m-2}, ..., e_1, n_1)
 * where mask = sum_j 2^{n_j}.  That is: fewest segments, then lowest node-set mask,
 * then lowest last node, then walking backwards lowest cut, then lowest node id.
 *
 * Pins (see tests/test_oracle_pins.py): the 10.2 Mbit / 6 Mbps = 1.7 s example of
 * Section 1, hand-worked plans, an exact-rational enumerator written in Python,
 * closed forms for k = 2 and for uniform data, the Theorem 1 bound, monotonicity,
 * exact power-of-two scalings, relabelling and chain-reversal symmetries.
 *
 * Build: gcc -O2 -std=c11 -fno-fast-math -ffp-contract=off -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_INFEASIBLE 1
#define ORC_ERR_ARG (-1)
#define ORC_ERR_NOMEM (-3)

/* plan_status bit flags of the evaluator */
#define ORC_PLAN_BAD_NSEG 1
#define ORC_PLAN_BAD_ENDS 2
#define ORC_PLAN_BAD_NODE 4
#define ORC_PLAN_MEMORY 8
#define ORC_PLAN_DEAD_LINK 16

typedef struct {
    int L, k;
    const uint64_t *bits; /* [L] output size of each layer, bits */
    const uint64_t *mem;  /* [L] memory of each layer, bytes */
    const uint64_t *cap;  /* [k] capacity of each node, bytes */
    const uint32_t *bw;   /* [k*k] kbps, bw[v*k+w] is the link v -> w */
} orc_instance;

/* Eq. 3: latency = data / bandwidth, one correctly rounded fp64 division (ms). */
double orc_gamma(uint64_t bits, uint32_t kbps)
{
    if (kbps == 0) return INFINITY;
    return (double)bits / (double)kbps;
}

/* memory of layers first..last inclusive */
static uint64_t seg_mem(const orc_instance *I, int first, int last)
{
    uint64_t s = 0;
    for (int i = first; i <= last; ++i) s += I->mem[i];
    return s;
}

/*
 * Eq. 2 + Eq. 3 for one candidate plan.  cuts[0..nseg-2] are the last layers of
 * segments 1..nseg-1 (the last segment always ends at L-1); nodes[0..nseg-1] are
 * the nodes in pipeline order.  Returns the plan_status flags; *beta is +inf when
 * any flag is set.
 */
int orc_eval_plan(int L, const uint64_t *bits, const uint64_t *mem, int k, const uint64_t *cap,
                  const uint32_t *bw, int nseg, const int32_t *cuts, const int32_t *nodes,
                  double *beta)
{
    orc_instance I = {L, k, bits, mem, cap, bw};
    int flags = 0;
    *beta = INFINITY;
    int mmax = k < L ? k : L;
    if (nseg < 1 || nseg > mmax) return ORC_PLAN_BAD_NSEG;
    for (int j = 0; j < nseg - 1; ++j) {
        if (cuts[j] < 0 || cuts[j] > L - 2) flags |= ORC_PLAN_BAD_ENDS;
        if (j > 0 && cuts[j] <= cuts[j - 1]) flags |= ORC_PLAN_BAD_ENDS;
    }
    for (int j = 0; j < nseg; ++j) {
        if (nodes[j] < 0 || nodes[j] >= k) { flags |= ORC_PLAN_BAD_NODE; continue; }
        for (int i = 0; i < j; ++i)
            if (nodes[i] == nodes[j]) flags |= ORC_PLAN_BAD_NODE;
    }
    if (flags) return flags;
    double b = 0.0;
    int first = 0;
    for (int j = 0; j < nseg; ++j) {
        int last = (j == nseg - 1) ? L - 1 : cuts[j];
        if (seg_mem(&I, first, last) > cap[nodes[j]]) flags |= ORC_PLAN_MEMORY;
        if (j < nseg - 1) {
            uint32_t link = bw[nodes[j] * k + nodes[j + 1]];
            if (link == 0) flags |= ORC_PLAN_DEAD_LINK;
            double g = orc_gamma(bits[last], link);
            if (g > b) b = g;
        }
        first = last + 1;
    }
    if (flags) return flags;
    *beta = b;
    return 0;
}

/* ---- canonical key ------------------------------------------------------- */

typedef struct {
    double beta;
    int m;
    int e[32]; /* e[j] = last layer of segment j (0-based), e[m-1] = L-1 */
    int n[32]; /* n[j] = node of segment j */
} orc_plan;

static uint32_t plan_mask(const orc_plan *p)
{
    uint32_t s = 0;
    for (int j = 0; j < p->m; ++j) s |= 1u << p->n[j];
    return s;
}

/* <0 if a precedes b in (beta, m, mask, n_m, e_{m-1}, n_{m-1}, ..., e_1, n_1) */
static int plan_cmp(const orc_plan *a, const orc_plan *b)
{
    if (a->beta < b->beta) return -1;
    if (a->beta > b->beta) return 1;
    if (a->m != b->m) return a->m < b->m ? -1 : 1;
    uint32_t ma = plan_mask(a), mb = plan_mask(b);
    if (ma != mb) return ma < mb ? -1 : 1;
    int m = a->m;
    if (a->n[m - 1] != b->n[m - 1]) return a->n[m - 1] < b->n[m - 1] ? -1 : 1;
    for (int j = m - 2; j >= 0; --j) {
        if (a->e[j] != b->e[j]) return a->e[j] < b->e[j] ? -1 : 1;
        if (a->n[j] != b->n[j]) return a->n[j] < b->n[j] ? -1 : 1;
    }
    return 0;
}

static void plan_out(const orc_plan *p, int k, double *beta, int32_t *m, int32_t *cuts,
                     int32_t *placement)
{
    *beta = p->beta;
    *m = p->m;
    for (int j = 0; j < k - 1; ++j) cuts[j] = (j < p->m - 1) ? p->e[j] : -1;
    for (int j = 0; j < k; ++j) placement[j] = (j < p->m) ? p->n[j] : -1;
}

static void plan_none(int k, double *beta, int32_t *m, int32_t *cuts, int32_t *placement)
{
    *beta = INFINITY;
    *m = 0;
    for (int j = 0; j < k - 1; ++j) cuts[j] = -1;
    for (int j = 0; j < k; ++j) placement[j] = -1;
}

/* ---- brute force: every cut set times every injective placement ----------- */

typedef struct {
    const orc_instance *I;
    orc_plan cur, best;
    int have;
    uint64_t visited;
} bf_state;

/* extend cur (j segments fixed, next segment starts at layer `first`) */
static void bf_rec(bf_state *st, int j, int first, uint32_t used, double beta_so_far)
{
    const orc_instance *I = st->I;
    int mmax = I->k < I->L ? I->k : I->L;
    if (j >= mmax) return;
    for (int last = first; last < I->L; ++last) {
        uint64_t need = seg_mem(I, first, last);
        for (int n = 0; n < I->k; ++n) {
            if (used & (1u << n)) continue;
            if (need > I->cap[n]) continue;
            double b = beta_so_far;
            if (j > 0) {
                double g = orc_gamma(I->bits[first - 1], I->bw[st->cur.n[j - 1] * I->k + n]);
                if (g > b) b = g;
            }
            st->cur.e[j] = last;
            st->cur.n[j] = n;
            if (last == I->L - 1) {
                st->cur.m = j + 1;
                st->cur.beta = b;
                st->visited++;
                if (!isinf(b) && (!st->have || plan_cmp(&st->cur, &st->best) < 0)) {
                    st->best = st->cur;
                    st->have = 1;
                }
            } else {
                bf_rec(st, j + 1, last + 1, used | (1u << n), b);
            }
        }
    }
}

int orc_bruteforce(int L, const uint64_t *bits, const uint64_t *mem, int k, const uint64_t *cap,
                   const uint32_t *bw, double *beta, int32_t *m, int32_t *cuts,
                   int32_t *placement, uint64_t *plans_visited)
{
    if (L < 1 || k < 1 || k > 20) return ORC_ERR_ARG;
    orc_instance I = {L, k, bits, mem, cap, bw};
    bf_state st;
    memset(&st, 0, sizeof st);
    st.I = &I;
    bf_rec(&st, 0, 0, 0, 0.0);
    if (plans_visited) *plans_visited = st.visited;
    if (!st.have) {
        plan_none(k, beta, m, cuts, placement);
        return ORC_INFEASIBLE;
    }
    plan_out(&st.best, k, beta, m, cuts, placement);
    return ORC_OK;
}

/* ---- dynamic programme over (used-node mask S, last node v, last layer c) -- */
/*
 * dp[S][v][c] = smallest bottleneck of a partial plan that covers layers 0..c with
 * exactly the nodes of S, one segment each, the last segment on v ending at c.
 *   |S| = 1:  dp[{v}][v][c] = +0.0 if layers 0..c fit on v, else +inf.
 *   else:     dp[S][w][c'] = min over v in S\{w}, c < c' with layers c+1..c' fitting
 *             on w, of max(dp[S\{w}][v][c], gamma(bits[c], bw[v][w])).
 * beta* = min over (S, v) of dp[S][v][L-1].
 * Rows are stored compactly: row(S, v) = rowoff[S] + (number of nodes of S below v).
 */

typedef struct {
    orc_instance I;
    uint64_t *M;     /* [L+1] prefix sums of mem */
    double *gam;     /* [L*k*k] gamma[c][v][w] */
    int64_t *rowoff; /* [2^k + 1] */
    double *dp;      /* [rows * L] */
} dp_state;

static int popc(uint32_t x) { return __builtin_popcount(x); }

static int64_t dp_row(const dp_state *D, uint32_t S, int v)
{
    return D->rowoff[S] + popc(S & ((1u << v) - 1));
}

static void dp_free(dp_state *D)
{
    free(D->M);
    free(D->gam);
    free(D->rowoff);
    free(D->dp);
}

static int dp_init(dp_state *D, int L, const uint64_t *bits, const uint64_t *mem, int k,
                   const uint64_t *cap, const uint32_t *bw)
{
    memset(D, 0, sizeof *D);
    D->I = (orc_instance){L, k, bits, mem, cap, bw};
    uint32_t nm = 1u << k;
    D->M = malloc(sizeof(uint64_t) * (L + 1));
    D->gam = malloc(sizeof(double) * (size_t)L * k * k);
    D->rowoff = malloc(sizeof(int64_t) * ((size_t)nm + 1));
    if (!D->M || !D->gam || !D->rowoff) { dp_free(D); return ORC_ERR_NOMEM; }
    D->M[0] = 0;
    for (int i = 0; i < L; ++i) D->M[i + 1] = D->M[i] + mem[i];
    for (int c = 0; c < L; ++c)
        for (int v = 0; v < k; ++v)
            for (int w = 0; w < k; ++w)
                D->gam[((size_t)c * k + v) * k + w] =
                    (v == w) ? INFINITY : orc_gamma(bits[c], bw[v * k + w]);
    D->rowoff[0] = 0;
    for (uint32_t S = 0; S < nm; ++S) D->rowoff[S + 1] = D->rowoff[S] + popc(S);
    D->dp = malloc(sizeof(double) * (size_t)D->rowoff[nm] * L);
    if (!D->dp) { dp_free(D); return ORC_ERR_NOMEM; }
    return ORC_OK;
}

/* layers first..last fit on node w */
static int fits(const dp_state *D, int first, int last, int w)
{
    return D->M[last + 1] - D->M[first] <= D->I.cap[w];
}

static void dp_base_row(dp_state *D, uint32_t S, int v)
{
    double *row = D->dp + dp_row(D, S, v) * D->I.L;
    for (int c = 0; c < D->I.L; ++c) row[c] = fits(D, 0, c, v) ? 0.0 : INFINITY;
}

/* the recurrence exactly as written above: every (v, c) pair tested on its own */
static void dp_row_naive(dp_state *D, uint32_t S, int w)
{
    int L = D->I.L, k = D->I.k;
    uint32_t P = S & ~(1u << w);
    double *out = D->dp + dp_row(D, S, w) * L;
    for (int c2 = 0; c2 < L; ++c2) {
        double best = INFINITY;
        for (int v = 0; v < k; ++v) {
            if (!(P & (1u << v))) continue;
            const double *src = D->dp + dp_row(D, P, v) * L;
            for (int c = 0; c < c2; ++c) {
                if (!fits(D, c + 1, c2, w)) continue;
                double g = D->gam[((size_t)c * k + v) * k + w];
                double cand = src[c] > g ? src[c] : g;
                if (cand < best) best = cand;
            }
        }
        out[c2] = best;
    }
}

/* same recurrence, min over v taken first (g), then the feasible run of c scanned */
static void dp_row_fact(dp_state *D, uint32_t S, int w, double *g)
{
    int L = D->I.L, k = D->I.k;
    uint32_t P = S & ~(1u << w);
    double *out = D->dp + dp_row(D, S, w) * L;
    for (int c = 0; c < L; ++c) {
        double best = INFINITY;
        for (int v = 0; v < k; ++v) {
            if (!(P & (1u << v))) continue;
            double d = D->dp[dp_row(D, P, v) * L + c];
            double x = D->gam[((size_t)c * k + v) * k + w];
            double cand = d > x ? d : x;
            if (cand < best) best = cand;
        }
        g[c] = best;
    }
    for (int c2 = 0; c2 < L; ++c2) {
        double best = INFINITY;
        for (int c = c2 - 1; c >= 0 && fits(D, c + 1, c2, w); --c)
            if (g[c] < best) best = g[c];
        out[c2] = best;
    }
}

static void dp_fill(dp_state *D, int factorised, int nthreads)
{
    int L = D->I.L, k = D->I.k;
    uint32_t nm = 1u << k;
    (void)nthreads;
    for (int j = 1; j <= k; ++j) {
        /* masks of one popcount only read masks of the previous popcount */
#ifdef _OPENMP
#pragma omp parallel num_threads(nthreads > 0 ? nthreads : 1)
#endif
        {
            double *g = malloc(sizeof(double) * L);
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 64)
#endif
            for (uint32_t S = 1; S < nm; ++S) {
                if (popc(S) != j) continue;
                for (int w = 0; w < k; ++w) {
                    if (!(S & (1u << w))) continue;
                    if (j == 1) dp_base_row(D, S, w);
                    else if (factorised) dp_row_fact(D, S, w, g);
                    else dp_row_naive(D, S, w);
                }
            }
            free(g);
        }
    }
}

/*
 * Pick the canonical optimum from a filled table.  Final state: lexicographic minimum
 * of (value, |S|, S, v) at c = L-1.  Walking back from (S, w, c') the predecessor is the
 * lowest c, then the lowest v, among those with max(dp[S\{w}][v][c], gamma) <= beta*:
 * dp is the best any prefix can do, so exactly those steps extend to an optimal plan,
 * and taking the smallest (c, v) at each step yields the smallest key.
 */
static int dp_extract(dp_state *D, double *beta, int32_t *m, int32_t *cuts, int32_t *placement)
{
    int L = D->I.L, k = D->I.k;
    uint32_t nm = 1u << k;
    double bbest = INFINITY;
    uint32_t Sbest = 0;
    int vbest = -1;
    for (uint32_t S = 1; S < nm; ++S)
        for (int v = 0; v < k; ++v) {
            if (!(S & (1u << v))) continue;
            double x = D->dp[dp_row(D, S, v) * L + (L - 1)];
            if (isinf(x)) continue;
            int better = 0;
            if (vbest < 0 || x < bbest) better = 1;
            else if (x == bbest) {
                if (popc(S) != popc(Sbest)) better = popc(S) < popc(Sbest);
                else if (S != Sbest) better = S < Sbest;
                else better = v < vbest;
            }
            if (better) { bbest = x; Sbest = S; vbest = v; }
        }
    if (vbest < 0) {
        plan_none(k, beta, m, cuts, placement);
        return ORC_INFEASIBLE;
    }
    orc_plan p;
    p.beta = bbest;
    p.m = popc(Sbest);
    uint32_t S = Sbest;
    int w = vbest, c2 = L - 1;
    for (int j = p.m - 1; j >= 0; --j) {
        p.e[j] = c2;
        p.n[j] = w;
        if (j == 0) break;
        uint32_t P = S & ~(1u << w);
        int found = 0;
        for (int c = 0; c < c2 && !found; ++c) {
            if (!fits(D, c + 1, c2, w)) continue;
            for (int v = 0; v < k && !found; ++v) {
                if (!(P & (1u << v))) continue;
                double d = D->dp[dp_row(D, P, v) * L + c];
                double x = D->gam[((size_t)c * k + v) * k + w];
                double cand = d > x ? d : x;
                if (cand <= bbest) { found = 1; S = P; w = v; c2 = c; }
            }
        }
        if (!found) return ORC_ERR_ARG; /* table inconsistent: cannot happen */
    }
    plan_out(&p, k, beta, m, cuts, placement);
    return ORC_OK;
}

static int dp_solve(int factorised, int nthreads, int L, const uint64_t *bits, const uint64_t *mem,
                    int k, const uint64_t *cap, const uint32_t *bw, double *beta, int32_t *m,
                    int32_t *cuts, int32_t *placement, double *table_out)
{
    if (L < 1 || k < 1 || k > 20) return ORC_ERR_ARG;
    dp_state D;
    int rc = dp_init(&D, L, bits, mem, k, cap, bw);
    if (rc != ORC_OK) return rc;
    dp_fill(&D, factorised, nthreads);
    rc = dp_extract(&D, beta, m, cuts, placement);
    if (table_out) {
        /* dense copy [S][v][c] with +inf where v is not in S, for element-wise comparison */
        uint32_t nm = 1u << k;
        for (uint32_t S = 0; S < nm; ++S)
            for (int v = 0; v < k; ++v)
                for (int c = 0; c < L; ++c)
                    table_out[((size_t)S * k + v) * L + c] =
                        (S & (1u << v)) ? D.dp[dp_row(&D, S, v) * L + c] : INFINITY;
    }
    dp_free(&D);
    return rc;
}

int orc_dp_naive(int L, const uint64_t *bits, const uint64_t *mem, int k, const uint64_t *cap,
                 const uint32_t *bw, double *beta, int32_t *m, int32_t *cuts, int32_t *placement,
                 double *table_out)
{
    return dp_solve(0, 1, L, bits, mem, k, cap, bw, beta, m, cuts, placement, table_out);
}

int orc_dp_fact(int L, const uint64_t *bits, const uint64_t *mem, int k, const uint64_t *cap,
                const uint32_t *bw, int nthreads, double *beta, int32_t *m, int32_t *cuts,
                int32_t *placement, double *table_out)
{
    return dp_solve(1, nthreads, L, bits, mem, k, cap, bw, beta, m, cuts, placement, table_out);
}

int orc_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
