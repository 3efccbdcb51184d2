/*
 * otlp_oracle.c -- slow, plain, double-precision CPU statement of the paper's other OTLP solvers and
 * of its offline analysis quantities.
 *
 * TEST INFRASTRUCTURE ONLY, like spec_oracle.c: this file is the checker the CUDA library is compared
 * against.  It shares no code with the CUDA path and is never called by the product path.
 *
 * What it computes, and the passage each function follows (p, q: sampling distributions of one node,
 * already normalised, as oracle_row_probs of spec_oracle.c makes them):
 *   otlp_solve            one call of an OTLP solver on a child list: NSS (Algorithm 1), Naive /
 *                         NaiveTree (Algorithm 2), SpecTr K-SEQ (Algorithm 3), in sampling mode with
 *                         caller-supplied uniforms.
 *   oracle_verify_otlp    the solver used top-down (Section 3.2 "OT-based algorithms": move to the
 *                         child whose token was output, stop when the output is not a child).
 *   oracle_acceptance     acceptance rates alpha(f) of Definition 5.1: Algorithms 6 (NSS), 7 (Naive),
 *                         8 (SpecTr), 9 (SpecInfer).
 *   oracle_divergences    L1(p,q), KL(p||q), KL(q||p) (the selector's scalar features, Section 6 /
 *                         Appendix E; the L1 curve of Section 5).
 *   oracle_branching      branching probabilities B(f, x, X_i) of Definition 5.3: Algorithms 11 (NSS),
 *                         12 (Naive), 13 (SpecTr), 14 (SpecInfer, children picked uniformly) and the
 *                         list-order SpecInfer this build's verifier runs.
 *   oracle_block_efficiency  the inner sum of equation (3), sum over the tree's nodes of the product
 *                         of branching probabilities along the path, for one given tree.
 *   oracle_latency_model  equation (8) of Appendix E (forward-pass time of an action) and the throughput
 *                         estimate of Section 6 (expected block efficiency over expected time).
 *
 * Readings (where the paper is silent): acceptance tests are strict (u < threshold) as in
 * spec_oracle.c; rho* of SpecTr is found by 60 bisection steps on [1, k] (the paper says "binary
 * search"); when the output token equals several children's tokens the walk moves to the first of
 * them in list order, and only that child gets the branching probability in the block-efficiency
 * sum (duplicates stay separate nodes here, Definition 3.1's multiplicities are not merged);
 * 0 log 0 = 0 and KL is +inf where the second law has no mass under the first.
 *
 * Pins (tests/test_otlp_pins.py): every solver's exact output law equals p (Definition 3.2) by
 * enumeration over child tuples and decision paths; acceptance rates against that enumeration;
 * branching probabilities against it for given child lists incl. duplicates, sum_t B <= 1 with
 * equality when the children cover the vocabulary; the block-efficiency sum against the exact
 * E[tau + 1] of the verifier on tiny trees; k = 1 reductions (SpecTr = Naive = SpecInfer);
 * divergences against scipy.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define OTLP_NSS 0
#define OTLP_NAIVE 1
#define OTLP_SPECTR 2
#define OTLP_SPECINFER 3        /* children tried in list order (this build's verifier) */
#define OTLP_SPECINFER_UNIFORM 4 /* Algorithm 4 as printed: the next child is picked uniformly */

#define OTLP_OK 0
#define OTLP_ERR_ARG (-1)
#define OTLP_ERR_ALLOC (-5)

/* provided by spec_oracle.c (same library) */
int32_t oracle_inverse_cdf(const double *w, int32_t V, double u, double *margin);
int oracle_row_probs(const double *z, int32_t V, double T, int32_t top_k, double top_p,
                     double *probs, double *stats);

static double ratio_unclipped(double P, double Q)
{
    if (!(P > 0.0)) return 0.0;
    if (!(Q > 0.0)) return INFINITY;
    return P / Q;
}
static double clip1(double r) { return r < 1.0 ? r : 1.0; }

/* ------------------------------------------------------------------------------------------ */
/* SpecTr: the division factor rho* (Appendix B, equations above Algorithm 3)                  */
/* ------------------------------------------------------------------------------------------ */
static double spectr_beta(const double *p, const double *q, int V, double rho)
{
    double b = 0.0;
    for (int t = 0; t < V; ++t) {
        double a = p[t] / rho;
        b += a < q[t] ? a : q[t];
    }
    return b;
}
/* root of rho -> p_acc(rho) - rho beta(rho) on [1, k] (monotone decreasing there): 60 bisection
 * steps; the value at 1 is >= 0, so rho* = 1 when k = 1 and when the function is already <= 0 */
double oracle_spectr_rho(const double *p, const double *q, int32_t V, int32_t k)
{
    double lo = 1.0, hi = (double)k;
    if (k <= 1) return 1.0;
    for (int it = 0; it < 60; ++it) {
        double mid = 0.5 * (lo + hi);
        double b = spectr_beta(p, q, V, mid);
        double f = (1.0 - pow(1.0 - b, (double)k)) - mid * b;
        if (f > 0.0) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}
/* beta, p_acc, gamma at rho and the residual law p_res ~ (p - min(p/rho, q) gamma)+ (Algorithm 3) */
static void spectr_residual(const double *p, const double *q, int V, int k, double rho, double *res,
                            double *beta_out, double *pacc_out)
{
    double beta = spectr_beta(p, q, V, rho);
    double pacc = 1.0 - pow(1.0 - beta, (double)k);
    double gamma = beta > 0.0 ? pacc / beta : 0.0;
    double S = 0.0;
    for (int t = 0; t < V; ++t) {
        double a = p[t] / rho;
        double m = a < q[t] ? a : q[t];
        double d = p[t] - m * gamma;
        res[t] = d > 0.0 ? d : 0.0;
        S += res[t];
    }
    if (S > 0.0)
        for (int t = 0; t < V; ++t) res[t] /= S;
    else
        memcpy(res, p, sizeof(double) * (size_t)V);
    if (beta_out) *beta_out = beta;
    if (pacc_out) *pacc_out = pacc;
}

/* ------------------------------------------------------------------------------------------ */
/* one solver call (sampling mode)                                                             */
/* ------------------------------------------------------------------------------------------ */
/*
 * x[k] child tokens, u_acc[k] one acceptance uniform per child, u_bonus the uniform of the residual
 * draw.  Returns the output token; *tested receives how many acceptance uniforms were consumed,
 * thr[j] the threshold child j's uniform was compared with (for the ones tested), *bonus_margin the
 * CDF margin of the residual draw (0 when no draw was made), *from_residual whether the token came
 * from a draw.  res (V doubles of scratch) holds the law the draw was made from.
 */
static int otlp_solve(int solver, const double *p, const double *q, int V, const int32_t *x,
                      const double *u_acc, int k, double u_bonus, double *res, int *tested, double *thr,
                      double *bonus_margin, int *from_residual)
{
    *tested = 0;
    *from_residual = 1;
    if (solver == OTLP_NSS || k == 0) {
        /* Algorithm 1: Y ~ p, the drafts are ignored */
        memcpy(res, p, sizeof(double) * (size_t)V);
    } else if (solver == OTLP_NAIVE) {
        /* Algorithm 2: test X_1 only; otherwise Y ~ norm((p - q)+), which may land on X_2..X_k */
        double r = clip1(ratio_unclipped(p[x[0]], q[x[0]]));
        thr[0] = r;
        *tested = 1;
        if (u_acc[0] < r) { *from_residual = 0; *bonus_margin = 0.0; return x[0]; }
        double S = 0.0;
        for (int t = 0; t < V; ++t) { double d = p[t] - q[t]; res[t] = d > 0.0 ? d : 0.0; S += res[t]; }
        if (S > 0.0) for (int t = 0; t < V; ++t) res[t] /= S;
        else memcpy(res, p, sizeof(double) * (size_t)V);
    } else { /* OTLP_SPECTR, Algorithm 3 */
        double rho = oracle_spectr_rho(p, q, V, k);
        for (int i = 0; i < k; ++i) {
            double r = clip1(ratio_unclipped(p[x[i]], q[x[i]]) / rho);
            thr[i] = r;
            *tested = i + 1;
            if (u_acc[i] < r) { *from_residual = 0; *bonus_margin = 0.0; return x[i]; }
        }
        spectr_residual(p, q, V, k, rho, res, NULL, NULL);
    }
    return oracle_inverse_cdf(res, V, u_bonus, bonus_margin);
}

/* ------------------------------------------------------------------------------------------ */
/* top-down verification with a solver (Section 3.2)                                           */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t B, N, V, logits_dtype;
    const void *target_logits, *draft_logits;
    int64_t seq_stride, node_stride;
    const int32_t *parent;
    int64_t topo_seq_stride;
    const int32_t *token;
    float temperature;
    int32_t top_k;
    float top_p;
    const float *temperature_per_seq;
    const float *u_accept, *u_bonus;
} OracleIn; /* same layout as in spec_oracle.c */

static double widen(const void *base, int dtype, int64_t idx)
{
    if (dtype == 0) return (double)((const float *)base)[idx];
    uint32_t w = (uint32_t)((const uint16_t *)base)[idx] << 16;
    float f;
    memcpy(&f, &w, 4);
    return (double)f;
}
static int node_law(const OracleIn *in, int b, int a, int which, double *out)
{
    const void *base = which ? in->draft_logits : in->target_logits;
    double *z = (double *)malloc(sizeof(double) * (size_t)in->V);
    if (!z) return OTLP_ERR_ALLOC;
    int64_t off = (int64_t)b * in->seq_stride + (int64_t)a * in->node_stride;
    for (int t = 0; t < in->V; ++t) z[t] = widen(base, in->logits_dtype, off + t);
    double T = (double)(in->temperature_per_seq ? in->temperature_per_seq[b] : in->temperature);
    int rc = oracle_row_probs(z, in->V, T, in->top_k, (double)in->top_p, out, NULL);
    free(z);
    return rc;
}
static int children_of(const int32_t *parent, int N, int a, int *out)
{
    int k = 0;
    for (int c = a + 1; c < N; ++c)
        if (parent[c] == a) out[k++] = c;
    return k;
}

/*
 * Per sequence: accepted_node, accept_len, out_tokens [B,N] (path tokens, the emitted token, -1...),
 * emitted token (bonus_token), bonus_margin (margin of the last residual draw, 0 if the last token was
 * an accepted child), min_margin (smallest |u - thr| over the acceptance tests made; 1 if none),
 * status.  A residual draw that lands on a child's token moves to the first such child in list order.
 */
int32_t oracle_verify_otlp(const OracleIn *in, int32_t solver, int32_t *accepted_node, int32_t *accept_len,
                           int32_t *out_tokens, int32_t *bonus_token, double *bonus_margin,
                           double *min_margin, int32_t *status)
{
    if (!in || !accepted_node || !accept_len || !out_tokens || !bonus_token || !status) return OTLP_ERR_ARG;
    if (solver != OTLP_NSS && solver != OTLP_NAIVE && solver != OTLP_SPECTR) return OTLP_ERR_ARG;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < in->B; ++b) {
        int N = in->N, V = in->V, rc = 0;
        const int32_t *parent = in->parent + (size_t)b * (size_t)in->topo_seq_stride;
        const int32_t *token = in->token + (size_t)b * N;
        double *P = (double *)malloc(sizeof(double) * (size_t)V), *Q = (double *)malloc(sizeof(double) * (size_t)V);
        double *res = (double *)malloc(sizeof(double) * (size_t)V);
        int *ch = (int *)malloc(sizeof(int) * (size_t)N);
        int32_t *x = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
        double *ua = (double *)malloc(sizeof(double) * (size_t)N), *thr = (double *)malloc(sizeof(double) * (size_t)N);
        int32_t *ot = out_tokens + (size_t)b * N;
        for (int i = 0; i < N; ++i) ot[i] = -1;
        double mm = 1.0, bm = 0.0;
        int cur = 0, len = 0, y = -1;
        if (!P || !Q || !res || !ch || !x || !ua || !thr) rc = OTLP_ERR_ALLOC;
        for (int i = 1; i < N && !rc; ++i)
            if (parent[i] < 0 || parent[i] >= i || token[i] < 0 || token[i] >= V) rc = OTLP_ERR_ARG;
        while (!rc) {
            rc = node_law(in, b, cur, 0, P);
            if (rc) break;
            int k = children_of(parent, N, cur, ch);
            if (k > 0 && solver != OTLP_NSS) { rc = node_law(in, b, cur, 1, Q); if (rc) break; }
            for (int j = 0; j < k; ++j) { x[j] = token[ch[j]]; ua[j] = (double)in->u_accept[(size_t)b * N + ch[j]]; }
            int tested = 0, from_res = 1;
            y = otlp_solve(solver, P, Q, V, x, ua, k, (double)in->u_bonus[(size_t)b * N + cur], res, &tested, thr,
                           &bm, &from_res);
            for (int j = 0; j < tested; ++j) { double m = fabs(ua[j] - thr[j]); if (m < mm) mm = m; }
            int next = -1;
            for (int j = 0; j < k && next < 0; ++j)
                if (x[j] == y) next = ch[j];
            if (next < 0) break;
            ot[len++] = y;
            cur = next;
            if (!from_res) bm = 0.0;
        }
        if (!rc) ot[len] = y;
        accepted_node[b] = rc ? -1 : cur; accept_len[b] = rc ? -1 : len; bonus_token[b] = rc ? -1 : y;
        if (bonus_margin) bonus_margin[b] = bm;
        if (min_margin) min_margin[b] = mm;
        status[b] = rc;
        free(P); free(Q); free(res); free(ch); free(x); free(ua); free(thr);
    }
    return OTLP_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* acceptance rates (Appendix C) and divergences                                               */
/* ------------------------------------------------------------------------------------------ */
/* out[0] NSS (Algorithm 6), out[1] Naive (7), out[2] SpecTr (8), out[3] SpecInfer (9) */
int32_t oracle_acceptance(const double *p, const double *q, int32_t V, int32_t k, double *out)
{
    if (!p || !q || !out || V <= 0 || k < 1) return OTLP_ERR_ARG;
    double nss = 0.0, naive = 0.0;
    for (int t = 0; t < V; ++t) {
        nss += p[t] * (1.0 - pow(1.0 - q[t], (double)k));
        double mn = p[t] < q[t] ? p[t] : q[t], d = p[t] - q[t];
        naive += mn + (d > 0.0 ? d : 0.0) * (1.0 - pow(1.0 - q[t], (double)(k - 1)));
    }
    out[0] = nss;
    out[1] = naive;
    /* Algorithm 8 */
    double *res = (double *)malloc(sizeof(double) * (size_t)V);
    double *pp = (double *)malloc(sizeof(double) * (size_t)V), *m = (double *)malloc(sizeof(double) * (size_t)V);
    if (!res || !pp || !m) { free(res); free(pp); free(m); return OTLP_ERR_ALLOC; }
    {
        double rho = oracle_spectr_rho(p, q, V, k), beta, pacc;
        spectr_residual(p, q, V, k, rho, res, &beta, &pacc);
        double s = 0.0;
        for (int t = 0; t < V; ++t) {
            double d = q[t] - p[t] / rho;
            double r = (d > 0.0 && beta < 1.0) ? d / (1.0 - beta) : 0.0;
            s += res[t] * (1.0 - pow(1.0 - r, (double)k));
        }
        out[2] = pacc + (1.0 - pacc) * s;
    }
    /* Algorithm 9 */
    {
        memcpy(pp, p, sizeof(double) * (size_t)V);
        for (int t = 0; t < V; ++t) m[t] = 1.0;
        double prej = 1.0;
        for (int i = 0; i < k; ++i) {
            double r = 0.0, S = 0.0;
            for (int t = 0; t < V; ++t) r += pp[t] < q[t] ? pp[t] : q[t];
            prej *= (1.0 - r);
            for (int t = 0; t < V; ++t) {
                double d = q[t] - pp[t];
                if (d > 0.0 && r < 1.0) m[t] *= 1.0 - d / (1.0 - r);
            }
            for (int t = 0; t < V; ++t) { double d = pp[t] - q[t]; res[t] = d > 0.0 ? d : 0.0; S += res[t]; }
            if (S > 0.0) for (int t = 0; t < V; ++t) pp[t] = res[t] / S;
        }
        double s = 0.0;
        for (int t = 0; t < V; ++t) s += pp[t] * (1.0 - m[t]);
        out[3] = (1.0 - prej) + prej * s;
    }
    free(res); free(pp); free(m);
    return OTLP_OK;
}

/* out[0] L1 = sum |p - q|, out[1] KL(p||q), out[2] KL(q||p) (nats; +inf where undefined) */
int32_t oracle_divergences(const double *p, const double *q, int32_t V, double *out)
{
    if (!p || !q || !out || V <= 0) return OTLP_ERR_ARG;
    double l1 = 0.0, kpq = 0.0, kqp = 0.0;
    for (int t = 0; t < V; ++t) {
        l1 += fabs(p[t] - q[t]);
        if (p[t] > 0.0) kpq += q[t] > 0.0 ? p[t] * (log(p[t]) - log(q[t])) : INFINITY;
        if (q[t] > 0.0) kqp += p[t] > 0.0 ? q[t] * (log(q[t]) - log(p[t])) : INFINITY;
    }
    out[0] = l1; out[1] = kpq; out[2] = kqp;
    return OTLP_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* branching probabilities (Appendix D)                                                        */
/* ------------------------------------------------------------------------------------------ */
/* out[i] = B(f, x, x[i]): probability that the solver outputs the token of child i */
int32_t oracle_branching(int32_t solver, const double *p, const double *q, int32_t V, const int32_t *x,
                         int32_t k, double *out)
{
    if (!p || !q || !x || !out || V <= 0 || k < 0) return OTLP_ERR_ARG;
    if (k == 0) return OTLP_OK;
    double *res = (double *)malloc(sizeof(double) * (size_t)V);
    if (!res) return OTLP_ERR_ALLOC;
    int rc = OTLP_OK;
    if (solver == OTLP_NSS) {
        for (int i = 0; i < k; ++i) out[i] = p[x[i]];                       /* Algorithm 11 */
    } else if (solver == OTLP_NAIVE) {                                       /* Algorithm 12 */
        double a = clip1(ratio_unclipped(p[x[0]], q[x[0]])), S = 0.0;
        for (int t = 0; t < V; ++t) { double d = p[t] - q[t]; res[t] = d > 0.0 ? d : 0.0; S += res[t]; }
        for (int i = 0; i < k; ++i)
            out[i] = (1.0 - a) * (S > 0.0 ? res[x[i]] / S : p[x[i]]) + (x[i] == x[0] ? a : 0.0);
    } else if (solver == OTLP_SPECTR) {                                      /* Algorithm 13 */
        double rho = oracle_spectr_rho(p, q, V, k);
        spectr_residual(p, q, V, k, rho, res, NULL, NULL);
        double *a = (double *)malloc(sizeof(double) * (size_t)k);
        if (!a) { free(res); return OTLP_ERR_ALLOC; }
        for (int i = 0; i < k; ++i) a[i] = clip1(ratio_unclipped(p[x[i]], q[x[i]]) / rho);
        double all = 1.0;
        for (int l = 0; l < k; ++l) all *= 1.0 - a[l];
        for (int i = 0; i < k; ++i) {
            double s = 0.0, pre = 1.0;
            for (int j = 0; j < k; ++j) {
                if (x[j] == x[i]) s += a[j] * pre;
                pre *= 1.0 - a[j];
            }
            out[i] = s + res[x[i]] * all;
        }
        free(a);
    } else if (solver == OTLP_SPECINFER || solver == OTLP_SPECINFER_UNIFORM) {
        /* residual laws p_0..p_k and the acceptance vectors a_i = min(1, p_i / q) at the children's tokens */
        double *pi = (double *)malloc(sizeof(double) * (size_t)V);
        double *A = (double *)malloc(sizeof(double) * (size_t)k * (size_t)k);   /* A[i*k + t]: round i, child t */
        double *pk = (double *)malloc(sizeof(double) * (size_t)k);
        if (!pi || !A || !pk) { free(pi); free(A); free(pk); free(res); return OTLP_ERR_ALLOC; }
        memcpy(pi, p, sizeof(double) * (size_t)V);
        for (int i = 0; i < k; ++i) {
            for (int t = 0; t < k; ++t) A[i * k + t] = clip1(ratio_unclipped(pi[x[t]], q[x[t]]));
            double S = 0.0;
            for (int t = 0; t < V; ++t) { double d = pi[t] - q[t]; res[t] = d > 0.0 ? d : 0.0; S += res[t]; }
            if (S > 0.0) for (int t = 0; t < V; ++t) pi[t] = res[t] / S;
        }
        for (int t = 0; t < k; ++t) pk[t] = pi[x[t]];
        if (solver == OTLP_SPECINFER) {
            /* list order: child j is tested in round j with a_j(x_j) */
            double all = 1.0;
            for (int l = 0; l < k; ++l) all *= 1.0 - A[l * k + l];
            for (int i = 0; i < k; ++i) {
                double s = 0.0, pre = 1.0;
                for (int j = 0; j < k; ++j) {
                    if (x[j] == x[i]) s += A[j * k + j] * pre;
                    pre *= 1.0 - A[j * k + j];
                }
                out[i] = s + pk[i] * all;
            }
        } else if (k > 20) {
            rc = OTLP_ERR_ARG;
        } else {
            /* Algorithm 14: dynamic programme over the sets of children still in S; bit t of the mask set
             * = child t still in S; |S| = k - i after i rejections */
            size_t nS = (size_t)1 << k;
            double *Bt = (double *)malloc(sizeof(double) * nS);
            if (!Bt) rc = OTLP_ERR_ALLOC;
            for (int xi = 0; xi < k && !rc; ++xi) {
                Bt[0] = pk[xi];
                for (size_t S = 1; S < nS; ++S) {
                    int cnt = 0;
                    for (int t = 0; t < k; ++t) cnt += (int)((S >> t) & 1);
                    int i = k - cnt;
                    double s = 0.0;
                    for (int t = 0; t < k; ++t)
                        if ((S >> t) & 1) {
                            double a = A[i * k + t];
                            s += a * (x[t] == x[xi] ? 1.0 : 0.0) + (1.0 - a) * Bt[S & ~((size_t)1 << t)];
                        }
                    Bt[S] = s / (double)cnt;
                }
                out[xi] = Bt[nS - 1];
            }
            free(Bt);
        }
        free(pi); free(A); free(pk);
    } else {
        rc = OTLP_ERR_ARG;
    }
    free(res);
    return rc;
}

/*
 * Equation (3), inner sum, for each given tree of the batch: E[tau + 1 | tree] = sum over nodes of the
 * probability that the top-down walk reaches the node = product of branching probabilities along its
 * path (the root counts 1).  node_reach [B,N] receives the per-node products, node_branch [B,N] the
 * branching probability into each node (root: 1), be [B] their sum.  A child whose token an earlier
 * sibling already carries is never moved to (the walk takes the first): its branching probability is 0.
 */
int32_t oracle_block_efficiency(const OracleIn *in, int32_t solver, double *be, double *node_reach,
                                double *node_branch, int32_t *status)
{
    if (!in || !be || !status) return OTLP_ERR_ARG;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < in->B; ++b) {
        int N = in->N, V = in->V, rc = 0;
        const int32_t *parent = in->parent + (size_t)b * (size_t)in->topo_seq_stride;
        const int32_t *token = in->token + (size_t)b * N;
        double *P = (double *)malloc(sizeof(double) * (size_t)V), *Q = (double *)malloc(sizeof(double) * (size_t)V);
        int *ch = (int *)malloc(sizeof(int) * (size_t)N);
        int32_t *x = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
        double *br = (double *)malloc(sizeof(double) * (size_t)N), *reach = (double *)malloc(sizeof(double) * (size_t)N);
        double *brn = (double *)malloc(sizeof(double) * (size_t)N);
        if (!P || !Q || !ch || !x || !br || !reach || !brn) rc = OTLP_ERR_ALLOC;
        for (int i = 1; i < N && !rc; ++i)
            if (parent[i] < 0 || parent[i] >= i || token[i] < 0 || token[i] >= V) rc = OTLP_ERR_ARG;
        double total = 0.0;
        if (!rc) { reach[0] = 1.0; brn[0] = 1.0; }
        for (int a = 0; a < N && !rc; ++a) {
            total += reach[a];
            int k = children_of(parent, N, a, ch);
            if (k == 0) continue;
            rc = node_law(in, b, a, 0, P);
            if (!rc) rc = node_law(in, b, a, 1, Q);
            if (rc) break;
            for (int j = 0; j < k; ++j) x[j] = token[ch[j]];
            rc = oracle_branching(solver, P, Q, V, x, k, br);
            for (int j = 0; j < k && !rc; ++j) {
                int dup = 0;
                for (int l = 0; l < j; ++l) dup |= x[l] == x[j];
                brn[ch[j]] = dup ? 0.0 : br[j];
                reach[ch[j]] = reach[a] * brn[ch[j]];
            }
        }
        be[b] = rc ? NAN : total;
        if (node_reach) for (int i = 0; i < N; ++i) node_reach[(size_t)b * N + i] = rc ? NAN : reach[i];
        if (node_branch) for (int i = 0; i < N; ++i) node_branch[(size_t)b * N + i] = rc ? NAN : brn[i];
        status[b] = rc;
        free(P); free(Q); free(ch); free(x); free(br); free(reach); free(brn);
    }
    return OTLP_OK;
}

/* Per-node analysis of a batch of trees: acc [B,N,4] (Algorithms 6-9 with k = the node's number of
 * children; NaN at childless nodes), div [B,N,3] (L1, KL(p||q), KL(q||p); NaN at childless nodes). */
int32_t oracle_node_analysis(const OracleIn *in, double *acc, double *dv, int32_t *status)
{
    if (!in || !acc || !dv || !status) return OTLP_ERR_ARG;
    for (int b = 0; b < in->B; ++b) status[b] = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < (int64_t)in->B * in->N; ++r) {
        int b = (int)(r / in->N), a = (int)(r % in->N), N = in->N, V = in->V;
        const int32_t *parent = in->parent + (size_t)b * (size_t)in->topo_seq_stride;
        int k = 0;
        for (int c = a + 1; c < N; ++c) k += parent[c] == a;
        double *o = acc + (size_t)r * 4, *d = dv + (size_t)r * 3;
        for (int i = 0; i < 4; ++i) o[i] = NAN;
        for (int i = 0; i < 3; ++i) d[i] = NAN;
        if (k == 0) continue;
        double *P = (double *)malloc(sizeof(double) * (size_t)V), *Q = (double *)malloc(sizeof(double) * (size_t)V);
        int rc = (!P || !Q) ? OTLP_ERR_ALLOC : node_law(in, b, a, 0, P);
        if (!rc) rc = node_law(in, b, a, 1, Q);
        if (!rc) rc = oracle_acceptance(P, Q, V, k, o);
        if (!rc) rc = oracle_divergences(P, Q, V, d);
        if (rc) {
#pragma omp critical
            status[b] = rc;
        }
        free(P); free(Q);
    }
    return OTLP_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* latency model (Appendix E, equation (8)) and the throughput estimate of Section 6            */
/* ------------------------------------------------------------------------------------------ */
/*
 * t_q[l], t_p[l]: measured draft / target forward times at context length l (tables of n_len
 * entries; a length beyond the table uses its last entry).  For action (K, L1, L2) at context length
 * ctx:  T = sum_{j<L1} t_q(ctx + j) + sum_{j<L2} t_q(ctx + L1 + j K) + t_p(ctx + L1 + K L2).
 */
static double tab(const double *t, int n, int l) { return t[l < 0 ? 0 : (l >= n ? n - 1 : l)]; }
int32_t oracle_latency_model(const double *t_q, const double *t_p, int32_t n_len, int32_t ctx,
                             const int32_t *actions /* [A,3] K,L1,L2 */, int32_t A, double *T_hat)
{
    if (!t_q || !t_p || !actions || !T_hat || n_len <= 0 || A <= 0) return OTLP_ERR_ARG;
    for (int a = 0; a < A; ++a) {
        int K = actions[3 * a], L1 = actions[3 * a + 1], L2 = actions[3 * a + 2];
        double s = 0.0;
        for (int j = 0; j < L1; ++j) s += tab(t_q, n_len, ctx + j);
        for (int j = 0; j < L2; ++j) s += tab(t_q, n_len, ctx + L1 + j * K);
        s += tab(t_p, n_len, ctx + L1 + K * L2);
        T_hat[a] = s;
    }
    return OTLP_OK;
}
/* Section 6, the policy's throughput estimate: sum_a pi(a) E[a] / sum_a pi(a) T[a] */
double oracle_tps_estimate(const double *pi, const double *E, const double *T_hat, int32_t A)
{
    double num = 0.0, den = 0.0;
    for (int a = 0; a < A; ++a) { num += pi[a] * E[a]; den += pi[a] * T_hat[a]; }
    return num / den;
}
