/*
 * spec_oracle.c -- slow, plain, double-precision CPU statement of draft-tree verification.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the checker the CUDA library is compared against.
 * It shares no code with the CUDA path, is never called by the product path, and is not tuned.
 *
 * What it computes, and the passage each function follows:
 *   oracle_row_probs      logits -> sampling distribution (temperature, top-k, top-p).  The paper
 *                         names temperature and nucleus sampling only (Section 4 experimental
 *                         setup); the tie rules are this build's reading (see the function).
 *   oracle_inverse_cdf    a draw from a weight vector by inverting its running sum
 *                         ("Sample Y ~ p", Algorithm 4 last line; Algorithm 2 residual draw).
 *   oracle_specinfer      Algorithm 4 (SpecInfer OTLP solver) used top-down as Section 3.2
 *                         "OT-based algorithms" states: solve at a node, move to the child whose
 *                         token was output, stop when the output is not a child.
 *   oracle_traversal      Traversal Verification, Section 3.2: bottom-up, reduces to block
 *                         verification for one path; the weight recursion is Section 3.1
 *                         "Block verification".  The sibling rule is a reconstruction that the
 *                         tests pin by exact enumeration (losslessness), not by a printed example.
 *   oracle_*_tables       the same per-node arithmetic evaluated at every node as if it were
 *                         reached (used to check the CUDA path's speculative per-node outputs).
 *
 * Pins (tests/test_oracle_*.py): exact output law == target law on tiny vocabularies for root
 * and delayed trees; k=1 reduces to naive speculative sampling with acceptance sum(min(p,q));
 * SpecInfer acceptance rate == Algorithm 9; uniform-order branching == Algorithm 14; one-path
 * Traversal == block verification and beats naive; depth-1 Traversal == SpecInfer; softmax and
 * sort-based truncation against numpy/scipy; invariants.  No function here is unpinned.
 *
 * Conventions.  Node 0 is the root.  parent[i] < i.  children(a) = nodes with parent a in
 * increasing index order; duplicates (equal tokens) are separate nodes.  Children are tried in
 * list order (for i.i.d. children this has the same output law as Algorithm 4's uniform pick).
 * Acceptance is the strict test u < threshold with u in [0,1).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)
#define ORACLE_ERR_TOKEN (-2)
#define ORACLE_ERR_TOPOLOGY (-3)
#define ORACLE_ERR_NAN (-4)
#define ORACLE_ERR_ALLOC (-5)

/* ------------------------------------------------------------------------------------------ */
/* input widening: the oracle consumes the same arrays as the device path, widened exactly     */
/* ------------------------------------------------------------------------------------------ */
static double widen_logit(const void *base, int dtype, int64_t idx)
{
    if (dtype == 0)
        return (double)((const float *)base)[idx];
    uint16_t h = ((const uint16_t *)base)[idx]; /* bf16 bit pattern */
    uint32_t w = (uint32_t)h << 16;
    float f;
    memcpy(&f, &w, 4);
    return (double)f;
}

/* ------------------------------------------------------------------------------------------ */
/* O1: logits -> sampling distribution                                                         */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    double z;
    int t;
} ZT;

static int cmp_zt_desc(const void *a, const void *b)
{
    const ZT *x = (const ZT *)a, *y = (const ZT *)b;
    if (x->z > y->z) return -1;
    if (x->z < y->z) return 1;
    return (x->t > y->t) - (x->t < y->t);
}

/*
 * z[V] logits (already widened).  T > 0.  top_k: 0 or >= V means off.  top_p: >= 1 means off.
 * Steps: y = z/T; m = max y; e = exp(y - m).
 *   top-k: v_k = k-th largest logit value counted with multiplicity; keep z >= v_k (ties at the
 *          k-th value are all kept, so the kept set does not depend on token order).
 *   top-p: within the kept set, tokens with equal logit form a group; groups ordered by value,
 *          largest first; with masses normalised over the kept set, keep the fewest leading
 *          groups whose cumulative mass is >= top_p (whole groups).
 *   p = e / sum(kept e) on kept tokens, 0 elsewhere.
 * stats[8]: 0 max y, 1 sum of kept e, 2 kept count, 3 entropy (nats), 4 largest p,
 *           5 nucleus margin (distance from top_p to the nearer neighbouring cumulative mass;
 *             1 when top-p is off), 6 threshold logit value of the kept set (-inf when nothing
 *             is cut), 7 sum of all e before truncation.
 */
int oracle_row_probs(const double *z, int32_t V, double T, int32_t top_k, double top_p,
                     double *probs, double *stats)
{
    if (!z || !probs || V <= 0 || !(T > 0.0) || top_k < 0 || !(top_p > 0.0))
        return ORACLE_ERR_ARG;
    double m = -INFINITY;
    for (int t = 0; t < V; ++t) {
        if (isnan(z[t])) return ORACLE_ERR_NAN;
        double y = z[t] / T;
        if (y > m) m = y;
    }
    if (!isfinite(m)) return ORACLE_ERR_NAN;
    double *e = (double *)malloc(sizeof(double) * (size_t)V);
    if (!e) return ORACLE_ERR_ALLOC;
    double sum_all = 0.0;
    for (int t = 0; t < V; ++t) {
        e[t] = exp(z[t] / T - m);
        sum_all += e[t];
    }
    double thr = -INFINITY; /* keep z >= thr */
    double margin = 1.0;
    int use_k = (top_k > 0 && top_k < V);
    int use_p = (top_p < 1.0);
    if (use_k || use_p) {
        ZT *s = (ZT *)malloc(sizeof(ZT) * (size_t)V);
        if (!s) { free(e); return ORACLE_ERR_ALLOC; }
        for (int t = 0; t < V; ++t) { s[t].z = z[t]; s[t].t = t; }
        qsort(s, (size_t)V, sizeof(ZT), cmp_zt_desc);
        int n_kept = V;
        if (use_k) {
            thr = s[top_k - 1].z;
            n_kept = top_k;
            while (n_kept < V && s[n_kept].z >= thr) ++n_kept; /* ties at the k-th value */
        }
        if (use_p) {
            double zk = 0.0;
            for (int i = 0; i < n_kept; ++i) zk += e[s[i].t];
            double cum = 0.0, prev = 0.0;
            int i = 0;
            while (i < n_kept) {
                double v = s[i].z;
                int j = i;
                while (j < n_kept && s[j].z == v) { cum += e[s[j].t]; ++j; }
                i = j;
                if (cum / zk >= top_p) {
                    double lo = top_p - prev / zk, hi = cum / zk - top_p;
                    margin = lo < hi ? lo : hi;
                    thr = v;
                    break;
                }
                prev = cum;
            }
            /* if rounding kept cum/zk below top_p to the end, everything kept stays */
        }
        free(s);
    }
    double zsum = 0.0;
    int kept = 0;
    for (int t = 0; t < V; ++t)
        if (z[t] >= thr) { zsum += e[t]; ++kept; }
    double H = 0.0, top1 = 0.0;
    for (int t = 0; t < V; ++t) {
        double p = (z[t] >= thr) ? e[t] / zsum : 0.0;
        probs[t] = p;
        if (p > 0.0) H -= p * log(p);
        if (p > top1) top1 = p;
    }
    if (stats) {
        stats[0] = m; stats[1] = zsum; stats[2] = (double)kept; stats[3] = H;
        stats[4] = top1; stats[5] = margin; stats[6] = thr; stats[7] = sum_all;
    }
    free(e);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* O4: inverse CDF                                                                             */
/* ------------------------------------------------------------------------------------------ */
/*
 * w[V] >= 0, not necessarily normalised.  W = sum w (index order).  target = u*W.
 * Returns the smallest t with C_t > target, C_t = w_0 + ... + w_t; if rounding leaves none, the
 * last t with w_t > 0.  margin = min(target - C_{t-1}, C_t - target) / W.  Returns -1 if W <= 0.
 */
int32_t oracle_inverse_cdf(const double *w, int32_t V, double u, double *margin)
{
    double W = 0.0;
    for (int t = 0; t < V; ++t) W += w[t];
    if (!(W > 0.0)) { if (margin) *margin = 0.0; return -1; }
    double target = u * W, c = 0.0;
    int last_pos = -1;
    for (int t = 0; t < V; ++t) {
        double prev = c;
        c += w[t];
        if (w[t] > 0.0) last_pos = t;
        if (c > target) {
            if (margin) {
                double lo = target - prev, hi = c - target;
                *margin = (lo < hi ? lo : hi) / W;
            }
            return t;
        }
    }
    if (margin) *margin = 0.0;
    return last_pos;
}

/* ------------------------------------------------------------------------------------------ */
/* one sequence: inputs                                                                        */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t N, V, dtype;
    const void *target_logits; /* row of node a starts at element a*node_stride */
    const void *draft_logits;
    int64_t node_stride;
    const int32_t *parent, *token;
    double T;
    int32_t top_k;
    double top_p;
    const float *u_accept, *u_bonus;
} Seq;

static int row_dist(const Seq *s, int which, int a, double *out, double *stats)
{
    const void *base = which ? s->draft_logits : s->target_logits;
    double *z = (double *)malloc(sizeof(double) * (size_t)s->V);
    if (!z) return ORACLE_ERR_ALLOC;
    for (int t = 0; t < s->V; ++t) z[t] = widen_logit(base, s->dtype, (int64_t)a * s->node_stride + t);
    int rc = oracle_row_probs(z, s->V, s->T, s->top_k, s->top_p, out, stats);
    free(z);
    return rc;
}

static int children_of(const Seq *s, int a, int *out)
{
    int k = 0;
    for (int c = a + 1; c < s->N; ++c)
        if (s->parent[c] == a) out[k++] = c;
    return k;
}

static int check_topology(const Seq *s)
{
    if (s->N <= 0 || s->V <= 0) return ORACLE_ERR_ARG;
    if (s->parent[0] != -1) return ORACLE_ERR_TOPOLOGY;
    for (int i = 1; i < s->N; ++i) {
        if (s->parent[i] < 0 || s->parent[i] >= i) return ORACLE_ERR_TOPOLOGY;
        if (s->token[i] < 0 || s->token[i] >= s->V) return ORACLE_ERR_TOKEN;
    }
    return ORACLE_OK;
}

/* acceptance ratio P(x)/Q(x) clipped at 1; P <= 0 never accepts; a token outside the draft
 * support (Q <= 0 < P) always does. */
static double ratio_clipped(double P, double Q)
{
    if (!(P > 0.0)) return 0.0;
    if (!(Q > 0.0)) return 1.0;
    double r = P / Q;
    return r < 1.0 ? r : 1.0;
}

/* per-sequence result record shared by the two verifiers */
typedef struct {
    int32_t *accepted_node; /* [1] */
    int32_t *accept_len;    /* [1] */
    int32_t *out_tokens;    /* [N]: path tokens, then the bonus token, then -1 */
    int32_t *bonus_token;   /* [1] */
    double *residual;       /* [V] or NULL: the distribution the bonus was drawn from */
    double *bonus_margin;   /* [1] or NULL */
    int32_t *trace_node;    /* [N] nodes whose uniform was consumed, in order */
    double *trace_thr;      /* [N] the threshold each was compared with */
    int32_t *trace_acc;     /* [N] 1 if u < threshold */
    int32_t *trace_len;     /* [1] */
} SeqOut;

static void emit_path(const Seq *s, const SeqOut *o, int node, int bonus)
{
    int len = 0;
    for (int a = node; a != 0; a = s->parent[a]) ++len;
    *o->accepted_node = node;
    *o->accept_len = len;
    *o->bonus_token = bonus;
    for (int i = 0; i < s->N; ++i) o->out_tokens[i] = -1;
    int i = len;
    o->out_tokens[len] = bonus;
    for (int a = node; a != 0; a = s->parent[a]) o->out_tokens[--i] = s->token[a];
}

/* ------------------------------------------------------------------------------------------ */
/* O2: SpecInfer (Algorithm 4) composed top-down (Section 3.2)                                 */
/* ------------------------------------------------------------------------------------------ */
/*
 * One OTLP solve at a node.  P (target) is replaced by the residual reached.  Children tried in
 * list order.  Returns the position of the accepted child or -1.  r_out[j] receives the
 * threshold used for child j (only the ones reached).  If never_accept is set every child is
 * rejected (table mode).
 */
static int specinfer_solve(double *P, const double *Q, int V, const int32_t *x, const double *u,
                           int k, int never_accept, double *r_out, int *n_tried)
{
    *n_tried = 0;
    for (int j = 0; j < k; ++j) {
        double r = ratio_clipped(P[x[j]], Q[x[j]]);
        r_out[j] = r;
        *n_tried = j + 1;
        if (!never_accept && u[j] < r) return j;
        double S = 0.0;
        for (int t = 0; t < V; ++t) {
            double d = P[t] - Q[t];
            if (d > 0.0) S += d;
        }
        if (S > 0.0)
            for (int t = 0; t < V; ++t) {
                double d = P[t] - Q[t];
                P[t] = d > 0.0 ? d / S : 0.0;
            }
        /* S == 0 would mean P == Q, whose ratio is 1 and cannot be rejected; P is left as is */
    }
    return -1;
}

static int specinfer_seq(const Seq *s, const SeqOut *o)
{
    int rc = check_topology(s);
    if (rc) return rc;
    int V = s->V, N = s->N;
    double *P = (double *)malloc(sizeof(double) * (size_t)V);
    double *Q = (double *)malloc(sizeof(double) * (size_t)V);
    int *ch = (int *)malloc(sizeof(int) * (size_t)N);
    int32_t *x = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    double *u = (double *)malloc(sizeof(double) * (size_t)N);
    double *r = (double *)malloc(sizeof(double) * (size_t)N);
    if (!P || !Q || !ch || !x || !u || !r) { rc = ORACLE_ERR_ALLOC; goto done; }
    *o->trace_len = 0;
    int cur = 0;
    for (;;) {
        rc = row_dist(s, 0, cur, P, NULL);
        if (rc) goto done;
        int k = children_of(s, cur, ch);
        int hit = -1;
        if (k > 0) {
            rc = row_dist(s, 1, cur, Q, NULL);
            if (rc) goto done;
            for (int j = 0; j < k; ++j) { x[j] = s->token[ch[j]]; u[j] = (double)s->u_accept[ch[j]]; }
            int tried = 0;
            hit = specinfer_solve(P, Q, V, x, u, k, 0, r, &tried);
            for (int j = 0; j < tried; ++j) {
                int n = (*o->trace_len)++;
                o->trace_node[n] = ch[j];
                o->trace_thr[n] = r[j];
                o->trace_acc[n] = (j == hit);
            }
        }
        if (hit >= 0) { cur = ch[hit]; continue; }
        double mg = 0.0;
        int y = oracle_inverse_cdf(P, V, (double)s->u_bonus[cur], &mg);
        if (o->bonus_margin) *o->bonus_margin = mg;
        if (o->residual) {
            double W = 0.0;
            for (int t = 0; t < V; ++t) W += P[t];
            for (int t = 0; t < V; ++t) o->residual[t] = P[t] / W;
        }
        emit_path(s, o, cur, y);
        break;
    }
done:
    free(P); free(Q); free(ch); free(x); free(u); free(r);
    return rc;
}

/* ------------------------------------------------------------------------------------------ */
/* O3: Traversal Verification (Section 3.2; weights as in Section 3.1 block verification)      */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    const Seq *s;
    const SeqOut *o;
    int never_accept;   /* table mode: reject everything, fill the tables */
    double *w_in;       /* [N] or NULL */
    double *w_fin;      /* [N] or NULL */
    int32_t *bonus_all; /* [N] or NULL: the bonus this node would draw if it were accepted */
    int rc;
} Trav;

/* weight handed to a child: min(1, w * P(x)/Q(x)); a zero incoming weight stays zero. */
static double child_weight(double w, double P, double Q)
{
    if (!(w > 0.0) || !(P > 0.0)) return 0.0;
    if (!(Q > 0.0)) return 1.0;
    double v = w * (P / Q);
    return v < 1.0 ? v : 1.0;
}

/* returns 1 if some node of the subtree of a (a included) was accepted */
static int trav_visit(Trav *tv, int a, double w)
{
    const Seq *s = tv->s;
    int V = s->V;
    int accepted = 0;
    double *P = (double *)malloc(sizeof(double) * (size_t)V);
    double *Q = NULL;
    int *ch = (int *)malloc(sizeof(int) * (size_t)s->N);
    if (!P || !ch) { tv->rc = ORACLE_ERR_ALLOC; goto out; }
    if (tv->w_in) tv->w_in[a] = w;
    tv->rc = row_dist(s, 0, a, P, NULL);
    if (tv->rc) goto out;
    int k = children_of(s, a, ch);
    if (k > 0) {
        Q = (double *)malloc(sizeof(double) * (size_t)V);
        if (!Q) { tv->rc = ORACLE_ERR_ALLOC; goto out; }
        tv->rc = row_dist(s, 1, a, Q, NULL);
        if (tv->rc) goto out;
    }
    for (int j = 0; j < k; ++j) {
        int c = ch[j];
        int xc = s->token[c];
        double wc = child_weight(w, P[xc], Q[xc]);
        if (trav_visit(tv, c, wc)) { accepted = 1; goto out; }
        if (tv->rc) goto out;
        /* the subtree of c was rejected: block-verification step on (w, P) */
        double S = 0.0;
        for (int t = 0; t < V; ++t) {
            double d = w * P[t] - Q[t];
            if (d > 0.0) S += d;
        }
        if (S > 0.0) {
            for (int t = 0; t < V; ++t) {
                double d = w * P[t] - Q[t];
                P[t] = d > 0.0 ? d / S : 0.0;
            }
            /* the sum is formed as S + (1 - w): 1 - w is exact for w in [1/2, 1], so a weight of exactly 1
             * stays exactly 1; (S + 1) - w would round S to the grid of 1 and the deviation of w from 1
             * grows by 1/S with every later step */
            w = S / (S + (1.0 - w));
        } else {
            w = (w >= 1.0) ? 1.0 : 0.0;
        }
    }
    /* every child subtree is gone: a is a leaf of what remains, with weight w and law P */
    if (tv->w_fin) tv->w_fin[a] = w;
    if (tv->bonus_all) {
        double mg;
        tv->bonus_all[a] = oracle_inverse_cdf(P, V, (double)s->u_bonus[a], &mg);
    }
    if (!tv->never_accept) {
        const SeqOut *o = tv->o;
        int hit = ((double)s->u_accept[a] < w) || a == 0;
        if (a != 0) {
            int n = (*o->trace_len)++;
            o->trace_node[n] = a;
            o->trace_thr[n] = w;
            o->trace_acc[n] = hit;
        }
        if (hit) {
            double mg = 0.0;
            int y = oracle_inverse_cdf(P, V, (double)s->u_bonus[a], &mg);
            if (o->bonus_margin) *o->bonus_margin = mg;
            if (o->residual) {
                double W = 0.0;
                for (int t = 0; t < V; ++t) W += P[t];
                for (int t = 0; t < V; ++t) o->residual[t] = P[t] / W;
            }
            emit_path(s, o, a, y);
            accepted = 1;
        }
    }
out:
    free(P); free(Q); free(ch);
    return accepted;
}

static int traversal_seq(const Seq *s, const SeqOut *o)
{
    int rc = check_topology(s);
    if (rc) return rc;
    *o->trace_len = 0;
    Trav tv = { s, o, 0, NULL, NULL, NULL, ORACLE_OK };
    int acc = trav_visit(&tv, 0, 1.0);
    if (tv.rc) return tv.rc;
    return acc ? ORACLE_OK : ORACLE_ERR_ARG;
}

/* ------------------------------------------------------------------------------------------ */
/* exported batch drivers (OpenMP over sequences: sequences are independent)                   */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t B, N, V, logits_dtype;
    const void *target_logits, *draft_logits; /* host */
    int64_t seq_stride, node_stride;          /* elements */
    const int32_t *parent;                    /* [N] or [B,N] */
    int64_t topo_seq_stride;                  /* 0: one topology for the batch */
    const int32_t *token;                     /* [B,N] */
    float temperature;
    int32_t top_k;
    float top_p;
    const float *temperature_per_seq; /* optional [B] */
    const float *u_accept, *u_bonus;  /* [B,N] */
} OracleIn;

typedef struct {
    int32_t *accepted_node, *accept_len; /* [B] */
    int32_t *out_tokens;                 /* [B,N] */
    int32_t *bonus_token;                /* [B] */
    double *residual;                    /* optional [B,V] */
    double *bonus_margin;                /* optional [B] */
    int32_t *trace_node;                 /* [B,N] */
    double *trace_thr;                   /* [B,N] */
    int32_t *trace_acc;                  /* [B,N] */
    int32_t *trace_len;                  /* [B] */
    int32_t *status;                     /* [B] */
} OracleOut;

static void make_seq(const OracleIn *in, int b, Seq *s)
{
    size_t esz = in->logits_dtype == 0 ? 4 : 2;
    s->N = in->N; s->V = in->V; s->dtype = in->logits_dtype;
    s->target_logits = (const char *)in->target_logits + (size_t)b * (size_t)in->seq_stride * esz;
    s->draft_logits = (const char *)in->draft_logits + (size_t)b * (size_t)in->seq_stride * esz;
    s->node_stride = in->node_stride;
    s->parent = in->parent + (size_t)b * (size_t)in->topo_seq_stride;
    s->token = in->token + (size_t)b * (size_t)in->N;
    s->T = (double)(in->temperature_per_seq ? in->temperature_per_seq[b] : in->temperature);
    s->top_k = in->top_k;
    s->top_p = (double)in->top_p;
    s->u_accept = in->u_accept + (size_t)b * (size_t)in->N;
    s->u_bonus = in->u_bonus + (size_t)b * (size_t)in->N;
}

static void make_out(const OracleIn *in, const OracleOut *out, int b, SeqOut *o)
{
    size_t N = (size_t)in->N;
    o->accepted_node = out->accepted_node + b;
    o->accept_len = out->accept_len + b;
    o->out_tokens = out->out_tokens + b * N;
    o->bonus_token = out->bonus_token + b;
    o->residual = out->residual ? out->residual + (size_t)b * (size_t)in->V : NULL;
    o->bonus_margin = out->bonus_margin ? out->bonus_margin + b : NULL;
    o->trace_node = out->trace_node + b * N;
    o->trace_thr = out->trace_thr + b * N;
    o->trace_acc = out->trace_acc + b * N;
    o->trace_len = out->trace_len + b;
}

static int check_in(const OracleIn *in, const OracleOut *out)
{
    if (!in || !out || in->B <= 0 || in->N <= 0 || in->V <= 0) return ORACLE_ERR_ARG;
    if (in->logits_dtype != 0 && in->logits_dtype != 1) return ORACLE_ERR_ARG;
    if (!in->target_logits || !in->draft_logits || !in->parent || !in->token) return ORACLE_ERR_ARG;
    if (!in->u_accept || !in->u_bonus) return ORACLE_ERR_ARG;
    if (!out->accepted_node || !out->accept_len || !out->out_tokens || !out->bonus_token) return ORACLE_ERR_ARG;
    if (!out->trace_node || !out->trace_thr || !out->trace_acc || !out->trace_len || !out->status) return ORACLE_ERR_ARG;
    return ORACLE_OK;
}

int32_t oracle_verify_specinfer(const OracleIn *in, const OracleOut *out)
{
    int rc = check_in(in, out);
    if (rc) return rc;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < in->B; ++b) {
        Seq s; SeqOut o;
        make_seq(in, b, &s);
        make_out(in, out, b, &o);
        out->status[b] = specinfer_seq(&s, &o);
    }
    return ORACLE_OK;
}

int32_t oracle_verify_traversal(const OracleIn *in, const OracleOut *out)
{
    int rc = check_in(in, out);
    if (rc) return rc;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < in->B; ++b) {
        Seq s; SeqOut o;
        make_seq(in, b, &s);
        make_out(in, out, b, &o);
        out->status[b] = traversal_seq(&s, &o);
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* per-node tables: every node evaluated as if reached                                         */
/* ------------------------------------------------------------------------------------------ */
/*
 * SpecInfer tables, all [B,N]:
 *   ratio[c]      threshold child c would be tested with if its parent were reached and all its
 *                 earlier siblings had been rejected (root: 1)
 *   next_child[a] first child c of a (list order) with u_accept[c] < ratio[c], else -1
 *   bonus_all[a]  token a would emit if the walk stopped at a: drawn with u_bonus[a] from the
 *                 residual after rejecting all children (from p itself at a leaf)
 */
int32_t oracle_specinfer_tables(const OracleIn *in, double *ratio, int32_t *next_child,
                                int32_t *bonus_all, int32_t *status)
{
    if (!in || !ratio || !next_child || !bonus_all || !status) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < in->B; ++b) {
        Seq s;
        make_seq(in, b, &s);
        int N = s.N, V = s.V;
        int rc = check_topology(&s);
        double *P = (double *)malloc(sizeof(double) * (size_t)V);
        double *Q = (double *)malloc(sizeof(double) * (size_t)V);
        int *ch = (int *)malloc(sizeof(int) * (size_t)N);
        int32_t *x = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
        double *u = (double *)malloc(sizeof(double) * (size_t)N);
        double *r = (double *)malloc(sizeof(double) * (size_t)N);
        if (!P || !Q || !ch || !x || !u || !r) rc = ORACLE_ERR_ALLOC;
        if (!rc) ratio[(size_t)b * N] = 1.0;
        for (int a = 0; a < N && !rc; ++a) {
            rc = row_dist(&s, 0, a, P, NULL);
            if (rc) break;
            int k = children_of(&s, a, ch);
            int first = -1;
            if (k > 0) {
                rc = row_dist(&s, 1, a, Q, NULL);
                if (rc) break;
                for (int j = 0; j < k; ++j) { x[j] = s.token[ch[j]]; u[j] = (double)s.u_accept[ch[j]]; }
                int tried;
                specinfer_solve(P, Q, V, x, u, k, 1, r, &tried);
                for (int j = 0; j < k; ++j) {
                    ratio[(size_t)b * N + ch[j]] = r[j];
                    if (first < 0 && u[j] < r[j]) first = ch[j];
                }
            }
            next_child[(size_t)b * N + a] = first;
            double mg;
            bonus_all[(size_t)b * N + a] = oracle_inverse_cdf(P, V, (double)s.u_bonus[a], &mg);
        }
        free(P); free(Q); free(ch); free(x); free(u); free(r);
        status[b] = rc;
    }
    return ORACLE_OK;
}

/*
 * Traversal tables, all [B,N]: w_in (weight handed down by the parent assuming every earlier
 * subtree was rejected), w_fin (weight the node is finally tested with), bonus_all (the draw
 * from the node's final law with u_bonus[node]).
 */
int32_t oracle_traversal_tables(const OracleIn *in, double *w_in, double *w_fin,
                                int32_t *bonus_all, int32_t *status)
{
    if (!in || !w_in || !w_fin || !bonus_all || !status) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < in->B; ++b) {
        Seq s;
        make_seq(in, b, &s);
        int rc = check_topology(&s);
        if (!rc) {
            size_t off = (size_t)b * (size_t)s.N;
            Trav tv = { &s, NULL, 1, w_in + off, w_fin + off, bonus_all + off, ORACLE_OK };
            trav_visit(&tv, 0, 1.0);
            rc = tv.rc;
        }
        status[b] = rc;
    }
    return ORACLE_OK;
}

/*
 * Row distributions and statistics for every node of every sequence.
 * which: 0 target, 1 draft.  probs: optional [B,N,V] doubles.  stats: optional [B,N,8] (layout
 * of oracle_row_probs).  Draft rows of leaves are computed too (the caller ignores them).
 */
int32_t oracle_tree_probs(const OracleIn *in, int32_t which, double *probs, double *stats,
                          int32_t *status)
{
    if (!in || !status) return ORACLE_ERR_ARG;
    int64_t rows = (int64_t)in->B * in->N;
    for (int b = 0; b < in->B; ++b) status[b] = ORACLE_OK;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
        int b = (int)(r / in->N), a = (int)(r % in->N);
        Seq s;
        make_seq(in, b, &s);
        double *tmp = probs ? probs + (size_t)r * (size_t)in->V
                            : (double *)malloc(sizeof(double) * (size_t)in->V);
        int rc = tmp ? row_dist(&s, which, a, tmp, stats ? stats + (size_t)r * 8 : NULL)
                     : ORACLE_ERR_ALLOC;
        if (!probs) free(tmp);
        if (rc) {
#pragma omp critical
            status[b] = rc;
        }
    }
    return ORACLE_OK;
}

/* batched inverse CDF over rows of float weights (the device entry point's counterpart) */
int32_t oracle_sample_bonus(const float *weights, int32_t R, int32_t V, const float *u,
                            int32_t *token, double *margin)
{
    if (!weights || !u || !token || R <= 0 || V <= 0) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < R; ++r) {
        double *w = (double *)malloc(sizeof(double) * (size_t)V);
        for (int t = 0; t < V; ++t) w[t] = (double)weights[(size_t)r * V + t];
        double mg = 0.0;
        token[r] = oracle_inverse_cdf(w, V, (double)u[r], &mg);
        if (margin) margin[r] = mg;
        free(w);
    }
    return ORACLE_OK;
}

int32_t oracle_max_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Number of threads the batch loops use from now on (n >= 1); arithmetic and results do not depend on it. */
void oracle_set_threads(int32_t n)
{
#ifdef _OPENMP
    extern void omp_set_num_threads(int);
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
