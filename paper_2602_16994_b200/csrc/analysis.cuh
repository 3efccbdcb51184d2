// Offline analysis of a draft tree on the resident node data of the every-node kernel (tree.cuh in its
// analysis instantiation): acceptance rates (Definition 5.1, Algorithms 6-9), the divergences between
// target and draft (Section 5's L1, the selector's KL features of Section 6), branching probabilities
// (Definition 5.3, Algorithms 11-14) and the block-efficiency sum of equation (3); and the forward-time
// model of equation (8).
//
// Division of work.  The every-node kernel holds a node's e_p, e_q on chip with its dominant tokens
// exact; in analysis mode it runs, before the SpecInfer recursion, read-only sweeps for the vocabulary-wide
// sums (the functors below) and SpecTr's bisection for rho*, and dumps per node the scalars everything
// else follows from (AnRec).  spec_branch_kernel (one warp per node) turns them into branching
// probabilities -- for SpecInfer with uniformly picked children the dynamic programme of Algorithm 14 over
// the sets of remaining children -- and spec_reach_kernel multiplies them down the tree.
//
// Algorithm 9's last term vanishes identically: a token with positive final residual p_k(t) was above
// q(t) in every round, so its m(t) stayed 1 and p_k(t) (1 - m(t)) = 0; SpecInfer's acceptance rate is
// 1 - prod_i S_i with S_i the residual mass of round i, which the recursion already has.
#pragma once
#include "common.cuh"

namespace specv {

constexpr int AN_KDP = 10;            // uniform-order SpecInfer: the DP covers up to 2^AN_KDP sets of children

// per node, dumped by the every-node kernel in analysis mode
struct __align__(16) AnRec {
    double A[KMAX + 1][KMAX];   // A[i][t] = min(1, p_i(x_t) / q(x_t)) for round i < k; row k: p_k(x_t)
    double S[KMAX];             // residual mass of round i (0 once the state equals q)
    double px[KMAX], qx[KMAX];  // p(x_t), q(x_t)
    double rho, beta, pacc, s_res;   // SpecTr: division factor, beta(rho*), p_acc, sum (p - min(p/rho, q) gamma)+
    int k, valid, pad[2];
};

// ---- functors of the read-only sweeps: tail in fp32, listed tokens in fp64 -----------------------------------
struct FnL1Min {        // a0: sum |p - q|, a1: sum min(p, q)
    float ipf, iqf; double ip, iq;
    __device__ __forceinline__ void tail(float ep, float eq, float &a0, float &a1) const
    { const float p = ep * ipf, q = eq * iqf; a0 += fabsf(p - q); a1 += fminf(p, q); }
    __device__ __forceinline__ void exact(double ep, double eq, double &a0, double &a1) const
    { const double p = ep * ip, q = eq * iq; a0 += fabs(p - q); a1 += fmin(p, q); }
};
struct FnNssNaive {     // a0: sum p (1 - (1-q)^k)  (Algorithm 6), a1: sum (p-q)+ (1 - (1-q)^(k-1))  (Algorithm 7)
    float ipf, iqf; double ip, iq; float kf; double kd;
    __device__ __forceinline__ void tail(float ep, float eq, float &a0, float &a1) const
    {
        const float p = ep * ipf, q = eq * iqf;
        const float l = log1pf(-fminf(q, 1.f));
        a0 += p * (-expm1f(kf * l));
        a1 += fmaxf(p - q, 0.f) * (kf > 1.f ? -expm1f((kf - 1.f) * l) : 0.f);
    }
    __device__ __forceinline__ void exact(double ep, double eq, double &a0, double &a1) const
    {
        const double p = ep * ip, q = eq * iq;
        const double l = log1p(-fmin(q, 1.0));
        a0 += p * (-expm1(kd * l));
        a1 += fmax(p - q, 0.0) * (kd > 1.0 ? -expm1((kd - 1.0) * l) : 0.0);
    }
};
struct FnBeta {         // a0: beta(rho) = sum min(p / rho, q)   (Appendix B, above Algorithm 3)
    float ipf, iqf; double ip, iq;   // ip already divided by rho
    __device__ __forceinline__ void tail(float ep, float eq, float &a0, float &) const { a0 += fminf(ep * ipf, eq * iqf); }
    __device__ __forceinline__ void exact(double ep, double eq, double &a0, double &) const { a0 += fmin(ep * ip, eq * iq); }
};
struct FnSpecTrRes {    // a0: sum d, a1: sum d (1 - (1-r)^k), d = (p - min(p/rho, q) gamma)+, r = (q - p/rho)+ / (1-beta)
    float ipf, iqf, irf, gf, ibf, kf; double ip, iq, ir, g, ib, kd;     // ir = 1/rho, ib = 1/(1-beta) (0 when beta = 1)
    __device__ __forceinline__ void tail(float ep, float eq, float &a0, float &a1) const
    {
        const float p = ep * ipf, q = eq * iqf, pr = p * irf;
        const float d = fmaxf(p - fminf(pr, q) * gf, 0.f);
        const float r = fminf(fmaxf(q - pr, 0.f) * ibf, 1.f);
        a0 += d;
        a1 += d * (-expm1f(kf * log1pf(-r)));
    }
    __device__ __forceinline__ void exact(double ep, double eq, double &a0, double &a1) const
    {
        const double p = ep * ip, q = eq * iq, pr = p * ir;
        const double d = fmax(p - fmin(pr, q) * g, 0.0);
        const double r = fmin(fmax(q - pr, 0.0) * ib, 1.0);
        a0 += d;
        a1 += d * (-expm1(kd * log1p(-r)));
    }
};

namespace analysis {

enum Solver { NSS = 0, NAIVE = 1, SPECTR = 2, SPECINFER = 3, SPECINFER_UNIFORM = 4, NSOLVER = 5 };

struct BParams {
    int B, N;
    const int *parent, *token;
    long long topo_stride;
    const AnRec *an;         // [B*N]
    float *acc;              // [B,N,4]: entry 3 (SpecInfer) is written here; NaN at childless nodes
    float *branch;           // [NSOLVER][B,N]: probability of moving from the parent into the node (root: 1)
};

__device__ __forceinline__ double clip1(double r) { return r < 1.0 ? r : 1.0; }
__device__ __forceinline__ double ratio(double P, double Q) { return !(P > 0.0) ? 0.0 : (!(Q > 0.0) ? CUDART_INF : P / Q); }

// One warp per node with children: branching probabilities of the five solvers into each child.
// A child whose token an earlier sibling carries is never moved to (the walk takes the first): 0.
__global__ void __launch_bounds__(128) spec_branch_kernel(const BParams P)
{
    __shared__ double dp[4][1 << AN_KDP];
    const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long node = (long long)blockIdx.x * 4 + wib;
    if (node >= (long long)P.B * P.N) return;
    const int b = (int)(node / P.N), a = (int)(node % P.N);
    const long long BN = (long long)P.B * P.N;
    if (a == 0 && lane < NSOLVER) P.branch[(long long)lane * BN + node] = 1.f;
    const AnRec &R = P.an[node];
    const int k = R.k;
    if (k <= 0 || !R.valid) {
        if (lane == 0) P.acc[node * 4 + 3] = CUDART_NAN_F;
        return;
    }
    const int *parent = P.parent + (long long)b * P.topo_stride;
    const int *token = P.token + (long long)b * P.N;
    // the children (list order) and their tokens: lane j holds child j
    int child = -1, tok = -1;
    {
        int seen = 0;
        for (int c0 = a + 1; c0 < P.N && seen < k; c0 += 32) {
            const int c = c0 + lane;
            const bool is = c < P.N && __ldg(parent + c) == a;
            const unsigned bal = __ballot_sync(0xffffffffu, is);
            // child number pos sits in lane pos
            for (int l = 0; l < 32; ++l) {
                if (!((bal >> l) & 1u)) continue;
                const int pos = seen + __popc(bal & ((1u << l) - 1u));
                const int cc = c0 + l;
                if (lane == pos) { child = cc; tok = __ldg(token + cc); }
            }
            seen += __popc(bal);
        }
    }
    // SpecInfer acceptance (Algorithm 9): 1 - prod S_i
    if (lane == 0) {
        double prej = 1.0;
        for (int i = 0; i < k; ++i) prej *= R.S[i];
        P.acc[node * 4 + 3] = (float)(1.0 - prej);
    }
    const bool mine = lane < k;
    bool dup = false;
    for (int l = 0; l < k; ++l) {
        const int tl = __shfl_sync(0xffffffffu, tok, l);
        if (mine && l < lane && tl == tok) dup = true;
    }
    const double pj = mine ? R.px[lane] : 0.0, qj = mine ? R.qx[lane] : 0.0;
    double out[NSOLVER] = {0.0, 0.0, 0.0, 0.0, 0.0};
    // NSS (Algorithm 11)
    out[NSS] = pj;
    // Naive (Algorithm 12): a = min(1, p(X_1)/q(X_1)); residual (p - q)+ / S_1
    {
        const double a1 = clip1(ratio(R.px[0], R.qx[0]));
        const double S1 = R.S[0];
        const double res = S1 > 0.0 ? fmax(pj - qj, 0.0) / S1 : pj;
        const int t0 = __shfl_sync(0xffffffffu, tok, 0);
        out[NAIVE] = (1.0 - a1) * res + (tok == t0 ? a1 : 0.0);
    }
    // SpecTr (Algorithm 13)
    {
        const double rho = R.rho;
        const double gamma = R.beta > 0.0 ? R.pacc / R.beta : 0.0;
        const double aj = mine ? clip1(ratio(pj, qj) / rho) : 0.0;
        double pre = 1.0, s = 0.0;
        for (int l = 0; l < k; ++l) {
            const double al = __shfl_sync(0xffffffffu, aj, l);
            const int tl = __shfl_sync(0xffffffffu, tok, l);
            if (tl == tok) s += al * pre;
            pre *= 1.0 - al;
        }
        const double res = R.s_res > 0.0 ? fmax(pj - fmin(pj / rho, qj) * gamma, 0.0) / R.s_res : pj;
        out[SPECTR] = s + res * pre;
    }
    // SpecInfer, children tried in list order: child l is tested in round l with A[l][l]
    {
        double pre = 1.0, s = 0.0;
        for (int l = 0; l < k; ++l) {
            const double al = R.A[l][l];
            const int tl = __shfl_sync(0xffffffffu, tok, l);
            if (tl == tok) s += al * pre;
            pre *= 1.0 - al;
        }
        out[SPECINFER] = s + (mine ? R.A[k][lane] : 0.0) * pre;
    }
    // SpecInfer, the next child picked uniformly (Algorithm 14): dynamic programme over the sets of children
    // still in S (bit t of the mask: child t), sets visited in increasing order, 32 per step
    if (k <= AN_KDP) {
        double *Bt = dp[wib];
        int toks[AN_KDP];
#pragma unroll
        for (int t = 0; t < AN_KDP; ++t) toks[t] = __shfl_sync(0xffffffffu, tok, t);
        for (int xi = 0; xi < k; ++xi) {
            const int tx = __shfl_sync(0xffffffffu, tok, xi);
            const double pkx = R.A[k][xi];
            const int nS = 1 << k;
            if (lane == 0) Bt[0] = pkx;
            __syncwarp();
            // all sets with cnt members depend only on sets with cnt - 1 members
            for (int cnt = 1; cnt <= k; ++cnt) {
                for (int S0 = 0; S0 < nS; S0 += 32) {
                    const int Sm = S0 + lane;
                    if (Sm < nS && __popc(Sm) == cnt) {
                        const int i = k - cnt;
                        double s = 0.0;
#pragma unroll
                        for (int t = 0; t < AN_KDP; ++t)
                            if (t < k && ((Sm >> t) & 1)) {
                                const double at = R.A[i][t];
                                s += at * (toks[t] == tx ? 1.0 : 0.0) + (1.0 - at) * Bt[Sm & ~(1 << t)];
                            }
                        Bt[Sm] = s / (double)cnt;
                    }
                }
                __syncwarp();
            }
            const double v = Bt[nS - 1];
            if (lane == xi) out[SPECINFER_UNIFORM] = v;
            __syncwarp();
        }
    } else {
        out[SPECINFER_UNIFORM] = CUDART_NAN;
    }
    if (mine) {
#pragma unroll
        for (int s = 0; s < NSOLVER; ++s) P.branch[(long long)s * BN + (long long)b * P.N + child] = dup ? 0.f : (float)out[s];
    }
}

struct RParams {
    int B, N;
    const int *parent;
    long long topo_stride;
    const float *branch;     // [NSOLVER][B,N]
    float *reach;            // [NSOLVER][B,N]: product of the branching probabilities along the node's path
    float *block_eff;        // [NSOLVER][B]: sum of reach over the nodes = E[tau + 1 | tree]  (equation (3))
};

// one thread per (solver, sequence): parents come before their children
__global__ void spec_reach_kernel(const RParams P)
{
    const int id = blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= NSOLVER * P.B) return;
    const int s = id / P.B, b = id % P.B;
    const int *parent = P.parent + (long long)b * P.topo_stride;
    const float *br = P.branch + ((long long)s * P.B + b) * P.N;
    float *re = P.reach + ((long long)s * P.B + b) * P.N;
    double total = 0.0;
    for (int a = 0; a < P.N; ++a) {
        const int pa = parent[a];
        const double r = a == 0 ? 1.0 : ((pa >= 0 && pa < a) ? (double)re[pa] * (double)br[a] : CUDART_NAN);
        re[a] = (float)r;
        total += r;
    }
    P.block_eff[(long long)s * P.B + b] = (float)total;
}

// Equation (8): forward-pass time of every action (K, L1, L2) at context length ctx from the measured
// tables t_q, t_p (a length beyond a table uses its last entry); one thread per action.
struct LParams {
    const double *t_q, *t_p;
    int n_len, ctx, A;
    const int *actions;      // [A,3]
    double *T_hat;           // [A]
};
__global__ void spec_latency_kernel(const LParams P)
{
    const int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= P.A) return;
    const int K = P.actions[3 * a], L1 = P.actions[3 * a + 1], L2 = P.actions[3 * a + 2];
    auto tab = [&](const double *t, int l) { return t[l < 0 ? 0 : (l >= P.n_len ? P.n_len - 1 : l)]; };
    double s = 0.0;
    for (int j = 0; j < L1; ++j) s += tab(P.t_q, P.ctx + j);
    for (int j = 0; j < L2; ++j) s += tab(P.t_q, P.ctx + L1 + j * K);
    s += tab(P.t_p, P.ctx + L1 + K * L2);
    P.T_hat[a] = s;
}

}  // namespace analysis
}  // namespace specv
