// SpecInfer verification as a walk (Algorithm 4 composed top-down, Section 3.2), one thread-block
// cluster per sequence, on top of the row statistics (stream.cuh / rowstat.cuh).
//
// With every row's normaliser known, the decision about a node's FIRST child needs no vocabulary-wide
// work: its threshold is min(1, p(x)/q(x)), two logits and two normalisers.  The cluster therefore walks
// down the tree with scalar arithmetic only, and brings a node's rows on chip (the same machinery as
// the every-node kernel of tree.cuh: producer warp + bulk-copy ring, e = 2^(z s - O) resident in registers and shared
// memory, one pass + one distributed-shared-memory exchange per sibling step, inverse-CDF search) only
// where Algorithm 4 needs a residual: at a node whose first child was rejected, and at the stop node
// for the bonus draw.  That is one or two resident nodes per sequence instead of every node of the tree.
//
// Before the walk the consumer threads of every CTA bring the sequence's scalars into shared memory in
// two batches of independent loads: topology, tokens, uniforms and the row records; then, for every
// non-root node, the two logits at its token in its parent's rows, exponentiated in fp64.
// After that a step down the tree is a few shared-memory reads.  The first child's test uses the
// normalisers of the statistics pass (fp32 exponentials: its threshold is good to a few 1e-7); a node
// that comes on chip gets its normalisers again from the resident e and the exact lists of verify.cuh.
//
// Every consumer warp of the cluster runs the same walk on the same numbers (the exchanges deliver
// bit-identical totals to all of them), so control flow agrees across the cluster without barriers.
// The thread that finds the bonus token writes all outputs of the sequence.
#pragma once
#include "analysis.cuh"
#include "stream.cuh"
#include "verify.cuh"

namespace specv {

constexpr int NWALK = 128;        // nodes per sequence the walk keeps in shared memory

struct WParams {
    int B, N, V, C, NSL;
    int slice_len, NS, nsm, off_x, off_list, off_es, off_ring;
    const void *zp, *zq;
    long long seq_stride, node_stride, topo_stride;
    const int *parent, *token;
    float T;
    const float *T_seq;
    const RowPart *part;      // [B*N*2][NSL]
    const float *u_accept, *u_bonus;
    SpecOut out;
    int solver;               // OT instantiation: 0 NSS (Algorithm 1), 1 NaiveTree (Algorithm 2), 2 SpecTr (Algorithm 3)
};

struct __align__(16) WHdr {
    uint64_t full[NSMAX], empty[NSMAX], xbar[2], cbar, req, ack;
    double wtile[NWMAX + 1][TMAX];
    WarpArea wa[NWMAX];
    int req_a, req_b, req_hq;
    int poison;
    // the sequence's scalars (written by the prologue of every sequence)
    int t_parent[NWALK], t_token[NWALK], t_fc[NWALK], t_kc[NWALK];
    float t_u[NWALK], t_ub[NWALK];
    double t_Z[2 * NWALK];        // normaliser of row (node, target / draft), in units of 2^O
    int t_O[2 * NWALK];
    float t_cut[2 * NWALK];
    double t_cp[NWALK], t_cq[NWALK];   // exact 2^(z s - O) of the node's token in its parent's target and draft rows
    int t_status;
};

// statistics of one row: normaliser, reference, cut
struct RowSum {
    double Z;
    int O;
    float cut;
};

// MINB: CTAs per SM the register budget is set for (1: up to 255 registers per thread, no spills)
// OT: the walk with one of the other OTLP solvers of Appendix B instead of SpecInfer (Section 3.2: move to the
// child whose token the solver put out, stop when the output is no child's token).  Every draw is then
// made known to the whole cluster (one more exchange), because the walk may go on from it.
template <int DT, int NW, int MINB, bool OT = false>
__global__ void __launch_bounds__((NW + 1) * 32, MINB) spec_walk_kernel(const WParams P)
{
    constexpr int NCONS = NW * 32;
    constexpr int TILE = NCONS * 8;
    constexpr int ESZ = DT == SPEC_BF16 ? 2 : 4;
    constexpr int ROWB = TILE * ESZ;
    constexpr int STAGE = 2 * ROWB;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    WHdr &S = *reinterpret_cast<WHdr *>(dyn_smem);
    double *xchg = reinterpret_cast<double *>(dyn_smem + P.off_x);   // [parity 2][rank C][warp NW][2]
    WarpList *lists = reinterpret_cast<WarpList *>(dyn_smem + P.off_list);   // [warp NW]
    float4 *es = reinterpret_cast<float4 *>(dyn_smem + P.off_es);    // [slot][p lo, p hi, q lo, q hi][NCONS]
    unsigned char *ring = dyn_smem + P.off_ring;
    const int C = P.C, NS = P.NS;
    const unsigned rank = cluster_ctarank();
    const int cid = blockIdx.x / C, NC = gridDim.x / C;
    const long long tok0 = (long long)rank * P.slice_len;
    const int n_slice = (int)max(0ll, min((long long)P.slice_len, (long long)P.V - tok0));
    const int ntiles = (n_slice + TILE - 1) / TILE;
    const int nsm = min(P.nsm, ntiles), nrg = ntiles - nsm;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&S.full[s], 1); mbar_init(&S.empty[s], NW); }
        mbar_init(&S.xbar[0], 1);
        mbar_init(&S.xbar[1], 1);
        mbar_init(&S.req, 1);
        mbar_init(&S.ack, 1);
        mbar_init(&S.cbar, NW);
        S.poison = 0;
        mbar_fence_init();
    }
    __syncthreads();
    cluster_sync_all();
    grid_dependency_wait();       // the row statistics come from the kernel before

    if (warp == NW) {
        // ======================= producer warp: loads the node the consumers ask for =====================
        int g = 0;
        uint32_t rphase = 0;
        for (;;) {
            int ok = 1;
            if (lane == 0) ok = mbar_wait(&S.req, rphase) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            rphase ^= 1u;
            if (!ok) { S.poison = 1; break; }
            const int a = *(volatile int *)&S.req_a, b = *(volatile int *)&S.req_b;
            const bool hq = *(volatile int *)&S.req_hq != 0;
            if (lane == 0) mbar_arrive(&S.ack);          // the request has been read: the next one may be posted
            if (a < 0) break;
            const long long row = (long long)b * P.seq_stride + (long long)a * P.node_stride + tok0;
            const unsigned char *src_p = (const unsigned char *)P.zp + row * ESZ;
            const unsigned char *src_q = (const unsigned char *)P.zq + row * ESZ;
            const bool aligned = ((((uintptr_t)src_p) | (hq ? (uintptr_t)src_q : 0)) & 15) == 0;
            bool fail = false;
            for (int i = 0; i < ntiles; ++i, ++g) {
                const int stage = g % NS, use = g / NS;
                if (use > 0) {
                    int w = 1;
                    if (lane == 0) w = mbar_wait(&S.empty[stage], (uint32_t)((use - 1) & 1)) ? 1 : 0;
                    w = __shfl_sync(0xffffffffu, w, 0);
                    if (!w || *(volatile int *)&S.poison) { S.poison = 1; fail = true; break; }
                }
                const int ntok = min(TILE, n_slice - i * TILE);
                unsigned char *dst_p = ring + (size_t)stage * STAGE, *dst_q = dst_p + ROWB;
                const unsigned char *sp = src_p + (size_t)i * ROWB, *sq = src_q + (size_t)i * ROWB;
                const uint32_t body = aligned ? (((uint32_t)ntok * ESZ) & ~15u) : 0u;
                if (ESZ == 2) {
                    for (int e = (int)(body / 2) + lane; e < ntok; e += 32) {
                        ((unsigned short *)dst_p)[e] = __ldg((const unsigned short *)sp + e);
                        if (hq) ((unsigned short *)dst_q)[e] = __ldg((const unsigned short *)sq + e);
                    }
                } else {
                    for (int e = (int)(body / 4) + lane; e < ntok; e += 32) {
                        ((float *)dst_p)[e] = __ldg((const float *)sp + e);
                        if (hq) ((float *)dst_q)[e] = __ldg((const float *)sq + e);
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    if (body) {
                        mbar_arrive_expect_tx(&S.full[stage], hq ? 2 * body : body);
                        bulk_g2s(dst_p, sp, body, &S.full[stage]);
                        if (hq) bulk_g2s(dst_q, sq, body, &S.full[stage]);
                    } else {
                        mbar_arrive(&S.full[stage]);
                    }
                }
            }
            if (fail) {
                if (lane == 0)
                    for (int k = 1; k <= NS && k <= g; ++k) {
                        const int gg = g - k;
                        mbar_wait(&S.full[gg % NS], (uint32_t)((gg / NS) & 1));
                    }
                break;
            }
        }
    } else {
        // ================================ consumer warps: the walk ==========================================
        WarpArea &W = S.wa[warp];
        const RingCtx rc = {S.full, S.empty, ring, NS, &S.poison};
        WarpList &L = lists[warp];
        int stage = 0;
        uint32_t phase = 0, cph = 0;
        int xn = 0;
        uint32_t aphase = 0;        // warp 0, lane 0: requests acknowledged so far (parity)
        bool posted = false;
        Resident R;

        for (int b = cid; b < P.B; b += NC) {
            const int *parent = P.parent + (long long)b * P.topo_stride;
            const int *token = P.token + (long long)b * P.N;
            NodeRows nr;
            nr.s_d = 1.4426950408889634 / (double)(P.T_seq ? __ldg(P.T_seq + b) : P.T);
            nr.s_hi = (float)nr.s_d;
            if ((double)nr.s_hi > nr.s_d) nr.s_hi = __uint_as_float(__float_as_uint(nr.s_hi) - 1u);
            nr.s_lo = (float)(nr.s_d - (double)nr.s_hi);
            if (!(nr.s_lo > 0.f)) nr.s_lo = 1.0e-30f;
            const double s_d = nr.s_d;

            // ---- first batch of loads: topology, tokens, uniforms, row records; the whole tree is checked ---------
            bar_sync(1, NCONS);                      // the previous sequence's scalars are no longer read
            if (tid == 0) S.t_status = 0;
            bar_sync(1, NCONS);
            {
                int st1 = 0;
                for (int i = tid; i < P.N; i += NCONS) {
                    const int pa = __ldg(parent + i);
                    if (i == 0 ? (pa != -1) : (pa < 0 || pa >= i)) st1 = max(st1, SPEC_DEV_TOPOLOGY);
                    int x = 0;
                    if (i > 0) {
                        x = __ldg(token + i);
                        if (x < 0 || x >= P.V) st1 = max(st1, SPEC_DEV_TOKEN);
                    }
                    S.t_parent[i] = pa; S.t_token[i] = x; S.t_fc[i] = P.N; S.t_kc[i] = 0;
                    S.t_u[i] = __ldg(P.u_accept + (long long)b * P.N + i);
                    S.t_ub[i] = __ldg(P.u_bonus + (long long)b * P.N + i);
                }
                for (int r2 = tid; r2 < 2 * P.N; r2 += NCONS) {
                    const RowPart *p = P.part + ((long long)b * 2 * P.N + r2);
                    const double Zr = __ldcg(&p->S);
                    const int Or = __ldcg(&p->O), bd = __ldcg(&p->bad);
                    // a row is not finite if it holds NaN / +inf, or no finite logit at all
                    if (bd == ROW_TIMEOUT)
                        st1 = max(st1, SPEC_DEV_TIMEOUT);
                    else if (bd != -1 && (bd == 1 || !(Or > ROWPART_EMPTY) || !(Zr > 0.0) || !(Zr < CUDART_INF)))
                        st1 = max(st1, SPEC_DEV_NONFINITE);
                    S.t_Z[r2] = Zr; S.t_O[r2] = Or; S.t_cut[r2] = __ldcg(&p->cut);
                }
                if (st1) atomicMax(&S.t_status, st1);
            }
            bar_sync(1, NCONS);
            // ---- second batch of loads: children, and the exponential of every node's token in its parent's rows
            if (S.t_status == 0) {
                int st2 = 0;
                for (int c = 1 + tid; c < P.N; c += NCONS) {
                    const int a = S.t_parent[c], xt = S.t_token[c];
                    atomicMin(&S.t_fc[a], c);
                    if (atomicAdd(&S.t_kc[a], 1) >= KMAX) st2 = SPEC_DEV_TOPOLOGY;
                    const long long rowb = (long long)b * P.seq_stride + (long long)a * P.node_stride;
                    const float zp_x = load_logit(P.zp, DT, rowb + xt), zq_x = load_logit(P.zq, DT, rowb + xt);
                    double pr[2];
#pragma unroll 1
                    for (int h = 0; h < 2; ++h) {
                        const float z = h ? zq_x : zp_x;
                        const double xd = (double)z * s_d - (double)S.t_O[2 * a + h];
                        pr[h] = 0.0;
                        if (z >= S.t_cut[2 * a + h] && xd > -1000.0) {
                            const double nd = rint(xd);
                            pr[h] = exp2_frac_once(xd - nd) * pow2d((int)nd);
                        }
                    }
                    S.t_cp[c] = pr[0]; S.t_cq[c] = pr[1];
                }
                if (st2) atomicMax(&S.t_status, st2);
            }
            bar_sync(1, NCONS);
            int status = S.t_status;
            int cur = 0, len = 0;
            int bonus = -1;
            bool writer = false;          // this lane writes the sequence's outputs
            bool done = status != 0;
            if (done && rank == 0 && warp == 0 && lane == 0) { writer = true; cur = -1; len = -1; }

            while (!done) {
                const int a = cur;
                const int c_first = S.t_fc[a];
                const bool hq = c_first < P.N;
                const int kc = S.t_kc[a];
                RowSum rp, rq;
                rp.Z = S.t_Z[2 * a]; rp.O = S.t_O[2 * a]; rp.cut = S.t_cut[2 * a];
                rq = rp;
                if (hq) { rq.Z = S.t_Z[2 * a + 1]; rq.O = S.t_O[2 * a + 1]; rq.cut = S.t_cut[2 * a + 1]; }
                if (OT) {
                    // ================= Algorithms 1-3 at node a =================================================
                    const int solver = P.solver;
                    const bool use_q = hq && solver != 0;            // Algorithm 1 ignores the drafts
                    // Algorithm 2 tests the first child only; Algorithm 3 with one child has rho = 1 and is the same
                    const bool one_test = use_q && (solver == 1 || kc == 1);
                    int acc = -1;
                    if (one_test) {
                        const double ep = S.t_cp[c_first], eq = S.t_cq[c_first];
                        const bool zero = !(ep > 0.0), one = !zero && !(eq > 0.0);
                        if (!zero && (one || (double)S.t_u[c_first] * eq * rp.Z < ep * rq.Z)) acc = c_first;
                    }
                    if (acc < 0) {
                        if (kc > 1) {
                            __syncwarp();
                            int seen = 0;
                            for (int c0 = a + 1; c0 < P.N && seen < kc; c0 += 32) {
                                const int c = c0 + lane;
                                const bool is = c < P.N && S.t_parent[c] == a;
                                const unsigned bal = __ballot_sync(0xffffffffu, is);
                                if (is) {
                                    const int pos = seen + __popc(bal & ((1u << lane) - 1u));
                                    W.child[pos] = c; W.cpm[pos] = S.t_cp[c]; W.cqm[pos] = S.t_cq[c]; W.cu[pos] = S.t_u[c];
                                }
                                seen += __popc(bal);
                            }
                            __syncwarp();
                        }
                        if (warp == 0 && lane == 0) {
                            if (posted) { if (!mbar_wait(&S.ack, aphase)) S.poison = 1; aphase ^= 1u; }
                            S.req_a = a; S.req_b = b; S.req_hq = use_q ? 1 : 0;
                            mbar_arrive(&S.req);
                            posted = true;
                        }
                        bool poisoned = *(volatile int *)&S.poison != 0;
                        nr.hq = use_q; nr.cut_p = rp.cut; nr.cut_q = rq.cut; nr.O_p = rp.O; nr.O_q = rq.O;
                        set_list_thresholds(nr, rp.Z, rq.Z);
                        int nl;
                        float zs_p, zs_q;
                        pass1<DT, NW>(rc, stage, phase, poisoned, nr, es, nsm, nrg, n_slice, tid, R, L, nl, zs_p, zs_q);
                        double Z_q = rq.Z, kappa, tot_r, Zr_q = 0.0;
                        {
                            const double v[2] = {warp_sum_once((double)zs_p + (lane < nl ? L.ep[lane] : 0.0)),
                                                 warp_sum_once((double)zs_q + (lane < nl ? L.eq[lane] : 0.0))};
                            double tot[2], mine[2];
                            cluster_exchange<NW, 2>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                            kappa = tot[0]; tot_r = mine[0];
                            if (use_q && tot[1] > 0.0) { Z_q = tot[1]; Zr_q = mine[1]; }
                        }
                        if (*(volatile int *)&S.poison) status = SPEC_DEV_TIMEOUT;
                        else if (!(kappa > 0.0)) status = SPEC_DEV_NONFINITE;
                        const double invZq = use_q ? __drcp_rn(Z_q) : 0.0;
                        bool is_q = false;
                        if (!status && one_test) {
                            // the first child was rejected: Y ~ norm((p - q)+), one step of the recursion of verify.cuh
                            const double g = __ddiv_rn(Z_q, kappa);
                            const double v[1] = {warp_sum_once(step_sweep<NW>(es, nsm, tid, R, L, nl, g))};
                            double tot[1], mine[1];
                            cluster_exchange<NW, 1>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                            if (*(volatile int *)&S.poison) status = SPEC_DEV_TIMEOUT;
                            else if (tot[0] * invZq > RESIDUAL_FLOOR) { kappa = tot[0]; tot_r = mine[0]; }
                            else { is_q = true; kappa = Z_q; tot_r = Zr_q; }      // S = 0: p = q, drawn from q's row
                        } else if (!status && use_q) {
                            // ---- Algorithm 3 with k >= 2 children: the division factor by bisection (Appendix B) ----
                            const double ip = __drcp_rn(kappa), kd = (double)kc;
                            auto sweep2 = [&](auto f, double &t0, double &t1) {
                                double o0, o1;
                                reduce_sweep<NW>(es, nsm, tid, R, L, nl, f, o0, o1);
                                const double v[2] = {warp_sum_once(o0), warp_sum_once(o1)};
                                double tot[2], mine[2];
                                cluster_exchange<NW, 2>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                                t0 = tot[0]; t1 = tot[1];
                            };
                            double lo = 1.0, hi = kd, dummy, beta;
                            for (int it = 0; it < 40; ++it) {
                                const double mid = 0.5 * (lo + hi), ipr = ip / mid;
                                sweep2(FnBeta{(float)ipr, (float)invZq, ipr, invZq}, beta, dummy);
                                const double f = (1.0 - pow(1.0 - beta, kd)) - mid * beta;
                                if (f > 0.0) lo = mid; else hi = mid;
                            }
                            const double rho = 0.5 * (lo + hi);
                            {
                                const double ipr = ip / rho;
                                sweep2(FnBeta{(float)ipr, (float)invZq, ipr, invZq}, beta, dummy);
                            }
                            const double pacc = 1.0 - pow(1.0 - beta, kd);
                            const double gamma = beta > 0.0 ? pacc / beta : 0.0;
                            // the children in list order, each against min(1, p(x) / (rho q(x)))
                            const double ux = lane < kc ? W.cpm[lane] : 0.0, eqx = lane < kc ? W.cqm[lane] : 0.0;
                            for (int j = 0; j < kc; ++j) {
                                const double Pp = __shfl_sync(0xffffffffu, ux, j) * ip;
                                const double Pq = __shfl_sync(0xffffffffu, eqx, j) * invZq;
                                double thr;
                                if (!(Pp > 0.0)) thr = 0.0;
                                else if (!(Pq > 0.0)) thr = 1.0;
                                else thr = fmin(1.0, (Pp / Pq) / rho);
                                if ((double)W.cu[j] < thr) {
                                    // the solver's output is the child's TOKEN: the walk moves to the first child,
                                    // in list order, that carries it (duplicates stay separate nodes)
                                    const int y = S.t_token[W.child[j]];
                                    for (int i = 0; i <= j && acc < 0; ++i)
                                        if (S.t_token[W.child[i]] == y) acc = W.child[i];
                                    break;
                                }
                            }
                            if (acc < 0) {
                                // all rejected: Y ~ norm((p - min(p / rho, q) gamma)+); p itself where that is empty
                                const double ib = beta < 1.0 ? 1.0 / (1.0 - beta) : 0.0;
                                double sres, sacc;
                                sweep2(FnSpecTrRes{(float)ip, (float)invZq, (float)(1.0 / rho), (float)gamma, (float)ib, (float)kd,
                                                   ip, invZq, 1.0 / rho, gamma, ib, kd}, sres, sacc);
                                if (sres > 0.0) {
                                    const double v[1] = {warp_sum_once(
                                        spectr_sweep<NW>(es, nsm, tid, R, L, nl, gamma, 1.0 / rho, kappa * invZq))};
                                    double tot[1], mine[1];
                                    cluster_exchange<NW, 1>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                                    kappa = tot[0]; tot_r = mine[0];
                                    if (!(kappa > 0.0)) status = SPEC_DEV_NONFINITE;
                                }
                            }
                            if (*(volatile int *)&S.poison) status = SPEC_DEV_TIMEOUT;
                        }
                        if (!status && acc < 0) {
                            // ---- the draw, and its token made known to every warp of the cluster ---------------------
                            const double E_tot = warp_sum_once(lane < C ? tot_r : 0.0);
                            const double target = (double)S.t_ub[a] * E_tot;
                            double tau;
                            const int owner = pick_lane(lane < C ? tot_r : 0.0, target, tau);
                            double say = 0.0;             // token + 1 from the one thread that found it; -role on a failure
                            if (owner < 0) {
                                status = SPEC_DEV_NONFINITE;
                            } else {
                                if (owner == (int)rank) {
                                    const BonusFind bf = bonus_search<NW>(S.wtile, &S.cbar, cph, &S.poison, es, nsm, tid, R, L, nl,
                                                                          is_q, tau);
                                    if (bf.role == 1) say = (double)(tok0 + bf.token) + 1.0;
                                    else if (bf.role >= 2) say = -(double)bf.role;
                                }
                                const double v[1] = {warp_sum_once(say)};
                                double tot[1], mine[1];
                                cluster_exchange<NW, 1>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                                if (*(volatile int *)&S.poison || tot[0] == -3.0) status = SPEC_DEV_TIMEOUT;
                                else if (!(tot[0] >= 1.0)) status = SPEC_DEV_NONFINITE;
                                else {
                                    const int y = (int)(tot[0] - 1.0);
                                    // the first child, in list order, that carries the token
                                    if (hq) {
                                        if (kc == 1) { if (S.t_token[c_first] == y) acc = c_first; }
                                        else
                                            for (int j = 0; j < kc && acc < 0; ++j)
                                                if (S.t_token[W.child[j]] == y) acc = W.child[j];
                                    }
                                    if (acc < 0) {
                                        done = true;
                                        bonus = y;
                                        if (rank == 0 && warp == 0 && lane == 0) writer = true;
                                    }
                                }
                            }
                        }
                        if (status) {
                            done = true;
                            if (rank == 0 && warp == 0 && lane == 0) { writer = true; cur = -1; len = -1; }
                        }
                    }
                    if (acc >= 0 && !done) { cur = acc; ++len; }
                    continue;
                }
                // ---- first child: needs no residual -------------------------------------------------------------------
                int acc = -1;
                int j0 = 0;
                if (hq) {
                    // p(x) / q(x) = (e_p / Z_p) / (e_q / Z_q), written without a division
                    const double ep = S.t_cp[c_first], eq = S.t_cq[c_first];
                    const bool zero = !(ep > 0.0), one = !zero && !(eq > 0.0);
                    if (!zero && (one || (double)S.t_u[c_first] * eq * rp.Z < ep * rq.Z)) acc = c_first;
                    j0 = 1;
                }
                if (acc < 0) {
                    // ---- the node comes on chip: e = 2^(z s - O) of both rows ----------------------------------------
                    // the warp's list of the node's children, in index order
                    if (kc > 1) {
                        __syncwarp();
                        int seen = 0;
                        for (int c0 = a + 1; c0 < P.N && seen < kc; c0 += 32) {
                            const int c = c0 + lane;
                            const bool is = c < P.N && S.t_parent[c] == a;
                            const unsigned bal = __ballot_sync(0xffffffffu, is);
                            if (is) {
                                const int pos = seen + __popc(bal & ((1u << lane) - 1u));
                                W.child[pos] = c; W.cpm[pos] = S.t_cp[c]; W.cqm[pos] = S.t_cq[c]; W.cu[pos] = S.t_u[c];
                            }
                            seen += __popc(bal);
                        }
                        __syncwarp();
                    }
                    if (warp == 0 && lane == 0) {
                        if (posted) { if (!mbar_wait(&S.ack, aphase)) S.poison = 1; aphase ^= 1u; }
                        S.req_a = a; S.req_b = b; S.req_hq = hq ? 1 : 0;
                        mbar_arrive(&S.req);
                        posted = true;
                    }
                    bool poisoned = *(volatile int *)&S.poison != 0;
                    nr.hq = hq; nr.cut_p = rp.cut; nr.cut_q = rq.cut; nr.O_p = rp.O; nr.O_q = rq.O;
                    set_list_thresholds(nr, rp.Z, rq.Z);
                    int nl;
                    float zs_p, zs_q;
                    pass1<DT, NW>(rc, stage, phase, poisoned, nr, es, nsm, nrg, n_slice, tid, R, L, nl, zs_p, zs_q);
                    // ---- the rows' totals from what is resident: the normalisers, and each rank's share of u_0 = e_p
                    double Z_q = rq.Z, kappa, tot_r, Zr_q = 0.0;
                    {
                        const double v[2] = {warp_sum_once((double)zs_p + (lane < nl ? L.ep[lane] : 0.0)),
                                             warp_sum_once((double)zs_q + (lane < nl ? L.eq[lane] : 0.0))};
                        double tot[2], mine[2];
                        cluster_exchange<NW, 2>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                        kappa = tot[0]; tot_r = mine[0];
                        if (hq && tot[1] > 0.0) { Z_q = tot[1]; Zr_q = mine[1]; }
                    }
                    if (*(volatile int *)&S.poison) status = SPEC_DEV_TIMEOUT;
                    else if (!(kappa > 0.0)) status = SPEC_DEV_NONFINITE;
                    const double invZq = hq ? __drcp_rn(Z_q) : 0.0;
                    // ---- the recursion of verify.cuh, step by step (the first child, if any, is already rejected);
                    // lane j < kc follows child j's token in fp64
                    double ux = 0.0, eqx = 0.0;
                    if (lane < kc) {
                        ux = kc > 1 ? W.cpm[lane] : S.t_cp[c_first];
                        eqx = kc > 1 ? W.cqm[lane] : S.t_cq[c_first];
                    }
                    bool is_q = false;
                    for (int j = 0; j < kc && !status; ++j) {
                        if (j >= j0) {
                            // child j from the current state
                            const double uxj = __shfl_sync(0xffffffffu, ux, j), eqj = __shfl_sync(0xffffffffu, eqx, j);
                            const double Pq = eqj * invZq;
                            const double Pp = is_q ? Pq : uxj / kappa;
                            double thr;
                            if (!(Pp > 0.0)) thr = 0.0;
                            else if (!(Pq > 0.0)) thr = 1.0;
                            else thr = fmin(1.0, Pp / Pq);
                            if ((double)W.cu[j] < thr) { acc = W.child[j]; break; }
                        }
                        if (is_q) continue;
                        // the step after rejecting child j: u <- (g u - e_q)+ , g = Z_q / kappa
                        const double g = __ddiv_rn(Z_q, kappa);
                        const double v[1] = {warp_sum_once(step_sweep<NW>(es, nsm, tid, R, L, nl, g))};
                        double tot[1], mine[1];
                        cluster_exchange<NW, 1>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                        if (*(volatile int *)&S.poison) { status = SPEC_DEV_TIMEOUT; break; }
                        ux = fmax(fma(g, ux, -eqx), 0.0);
                        if (tot[0] * invZq > RESIDUAL_FLOOR) { kappa = tot[0]; tot_r = mine[0]; }
                        else { is_q = true; kappa = Z_q; tot_r = Zr_q; }      // S = 0: the state equals q
                    }
                    if (status) { done = true; if (rank == 0 && warp == 0 && lane == 0) { writer = true; cur = -1; len = -1; } break; }
                    if (acc < 0) {
                        // ---- stop here: the bonus token from the final state ----------------------------------------------
                        done = true;
                        const double E_tot = warp_sum_once(lane < C ? tot_r : 0.0);
                        const double target = (double)S.t_ub[a] * E_tot;
                        double tau;
                        const int owner = pick_lane(lane < C ? tot_r : 0.0, target, tau);
                        if (owner < 0) {
                            status = SPEC_DEV_NONFINITE;
                            if (rank == 0 && warp == 0 && lane == 0) { writer = true; cur = -1; len = -1; }
                        } else if (owner == (int)rank) {
                            const BonusFind bf = bonus_search<NW>(S.wtile, &S.cbar, cph, &S.poison, es, nsm, tid, R, L, nl,
                                                                  is_q, tau);
                            if (bf.role == 1) {
                                bonus = (int)(tok0 + bf.token);
                                writer = true;
                            } else if (bf.role >= 2) {
                                status = bf.role == 3 ? SPEC_DEV_TIMEOUT : SPEC_DEV_NONFINITE;
                                writer = true; cur = -1; len = -1;
                            }
                        }
                    }
                }
                if (acc >= 0) { cur = acc; ++len; continue; }
            }

            // ---- outputs of the sequence (one thread) -----------------------------------------------------------------------
            if (writer) {
                const int st = status;
                const int accn = st ? -1 : cur, ln = st ? -1 : len, bn = st ? -1 : bonus;
                P.out.accepted_node[b] = accn;
                P.out.accept_len[b] = ln;
                P.out.bonus_token[b] = bn;
                P.out.status[b] = st;
                int *ot = P.out.out_tokens + (long long)b * P.N;
                for (int i = 0; i < P.N; ++i) ot[i] = -1;
                if (accn >= 0) {
                    ot[ln] = bn;
                    int i = ln;
                    for (int x = accn; x != 0 && i > 0; x = S.t_parent[x]) ot[--i] = S.t_token[x];
                }
            }
        }
        // tell the producer to leave
        if (warp == 0 && lane == 0) {
            if (posted) { if (!mbar_wait(&S.ack, aphase)) S.poison = 1; aphase ^= 1u; }
            S.req_a = -1;
            mbar_arrive(&S.req);
        }
    }
    __syncthreads();
    cluster_sync_all();
}

}  // namespace specv
