// Whole-tree verification on top of the row statistics (stream.cuh / rowstat.cuh): every node of
// every sequence is one work item of a thread-block cluster, as Traversal Verification needs (its
// weights are defined for every node, top-down: Section 3.2) and as SpecInfer's diagnostic outputs
// need (the threshold of every node, Algorithm 4).
//
// With a row's reference O and normaliser Z known before the node comes on chip, a node is:
//   scalars   children, their tokens and uniforms, the exact exponentials 2^(z s - O) of every child's
//             token in both rows -- gathered by the producer warp, one node ahead of the consumers,
//             into a double-buffered block of shared memory;
//   pass 1    e = 2^(z s - O) of both rows, resident in registers and shared memory, all threads in
//             the same units; the dominant tokens in fp64 on the warps' exact lists (verify.cuh);
//   Z         the rows' normalisers again, from the resident e and the lists (one exchange): the
//             statistics pass gives them to fp32 accuracy only, too coarse for the differences below;
//   weight    Traversal: the weight the parent published for this node (bounded poll);
//   siblings  the residual recursion of verify.cuh, step by step: u <- (g u - e_q)+ in place, one sweep
//             over the resident data and one distributed-shared-memory exchange per rejected child;
//             child j is handed min(1, w P(x_j) / q(x_j)) from the state before its step, published at once;
//   outcome   the node's final weight; where the node can be the accepted one, the bonus token by an
//             inverse-CDF search over the final state.
// Records, published weights, arrival counting and the writing of a sequence's outputs are those of
// verify.cuh.
#pragma once
#include "stream.cuh"
#include "verify.cuh"

namespace specv {

struct TParams {
    VParams v;                // shapes, inputs, records, published weights, arrival counters, outputs
    const RowPart *part;      // [B*N*2] statistics of every row the verifier reads
    double *gseq;             // optional [B*N][KMAX]: the step coefficients g_j of every node (for the residual output)
};

// what the consumers need to know about a node besides its rows
struct __align__(16) NodeScalars {
    double Z_p, Z_q;
    double cpm[KMAX], cqm[KMAX];   // exact 2^(z s - O) of the children's tokens in the node's target and draft rows
    float cu[KMAX];                // the children's acceptance uniforms
    int child[KMAX];
    int kc, err, O_p, O_q;
    float cut_p, cut_q, u_a, ub_a;
};

struct __align__(16) THdr {
    uint64_t full[NSMAX], empty[NSMAX], xbar[2], cbar, sfull[2], sempty[2];
    double wtile[NWMAX + 1][TMAX];
    NodeScalars sc[2];
    int poison;
};

static_assert(sizeof(THdr) <= sizeof(Hdr), "the launch plan reserves sizeof(Hdr) bytes for the header");

template <int DT, int NW>
__global__ void __launch_bounds__((NW + 1) * 32, NW <= 7 ? 2 : 1) spec_tree_kernel(const TParams TP)
{
    const VParams &P = TP.v;
    constexpr int NCONS = NW * 32;
    constexpr int TILE = NCONS * 8;
    constexpr int ESZ = DT == SPEC_BF16 ? 2 : 4;
    constexpr int ROWB = TILE * ESZ;
    constexpr int STAGE = 2 * ROWB;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    THdr &S = *reinterpret_cast<THdr *>(dyn_smem);
    double *xchg = reinterpret_cast<double *>(dyn_smem + P.off_x);   // [parity 2][rank C][warp NW][2]
    WarpList *lists = reinterpret_cast<WarpList *>(dyn_smem + P.off_list);   // [warp NW]
    float4 *es = reinterpret_cast<float4 *>(dyn_smem + P.off_es);    // [slot][p lo, p hi, q lo, q hi][NCONS]
    unsigned char *ring = dyn_smem + P.off_ring;
    const int C = P.C, NS = P.NS;
    const unsigned rank = cluster_ctarank();
    const int cid = blockIdx.x / C, NC = gridDim.x / C;
    const long long total = (long long)P.B * P.N;
    const long long tok0 = (long long)rank * P.slice_len;
    const int n_slice = (int)max(0ll, min((long long)P.slice_len, (long long)P.V - tok0));
    const int ntiles = (n_slice + TILE - 1) / TILE;
    const int nsm = min(P.nsm, ntiles), nrg = ntiles - nsm;
    const bool trav = P.mode == MODE_TRAVERSAL;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&S.full[s], 1); mbar_init(&S.empty[s], NW); }
        mbar_init(&S.xbar[0], 1);
        mbar_init(&S.xbar[1], 1);
        mbar_init(&S.sfull[0], 1);
        mbar_init(&S.sfull[1], 1);
        mbar_init(&S.sempty[0], NW);
        mbar_init(&S.sempty[1], NW);
        mbar_init(&S.cbar, NW);
        S.poison = 0;
        mbar_fence_init();
    }
    __syncthreads();
    cluster_sync_all();

    if (warp == NW) {
        // ======================= producer warp: fills the ring, node after node, and gathers the =======
        // ======================= scalars of the node after the one whose rows it has just issued =======
        int g = 0;
        bool ok = true;
        // scalars of item `id` (the kidx-th item of this cluster) into block kidx & 1
        auto scalars = [&](long long id, int kidx) {
            const int a = (int)(id / P.B), b = (int)(id % P.B);
            const int buf = kidx & 1;
            if (kidx >= 2) {
                int w = 1;
                if (lane == 0) w = mbar_wait(&S.sempty[buf], (uint32_t)(((kidx >> 1) - 1) & 1)) ? 1 : 0;
                w = __shfl_sync(0xffffffffu, w, 0);
                if (!w || *(volatile int *)&S.poison) { S.poison = 1; ok = false; return; }
            }
            NodeScalars &N = S.sc[buf];
            const int *parent = P.parent + (long long)b * P.topo_stride;
            const int *token = P.token + (long long)b * P.N;
            const double s_d = 1.4426950408889634 / (double)(P.T_seq ? __ldg(P.T_seq + b) : P.T);
            int kc = 0, err = 0;
            if (lane == 0) {
                const int pa = __ldg(parent + a);
                if (a == 0 ? (pa != -1) : (pa < 0 || pa >= a)) err = SPEC_DEV_TOPOLOGY;
                if (a > 0) {
                    const int x = __ldg(token + a);
                    if (x < 0 || x >= P.V) err = SPEC_DEV_TOKEN;
                }
                N.u_a = __ldg(P.u_accept + (long long)b * P.N + a);
                N.ub_a = __ldg(P.u_bonus + (long long)b * P.N + a);
            }
            int my_tok = 0;              // lanes j and 16 + j: token of child j
            for (int c0 = a + 1; c0 < P.N; c0 += 32) {
                const int c = c0 + lane;
                const bool is = c < P.N && __ldg(parent + c) == a;
                const unsigned bal = __ballot_sync(0xffffffffu, is);
                if (is) {
                    const int pos = kc + __popc(bal & ((1u << lane) - 1u));
                    if (pos < KMAX) {
                        const int x = __ldg(token + c);
                        N.child[pos] = c;
                        N.cu[pos] = __ldg(P.u_accept + (long long)b * P.N + c);
                        N.cpm[pos] = (double)x;          // parked here until the probabilities are known
                        if (x < 0 || x >= P.V) err = SPEC_DEV_TOKEN;
                    }
                }
                kc += __popc(bal);
            }
            if (kc > KMAX) err = SPEC_DEV_TOPOLOGY;
            const bool hq = kc > 0;
            const RowPart *rp = TP.part + ((long long)b * P.N + a) * 2;
            const double Z_p = __ldcg(&rp[0].S);
            const int O_p = __ldcg(&rp[0].O);
            const float cut_p = __ldcg(&rp[0].cut);
            double Z_q = 0.0;
            int O_q = ROWPART_EMPTY;
            float cut_q = -CUDART_INF_F;
            bool bad = __ldcg(&rp[0].bad) != 0 || !(O_p > ROWPART_EMPTY) || !(Z_p > 0.0) || !(Z_p < CUDART_INF);
            if (hq) {
                Z_q = __ldcg(&rp[1].S); O_q = __ldcg(&rp[1].O); cut_q = __ldcg(&rp[1].cut);
                bad = bad || __ldcg(&rp[1].bad) != 0 || !(O_q > ROWPART_EMPTY) || !(Z_q > 0.0) || !(Z_q < CUDART_INF);
            }
            err = __reduce_max_sync(0xffffffffu, err);
            if (bad && !err) err = SPEC_DEV_NONFINITE;
            __syncwarp();
            {
                const int j = lane & 15;
                const bool mine = !err && j < kc;
                my_tok = mine ? (int)N.cpm[j] : 0;
                __syncwarp();
                double pr = 0.0;
                if (mine) {
                    const long long rowb = (long long)b * P.seq_stride + (long long)a * P.node_stride;
                    const float z = load_logit(lane < 16 ? P.zp : P.zq, DT, rowb + my_tok);
                    const double xd = (double)z * s_d - (double)(lane < 16 ? O_p : O_q);
                    if (z >= (lane < 16 ? cut_p : cut_q) && xd > -1000.0) {
                        const double nd = rint(xd);
                        pr = exp2_frac_once(xd - nd) * pow2d((int)nd);
                    }
                }
                if (j < KMAX) { if (lane < 16) N.cpm[j] = pr; else N.cqm[j] = pr; }
            }
            if (lane == 0) {
                N.Z_p = Z_p; N.Z_q = Z_q; N.O_p = O_p; N.O_q = O_q; N.cut_p = cut_p; N.cut_q = cut_q;
                N.kc = kc; N.err = err;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.sfull[buf]);
        };
        // pass 1 needs a node's references and cuts, so its scalars come before its rows: the first
        // node's before anything else, from then on one node ahead
        int kidx = 0;
        if (cid < total) scalars(cid, 0);
        for (long long id = cid; id < total && ok; id += NC, ++kidx) {
            const int a = (int)(id / P.B), b = (int)(id % P.B);
            const bool hq = warp_has_children(P.parent + (long long)b * P.topo_stride, P.N, a, lane);
            const long long row = (long long)b * P.seq_stride + (long long)a * P.node_stride + tok0;
            const unsigned char *src_p = (const unsigned char *)P.zp + row * ESZ;
            const unsigned char *src_q = (const unsigned char *)P.zq + row * ESZ;
            const bool aligned = ((((uintptr_t)src_p) | (hq ? (uintptr_t)src_q : 0)) & 15) == 0;
            for (int i = 0; i < ntiles; ++i, ++g) {
                const int stage = g % NS, use = g / NS;
                if (use > 0) {
                    int w = 1;
                    if (lane == 0) w = mbar_wait(&S.empty[stage], (uint32_t)((use - 1) & 1)) ? 1 : 0;
                    w = __shfl_sync(0xffffffffu, w, 0);
                    if (!w || *(volatile int *)&S.poison) { S.poison = 1; ok = false; break; }
                }
                const int ntok = min(TILE, n_slice - i * TILE);
                unsigned char *dst_p = ring + (size_t)stage * STAGE, *dst_q = dst_p + ROWB;
                const unsigned char *sp = src_p + (size_t)i * ROWB, *sq = src_q + (size_t)i * ROWB;
                const uint32_t body = aligned ? (((uint32_t)ntok * ESZ) & ~15u) : 0u;
                // what the bulk copy cannot take (a misaligned row, the last few bytes): plain loads
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
            if (!ok) break;
            if (id + NC < total) scalars(id + NC, kidx + 1);
        }
        if (!ok && lane == 0) {
            // gave up: wait (bounded) for the copies still in flight before leaving
            for (int k = 1; k <= NS && k <= g; ++k) {
                const int gg = g - k;
                mbar_wait(&S.full[gg % NS], (uint32_t)((gg / NS) & 1));
            }
        }
    } else {
        // ================================ consumer warps ================================================
        const bool scribe = rank == 0 && warp == 0;     // the one warp that writes the node's record
        const RingCtx rc = {S.full, S.empty, ring, NS, &S.poison};
        WarpList &L = lists[warp];
        int stage = 0;
        uint32_t phase = 0, cph = 0;
        int xn = 0;
        int kidx = 0;
        Resident R;

        for (long long id = cid; id < total; id += NC, ++kidx) {
            const int a = (int)(id / P.B), b = (int)(id % P.B);
            const int *parent = P.parent + (long long)b * P.topo_stride;
            NodeRows nr;
            nr.s_d = 1.4426950408889634 / (double)(P.T_seq ? __ldg(P.T_seq + b) : P.T);
            nr.s_hi = (float)nr.s_d;
            if ((double)nr.s_hi > nr.s_d) nr.s_hi = __uint_as_float(__float_as_uint(nr.s_hi) - 1u);
            nr.s_lo = (float)(nr.s_d - (double)nr.s_hi);
            if (!(nr.s_lo > 0.f)) nr.s_lo = 1.0e-30f;

            // ---- the node's scalars, gathered by the producer warp --------------------------------------------
            bool poisoned = *(volatile int *)&S.poison != 0;
            const NodeScalars &W = S.sc[kidx & 1];
            if (!poisoned && !mbar_wait(&S.sfull[kidx & 1], (uint32_t)((kidx >> 1) & 1))) { S.poison = 1; poisoned = true; }
            int err = poisoned ? SPEC_DEV_TIMEOUT : W.err;
            const int kc = poisoned ? 0 : W.kc;
            const bool hq = kc > 0;
            nr.hq = hq; nr.cut_p = W.cut_p; nr.cut_q = W.cut_q; nr.O_p = W.O_p; nr.O_q = W.O_q;
            set_list_thresholds(nr, W.Z_p, W.Z_q);

            // ---- pass 1: e = 2^(z s - O) of both rows, resident; dominant tokens to the exact lists -------------
            int nl;
            float zs_p, zs_q;
            pass1<DT, NW>(rc, stage, phase, poisoned, nr, es, nsm, nrg, n_slice, tid, R, L, nl, zs_p, zs_q);
            if (poisoned && !err) err = SPEC_DEV_TIMEOUT;

            // ---- the rows' normalisers from what is resident (one exchange; a childless node needs none:
            // its weight is its parent's, and the bonus search works on unnormalised totals) -----------------
            double Z_p = W.Z_p, Z_q = W.Z_q;
            double Zr_p = 0.0, Zr_q = 0.0;        // lane r: rank r's share of the normalisers
            if (hq && !err) {
                const double v[2] = {warp_sum_once((double)zs_p + (lane < nl ? L.ep[lane] : 0.0)),
                                     warp_sum_once((double)zs_q + (lane < nl ? L.eq[lane] : 0.0))};
                double tot[2], mine[2];
                cluster_exchange<NW, 2>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                if (*(volatile int *)&S.poison) err = SPEC_DEV_TIMEOUT;
                else if (!(tot[0] > 0.0) || !(tot[1] > 0.0)) err = SPEC_DEV_NONFINITE;
                else { Z_p = tot[0]; Z_q = tot[1]; Zr_p = mine[0]; Zr_q = mine[1]; }
            }
            const double invZq = (err || !hq) ? 0.0 : __drcp_rn(Z_q);

            // ---- Traversal: the weight handed down by the parent (bounded poll, every warp for itself) ------
            double w_in = 1.0;
            if (trav && a > 0 && !err) {
                unsigned long long bits = W_PENDING;
                if (lane == 0) {
                    volatile unsigned long long *slot = P.w_pub + (long long)b * P.N + a;
                    const long long t0 = clock64();
                    for (;;) {
                        bits = *slot;
                        if (bits != W_PENDING || clock64() - t0 > WAIT_CYCLES || *(volatile int *)&S.poison) break;
                        __nanosleep(32);
                    }
                }
                bits = __shfl_sync(0xffffffffu, bits, 0);
                if (bits == W_PENDING) { err = SPEC_DEV_TIMEOUT; S.poison = 1; w_in = 0.0; }
                else w_in = __longlong_as_double((long long)bits);
            }

            // ---- the recursion, step by step (identical in every warp of the cluster) ---------------------------
            // state: the resident u (total kappa), the node's weight w, and in lane j < kc the value of u at
            // child j's token with its e_q (fp64, the same recursion as the vocabulary)
            const bool live = !err && w_in > 0.0;
            double w = live ? w_in : 0.0, kappa = Z_p;
            bool dead = !live, is_q = false;      // is_q: a step with S = 0 at weight 1 showed that the state equals q
            int nsteps = 0;
            const int kce = min(kc, KMAX);
            double ux = (lane < kce) ? W.cpm[lane] : 0.0;
            const double eqx = (lane < kce) ? W.cqm[lane] : 0.0;
            double tot_r = hq ? Zr_p : 0.0;       // lane r: rank r's share of kappa (childless node: exchanged below)
            double *gs = TP.gseq ? TP.gseq + ((long long)b * P.N + a) * KMAX : nullptr;
            int acc = -1;
            if (err && scribe && lane == 0) {
                // nothing below a faulty node is evaluated: every child gets weight / threshold 0
                NodeRec *rec = P.rec + (long long)b * P.N;
                for (int c = a + 1; c < P.N; ++c)
                    if (__ldg(parent + c) == a) {
                        if (trav) {
                            rec[c].w_in = 0.0;
                            *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + c) = 0ull;
                        } else {
                            rec[c].thr = 0.0;
                        }
                    }
            }
            for (int j = 0; j < kce && !err; ++j) {
                // child j from the current state: P(x) = u(x) / kappa, q(x) = e_q(x) / Z_q
                const double uxj = __shfl_sync(0xffffffffu, ux, j), eqj = __shfl_sync(0xffffffffu, eqx, j);
                const double Pq = eqj * invZq;
                const double Pp = is_q ? Pq : uxj / kappa;
                double thr;
                if (dead || !(Pp > 0.0)) thr = 0.0;
                else if (!(Pq > 0.0)) thr = 1.0;
                else thr = fmin(1.0, w * (Pp / Pq));
                // Traversal: a weight within a rounding of 1 is 1.  The step after it is discontinuous at
                // w = 1 when P = q (S = 0 gives weight 1 for w = 1 and weight 0 for any w < 1).
                if (trav && thr > 1.0 - WEIGHT_SNAP) thr = 1.0;
                if (scribe && lane == 0) {
                    NodeRec *rec = P.rec + (long long)b * P.N;
                    const int cj = W.child[j];
                    if (trav) {
                        // the child polls the published slot only; the record is read after all of the
                        // sequence's arrivals (each fenced), so no fence is needed between the two stores
                        rec[cj].w_in = thr;
                        *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + cj) =
                            (unsigned long long)__double_as_longlong(thr);
                    } else {
                        rec[cj].thr = thr;
                    }
                }
                if (!trav && acc < 0 && (double)W.cu[j] < thr) {
                    acc = W.child[j];
                    if (!P.all_thr) {
                        if (scribe && lane == 0)
                            for (int jj = j + 1; jj < kce; ++jj) P.rec[(long long)b * P.N + W.child[jj]].thr = CUDART_NAN;
                        break;
                    }
                }
                if (dead || is_q) continue;       // weight 0, or P = q (every further step has S = 0 again)
                // the step after rejecting child j: u <- (g u - e_q)+ , g = w Z_q / kappa
                const double g = __ddiv_rn(w * Z_q, kappa);
                const double v[1] = {warp_sum_once(step_sweep<NW>(es, nsm, tid, R, L, nl, g))};
                double tot[1], mine[1];
                cluster_exchange<NW, 1>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                if (*(volatile int *)&S.poison) { err = SPEC_DEV_TIMEOUT; break; }
                ux = fmax(fma(g, ux, -eqx), 0.0);
                const double Sj = tot[0] * invZq;
                // A step whose mass is below 1e-13 of the weight before it counts as S = 0: P equals q, and what
                // is left is the rounding of g.
                if (Sj > RESIDUAL_FLOOR * w) {
                    kappa = tot[0];
                    tot_r = mine[0];
                    if (trav) w = Sj / (Sj + (1.0 - w));
                    if (gs && scribe && lane == 0) gs[nsteps] = g;
                    ++nsteps;
                } else if (w >= 1.0) {
                    is_q = true;       // S = 0 with w = 1: the state is q itself (the stored u is no longer used)
                    tot_r = Zr_q;
                    kappa = Z_q;
                } else {
                    dead = true;       // S = 0 with w < 1: the weight drops to 0 (Traversal only)
                    w = 0.0;
                }
            }

            // ---- the node's outcome -----------------------------------------------------------------------------
            const double w_fin = (dead || err) ? 0.0 : w;
            bool want_bonus;
            if (trav) want_bonus = (a == 0) || ((double)W.u_a < w_fin);
            else want_bonus = acc < 0;
            if (dead || err) want_bonus = false;
            int owner = -1;
            double tau = 0.0, E_tot = 0.0;
            if (want_bonus && !hq) {
                // a childless node: the totals of u_0 = e_p per rank (pass 1 summed them already)
                const double v[1] = {warp_sum_once((double)zs_p + (lane < nl ? L.ep[lane] : 0.0))};
                double tot[1], mine[1];
                cluster_exchange<NW, 1>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                tot_r = mine[0];
                kappa = tot[0];
                if (*(volatile int *)&S.poison) { err = SPEC_DEV_TIMEOUT; want_bonus = false; }
            }
            if (want_bonus) {
                E_tot = warp_sum_once(lane < C ? tot_r : 0.0);
                const double target = (double)W.ub_a * E_tot;
                owner = pick_lane(lane < C ? tot_r : 0.0, target, tau);
            }
            if (scribe) {
                if (lane == 0) {
                    NodeRec &Rc = P.rec[(long long)b * P.N + a];
                    Rc.O_p = (double)nr.O_p; Rc.Z_p = Z_p; Rc.O_q = (double)nr.O_q; Rc.Z_q = Z_q;
                    Rc.kappa = (dead || err) ? 0.0 : kappa;
                    Rc.nsteps = is_q ? STATE_IS_Q : nsteps;
                    Rc.cut_p = nr.cut_p; Rc.cut_q = nr.cut_q;
                    Rc.next_child = acc;
                    Rc.status = err;
                    if (trav) { Rc.thr = (a == 0) ? 1.0 : w_fin; if (a == 0) Rc.w_in = 1.0; }
                    else { Rc.w_in = 1.0; if (a == 0) Rc.thr = 1.0; }
                    if (owner < 0) { Rc.bonus = -1; Rc.bonus_margin = 0.f; }
                }
                arrive_sequence(P, b, owner < 0 ? 2u : 1u);
            }

            // ---- bonus token: inverse CDF over the owner CTA's share of the state ----------------------------------
            if (owner == (int)rank) {
                const BonusFind bf = bonus_search<NW>(S.wtile, &S.cbar, cph, &S.poison, es, nsm, tid, R, L, nl, is_q, tau);
                if (bf.role) {
                    NodeRec &Rc = P.rec[(long long)b * P.N + a];
                    Rc.bonus = bf.role == 1 ? (int)(tok0 + bf.token) : (bf.role == 3 ? BONUS_TIMEOUT : -1);
                    Rc.bonus_margin = bf.role == 1 ? (float)(bf.edge / E_tot) : 0.f;
                }
                // the arrival is made by lane 0 of the warp that holds the reporting thread
                __syncwarp();
                if (__any_sync(0xffffffffu, bf.role != 0)) arrive_sequence(P, b, 1u);
            }
            // the scalars block may be rewritten
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.sempty[kidx & 1]);
        }
    }
    __syncthreads();
    cluster_sync_all();        // nobody leaves while a peer may still write to its shared memory
}

}  // namespace specv
