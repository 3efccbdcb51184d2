// Whole-tree verification on top of the row statistics (stream.cuh / rowstat.cuh): every node of
// every sequence is one work item of a thread-block cluster, as Traversal Verification needs (its
// weights are defined for every node, top-down: Section 3.2) and as SpecInfer's diagnostic outputs
// need (the threshold of every node, Algorithm 4).
//
// Items are handed out at run time: the producer warp of a cluster's first CTA draws a ticket from a
// counter in the workspace and passes it to the other CTAs' producers through distributed shared
// memory.  Tickets 0 .. B N - 1 are the nodes in node-major order (parents first), tickets B N ..
// B N + B - 1 one FINISH item per sequence.  A node waits only for the weight its parent publishes,
// the parent holds a smaller ticket, and a ticket is drawn only by a running cluster, so the smallest
// unfinished ticket never waits on anything unfinished -- whatever share of the grid is resident.
//
// With a row's reference O and normaliser Z known before the node comes on chip, a node is:
//   scalars   children, their tokens and uniforms, the exact exponentials 2^(z s - O) of every child's
//             token in both rows -- gathered by the producer warp, ahead of the consumers, into a
//             double-buffered block of shared memory;
//   pass 1    e = 2^(z s - O) of both rows, resident in registers and shared memory, all threads in
//             the same units; the dominant tokens in fp64 on the warps' exact lists (verify.cuh);
//   Z         the rows' normalisers again, from the resident e and the lists (one exchange): the
//             statistics pass gives them to fp32 accuracy only, too coarse for the differences below;
//   weight    Traversal: the weight the parent published for this node (bounded poll);
//   siblings  the residual recursion of verify.cuh, step by step: u <- (g u - e_q)+ in place, one sweep
//             over the resident data and one distributed-shared-memory exchange per rejected child;
//             child j is handed min(1, w P(x_j) / q(x_j)) from the state before its step, published at once;
//   outcome   the node's final weight and the coefficients g_j of its steps, recorded.
// A childless node needs no rows and no item of its own: its weight is the one it is handed, so the
// parent's scribe warp writes its record and makes its arrival when it publishes that weight (its ticket
// is skipped by every producer).  A node whose weight is already known to be 0 when its ticket is drawn
// needs no rows either (nothing below it can be accepted).
// The warp that makes the last of a sequence's arrivals selects the accepted node and publishes it;
// the sequence's FINISH item brings that one node back on chip, replays its recorded steps (no
// exchange: the coefficients are known) and draws the bonus token by the inverse-CDF search.
#pragma once
#include "analysis.cuh"
#include "stream.cuh"
#include "verify.cuh"

namespace specv {

struct TParams {
    VParams v;                // shapes, inputs, records, published weights, arrival counters, outputs
    const RowPart *part;      // [B*N*2] statistics of every row the verifier reads
    double *gseq;             // [B*N][KMAX]: the step coefficients g_j of every node
    unsigned int *ticket;     // item counter (0 at launch)
    // analysis instantiation only (SpecInfer mode, every threshold evaluated)
    AnRec *an;                // [B*N] per-node scalars for the branching probabilities
    float *an_acc;            // [B,N,4] acceptance rates: NSS, Naive, SpecTr written here (SpecInfer by spec_branch_kernel)
    float *an_div;            // [B,N,3] L1, KL(p||q), KL(q||p)
};

// ITEM_LEAF: a childless root (a tree of one node); other childless nodes are never items
enum ItemKind { ITEM_NODE = 0, ITEM_LEAF = 1, ITEM_DEAD = 2, ITEM_FINISH = 3, ITEM_IDLE = 4, ITEM_EXIT = 5 };

// what the consumers need to know about an item besides its rows
struct __align__(16) NodeScalars {
    double Z_p, Z_q;
    double cpm[KMAX], cqm[KMAX];   // node: exact 2^(z s - O) of the children's tokens in the node's target and draft
                                   // rows; FINISH item: cpm = the recorded coefficients g_j
    float cu[KMAX];                // the children's acceptance uniforms
    int child[KMAX];
    int kc, err, O_p, O_q;
    float cut_p, cut_q, u_a, ub_a;
    int kind, a, b, nsteps;
    unsigned leaf_mask;            // bit j: child j has no children
    int len;                       // FINISH item: the accepted path's length
    int pruned;                    // the node lies wholly after a known acceptance: weight 0 without waiting for it
    unsigned ord_a;                // the node's entry of the post-order table (0: not known)
    unsigned cord[KMAX];           // ... and its children's
};

struct __align__(16) THdr {
    uint64_t full[NSMAX], empty[NSMAX], xbar[2], cbar, sfull[2], sempty[2], tbar[2], abar[2];
    unsigned long long item[2];    // ticket | (weight already 0) << 32, written by the first CTA's producer
    double wtile[NWMAX + 1][TMAX];
    NodeScalars sc[2];
    NodeScalars scd;               // the producer's own block for a node it finishes by itself (weight known to be 0)
    int poison;
};

static_assert(sizeof(THdr) <= sizeof(Hdr), "the launch plan reserves sizeof(Hdr) bytes for the header");

__device__ __forceinline__ void st_async_u64(unsigned long long *slot, uint64_t *bar, uint32_t rank, unsigned long long v)
{
    asm volatile(
        "{\n\t.reg .b32 ra, rb;\n\tmapa.shared::cluster.u32 ra, %0, %2;\n\tmapa.shared::cluster.u32 rb, %1, %2;\n\t"
        "st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b64 [ra], %3, [rb];\n\t}" ::"r"(smem_u32(slot)),
        "r"(smem_u32(bar)), "r"(rank), "l"(v)
        : "memory");
}
// one arrival on the mbarrier at the same offset in CTA `rank` of the cluster
__device__ __forceinline__ void mbar_arrive_remote(uint64_t *bar, uint32_t rank)
{
    asm volatile(
        "{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t}" ::"r"(smem_u32(bar)), "r"(rank)
        : "memory");
}
// Entry `lane` of the post-order table of one tree of at most 32 nodes (children visited in index order, a
// node after its subtree: the order in which Traversal Verification tests the nodes).  Low word:
// 0x80000000 | rank << 8 | F, with F the number of nodes that come wholly before the node's subtree; high word:
// the node's ancestors, itself included, as a bit mask.  0 for every node of a tree whose parents do not come first.  From ancestor masks: F(v) sums, over v and its
// ancestors, the sizes of the subtrees of their earlier siblings, and rank(v) = F(v) + size(v) - 1.
__device__ __noinline__ unsigned long long post_order_entry(const int *parent, int N, int lane)
{
    const bool own = lane < N;
    const int par = own ? __ldg(parent + lane) : -2;
    if (__any_sync(0xffffffffu, own && (lane == 0 ? par != -1 : (par < 0 || par >= lane)))) return 0ull;
    unsigned anc = own ? 1u << lane : 0u;
    int jump = own ? par : -1;
#pragma unroll
    for (int it = 0; it < 5; ++it) {
        const int src = jump < 0 ? lane : jump;
        const unsigned up = __shfl_sync(0xffffffffu, anc, src);
        const int jj = __shfl_sync(0xffffffffu, jump, src);
        if (jump >= 0) { anc |= up; jump = jj; }
    }
    unsigned D = 0;                 // the node's subtree: the lanes whose ancestor mask holds it
    for (int v = 0; v < N; ++v) {
        const unsigned m = __ballot_sync(0xffffffffu, (anc >> v) & 1u);
        if (lane == v) D = m;
    }
    unsigned Em = 0;                // the subtrees of the node's earlier siblings
    for (int sb = 1; sb < N; ++sb) {
        const unsigned Ds = __shfl_sync(0xffffffffu, D, sb);
        const int ps = __shfl_sync(0xffffffffu, par, sb);
        if (own && sb < lane && ps == par) Em |= Ds;
    }
    const int E = __popc(Em);
    int F = 0;
    for (int x = 1; x < N; ++x) {
        const int Ex = __shfl_sync(0xffffffffu, E, x);
        if ((anc >> x) & 1u) F += Ex;
    }
    const int rank = F + __popc(D) - 1;
    return own ? (((unsigned long long)anc << 32) | 0x80000000u | ((unsigned)rank << 8) | (unsigned)F) : 0ull;
}

// The record of a childless node c of sequence b, finished by whoever hands it its weight thr_c (lane 0 of a
// converged warp writes; the node's arrival is counted by the caller).  Accepted if reached (Traversal without
// diagnostics, `ord` its post-order entry, u its uniform): nothing after it in the traversal order matters.
__device__ __noinline__ void leaf_record(const VParams &P, const RowPart *part, int b, int c, double thr_c, unsigned ord,
                                         float u)
{
    if ((threadIdx.x & 31) != 0) return;
    const bool trav = P.mode == MODE_TRAVERSAL;
    NodeRec &Rl = P.rec[(long long)b * P.N + c];
    const RowPart *rpl = part + ((long long)b * P.N + c) * 2;
    const double Zl = __ldcg(&rpl->S);
    const int Ol = __ldcg(&rpl->O);
    const bool badl = __ldcg(&rpl->bad) != 0 || !(Ol > ROWPART_EMPTY) || !(Zl > 0.0) || !(Zl < CUDART_INF);
    Rl.O_p = (double)Ol; Rl.Z_p = Zl; Rl.O_q = 0.0; Rl.Z_q = 0.0;
    Rl.kappa = Zl; Rl.nsteps = 0;
    Rl.cut_p = __ldcg(&rpl->cut); Rl.cut_q = -CUDART_INF_F;
    Rl.next_child = -1;
    Rl.status = badl ? (__ldcg(&rpl->bad) == ROW_TIMEOUT ? SPEC_DEV_TIMEOUT : SPEC_DEV_NONFINITE) : 0;
    Rl.bonus = -1; Rl.bonus_margin = 0.f;
    Rl.w_in = trav ? thr_c : 1.0;
    Rl.thr = thr_c;
    if (P.prune && (ord >> 31) && (double)u < thr_c) atomicMin(P.best + b, (ord >> 8) & 255u);
}

// A node of weight 0 (Traversal), finished by the warp that found it out: its record, weight 0 for its children
// (childless ones are finished on the spot), and the arrival of all of them.  W: the node's scalars.
__device__ __noinline__ void dead_node(const VParams &P, const RowPart *part, const NodeScalars &W)
{
    const int lane = threadIdx.x & 31;
    const int a = W.a, b = W.b;
    NodeRec *rec = P.rec + (long long)b * P.N;
    if (lane == 0) {
        NodeRec &Rc = rec[a];
        Rc.O_p = (double)W.O_p; Rc.Z_p = W.Z_p; Rc.O_q = (double)W.O_q; Rc.Z_q = W.Z_q;
        Rc.kappa = W.Z_p; Rc.nsteps = 0;
        Rc.cut_p = W.cut_p; Rc.cut_q = W.cut_q;
        Rc.next_child = -1;
        Rc.status = 0;
        Rc.bonus = -1; Rc.bonus_margin = 0.f;
        Rc.thr = 0.0;
    }
    unsigned narr = 1u;
    for (int j = 0; j < W.kc; ++j) {
        const int c = W.child[j];
        if ((W.leaf_mask >> j) & 1u) { leaf_record(P, part, b, c, 0.0, 0u, 0.f); ++narr; continue; }
        if (lane == 0) {
            rec[c].w_in = 0.0;
            *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + c) = 0ull;
        }
    }
    __syncwarp();
    arrive_sequence(P, b, narr);
}

// bounded poll of a published weight; W_PENDING when the limit ran out
__device__ __forceinline__ unsigned long long poll_weight(const unsigned long long *slot_, const int *poison)
{
    volatile const unsigned long long *slot = slot_;
    const long long t0 = clock64();
    unsigned long long bits;
    for (;;) {
        bits = *slot;
        if (bits != W_PENDING || clock64() - t0 > WAIT_CYCLES || *(volatile const int *)poison) break;
        __nanosleep(32);
    }
    return bits;
}

// AN: the analysis instantiation (read-only sweeps for acceptance rates and divergences, SpecTr's bisection,
// the per-node scalars of the branching probabilities) -- a separate instantiation, so that the verifiers'
// kernels carry none of it
template <int DT, int NW, bool AN>
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
        for (int i = 0; i < 2; ++i) {
            mbar_init(&S.sfull[i], 1);
            mbar_init(&S.sempty[i], NW);
            mbar_init(&S.tbar[i], 1);
            mbar_init(&S.abar[i], C);
        }
        mbar_init(&S.cbar, NW);
        S.poison = 0;
        mbar_fence_init();
    }
    __syncthreads();
    cluster_sync_all();

    if (warp == NW) {
        // ======================= producer warp: draws items, gathers their scalars, fills the ring ==============
        int g = 0, sidx = 0;          // ring uses so far; scalars blocks handed to the consumers so far
        bool ok = true;
        for (int kidx = 0; ok; ++kidx) {
            const int buf = kidx & 1;
            // once its first item is under way, one producer of the cluster writes the post-order tables of its
            // share of the sequences (a hint for the item hand-out below: absent entries only mean no skipping)
            if (kidx == 1 && trav && P.N <= 32 && rank == (unsigned)(C > 1 ? 1 : 0)) {
                const int ncl = (int)(gridDim.x / (unsigned)C);
                for (int bb = (int)(blockIdx.x / (unsigned)C); bb < P.B; bb += ncl) {
                    const unsigned long long e = post_order_entry(P.parent + (long long)bb * P.topo_stride, P.N, lane);
                    if (lane < P.N) *(volatile unsigned long long *)(P.order + (long long)bb * P.N + lane) = e;
                }
            }
            // ---- the item: drawn by the first CTA's producer, passed on to the others ---------------------------
            if (rank == 0) {
                unsigned long long val = 0;
                int w = 1;
                unsigned t = 0;
                if (lane == 0) {
                    // every producer has read the item that used this slot before
                    if (kidx >= 2) w = mbar_wait_cluster(&S.abar[buf], (uint32_t)(((kidx >> 1) - 1) & 1)) ? 1 : 0;
                    t = atomicAdd(TP.ticket, 1u);
                }
                t = __shfl_sync(0xffffffffu, t, 0);
                unsigned hint = 0;
                if (trav && (long long)t < total && t >= (unsigned)P.B) {
                    const int a = (int)(t / (unsigned)P.B), b = (int)(t % (unsigned)P.B);
                    // A node whose weight is already known to be 0 needs no rows, and the weight is 0 as soon as
                    // an ancestor's is (one load per lane: the weights of the tree's first 32 nodes).  Neither
                    // does a subtree that comes wholly after a node known to be accepted.
                    const unsigned long long e = *(volatile unsigned long long *)(P.order + (long long)b * P.N + a);
                    const unsigned ord = (unsigned)e;
                    unsigned anc = (ord >> 31) ? (unsigned)(e >> 32) : 0u;
                    if (a < 32) anc |= 1u << a;
                    const bool zero = lane < P.N && ((anc >> lane) & 1u) &&
                                      *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + lane) == 0ull;
                    const unsigned zm = __ballot_sync(0xffffffffu, zero);
                    if (zm) hint = (zm >> (a < 32 ? a : 0)) & 1u ? 1 : 3;
                    if (a >= 32 && *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + a) == 0ull) hint = 1;
                    if (P.prune && (ord >> 31) && *(volatile unsigned *)(P.best + b) < (ord & 255u)) hint = 2;
                }
                val = (unsigned long long)t | ((unsigned long long)hint << 32);
                w = __shfl_sync(0xffffffffu, w, 0);
                val = __shfl_sync(0xffffffffu, val, 0);
                if (!w) { S.poison = 1; val = 0xFFFFFFFFull; }       // gave up: everybody leaves
                if (lane < C) st_async_u64(&S.item[buf], &S.tbar[buf], (uint32_t)lane, val);
            }
            unsigned long long item = 0;
            {
                int w = 1;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&S.tbar[buf], 8u);
                    w = mbar_wait_cluster(&S.tbar[buf], (uint32_t)((kidx >> 1) & 1)) ? 1 : 0;
                    item = *(volatile unsigned long long *)&S.item[buf];
                    mbar_arrive_remote(&S.abar[buf], 0u);
                }
                w = __shfl_sync(0xffffffffu, w, 0);
                item = __shfl_sync(0xffffffffu, item, 0);
                if (!w) { S.poison = 1; item = 0xFFFFFFFFull; }
            }
            const long long t = (long long)(item & 0xFFFFFFFFull);
            // (1: its own weight is 0; 2, 3: wholly after an accepted node, or below a node of weight 0 -- its weight
            // is, or may as well be, 0, and is not waited for)
            const bool hint_dead = (item >> 32) != 0, hint_pruned = (item >> 32) >= 2;

            // a childless node other than the root is finished by its parent: its ticket is skipped by everybody
            // (one whose parent index is not valid is nobody's child: it stays an item and reports the fault)
            if (t >= P.B && t < total) {
                const int a_ = (int)(t / P.B), b_ = (int)(t % P.B);
                const int *par_ = P.parent + (long long)b_ * P.topo_stride;
                const int pa_ = __ldg(par_ + a_);
                if (pa_ >= 0 && pa_ < a_ && !warp_has_children(par_, P.N, a_, lane)) continue;
            }

            // ---- the scalars block of this item -----------------------------------------------------------------
            // A node whose weight is known to be 0 never reaches the consumers: its scalars go to the producer's
            // own block, and the first CTA's producer finishes it at once (behind the consumers' current item it
            // would hold up its sequence's arrivals for nothing).  Every CTA takes the same decision.
            const bool own_block = trav && hint_dead && t >= P.B && t < total;
            const int sbuf = sidx & 1;
            auto claim_block = [&]() {
                if (sidx >= 2) {
                    int w = 1;
                    if (lane == 0) w = mbar_wait(&S.sempty[sbuf], (uint32_t)(((sidx >> 1) - 1) & 1)) ? 1 : 0;
                    w = __shfl_sync(0xffffffffu, w, 0);
                    if (!w) S.poison = 1;
                }
                ++sidx;
            };
            if (!own_block) claim_block();
            NodeScalars &N = own_block ? S.scd : S.sc[sbuf];
            int kind, a = 0, b = 0;
            bool hq = false;
            if (t >= total + P.B || *(volatile int *)&S.poison) {
                kind = ITEM_EXIT;
                ok = false;
            } else if (t >= total) {
                // FINISH: wait (bounded) until the sequence's accepted node is published
                kind = ITEM_FINISH;
                b = (int)(t - total);
                int acc = FIN_PENDING;
                if (lane == 0) {
                    volatile int *slot = P.fin + b;
                    const long long t0 = clock64();
                    for (;;) {
                        acc = *slot;
                        if (acc != FIN_PENDING || clock64() - t0 > WAIT_CYCLES || *(volatile int *)&S.poison) break;
                        __nanosleep(64);
                    }
                    __threadfence();       // the records written before the publication are read below
                }
                acc = __shfl_sync(0xffffffffu, acc, 0);
                int err = 0;
                if (acc == FIN_PENDING) { err = SPEC_DEV_TIMEOUT; S.poison = 1; }
                const int len = acc >> FIN_LEN_SHIFT;
                if (acc >= 0) acc &= (1 << FIN_LEN_SHIFT) - 1;
                if (acc < 0 || err) {
                    kind = ITEM_IDLE;           // a faulty sequence has no bonus draw
                    if (lane == 0) { N.err = err; N.b = b; N.a = -1; }
                } else {
                    a = acc;
                    const NodeRec *rc = P.rec + (long long)b * P.N + a;
                    // (all coefficient slots are fetched, in the same round of loads as the step count: only the first
                    // nsteps are read by the consumers)
                    const double gj = lane < KMAX ? __ldcg(TP.gseq + ((long long)b * P.N + a) * KMAX + lane) : 0.0;
                    const int nsteps = __ldcg(&rc->nsteps);
                    hq = nsteps != 0;
                    if (lane < KMAX) N.cpm[lane] = gj;
                    if (lane == 0) {
                        N.Z_p = __ldcg(&rc->Z_p); N.Z_q = __ldcg(&rc->Z_q);
                        N.O_p = (int)__ldcg(&rc->O_p); N.O_q = (int)__ldcg(&rc->O_q);
                        N.cut_p = __ldcg(&rc->cut_p); N.cut_q = __ldcg(&rc->cut_q);
                        N.nsteps = nsteps; N.kc = hq ? 1 : 0; N.err = 0; N.a = a; N.b = b; N.len = len;
                        N.ub_a = __ldg(P.u_bonus + (long long)b * P.N + a);
                    }
                }
            } else {
                a = (int)(t / P.B);
                b = (int)(t % P.B);
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
                    N.pruned = hint_pruned ? 1 : 0;
                    N.ord_a = P.prune ? (unsigned)*(volatile unsigned long long *)(P.order + (long long)b * P.N + a) : 0u;
                    N.ub_a = __ldg(P.u_bonus + (long long)b * P.N + a);
                    N.a = a; N.b = b; N.nsteps = 0;
                }
                for (int c0 = a + 1; c0 < P.N; c0 += 32) {
                    const int c = c0 + lane;
                    const bool is = c < P.N && __ldg(parent + c) == a;
                    const unsigned bal = __ballot_sync(0xffffffffu, is);
                    if (is) {
                        const int pos = kc + __popc(bal & ((1u << lane) - 1u));
                        if (pos < KMAX) {
                            const int x = __ldg(token + c);
                            N.child[pos] = c;
                            N.cord[pos] = P.prune ? (unsigned)*(volatile unsigned long long *)(P.order + (long long)b * P.N + c) : 0u;
                            N.cu[pos] = __ldg(P.u_accept + (long long)b * P.N + c);
                            N.cpm[pos] = (double)x;          // parked here until the exponentials are known
                            if (x < 0 || x >= P.V) err = SPEC_DEV_TOKEN;
                        }
                    }
                    kc += __popc(bal);
                }
                if (kc > KMAX) err = SPEC_DEV_TOPOLOGY;
                hq = kc > 0;
                // which children are childless (their grandchildren name them as parent)
                unsigned nonleaf = 0;
                __syncwarp();
                for (int d0 = a + 2; d0 < P.N; d0 += 32) {
                    const int d = d0 + lane;
                    const int pd = d < P.N ? __ldg(parent + d) : -1;
                    for (int j = 0; j < min(kc, KMAX); ++j)
                        if (pd == N.child[j]) nonleaf |= 1u << j;
                }
                nonleaf = __reduce_or_sync(0xffffffffu, nonleaf);
                const RowPart *rp = TP.part + ((long long)b * P.N + a) * 2;
                const double Z_p = __ldcg(&rp[0].S);
                const int O_p = __ldcg(&rp[0].O);
                const float cut_p = __ldcg(&rp[0].cut);
                double Z_q = 0.0;
                int O_q = ROWPART_EMPTY;
                float cut_q = -CUDART_INF_F;
                bool bad = __ldcg(&rp[0].bad) != 0 || !(O_p > ROWPART_EMPTY) || !(Z_p > 0.0) || !(Z_p < CUDART_INF);
                bool slow = __ldcg(&rp[0].bad) == ROW_TIMEOUT || (hq && __ldcg(&rp[1].bad) == ROW_TIMEOUT);
                if (hq) {
                    Z_q = __ldcg(&rp[1].S); O_q = __ldcg(&rp[1].O); cut_q = __ldcg(&rp[1].cut);
                    bad = bad || __ldcg(&rp[1].bad) != 0 || !(O_q > ROWPART_EMPTY) || !(Z_q > 0.0) || !(Z_q < CUDART_INF);
                }
                err = __reduce_max_sync(0xffffffffu, err);
                if (bad && !err) err = slow ? SPEC_DEV_TIMEOUT : SPEC_DEV_NONFINITE;
                kind = (hint_dead || err) ? ITEM_DEAD : (hq ? ITEM_NODE : ITEM_LEAF);
                __syncwarp();
                if (kind == ITEM_NODE) {
                    const int j = lane & 15;
                    const bool mine = j < kc;
                    const int my_tok = mine ? (int)N.cpm[j] : 0;
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
                    N.kc = kc; N.err = err; N.leaf_mask = ~nonleaf;
                }
            }
            if (lane == 0) N.kind = kind;
            __syncwarp();
            if (own_block) {
                if (kind == ITEM_DEAD && N.err == 0 && N.kc <= KMAX) {
                    if (rank == 0) dead_node(P, TP.part, N);
                    continue;
                }
                // (a faulty node after all: it goes to the consumers like any other item)
                claim_block();
                {
                    const int *src = reinterpret_cast<const int *>(&S.scd);
                    int *dst = reinterpret_cast<int *>(&S.sc[sbuf]);
                    for (int i = lane; i < (int)(sizeof(NodeScalars) / 4); i += 32) dst[i] = src[i];
                }
                __syncwarp();
            }
            if (lane == 0) mbar_arrive(&S.sfull[sbuf]);
            if (kind != ITEM_NODE && kind != ITEM_FINISH) continue;

            // ---- the item's rows through the ring -------------------------------------------------------------------
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
        }
        if (*(volatile int *)&S.poison && lane == 0) {
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
        Resident R;

        for (int kidx = 0;; ++kidx) {
            // ---- the item's scalars, gathered by the producer warp ------------------------------------------------
            bool poisoned = *(volatile int *)&S.poison != 0;
            const NodeScalars &W = S.sc[kidx & 1];
            if (!poisoned && !mbar_wait(&S.sfull[kidx & 1], (uint32_t)((kidx >> 1) & 1))) { S.poison = 1; poisoned = true; }
            const int kind = poisoned ? ITEM_EXIT : W.kind;
            if (kind == ITEM_EXIT) break;
            const int a = W.a, b = W.b;
            int err = W.err;
            const int *parent = P.parent + (long long)b * P.topo_stride;

            // a childless child is finished here, by the scribe warp: its record; its arrival is made with the node's
            unsigned narr = 1u;
            auto finish_leaf = [&](int c, double thr_c, int j = -1) {
                leaf_record(P, TP.part, b, c, thr_c, j >= 0 ? W.cord[j] : 0u, j >= 0 ? W.cu[j] : 0.f);
                ++narr;
            };

            if (kind == ITEM_IDLE) {
                // a sequence without a bonus draw: its status says why (a timeout met here is added)
                if (scribe && lane == 0 && err) P.out.status[b] = err;
            } else if (kind == ITEM_LEAF || kind == ITEM_DEAD) {
                // ---- no rows: a childless node is tested with the weight it was handed; nothing under a node of
                // weight 0 (or under a faulty node) can be accepted -----------------------------------------------
                if (scribe) {
                    double w_in = 1.0;
                    if (W.pruned) {
                        w_in = 0.0;        // whatever its weight, it cannot be the accepted node
                    } else if (trav && a > 0 && !err) {
                        unsigned long long bits = W_PENDING;
                        if (lane == 0) bits = poll_weight(P.w_pub + (long long)b * P.N + a, &S.poison);
                        bits = __shfl_sync(0xffffffffu, bits, 0);
                        if (bits == W_PENDING) { err = SPEC_DEV_TIMEOUT; S.poison = 1; w_in = 0.0; }
                        else w_in = __longlong_as_double((long long)bits);
                    }
                    if (lane == 0) {
                        NodeRec *rec = P.rec + (long long)b * P.N;
                        NodeRec &Rc = rec[a];
                        Rc.O_p = (double)W.O_p; Rc.Z_p = W.Z_p; Rc.O_q = (double)W.O_q; Rc.Z_q = W.Z_q;
                        Rc.kappa = W.Z_p; Rc.nsteps = 0;
                        Rc.cut_p = W.cut_p; Rc.cut_q = W.cut_q;
                        Rc.next_child = -1;
                        Rc.status = err;
                        Rc.bonus = -1; Rc.bonus_margin = 0.f;
                        if (trav) { Rc.thr = (a == 0) ? 1.0 : (err ? 0.0 : w_in); if (a == 0) Rc.w_in = 1.0; }
                        else { Rc.w_in = 1.0; if (a == 0) Rc.thr = 1.0; }
                    }
                    // the children of a node of weight 0 (or of a faulty one) get weight / threshold 0 at once
                    if (kind == ITEM_DEAD && W.kc > KMAX) {
                        // too many children to list: found by scanning
                        for (int c = a + 1; c < P.N; ++c) {
                            if (__ldg(parent + c) != a) continue;
                            if (!warp_has_children(parent, P.N, c, lane)) { finish_leaf(c, 0.0); continue; }
                            if (lane == 0) {
                                NodeRec *rec = P.rec + (long long)b * P.N;
                                if (trav) {
                                    rec[c].w_in = 0.0;
                                    *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + c) = 0ull;
                                } else {
                                    rec[c].thr = 0.0;
                                }
                            }
                        }
                    } else if (kind == ITEM_DEAD)
                        for (int j = 0; j < W.kc; ++j) {
                            const int c = W.child[j];
                            if ((W.leaf_mask >> j) & 1u) { finish_leaf(c, 0.0); continue; }
                            if (lane == 0) {
                                NodeRec *rec = P.rec + (long long)b * P.N;
                                if (trav) {
                                    rec[c].w_in = 0.0;
                                    *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + c) = 0ull;
                                } else {
                                    rec[c].thr = 0.0;
                                }
                            }
                        }
                    arrive_sequence(P, b, narr);
                }
            } else {
              // ---- a node, or a sequence's FINISH item: pass 1 (one copy of its code for both): e = 2^(z s - O) of
              // the rows, resident; dominant tokens to the exact lists ----------------------------------------------
              NodeRows nr;
              nr.s_d = 1.4426950408889634 / (double)(P.T_seq ? __ldg(P.T_seq + b) : P.T);
              nr.s_hi = (float)nr.s_d;
              if ((double)nr.s_hi > nr.s_d) nr.s_hi = __uint_as_float(__float_as_uint(nr.s_hi) - 1u);
              nr.s_lo = (float)(nr.s_d - (double)nr.s_hi);
              if (!(nr.s_lo > 0.f)) nr.s_lo = 1.0e-30f;
              // (a FINISH item reads the draft row only if the accepted node's state is not its target row)
              nr.hq = kind == ITEM_NODE || W.nsteps != 0;
              nr.cut_p = W.cut_p; nr.cut_q = W.cut_q; nr.O_p = W.O_p; nr.O_q = W.O_q;
              set_list_thresholds(nr, W.Z_p, W.Z_q);
              int nl;
              float zs_p, zs_q;
              KlSums kls = {0.f, 0.f, 0.f, 0.f};
              pass1<DT, NW, AN>(rc, stage, phase, poisoned, nr, es, nsm, nrg, n_slice, tid, R, L, nl, zs_p, zs_q, &kls);
              if (kind == ITEM_NODE) {
                const int kc = W.kc;
                if (poisoned && !err) err = SPEC_DEV_TIMEOUT;

                // ---- the rows' normalisers from what is resident (one exchange) -----------------------------------
                double Z_p = W.Z_p, Z_q = W.Z_q;
                {
                    const double v[2] = {warp_sum_once((double)zs_p + (lane < nl ? L.ep[lane] : 0.0)),
                                         warp_sum_once((double)zs_q + (lane < nl ? L.eq[lane] : 0.0))};
                    double tot[2], mine[2];
                    cluster_exchange<NW, 2>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                    if (*(volatile int *)&S.poison) err = SPEC_DEV_TIMEOUT;
                    else if (!(tot[0] > 0.0) || !(tot[1] > 0.0)) err = SPEC_DEV_NONFINITE;
                    else { Z_p = tot[0]; Z_q = tot[1]; }
                }
                const double invZq = err ? 0.0 : __drcp_rn(Z_q);

                // ---- Traversal: the weight handed down by the parent (bounded poll, every warp for itself) ------
                double w_in = 1.0;
                if (trav && a > 0 && !err) {
                    unsigned long long bits = W_PENDING;
                    if (lane == 0) bits = poll_weight(P.w_pub + (long long)b * P.N + a, &S.poison);
                    bits = __shfl_sync(0xffffffffu, bits, 0);
                    if (bits == W_PENDING) { err = SPEC_DEV_TIMEOUT; S.poison = 1; w_in = 0.0; }
                    else w_in = __longlong_as_double((long long)bits);
                }

                // ---- offline analysis on the untouched rows (read-only sweeps, totals identical in every warp) ----------
                double an_rho = 1.0, an_beta = 0.0, an_pacc = 0.0, an_sres = 0.0;
                if (AN && !err) {
                    const double ip = __drcp_rn(Z_p), iq = invZq;
                    const double kd = (double)kc;
                    auto sweep2 = [&](auto f, double &t0, double &t1) {
                        double o0, o1;
                        reduce_sweep<NW>(es, nsm, tid, R, L, nl, f, o0, o1);
                        const double v[2] = {warp_sum_once(o0), warp_sum_once(o1)};
                        double tot[2], mine[2];
                        cluster_exchange<NW, 2>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                        t0 = tot[0]; t1 = tot[1];
                    };
                    double l1, smin, klpq, klqp, nss, naive2;
                    sweep2(FnL1Min{(float)ip, (float)iq, ip, iq}, l1, smin);
                    {
                        // KL(p||q) = ln 2 (sum e_p x_p - sum e_p x_q) / Z_p - ln Z_p + ln Z_q, and the mirror image
                        const double v1[2] = {warp_sum_once((double)kls.pp), warp_sum_once((double)kls.pq)};
                        const double v2[2] = {warp_sum_once((double)kls.qq), warp_sum_once((double)kls.qp)};
                        double t1[2], t2[2], mine[2];
                        cluster_exchange<NW, 2>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v1, t1, mine);
                        cluster_exchange<NW, 2>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v2, t2, mine);
                        const double lz = log(Z_p) - log(Z_q);
                        klpq = 0.6931471805599453 * (t1[0] - t1[1]) * ip - lz;
                        klqp = 0.6931471805599453 * (t2[0] - t2[1]) * iq + lz;
                    }
                    sweep2(FnNssNaive{(float)ip, (float)iq, ip, iq, (float)kd, kd}, nss, naive2);
                    // SpecTr's division factor: root of 1 - (1 - beta)^k - rho beta on [1, k] by bisection (Appendix B)
                    double lo = 1.0, hi = kd, dummy;
                    if (kc > 1) {
                        for (int it = 0; it < 40; ++it) {
                            const double mid = 0.5 * (lo + hi), ipr = ip / mid;
                            double beta;
                            sweep2(FnBeta{(float)ipr, (float)iq, ipr, iq}, beta, dummy);
                            const double f = (1.0 - pow(1.0 - beta, kd)) - mid * beta;
                            if (f > 0.0) lo = mid; else hi = mid;
                        }
                        an_rho = 0.5 * (lo + hi);
                    }
                    {
                        const double ipr = ip / an_rho;
                        sweep2(FnBeta{(float)ipr, (float)iq, ipr, iq}, an_beta, dummy);
                    }
                    an_pacc = 1.0 - pow(1.0 - an_beta, kd);
                    const double gamma = an_beta > 0.0 ? an_pacc / an_beta : 0.0;
                    const double ib = an_beta < 1.0 ? 1.0 / (1.0 - an_beta) : 0.0;
                    double sacc;
                    sweep2(FnSpecTrRes{(float)ip, (float)iq, (float)(1.0 / an_rho), (float)gamma, (float)ib, (float)kd,
                                       ip, iq, 1.0 / an_rho, gamma, ib, kd}, an_sres, sacc);
                    if (*(volatile int *)&S.poison) err = SPEC_DEV_TIMEOUT;
                    if (scribe && lane == 0 && !err) {
                        float *ao = TP.an_acc + ((long long)b * P.N + a) * 4, *dv = TP.an_div + ((long long)b * P.N + a) * 3;
                        ao[0] = (float)nss;
                        ao[1] = (float)(smin + naive2);
                        ao[2] = (float)(an_pacc + (1.0 - an_pacc) * (an_sres > 0.0 ? sacc / an_sres : 0.0));
                        dv[0] = (float)l1; dv[1] = (float)klpq; dv[2] = (float)klqp;
                    }
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
                double *gs = TP.gseq + ((long long)b * P.N + a) * KMAX;
                int acc = -1;
                if (err && scribe) {
                    // nothing below a faulty node is evaluated: every child gets weight / threshold 0
                    for (int j = 0; j < kce; ++j) {
                        const int c = W.child[j];
                        if ((W.leaf_mask >> j) & 1u) { finish_leaf(c, 0.0); continue; }
                        if (lane == 0) {
                            NodeRec *rec = P.rec + (long long)b * P.N;
                            if (trav) {
                                rec[c].w_in = 0.0;
                                *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + c) = 0ull;
                            } else {
                                rec[c].thr = 0.0;
                            }
                        }
                    }
                }
                for (int j = 0; j < kce && !err; ++j) {
                    // child j from the current state: P(x) = u(x) / kappa, q(x) = e_q(x) / Z_q
                    const double uxj = __shfl_sync(0xffffffffu, ux, j), eqj = __shfl_sync(0xffffffffu, eqx, j);
                    const double Pq = eqj * invZq;
                    const double Pp = is_q ? Pq : uxj / kappa;
                    if (AN && scribe && lane < kce) {
                        // round j's acceptance probability of every child's token: min(1, p_j(x_t) / q(x_t))
                        const double q_t = eqx * invZq, p_t = is_q ? q_t : ux / kappa;
                        TP.an[(long long)b * P.N + a].A[j][lane] =
                            !(p_t > 0.0) ? 0.0 : (!(q_t > 0.0) ? 1.0 : fmin(1.0, p_t / q_t));
                    }
                    double thr;
                    if (dead || !(Pp > 0.0)) thr = 0.0;
                    else if (!(Pq > 0.0)) thr = 1.0;
                    else thr = fmin(1.0, w * (Pp / Pq));
                    // Traversal: a weight within a rounding of 1 is 1.  The step after it is discontinuous at
                    // w = 1 when P = q (S = 0 gives weight 1 for w = 1 and weight 0 for any w < 1).
                    if (trav && thr > 1.0 - WEIGHT_SNAP) thr = 1.0;
                    if (scribe) {
                        const int cj = W.child[j];
                        if ((W.leaf_mask >> j) & 1u) {
                            finish_leaf(cj, thr, j);
                        } else if (lane == 0) {
                            NodeRec *rec = P.rec + (long long)b * P.N;
                            if (trav) {
                                // the child polls the published slot only; the record is read after all of the
                                // sequence's arrivals (each fenced), so no fence is needed between the two stores
                                rec[cj].w_in = thr;
                                if (b * P.N + cj != c_hold_slot)      // (a test may ask for one slot to stay pending)
                                    *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + cj) =
                                        (unsigned long long)__double_as_longlong(thr);
                            } else {
                                rec[cj].thr = thr;
                            }
                        }
                    }
                    if (!trav && acc < 0 && (double)W.cu[j] < thr) {
                        acc = W.child[j];
                        if (!P.all_thr) {
                            if (scribe)
                                for (int jj = j + 1; jj < kce; ++jj) {
                                    if ((W.leaf_mask >> jj) & 1u) finish_leaf(W.child[jj], CUDART_NAN);
                                    else if (lane == 0) P.rec[(long long)b * P.N + W.child[jj]].thr = CUDART_NAN;
                                }
                            break;
                        }
                    }
                    if (AN && scribe && lane == 0 && (dead || is_q)) TP.an[(long long)b * P.N + a].S[j] = 0.0;
                    if (dead || is_q) continue;       // weight 0, or P = q (every further step has S = 0 again)
                    // the step after rejecting child j: u <- (g u - e_q)+ , g = w Z_q / kappa
                    const double g = __ddiv_rn(w * Z_q, kappa);
                    const double v[1] = {warp_sum_once(step_sweep<NW>(es, nsm, tid, R, L, nl, g))};
                    double tot[1], mine[1];
                    cluster_exchange<NW, 1>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                    if (*(volatile int *)&S.poison) { err = SPEC_DEV_TIMEOUT; break; }
                    ux = fmax(fma(g, ux, -eqx), 0.0);
                    const double Sj = tot[0] * invZq;
                    if (AN && scribe && lane == 0) TP.an[(long long)b * P.N + a].S[j] = Sj > RESIDUAL_FLOOR * w ? Sj : 0.0;
                    // A step whose mass is below 1e-13 of the weight before it counts as S = 0: P equals q, and what
                    // is left is the rounding of g.
                    if (Sj > RESIDUAL_FLOOR * w) {
                        kappa = tot[0];
                        if (trav) w = Sj / (Sj + (1.0 - w));
                        if (scribe && lane == 0) gs[nsteps] = g;
                        ++nsteps;
                    } else if (w >= 1.0) {
                        is_q = true;       // S = 0 with w = 1: the state is q itself (the stored u is no longer used)
                        kappa = Z_q;
                    } else {
                        dead = true;       // S = 0 with w < 1: the weight drops to 0 (Traversal only)
                        w = 0.0;
                    }
                }

                if (AN && scribe) {
                    AnRec &Ar = TP.an[(long long)b * P.N + a];
                    if (lane < kce) {
                        const double q_t = eqx * invZq;
                        Ar.A[kce][lane] = err ? 0.0 : (is_q ? q_t : ux / kappa);      // p_k(x_t)
                        Ar.px[lane] = W.cpm[lane] / Z_p;
                        Ar.qx[lane] = q_t;
                    }
                    if (lane == 0) {
                        Ar.rho = an_rho; Ar.beta = an_beta; Ar.pacc = an_pacc; Ar.s_res = an_sres;
                        Ar.k = kce; Ar.valid = err ? 0 : 1;
                    }
                }

                // ---- the node's outcome -----------------------------------------------------------------------------
                const double w_fin = (dead || err) ? 0.0 : w;
                if (scribe) {
                    if (lane == 0) {
                        NodeRec &Rc = P.rec[(long long)b * P.N + a];
                        Rc.O_p = (double)nr.O_p; Rc.Z_p = Z_p; Rc.O_q = (double)nr.O_q; Rc.Z_q = Z_q;
                        Rc.kappa = (dead || err) ? 0.0 : kappa;
                        Rc.nsteps = is_q ? STATE_IS_Q : nsteps;
                        Rc.cut_p = nr.cut_p; Rc.cut_q = nr.cut_q;
                        Rc.next_child = acc;
                        Rc.status = err;
                        Rc.bonus = -1; Rc.bonus_margin = 0.f;
                        if (trav) { Rc.thr = (a == 0) ? 1.0 : w_fin; if (a == 0) Rc.w_in = 1.0; }
                        else { Rc.w_in = 1.0; if (a == 0) Rc.thr = 1.0; }
                        if (P.prune && a > 0 && !err && (W.ord_a >> 31) && (double)W.u_a < w_fin)
                            atomicMin(P.best + b, (W.ord_a >> 8) & 255u);
                    }
                    arrive_sequence(P, b, narr);
                }
              } else {
                // ---- FINISH: the accepted node back on chip, its recorded steps replayed, the bonus token drawn ---------
                const int nsteps = W.nsteps;
                const bool is_q = nsteps == STATE_IS_Q;
                double part = (double)zs_p + (lane < nl ? L.ep[lane] : 0.0);
                if (is_q) part = (double)zs_q + (lane < nl ? L.eq[lane] : 0.0);
                for (int j = 0; j < nsteps; ++j) part = step_sweep<NW>(es, nsm, tid, R, L, nl, W.cpm[j]);
                const double v[1] = {warp_sum_once(part)};
                double tot[1], mine[1];
                cluster_exchange<NW, 1>(xchg, S.xbar, xn, C, rank, warp, lane, &S.poison, v, tot, mine);
                int ferr = (poisoned || *(volatile int *)&S.poison) ? SPEC_DEV_TIMEOUT : 0;
                double tau = 0.0;
                int owner = -1;
                if (!ferr) {
                    const double target = (double)W.ub_a * tot[0];
                    owner = pick_lane(lane < C ? mine[0] : 0.0, target, tau);
                    if (owner < 0) ferr = SPEC_DEV_NONFINITE;
                }
                int role = 0, tokn = -1;
                float mg = 0.f;
                if (ferr) {
                    role = (scribe && lane == 0) ? (ferr == SPEC_DEV_TIMEOUT ? 3 : 2) : 0;
                } else if (owner == (int)rank) {
                    const BonusFind bf = bonus_search<NW>(S.wtile, &S.cbar, cph, &S.poison, es, nsm, tid, R, L, nl, is_q, tau);
                    role = bf.role;
                    tokn = (int)(tok0 + bf.token);
                    mg = (float)(bf.edge / tot[0]);
                }
                if (role == 1) {
                    const int len = W.len;
                    P.out.bonus_token[b] = tokn;
                    P.out.out_tokens[(long long)b * P.N + len] = tokn;
                    if (P.out.margin) P.out.margin[(long long)b * (P.N + 1) + P.N] = mg;
                } else if (role >= 2) {
                    P.out.status[b] = role == 3 ? SPEC_DEV_TIMEOUT : SPEC_DEV_NONFINITE;
                    P.out.accepted_node[b] = -1; P.out.accept_len[b] = -1; P.out.bonus_token[b] = -1;
                    int *ot = P.out.out_tokens + (long long)b * P.N;
                    for (int i = 0; i < P.N; ++i) ot[i] = -1;
                }
              }
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
