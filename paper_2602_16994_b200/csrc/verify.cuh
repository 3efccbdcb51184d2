// Pieces shared by the verification kernels (walk.cuh: SpecInfer along the accepted path, Algorithm 4
// composed top-down, Section 3.2; tree.cuh: every node, Traversal Verification of Section 3.2 with the
// block-verification weights of Section 3.1): constants and shared-memory layouts, the handling of
// one chunk of 8 logits (unpack, mask, exponentiate), the residual pass over resident e, prefix picks,
// the inverse-CDF search for the bonus token, and the writing of a sequence's outputs from the node
// records.
//
// Common ground of both kernels.  Each CTA of a cluster owns a contiguous vocabulary slice; each
// consumer thread owns 8 consecutive tokens of every tile of that slice.  A logit becomes
// e = 2^(z s - O) with s = log2(e)/T and O the row's integer reference, so every scale factor is an
// exact power of two.  The e of the last RT tiles of a slice stay in registers, the others in shared
// memory; nothing is written back to HBM.
//
// The recursion is the paper's own, step by step.  A node's state after j rejected children is the
// residual law P_j with P_0 = p, held as u_j(t) = kappa_j P_j(t) in place of the resident e_p:
//     u_j(t) = (g_j u_{j-1}(t) - e_q(t))+ ,   g_j = w_{j-1} Z_q / kappa_{j-1} ,   kappa_j = sum_t u_j(t) ,
// which is Z_q (w_{j-1} P_{j-1} - q)+, so kappa_j = Z_q S_j with S_j the step's residual mass
// (SpecInfer: w = 1 throughout and child j is accepted with min(1, P_{j-1}(x) / q(x)); Traversal
// Verification: w_j = S_j / (S_j + 1 - w_{j-1}) and child j is handed min(1, w_{j-1} P_{j-1}(x) / q(x))).
// One sibling step is one sweep over the resident data (subtract, clamp, store, sum) plus one scalar
// exchange through distributed shared memory.  Every step renormalises, as the paper's
// P <- norm((P - q)+) does, so a state that is reached with probability 1e-15 is as well conditioned
// as the first one; a closed form in the original units, (w P_0 - c_j q)+ with accumulated c_j, is
// not: its difference cancels to the rounding of fp64 once the accumulated mass drops below 1e-11.
// The children's tokens follow the same recursion as scalars in fp64.
//
// Precision.  The e are fp32 (one ex2.approx each, relative error about 2^-22), which is not enough
// where a residual mass E_j is small against the probabilities it is the difference of (two peaked
// laws on the same token: near-greedy temperatures, top-k / top-p): w_in P0(x) - c_j q(x) then cancels
// to a few 1e-7 of its terms.  The few tokens that carry a row's mass are therefore kept exactly: every
// consumer warp owns a short list of DOMINANT tokens of its part of the slice (above 2^-DOM_A of the
// row's mass always; above 2^-DOM_B while the list has room), whose exponentials are evaluated in fp64
// and whose fp32 copies are set to zero.  Every sum over the vocabulary is then (fp32 over the tail,
// accumulated in fp64 above a thread) + (fp64 over the lists), and so are the rows' normalisers, which
// the cluster recomputes from the resident e instead of taking them from the statistics pass.
//
// Exchanges.  Every consumer warp of every CTA of the cluster sends its partial sum straight into
// the shared memory of all CTAs (st.async, which counts the bytes on the receiver's mbarrier); every
// warp waits on its own CTA's mbarrier and reduces all partials itself, in one fixed order, so all
// warps of the cluster hold bit-identical totals and take identical decisions without any CTA-wide
// barrier.
#pragma once
#include "common.cuh"

namespace specv {

constexpr int RT = 4;        // tiles per thread whose e may live in registers
constexpr int SMT = 10;      // tiles per thread whose e may live in shared memory
constexpr int TMAX = RT + SMT;
constexpr int CMAX = 16;     // CTAs per cluster (above 8: non-portable size)
constexpr int NSMAX = 16;    // ring stages
constexpr int NWMAX = 15;    // consumer warps
constexpr int OMIN = -(1 << 30);
constexpr int FAST_N = 32;   // trees up to this size are finished warp-parallel
constexpr int FIN_PENDING = -1;     // VParams::fin of a sequence whose nodes are not all done
constexpr int FIN_FAULTY = -2;      // ... of a sequence with a device-detected fault: no bonus draw
constexpr int FIN_LEN_SHIFT = 12;   // a selected node is published as node | (accepted length << FIN_LEN_SHIFT)
static_assert(SPEC_MAX_NODES <= (1 << FIN_LEN_SHIFT) && SPEC_MAX_NODES < (1 << (30 - FIN_LEN_SHIFT)), "packing of the published node");
// A residual step whose mass is below this fraction of the mass before it is treated as S = 0: where P
// equals q (the same row twice, two one-token nuclei on the same token) the exact difference is 0 and
// the computed one a few 1e-16 of the mass (the rounding of the coefficient g).
constexpr double RESIDUAL_FLOOR = 1.0e-13;
// Traversal: a handed-down weight this close to 1 is 1 (a ratio that is exactly 1 may come out one
// rounding below; the step after it is discontinuous at w = 1 when S = 0)
constexpr double WEIGHT_SNAP = 1.0e-12;

// exact list of dominant tokens, one per consumer warp
constexpr int MW = 32;       // entries (one per lane in a pass)
constexpr int MW_RES = 8;    // entries kept free for tokens above 2^-DOM_A of a row's mass
constexpr int DOM_A = 6;     // such a token is always listed: at most 64 per row, and they are what bounds the tail's error
constexpr int DOM_B = 34;    // tokens above 2^-DOM_B of a row's mass are listed while the list has room

enum Mode { MODE_SPECINFER = 0, MODE_TRAVERSAL = 1 };

struct VParams {
    int B, N, V, C, mode, all_thr;
    int slice_len;            // tokens per CTA slice: a multiple of 8, at most TMAX tiles
    int NS;                   // ring stages
    int nsm;                  // tiles of a slice kept in shared memory (the others, at most RT, in registers)
    int off_x, off_list, off_es, off_ring;   // byte offsets inside dynamic shared memory
    const void *zp, *zq;
    long long seq_stride, node_stride, topo_stride;
    const int *parent, *token;
    float T;
    const float *T_seq;
    const float *u_accept, *u_bonus;
    NodeRec *rec;
    unsigned long long *w_pub;   // [B*N] weight handed to a node by its parent (Traversal), W_PENDING until known
    unsigned int *done;          // [B] arrivals per sequence (one per node); the last one selects the accepted node
    int *fin;                    // [B] the accepted node once it is selected (FIN_PENDING before, FIN_FAULTY for a faulty sequence)
    unsigned int *best;          // [B] smallest post-order rank of a node known to be accepted if reached (all-ones: none)
    unsigned long long *order;   // [B*N] low word: 0x80000000 | post-order rank << 8 | nodes wholly before the node's
                                 // subtree; high word: the node's ancestors (itself included) as a bit mask; 0: not computed
    int prune;                   // Traversal: skip subtrees that lie wholly after a known acceptance
    SpecOut out;
};

// per consumer warp: the children of the current node and the scalar state of its recursion
struct __align__(16) WarpList {
    double ep[MW], eq[MW];         // exact 2^(z s - O) of the token in the target / draft row (0: cut, or no draft row)
    int pos[MW];                   // (slot << 8) | (lane << 3) | position in the chunk; slot as in bonus_search
};

// the e of the RT register tiles of a thread
struct Resident {
    float p[RT][8], q[RT][8];
};

struct __align__(16) WarpArea {
    double cpm[KMAX], cqm[KMAX];   // exact 2^(z s - O) of the children's tokens in the node's target and draft rows
    float cu[KMAX];
    int child[KMAX];
    double c, E, G;                // committed state (see the file header); identical in every warp of the cluster
    double A, w_in, invZp, invZq;  // A = w_in / Z_p
    double Rg;                     // pass coefficient g = (c + G) Rg, Rg = Z_p / (w_in Z_q)
    double g_commit;               // coefficient of the pass the committed state came from (0: none)
    double Z_p, Z_q;
    int O_p, O_q;
};

struct __align__(16) Hdr {
    uint64_t full[NSMAX], empty[NSMAX], xbar[2], cbar;
    double wtile[NWMAX + 1][TMAX];
    WarpArea wa[NWMAX];
    int poison;
};

// ------------------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool warp_has_children(const int *parent, int N, int a, int lane)
{
    for (int c0 = a + 1; c0 < N; c0 += 32) {
        int c = c0 + lane;
        bool is = c < N && __ldg(parent + c) == a;
        if (__any_sync(0xffffffffu, is)) return true;
    }
    return false;
}

// the 8 logits a thread owns in one tile of one row, as they sit in the ring
template <int DT>
struct RawChunk {
    uint4 a, b;      // bf16: a only
};
template <int DT>
__device__ __forceinline__ RawChunk<DT> read_raw(const unsigned char *sp)
{
    RawChunk<DT> r;
    r.a = *reinterpret_cast<const uint4 *>(sp);
    if (DT == SPEC_F32) r.b = reinterpret_cast<const uint4 *>(sp)[1];
    return r;
}
template <int DT>
__device__ __forceinline__ void unpack_chunk(const RawChunk<DT> &r, float (&z)[8])
{
    if (DT == SPEC_BF16) {
        z[0] = bf16_lo(r.a.x); z[1] = bf16_hi(r.a.x); z[2] = bf16_lo(r.a.y); z[3] = bf16_hi(r.a.y);
        z[4] = bf16_lo(r.a.z); z[5] = bf16_hi(r.a.z); z[6] = bf16_lo(r.a.w); z[7] = bf16_hi(r.a.w);
    } else {
        z[0] = __uint_as_float(r.a.x); z[1] = __uint_as_float(r.a.y); z[2] = __uint_as_float(r.a.z); z[3] = __uint_as_float(r.a.w);
        z[4] = __uint_as_float(r.b.x); z[5] = __uint_as_float(r.b.y); z[6] = __uint_as_float(r.b.z); z[7] = __uint_as_float(r.b.w);
    }
}
// logits beyond the slice (nvalid < 8) or below the row's cut become -inf
__device__ __forceinline__ void mask_chunk(float (&z)[8], int nvalid, bool has_cut, float cut)
{
    if (nvalid < 8) {
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (k >= nvalid) z[k] = -CUDART_INF_F;
    }
    if (has_cut) {
#pragma unroll
        for (int k = 0; k < 8; ++k) z[k] = z[k] >= cut ? z[k] : -CUDART_INF_F;
    }
}

// e[k] = 2^(z[k] s - of) for the 8 logits of a chunk (the large product z s_hi - of is formed first, in
// one rounding, so that the exponent's error is relative to the exponent and not to of), of the thread's reference for this row (an
// integer-valued float); returns sum e.  FEAT: also sx += sum e x with x the exponent.
template <bool FEAT>
__device__ __forceinline__ float exp_chunk(const float (&z)[8], float s_hi, float s_lo, float of, float (&e)[8],
                                           float &sx)
{
    float sum = 0.f;
    if (FEAT) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float x = fmaxf(fmaf(z[k], s_lo, fmaf(z[k], s_hi, -of)), -200.f);
            e[k] = ex2_approx(x);
            sum += e[k];
            sx = fmaf(e[k], x, sx);
        }
    } else {
        // two exponents per instruction (fp32 pairs; each half is the scalar operation)
        const unsigned long long sh2 = pack_f32x2(s_hi, s_hi), sl2 = pack_f32x2(s_lo, s_lo), no2 = pack_f32x2(-of, -of);
#pragma unroll
        for (int k = 0; k < 8; k += 2) {
            const unsigned long long z2 = pack_f32x2(z[k], z[k + 1]);
            float x0, x1;
            unpack_f32x2(fma_f32x2(z2, sl2, fma_f32x2(z2, sh2, no2)), x0, x1);
            e[k] = ex2_approx(x0);
            e[k + 1] = ex2_approx(x1);
            sum += e[k] + e[k + 1];
        }
    }
    return sum;
}
__device__ __forceinline__ void load_e8(const float4 *d, int stride, float (&e)[8])
{
    const float4 lo = d[0], hi = d[stride];
    e[0] = lo.x; e[1] = lo.y; e[2] = lo.z; e[3] = lo.w; e[4] = hi.x; e[5] = hi.y; e[6] = hi.z; e[7] = hi.w;
}

// first lane whose running sum of v exceeds tau (v >= 0 in every lane); if rounding leaves none, the
// last lane with v > 0 and tau_res = +inf; -1 if no lane has weight.  All lanes get the same answer.
// Not inlined on purpose: it runs a handful of times per sequence, and one copy that is already in the
// instruction cache after its first call is faster than several cold ones.
__device__ __noinline__ int pick_lane(double v, double tau, double &tau_res)
{
    const int lane = threadIdx.x & 31;
    double incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    const double excl = incl - v;
    const unsigned hit = __ballot_sync(0xffffffffu, incl > tau && v > 0.0);
    if (hit) {
        const int idx = __ffs(hit) - 1;
        tau_res = tau - __shfl_sync(0xffffffffu, excl, idx);
        return idx;
    }
    const unsigned pos = __ballot_sync(0xffffffffu, v > 0.0);
    tau_res = CUDART_INF;
    return pos ? 31 - __clz(pos) : -1;
}

// 2^(z s - O) in fp64 (about 1e-15 relative); 0 for -inf and for exponents below the double range
__device__ __forceinline__ double exp2_exact(float z, double s_d, int O)
{
    const double xd = (double)z * s_d - (double)O;
    if (!(xd > -1000.0)) return 0.0;
    const double nd = rint(xd);
    return exp2_frac(xd - nd) * pow2d((int)nd);
}

// ------------------------------------------------------------------------------------------------
// pass 1: a node's rows from the ring into resident e, its dominant tokens into the warp's exact list
// ------------------------------------------------------------------------------------------------
// what pass 1 has to know about the two rows of a node
struct NodeRows {
    bool hq;                  // the node has children: its draft row is read too
    float cut_p, cut_q;       // smallest kept logit (-inf: nothing cut)
    int O_p, O_q;             // integer references of the rows
    float s_hi, s_lo;         // log2(e) / T = s_hi + s_lo
    double s_d;
    float thrA_p, thrA_q;     // e above this: always listed (2^-DOM_A of the row's mass)
    float thrB_p, thrB_q;     // e above this: listed while the list has room (2^-DOM_B)
};
// Z: the row's normaliser from the statistics pass (fp32 exponentials: good enough for a threshold).
// The second tier pays only where it can hold nearly all of a row's mass, that is on laws that are
// peaked (near-greedy temperatures, short nuclei), and it is needed only where a residual mass is small
// against the weight, which takes two laws that nearly agree on their heavy tokens: both rows peaked.
// The largest e of a row lies in (1/2, 1], so Z > LIST_FLAT_Z means that no token holds more than
// 1/LIST_FLAT_Z of the row's mass.  On such a row the tier would fill with the first tokens it meets and
// buy nothing, so it is left out; a node without a draft row (nothing is subtracted there) has no use
// for it either.
constexpr double LIST_FLAT_Z = 4.0;
__device__ __forceinline__ void set_list_thresholds(NodeRows &nr, double Z_p, double Z_q)
{
    const double a = 1.0 / (double)(1ull << DOM_A), b = 1.0 / (double)(1ull << DOM_B);
    const bool flat = !nr.hq || Z_p > LIST_FLAT_Z || Z_q > LIST_FLAT_Z;
    nr.thrA_p = (float)(Z_p * a);
    nr.thrB_p = flat ? nr.thrA_p : (float)(Z_p * b);
    nr.thrA_q = nr.hq ? (float)(Z_q * a) : CUDART_INF_F;
    nr.thrB_q = nr.hq ? (flat ? nr.thrA_q : (float)(Z_q * b)) : CUDART_INF_F;
}
struct RingCtx {
    uint64_t *full, *empty;
    unsigned char *ring;
    int NS;
    int *poison;
};

// the e of the 8 tokens a thread owns in one tile, both rows (passed by value to list_append)
struct Chunk16 {
    float p[8], q[8];
};

// Warp-collective, and out of line on purpose (it runs on a few per cent of the tiles, and the kernels
// are short of instruction cache): the tokens of the lane's chunk whose e exceeds the always-listed
// threshold (thrA), or the while-there-is-room threshold (tp, tq), are appended to the warp's list while
// it has room, as raw logits (pass1 evaluates the exponentials in fp64 once all tiles are in).  n is the
// list's fill, the same in every lane.  Returns (new fill << 8) | the lane's mask of appended tokens
// (the caller zeroes their fp32 copies).
template <int DT>
__device__ __noinline__ unsigned list_append(WarpList &L, int n, const RawChunk<DT> raw_p, const RawChunk<DT> raw_q,
                                             const Chunk16 e, float thrA_p, float thrA_q, float tp, float tq, int nvalid,
                                             float cut_p, float cut_q, bool hq, int slot)
{
    const int lane = threadIdx.x & 31;
    const unsigned lt = (1u << lane) - 1u;
    unsigned m_any = 0, m_a = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const bool a = e.p[k] > thrA_p || e.q[k] > thrA_q;
        const bool any = a || e.p[k] > tp || e.q[k] > tq;
        m_any |= (any ? 1u : 0u) << k;
        m_a |= (a ? 1u : 0u) << k;
    }
    float zp[8], zq[8];
    unpack_chunk<DT>(raw_p, zp);
    unpack_chunk<DT>(raw_q, zq);
    unsigned adm = 0;
#pragma unroll 1
    for (int k = 0; k < 8; ++k) {
        if (n >= MW - MW_RES) m_any &= m_a;           // no room left in the second tier
        if (!__any_sync(0xffffffffu, (m_any >> k) != 0u)) break;
        const bool a = (m_a >> k) & 1u, b = ((m_any >> k) & 1u) && !a;
        const unsigned balA = __ballot_sync(0xffffffffu, a), balB = __ballot_sync(0xffffffffu, b);
        if (!(balA | balB)) continue;
        const int nA = min(n + __popc(balA), MW);
        const int capB = MW - MW_RES;
        const int nB = max(nA, min(nA + __popc(balB), capB));
        int idx = -1;
        if (a) { const int i = n + __popc(balA & lt); if (i < MW) idx = i; }
        else if (b) { const int i = nA + __popc(balB & lt); if (i < capB) idx = i; }
        n = nB;
        if (idx >= 0) {
            float z0 = zp[0], z1 = zq[0];
#pragma unroll
            for (int kk = 1; kk < 8; ++kk)
                if (kk == k) { z0 = zp[kk]; z1 = zq[kk]; }
            // the raw logits for now (-inf: cut, or no draft row); pass1 turns every entry into its
            // exponential at the end, all lanes at once, instead of one long fp64 chain per admission
            const bool valid = k < nvalid;
            L.ep[idx] = (valid && z0 >= cut_p) ? (double)z0 : -CUDART_INF;
            L.eq[idx] = (valid && hq && z1 >= cut_q) ? (double)z1 : -CUDART_INF;
            L.pos[idx] = (slot << 8) | (lane << 3) | k;
            adm |= 1u << k;
        }
    }
    __syncwarp();
    return ((unsigned)n << 8) | adm;
}

// cross sums of the two rows for the Kullback-Leibler divergences (analysis instantiation only):
// sum e_p x_p, sum e_p x_q, sum e_q x_p, sum e_q x_q with x = z s - O the exponents (a token cut from one row
// has x = -inf there, which makes the divergence from the other row infinite, as it is)
struct KlSums {
    float pp, pq, qp, qq;
};

// One tile: wait for the stage, take the thread's 8 logits of both rows, hand the stage back, turn them
// into e (EP, EQ), move dominant tokens to the list.  The thread's tail sums of e go to zs_p / zs_q.
template <int DT, int NW, bool KLS = false>
__device__ __forceinline__ void pass1_tile(const RingCtx &rc, int &stage, uint32_t &phase, bool &poisoned,
                                           const NodeRows &nr, int tile_index, int slot, int n_slice, int tid,
                                           float (&EP)[8], float (&EQ)[8], WarpList &L, int &nl, float &zs_p, float &zs_q,
                                           KlSums *kl = nullptr)
{
    constexpr int NCONS = NW * 32;
    constexpr int TILE = NCONS * 8;
    constexpr int ESZ = DT == SPEC_BF16 ? 2 : 4;
    constexpr int ROWB = TILE * ESZ;
    constexpr int STAGE = 2 * ROWB;
    if (!poisoned && !mbar_wait(&rc.full[stage], phase)) { *rc.poison = 1; poisoned = true; }
    const unsigned char *sp = rc.ring + (size_t)stage * STAGE + (size_t)tid * 8 * ESZ;
    const RawChunk<DT> raw_p = read_raw<DT>(sp);
    RawChunk<DT> raw_q = raw_p;
    if (nr.hq) raw_q = read_raw<DT>(sp + ROWB);
    __syncwarp();
    if ((tid & 31) == 0) mbar_arrive(&rc.empty[stage]);
    if (++stage == rc.NS) { stage = 0; phase ^= 1u; }
    const int nvalid = poisoned ? 0 : n_slice - (tile_index * TILE + tid * 8);
    float z[8], dsx = 0.f;
    float sum_p, sum_q = 0.f;
    if (KLS) {
        // the exponents themselves are needed: scalar form
        float xp[8], xq[8];
        unpack_chunk<DT>(raw_p, z);
        mask_chunk(z, nvalid, nr.cut_p > -CUDART_INF_F, nr.cut_p);
        sum_p = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) { xp[k] = fmaf(z[k], nr.s_lo, fmaf(z[k], nr.s_hi, -(float)nr.O_p)); EP[k] = ex2_approx(xp[k]); sum_p += EP[k]; }
        unpack_chunk<DT>(raw_q, z);
        mask_chunk(z, nvalid, nr.cut_q > -CUDART_INF_F, nr.cut_q);
#pragma unroll
        for (int k = 0; k < 8; ++k) { xq[k] = fmaf(z[k], nr.s_lo, fmaf(z[k], nr.s_hi, -(float)nr.O_q)); EQ[k] = ex2_approx(xq[k]); sum_q += EQ[k]; }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            if (EP[k] > 0.f) { kl->pp = fmaf(EP[k], xp[k], kl->pp); kl->pq = fmaf(EP[k], xq[k], kl->pq); }
            if (EQ[k] > 0.f) { kl->qp = fmaf(EQ[k], xp[k], kl->qp); kl->qq = fmaf(EQ[k], xq[k], kl->qq); }
        }
    } else {
        unpack_chunk<DT>(raw_p, z);
        mask_chunk(z, nvalid, nr.cut_p > -CUDART_INF_F, nr.cut_p);
        sum_p = exp_chunk<false>(z, nr.s_hi, nr.s_lo, (float)nr.O_p, EP, dsx);
        if (nr.hq) {
            unpack_chunk<DT>(raw_q, z);
            mask_chunk(z, nvalid, nr.cut_q > -CUDART_INF_F, nr.cut_q);
            sum_q = exp_chunk<false>(z, nr.s_hi, nr.s_lo, (float)nr.O_q, EQ, dsx);
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) EQ[k] = 0.f;
        }
    }
    // dominant tokens: a chunk whose sum stays below the threshold holds none (e >= 0)
    const bool room = nl < MW - MW_RES;
    const float tp = room ? nr.thrB_p : nr.thrA_p, tq = room ? nr.thrB_q : nr.thrA_q;
    if (__any_sync(0xffffffffu, sum_p > tp || sum_q > tq)) {
        Chunk16 e;
#pragma unroll
        for (int k = 0; k < 8; ++k) { e.p[k] = EP[k]; e.q[k] = EQ[k]; }
        const unsigned r = list_append<DT>(L, nl, raw_p, raw_q, e, nr.thrA_p, nr.thrA_q, tp, tq, nvalid, nr.cut_p,
                                           nr.cut_q, nr.hq, slot);
        nl = (int)(r >> 8);
        const unsigned adm = r & 255u;
        if (adm) {
            sum_p = 0.f; sum_q = 0.f;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if ((adm >> k) & 1u) { EP[k] = 0.f; EQ[k] = 0.f; }
                sum_p += EP[k]; sum_q += EQ[k];
            }
        }
    }
    zs_p += sum_p;
    zs_q += sum_q;
}

// Pass 1 of a node.  es: [slot][p lo, p hi, q lo, q hi][NCONS] for the nsm shared-memory tiles; the last
// nrg tiles of the slice stay in R.  On return nl is the fill of the warp's list and zs_p / zs_q the
// thread's sums of the fp32 e it keeps (listed tokens excluded).
template <int DT, int NW, bool KLS = false>
__device__ __forceinline__ void pass1(const RingCtx &rc, int &stage, uint32_t &phase, bool &poisoned, const NodeRows &nr,
                                      float4 *es, int nsm, int nrg, int n_slice, int tid, Resident &R, WarpList &L,
                                      int &nl, float &zs_p, float &zs_q, KlSums *kl = nullptr)
{
    constexpr int NCONS = NW * 32;
    nl = 0; zs_p = 0.f; zs_q = 0.f;
    for (int i = 0; i < nsm; ++i) {
        float ep[8], eq[8];
        pass1_tile<DT, NW, KLS>(rc, stage, phase, poisoned, nr, i, i, n_slice, tid, ep, eq, L, nl, zs_p, zs_q, kl);
        float4 *d = es + (size_t)(i * 4) * NCONS + tid;
        d[0] = make_float4(ep[0], ep[1], ep[2], ep[3]);
        d[NCONS] = make_float4(ep[4], ep[5], ep[6], ep[7]);
        d[2 * NCONS] = make_float4(eq[0], eq[1], eq[2], eq[3]);
        d[3 * NCONS] = make_float4(eq[4], eq[5], eq[6], eq[7]);
    }
#pragma unroll
    for (int j = 0; j < RT; ++j) {
        if (j < nrg) {
            pass1_tile<DT, NW, KLS>(rc, stage, phase, poisoned, nr, nsm + j, SMT + j, n_slice, tid, R.p[j], R.q[j], L, nl, zs_p, zs_q, kl);
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) { R.p[j][k] = 0.f; R.q[j][k] = 0.f; }
        }
    }
    // the listed tokens' exponentials in fp64, entry `lane` (list_append left the raw logits)
    __syncwarp();
    if ((tid & 31) < nl) {
        const int i = tid & 31;
        const double zp = L.ep[i], zq = L.eq[i];
        L.ep[i] = zp > -CUDART_INF ? exp2_exact((float)zp, nr.s_d, nr.O_p) : 0.0;
        L.eq[i] = zq > -CUDART_INF ? exp2_exact((float)zq, nr.s_d, nr.O_q) : 0.0;
    }
    __syncwarp();
}

// hand a node's stages back unread (the node turned out not to need its rows)
__device__ __forceinline__ void drain_tiles(const RingCtx &rc, int &stage, uint32_t &phase, bool &poisoned, int ntiles)
{
    for (int i = 0; i < ntiles; ++i) {
        if (!poisoned && !mbar_wait(&rc.full[stage], phase)) { *rc.poison = 1; poisoned = true; }
        __syncwarp();
        if ((threadIdx.x & 31) == 0) mbar_arrive(&rc.empty[stage]);
        if (++stage == rc.NS) { stage = 0; phase ^= 1u; }
    }
}

// One step on a chunk: u <- (g u - q)+ for its 8 tokens, g = gh + gl; returns the sum of the new u
// (two tokens per fused multiply-add; q - g u is formed and its negation clamped)
__device__ __forceinline__ float step_chunk(float (&u)[8], const float (&q)[8], float gh, float gl)
{
    const unsigned long long ngh2 = pack_f32x2(-gh, -gh), ngl2 = pack_f32x2(-gl, -gl);
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < 8; k += 2) {
        const unsigned long long u2 = pack_f32x2(u[k], u[k + 1]);
        float d0, d1;
        unpack_f32x2(fma_f32x2(ngl2, u2, fma_f32x2(ngh2, u2, pack_f32x2(q[k], q[k + 1]))), d0, d1);
        u[k] = fmaxf(-d0, 0.f);
        u[k + 1] = fmaxf(-d1, 0.f);
        acc += u[k] + u[k + 1];
    }
    return acc;
}
__device__ __forceinline__ float sum_chunk(const float (&u)[8])
{
    return ((u[0] + u[1]) + (u[2] + u[3])) + ((u[4] + u[5]) + (u[6] + u[7]));
}

// One sibling step over the thread's share of the resident node, in place: u <- (g u - e_q)+ for its
// fp32 tail tokens and for the entry of the warp's exact list that falls to its lane.  Returns the
// thread's sum of the new u.
template <int NW>
__device__ __forceinline__ double step_sweep(float4 *es, int nsm, int tid, Resident &R, WarpList &L, int nl, double g)
{
    constexpr int NCONS = NW * 32;
    float g_hi, g_lo;
    split_float(g, g_hi, g_lo);
    float tot = 0.f;
    for (int i = 0; i < nsm; ++i) {
        float u[8], q[8];
        float4 *d = es + (size_t)(i * 4) * NCONS + tid;
        load_e8(d, NCONS, u);
        load_e8(d + 2 * NCONS, NCONS, q);
        tot += step_chunk(u, q, g_hi, g_lo);
        d[0] = make_float4(u[0], u[1], u[2], u[3]);
        d[NCONS] = make_float4(u[4], u[5], u[6], u[7]);
    }
    tot += (step_chunk(R.p[0], R.q[0], g_hi, g_lo) + step_chunk(R.p[1], R.q[1], g_hi, g_lo)) +
           (step_chunk(R.p[2], R.q[2], g_hi, g_lo) + step_chunk(R.p[3], R.q[3], g_hi, g_lo));
    double d = (double)tot;
    const int lane = tid & 31;
    if (lane < nl) {
        const double v = fmax(fma(g, L.ep[lane], -L.eq[lane]), 0.0);
        L.ep[lane] = v;
        d += v;
    }
    return d;
}

// SpecTr's residual (Algorithm 3) in place, in the units of the resident e_p: u <- (u - gm min(u ir, e_q r))+
// with ir = 1 / rho, r = Z_p / Z_q, gm = gamma, for the thread's fp32 tail tokens and for the entry of the
// warp's exact list that falls to its lane.  Returns the thread's sum of the new u.
template <int NW>
__device__ __forceinline__ double spectr_sweep(float4 *es, int nsm, int tid, Resident &R, WarpList &L, int nl, double gm,
                                               double ir, double r)
{
    constexpr int NCONS = NW * 32;
    const float gf = (float)gm, irf = (float)ir, rf = (float)r;
    float tot = 0.f;
    for (int i = 0; i < nsm; ++i) {
        float u[8], q[8];
        float4 *d = es + (size_t)(i * 4) * NCONS + tid;
        load_e8(d, NCONS, u);
        load_e8(d + 2 * NCONS, NCONS, q);
#pragma unroll
        for (int k = 0; k < 8; ++k) { u[k] = fmaxf(u[k] - gf * fminf(u[k] * irf, q[k] * rf), 0.f); tot += u[k]; }
        d[0] = make_float4(u[0], u[1], u[2], u[3]);
        d[NCONS] = make_float4(u[4], u[5], u[6], u[7]);
    }
#pragma unroll
    for (int j = 0; j < RT; ++j) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            R.p[j][k] = fmaxf(R.p[j][k] - gf * fminf(R.p[j][k] * irf, R.q[j][k] * rf), 0.f);
            tot += R.p[j][k];
        }
    }
    double d = (double)tot;
    const int lane = tid & 31;
    if (lane < nl) {
        const double v = fmax(L.ep[lane] - gm * fmin(L.ep[lane] * ir, L.eq[lane] * r), 0.0);
        L.ep[lane] = v;
        d += v;
    }
    return d;
}

// A read-only sweep over the thread's share of the resident node for the offline analysis: f.tail(e_p, e_q,
// a0, a1) on every fp32 token (two running sums), f.exact(...) in fp64 on the entry of the warp's exact
// list that falls to the lane.  Listed tokens are zero in the fp32 arrays; every f maps (0, 0) to nothing.
template <int NW, typename F>
__device__ __forceinline__ void reduce_sweep(const float4 *es, int nsm, int tid, const Resident &R, const WarpList &L,
                                             int nl, const F &f, double &o0, double &o1)
{
    constexpr int NCONS = NW * 32;
    float a0 = 0.f, a1 = 0.f;
    for (int i = 0; i < nsm; ++i) {
        float p[8], q[8];
        const float4 *d = es + (size_t)(i * 4) * NCONS + tid;
        load_e8(d, NCONS, p);
        load_e8(d + 2 * NCONS, NCONS, q);
#pragma unroll
        for (int k = 0; k < 8; ++k) f.tail(p[k], q[k], a0, a1);
    }
#pragma unroll
    for (int j = 0; j < RT; ++j) {
#pragma unroll
        for (int k = 0; k < 8; ++k) f.tail(R.p[j][k], R.q[j][k], a0, a1);
    }
    o0 = (double)a0;
    o1 = (double)a1;
    if ((tid & 31) < nl) f.exact(L.ep[tid & 31], L.eq[tid & 31], o0, o1);
}

// All-to-all of NV doubles per consumer warp of the cluster: tot[i] is the sum over every warp of every
// CTA (bit-identical in all of them: one fixed order), mine[i] in lane r < C the sum over CTA r's warps.
// xchg: [parity 2][rank C][warp NW][2] doubles in every CTA's shared memory, xbar: two mbarriers.
template <int NW, int NV>
__device__ __forceinline__ void cluster_exchange(double *xchg, uint64_t *xbar, int &xn, int C, unsigned rank, int warp,
                                                 int lane, int *poison, const double (&v)[NV], double (&tot)[NV],
                                                 double (&mine)[NV])
{
    static_assert(NV <= 2, "two doubles per warp and exchange at most");
    const int par = xn & 1;
    if (warp == 0 && lane == 0) mbar_arrive_expect_tx(&xbar[par], (uint32_t)(C * NW * 8 * NV));
    if (lane < C) {
#pragma unroll
        for (int i = 0; i < NV; ++i)
            st_async_f64(xchg + ((size_t)(par * C + rank) * NW + warp) * 2 + i, &xbar[par], (uint32_t)lane, v[i]);
    }
    if (!*(volatile int *)poison && !mbar_wait_cluster(&xbar[par], (uint32_t)((xn >> 1) & 1))) *poison = 1;
    ++xn;
#pragma unroll
    for (int i = 0; i < NV; ++i) mine[i] = 0.0;
    if (lane < C) {
        const double *src = xchg + (size_t)(par * C + lane) * NW * 2;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
#pragma unroll
            for (int i = 0; i < NV; ++i) mine[i] += src[w * 2 + i];
        }
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) tot[i] = warp_sum_once(mine[i]);
}

// barrier of the consumer warps of a CTA on an mbarrier (one arrival per warp), with a bounded wait
__device__ __forceinline__ void consumer_sync(uint64_t *bar, uint32_t &ph, int *poison)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
    if (!*(volatile int *)poison && !mbar_wait(bar, ph)) *poison = 1;
    ph ^= 1u;
}

// Inverse-CDF search over one CTA's share of the node's current state u (from_q: of the draft row e_q
// instead, for a state that equals q), run by all consumer warps of the CTA that owns the target
// (tau_rel, in units of e).  Token order is (tile, warp, lane, position
// in the chunk): the tile, then the warp inside the tile, then the lane, then the token.  The per-tile
// totals of a warp are reduced together, so that the shuffles of the ten tiles overlap; warp 0 alone
// picks tile and warp.  Listed tokens enter with their exact values.
// role: 1 = this thread found the token (index inside the slice in `token`, distance to the nearer
// CDF edge in `edge`, both in units of e); 2 = this thread reports that no token carries weight;
// 3 = this thread reports that a bounded wait ran out; 0 = nothing to do.  wtile is [NW + 1][TMAX] in shared memory; cbar / cph: the consumers' barrier.
struct BonusFind {
    int role, token;
    double edge;
};
template <int NW>
__device__ __forceinline__ BonusFind bonus_search(double (*wtile)[TMAX], uint64_t *cbar, uint32_t &cph, int *poison,
                                                  const float4 *es, int nsm, int tid, const Resident &R,
                                                  const WarpList &L, int nl, bool from_q, double tau_rel)
{
    constexpr int NCONS = NW * 32;
    constexpr int TILE = NCONS * 8;
    const int warp = tid >> 5, lane = tid & 31;
    const int qoff = from_q ? 2 * NCONS : 0;
    BonusFind out = {0, -1, 0.0};
    // slot s < SMT: shared-memory tile s (empty beyond nsm); slot SMT + j: register tile j
    float r[TMAX];
#pragma unroll
    for (int i = 0; i < SMT; ++i) {
        r[i] = 0.f;
        if (i < nsm) {
            float p[8];
            load_e8(es + (size_t)(i * 4) * NCONS + tid + qoff, NCONS, p);
            r[i] = sum_chunk(p);
        }
    }
#pragma unroll
    for (int j = 0; j < RT; ++j) r[SMT + j] = from_q ? sum_chunk(R.q[j]) : sum_chunk(R.p[j]);
    // a warp's total of one tile: 256 tokens, summed in fp32 like the chunks themselves; every level
    // above works in fp64 on these stored values, so the levels agree with each other exactly
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int i = 0; i < TMAX; ++i) r[i] += __shfl_xor_sync(0xffffffffu, r[i], o);
    }
    // the warp's listed tokens, exactly: entry `lane`
    const double lr = lane < nl ? (from_q ? L.eq[lane] : L.ep[lane]) : 0.0;
    const int lpos = lane < nl ? L.pos[lane] : -1;
    double mine = 0.0;
#pragma unroll
    for (int i = 0; i < TMAX; ++i)
        if (lane == i) mine = (double)r[i];
    if (nl > 0) {
#pragma unroll 1
        for (int i = 0; i < TMAX; ++i) {
            const double add = warp_sum_once((lpos >= 0 && (lpos >> 8) == i) ? lr : 0.0);
            if (lane == i) mine += add;
        }
    }
    if (lane < TMAX) wtile[warp][lane] = mine;
    consumer_sync(cbar, cph, poison);
    // warp 0 picks the tile and the warp inside it; the others wait for its answer in row NW
    if (warp == 0) {
        double Ti = 0.0;
        if (lane < TMAX)
            for (int w = 0; w < NW; ++w) Ti += wtile[w][lane];
        double tau2, tau3;
        const int s_pick = pick_lane(Ti, tau_rel, tau2);
        const double Ww = (s_pick >= 0 && lane < NW) ? wtile[lane][s_pick] : 0.0;
        const int w_pick = s_pick >= 0 ? pick_lane(Ww, tau2, tau3) : -1;
        if (lane == 0) { wtile[NW][0] = (double)s_pick; wtile[NW][1] = (double)w_pick; wtile[NW][2] = tau3; }
    }
    consumer_sync(cbar, cph, poison);
    if (*(volatile int *)poison) {
        if (tid == 0) out.role = 3;
        return out;
    }
    const int s_star = (int)wtile[NW][0], w_star = (int)wtile[NW][1];
    const double tau3 = wtile[NW][2];
    double tau4;
    if (w_star < 0) {
        if (tid == 0) out.role = 2;
        return out;
    }
    if (warp != w_star) return out;
    float p[8];
    if (s_star < SMT) {
        load_e8(es + (size_t)(s_star * 4) * NCONS + tid + qoff, NCONS, p);
    } else {
        const int jr = s_star - SMT;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float pv = jr == 0 ? R.p[0][k] : (jr == 1 ? R.p[1][k] : (jr == 2 ? R.p[2][k] : R.p[3][k]));
            const float qv = jr == 0 ? R.q[0][k] : (jr == 1 ? R.q[1][k] : (jr == 2 ? R.q[2][k] : R.q[3][k]));
            p[k] = from_q ? qv : pv;
        }
    }
    double wk[8], v = 0.0;
#pragma unroll
    for (int k = 0; k < 8; ++k) wk[k] = (double)p[k];
    // the listed tokens of this tile: each goes to the lane and position it was taken from
#pragma unroll 1
    for (int i = 0; i < nl; ++i) {
        const int ps = __shfl_sync(0xffffffffu, lpos, i);
        const double rv = __shfl_sync(0xffffffffu, lr, i);
        if ((ps >> 8) == s_star && ((ps >> 3) & 31) == lane) {
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if ((ps & 7) == k) wk[k] = rv;
        }
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) v += wk[k];
    const int l_star = pick_lane(v, tau3, tau4);
    if (l_star < 0) {
        if (lane == 0) out.role = 2;
        return out;
    }
    if (lane == l_star) {
        double run = 0.0, dlo = 0.0, dhi = 0.0;
        int found = -1, last_pos = -1;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const double before = run;
            run += wk[k];
            if (wk[k] > 0.0) last_pos = k;
            if (found < 0 && run > tau4) { found = k; dlo = tau4 - before; dhi = run - tau4; }
        }
        if (found < 0) { found = last_pos; dlo = 0.0; dhi = 0.0; }
        const int tile = s_star < SMT ? s_star : nsm + (s_star - SMT);
        out.role = found >= 0 ? 1 : 2;
        out.token = found >= 0 ? tile * TILE + tid * 8 + found : -1;
        out.edge = fmin(dlo, dhi);
    }
    return out;
}

// ------------------------------------------------------------------------------------------------
// selecting the accepted node of one sequence: run by the whole warp whose lane made the last arrival
// ------------------------------------------------------------------------------------------------
// Writes every output of the sequence except the bonus token (accepted node, length, path tokens, status,
// the per-node diagnostics) and publishes the accepted node in P.fin for the sequence's FINISH item.
__device__ __noinline__ void finalize_sequence(const VParams &P, int b)
{
    const int lane = threadIdx.x & 31;
    const int N = P.N;
    const int *parent = P.parent + (long long)b * P.topo_stride;
    const int *token = P.token + (long long)b * N;
    const NodeRec *rec = P.rec + (long long)b * N;
    const float *ua = P.u_accept + (long long)b * N;
    int acc = -1, len = 0;
    const bool fast = N <= FAST_N;
    // a lane's own node, everything the selection needs of it fetched in one round of loads
    const bool own = fast && lane < N;
    const int par = own ? __ldg(parent + lane) : -2;
    const int tok = own ? __ldg(token + lane) : -1;
    const int nx = own ? __ldcg(&rec[lane].next_child) : -1;
    const double thr_l = own ? __ldcg(&rec[lane].thr) : 0.0;
    const float ua_l = own ? __ldg(ua + lane) : 0.f;
    int status = 0;
    for (int i = lane; i < N; i += 32) status = max(status, __ldcg(&rec[i].status));
    status = __reduce_max_sync(0xffffffffu, status);
    // (fast path) the ancestors of the lane's node, itself included, as a bit mask: pointer doubling, five
    // rounds for up to 32 levels; on a tree whose parents come first (checked by the nodes: status)
    unsigned anc = own ? 1u << lane : 0u;
    if (fast) {
        int jump = own ? par : -1;
#pragma unroll
        for (int it = 0; it < 5; ++it) {
            const int src = jump < 0 ? lane : jump;
            const unsigned up = __shfl_sync(0xffffffffu, anc, src);
            const int jj = __shfl_sync(0xffffffffu, jump, src);
            if (jump >= 0) { anc |= up; jump = jj; }
        }
    }
    if (!status) {
        if (fast) {
            if (P.mode == MODE_SPECINFER) {
                acc = 0;
                for (int hop = 0; hop < N; ++hop) {
                    const int n = __shfl_sync(0xffffffffu, nx, acc);
                    if (n < 0 || n >= N) break;
                    acc = n;
                }
            } else {
                // Depth-first post-order; the first node with u < w_fin (the root always) is accepted.  With H the
                // set of nodes whose subtree holds such a node: from the root, step to the first child in H
                // while there is one (the subtrees of the children before it are rejected as a whole).
                const bool hit = own && (lane == 0 || (double)ua_l < thr_l);
                const unsigned H = __reduce_or_sync(0xffffffffu, hit ? anc : 0u);
                int cur = 0;
                for (int d = 0; d < N; ++d) {
                    const unsigned m = __ballot_sync(0xffffffffu, own && par == cur && ((H >> lane) & 1u));
                    if (!m) break;
                    cur = __ffs(m) - 1;
                }
                acc = cur;
            }
            // the path's length is the accepted node's depth
            len = __popc(__shfl_sync(0xffffffffu, anc, acc)) - 1;
        } else {
            if (lane == 0) {
                if (P.mode == MODE_SPECINFER) {
                    acc = 0;
                    for (int hop = 0; hop < N; ++hop) {
                        int nx = __ldcg(&rec[acc].next_child);
                        if (nx < 0) break;
                        acc = nx;
                    }
                } else {
                    int cur = 0;
                    for (int guard = 0; guard < 4 * N + 4 && acc < 0; ++guard) {
                        for (;;) {
                            int fc = -1;
                            for (int c = cur + 1; c < N; ++c)
                                if (parent[c] == cur) { fc = c; break; }
                            if (fc < 0) break;
                            cur = fc;
                        }
                        for (;;) {
                            if (cur == 0 || (double)ua[cur] < __ldcg(&rec[cur].thr)) { acc = cur; break; }
                            const int p = parent[cur];
                            int sib = -1;
                            for (int d = cur + 1; d < N; ++d)
                                if (parent[d] == p) { sib = d; break; }
                            if (sib >= 0) { cur = sib; break; }
                            cur = p;
                        }
                    }
                }
                if (acc >= 0)
                    for (int x = acc; x != 0; x = parent[x]) ++len;
            }
            acc = __shfl_sync(0xffffffffu, acc, 0);
            len = __shfl_sync(0xffffffffu, len, 0);
        }
        if (acc < 0) status = SPEC_DEV_TOPOLOGY;
    }
    if (status) { acc = -1; len = -1; }
    int *ot = P.out.out_tokens + (long long)b * N;
    if (fast) {
        // a node on the accepted path (an ancestor of the accepted node, or that node; not the root) puts its
        // token at its depth - 1
        const unsigned path = acc >= 0 ? __shfl_sync(0xffffffffu, anc, acc) : 0u;
        const int mine = (own && lane > 0 && ((path >> lane) & 1u)) ? __popc(anc) - 1 : 0;
        for (int j = lane; j < N; j += 32) ot[j] = -1;
        __syncwarp();
        if (mine > 0) ot[mine - 1] = tok;
    } else {
        for (int i = lane; i < N; i += 32) ot[i] = -1;
        __syncwarp();
        if (lane == 0 && acc >= 0) {
            int i = len;
            for (int x = acc; x != 0 && i > 0; x = parent[x]) ot[--i] = token[x];
        }
    }
    if (lane == 0) {
        P.out.accepted_node[b] = acc;
        P.out.accept_len[b] = len;
        P.out.bonus_token[b] = -1;         // the FINISH item draws it
        P.out.status[b] = status;
        if (P.out.margin) P.out.margin[(long long)b * (N + 1) + N] = CUDART_NAN_F;   // (the FINISH item's slot)
    }
    // publication: the outputs above are visible to whoever sees the accepted node (the diagnostics below
    // are read by nobody on the device)
    __syncwarp();
    if (lane == 0) {
        __threadfence();
        *(volatile int *)(P.fin + b) = status ? FIN_FAULTY : (acc | (len << FIN_LEN_SHIFT));
    }
    if (P.out.node_thr)
        for (int i = lane; i < N; i += 32) P.out.node_thr[(long long)b * N + i] = (float)__ldcg(&rec[i].thr);
    if (P.out.node_w_in && P.mode == MODE_TRAVERSAL)
        for (int i = lane; i < N; i += 32) P.out.node_w_in[(long long)b * N + i] = (float)__ldcg(&rec[i].w_in);
    if (P.out.margin) {
        float *mg = P.out.margin + (long long)b * (N + 1);
        for (int i = lane; i < N; i += 32)
            mg[i] = i == 0 ? CUDART_NAN_F : (float)fabs((double)ua[i] - __ldcg(&rec[i].thr));
    }
}

// The arrival of `count` nodes at their sequence (a node and the childless children it finished), made
// by lane 0 of a converged warp; the warp that makes the last of the N arrivals selects the accepted node.
__device__ __forceinline__ void arrive_sequence(const VParams &P, int b, unsigned count = 1u)
{
    int last = 0;
    if ((threadIdx.x & 31) == 0) {
        // release: the node's record (written by this warp, ordered before by __syncwarp where another
        // lane wrote it) is visible to whoever sees the count; acquire: the last arrival sees all records
        unsigned prev;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(prev) : "l"(P.done + b), "r"(count) : "memory");
        last = (prev + count == (unsigned)P.N) ? 1 : 0;
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) finalize_sequence(P, b);
}

}  // namespace specv
