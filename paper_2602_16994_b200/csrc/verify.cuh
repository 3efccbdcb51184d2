// The fused verification kernel: SpecInfer (Algorithm 4 composed top-down, Section 3.2) and
// Traversal Verification (Section 3.2; block-verification weights of Section 3.1), one tree node
// per thread-block cluster, clusters persistent over the (node, sequence) list.
//
// Data flow of one node.  Its target row (and its draft row when it has children) streams from HBM
// through a ring of shared-memory stages filled by bulk asynchronous copies that a producer warp
// issues (it runs ahead into the next node while the consumers finish the current one).  Each CTA
// of the cluster owns a contiguous vocabulary slice; each consumer thread owns 8 consecutive tokens
// of every tile of that slice.  A logit becomes e = 2^(z s - o) with s = log2(e)/T and o the thread's
// reference for the row, an integer, so every scale factor between threads, warps and CTAs is an
// exact power of two.  The e of the last RT tiles of a slice stay in registers, the others in shared
// memory; nothing is written back to HBM.
//
// After j rejected children the unnormalised target law of the node is
//     U_j(t) = (w_in P0(t) - c_j q(t))+ ,   c_0 = 0,  c_{j+1} = c_j + G_j,
//     E_j = sum_t U_j(t),  G_{j+1} = E_{j+1} + G_j - E_j   (G_0 = 1, E_0 = w_in).
// SpecInfer has w_in = 1, G_j = E_j: U_j / E_j is the residual after j updates P <- norm((P - q)+)
// and child j is accepted with min(1, U_j(x) / (E_j q(x))).  In Traversal Verification E_j / G_j is
// the node's weight after j rejected subtrees (w <- S / (S + 1 - w), P <- (wP - q)+ / S without the
// renormalisation) and child j is handed min(1, U_j(x) / (G_j q(x))).  One sibling step is one pass
// over the resident e computing sum (e_p - g e_q)+ plus one scalar exchange through distributed
// shared memory.  The bonus token is an inverse-CDF search over the resident slice.
//
// Exchanges.  Every consumer warp of every CTA of the cluster sends its partial sums straight into
// the shared memory of all CTAs (st.async, which counts the bytes on the receiver's mbarrier); every
// warp waits on its own CTA's mbarrier and reduces all partials itself, in one fixed order, so all
// warps of the cluster hold bit-identical totals and take identical decisions without any CTA-wide
// barrier.  The scalar recursion is therefore replicated per warp; only warp 0 of CTA rank 0 (the
// "scribe") writes the node's record, publishes the children's weights (Traversal) and counts the
// node as done.
#pragma once
#include "common.cuh"

namespace specv {

constexpr int RT = 4;        // tiles per thread whose e live in registers (the kernel names them one by one)
constexpr int SMT = 6;       // further tiles per thread whose e live in shared memory
constexpr int TMAX = RT + SMT;
constexpr int CMAX = 16;     // CTAs per cluster (above 8: non-portable size)
constexpr int NSMAX = 16;    // ring stages
constexpr int NWMAX = 15;    // consumer warps
constexpr int OMIN = -(1 << 30);
constexpr int FAST_N = 32;   // trees up to this size are finished warp-parallel

enum Mode { MODE_SPECINFER = 0, MODE_TRAVERSAL = 1 };

struct VParams {
    int B, N, V, C, mode, all_thr;
    int slice_len;            // tokens per CTA slice: a multiple of 8, at most TMAX tiles
    int NS;                   // ring stages
    int off_x, off_es, off_ring;   // byte offsets inside dynamic shared memory
    const void *zp, *zq;
    long long seq_stride, node_stride, topo_stride;
    const int *parent, *token;
    float T;
    const float *T_seq;
    const float *cut;         // optional [B*N*2]: smallest kept logit of the target / draft row
    const float *u_accept, *u_bonus;
    NodeRec *rec;
    unsigned long long *w_pub;   // [B*N] weight handed to a node by its parent (Traversal), W_PENDING until known
    unsigned int *done;          // [B] arrivals per sequence (two per node); the last one writes the outputs
    float *features;
    SpecOut out;
};

// per consumer warp: the children of the current node and the scalar state of its recursion
struct __align__(16) WarpArea {
    double cpm[KMAX], cqm[KMAX];   // 2^frac of the child token's exponent z s (0: token cut away)
    int cpn[KMAX], cqn[KMAX];      // its integer part
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
    uint64_t full[NSMAX], empty[NSMAX], xbar[2];
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
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        float x = fmaf(z[k], s_lo, fmaf(z[k], s_hi, -of));
        if (FEAT) x = fmaxf(x, -200.f);
        e[k] = ex2_approx(x);
        sum += e[k];
        if (FEAT) sx = fmaf(e[k], x, sx);
    }
    return sum;
}
__device__ __forceinline__ float max8(const float (&z)[8])
{
    return fmaxf(fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])), fmaxf(fmaxf(z[4], z[5]), fmaxf(z[6], z[7])));
}
__device__ __forceinline__ void scale_f4(float4 *d, float f)
{
    float4 v = *d;
    v.x *= f; v.y *= f; v.z *= f; v.w *= f;
    *d = v;
}
__device__ __forceinline__ void load_e8(const float4 *d, int stride, float (&e)[8])
{
    const float4 lo = d[0], hi = d[stride];
    e[0] = lo.x; e[1] = lo.y; e[2] = lo.z; e[3] = lo.w; e[4] = hi.x; e[5] = hi.y; e[6] = hi.z; e[7] = hi.w;
}

// first lane whose running sum of v exceeds tau (v >= 0 in every lane); if rounding leaves none, the
// last lane with v > 0 and tau_res = +inf; -1 if no lane has weight.  All lanes get the same answer.
__device__ __forceinline__ int pick_lane(double v, double tau, double &tau_res)
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

// sum over one chunk of (e_p - g e_q)+
__device__ __forceinline__ float residual_chunk(const float (&p)[8], const float (&q)[8], float gh, float gl)
{
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) acc += fmaxf(fmaf(-gl, q[k], fmaf(-gh, q[k], p[k])), 0.f);
    return acc;
}

// Inverse-CDF search over one CTA's resident residual (e_p - g e_q)+, run by all consumer warps of
// the CTA that owns the target (tau_rel, in units of e).  Token order is (tile, warp, lane, position
// in the chunk): the tile, then the warp inside the tile, then the lane, then the token.  The per-tile
// totals of a warp are reduced together, so that the shuffles of the ten tiles overlap.
// role: 1 = this thread found the token (index inside the slice in `token`, distance to the nearer
// CDF edge in `edge`, both in units of e); 2 = this thread reports that no token carries weight;
// 0 = nothing to do.  wtile is [NW + 1][TMAX] in shared memory; named barrier 1 is used twice.
struct BonusFind {
    int role, token;
    double edge;
};
template <int NW>
__device__ __forceinline__ BonusFind bonus_search(double (*wtile)[TMAX], const float4 *es, int nsm, int tid,
                                                  const float (&ep0)[8], const float (&ep1)[8], const float (&ep2)[8],
                                                  const float (&ep3)[8], const float (&eq0)[8], const float (&eq1)[8],
                                                  const float (&eq2)[8], const float (&eq3)[8], float gh, float gl,
                                                  double tau_rel)
{
    constexpr int NCONS = NW * 32;
    constexpr int TILE = NCONS * 8;
    const int warp = tid >> 5, lane = tid & 31;
    BonusFind out = {0, -1, 0.0};
    // slot s < SMT: shared-memory tile s (empty beyond nsm); slot SMT + j: register tile j
    double r[TMAX];
#pragma unroll
    for (int i = 0; i < SMT; ++i) {
        r[i] = 0.0;
        if (i < nsm) {
            float p[8], q[8];
            const float4 *d = es + (size_t)(i * 4) * NCONS + tid;
            load_e8(d, NCONS, p);
            load_e8(d + 2 * NCONS, NCONS, q);
            r[i] = (double)residual_chunk(p, q, gh, gl);
        }
    }
    r[SMT + 0] = (double)residual_chunk(ep0, eq0, gh, gl);
    r[SMT + 1] = (double)residual_chunk(ep1, eq1, gh, gl);
    r[SMT + 2] = (double)residual_chunk(ep2, eq2, gh, gl);
    r[SMT + 3] = (double)residual_chunk(ep3, eq3, gh, gl);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int i = 0; i < TMAX; ++i) r[i] += __shfl_xor_sync(0xffffffffu, r[i], o);
    }
#pragma unroll
    for (int i = 0; i < TMAX; ++i)
        if (lane == i) wtile[warp][i] = r[i];
    bar_sync(1, NCONS);
    double Ti = 0.0;
    if (lane < TMAX)
        for (int w = 0; w < NW; ++w) Ti += wtile[w][lane];
    double tau2, tau3, tau4;
    const int s_star = pick_lane(Ti, tau_rel, tau2);
    const double Ww = (s_star >= 0 && lane < NW) ? wtile[lane][s_star] : 0.0;
    const int w_star = s_star >= 0 ? pick_lane(Ww, tau2, tau3) : -1;
    bar_sync(1, NCONS);          // wtile may be rewritten only after everyone has read it
    if (w_star < 0) {
        if (tid == 0) out.role = 2;
        return out;
    }
    if (warp != w_star) return out;
    float p[8], q[8];
    if (s_star < SMT) {
        const float4 *d = es + (size_t)(s_star * 4) * NCONS + tid;
        load_e8(d, NCONS, p);
        load_e8(d + 2 * NCONS, NCONS, q);
    } else {
        const int jr = s_star - SMT;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            p[k] = jr == 0 ? ep0[k] : (jr == 1 ? ep1[k] : (jr == 2 ? ep2[k] : ep3[k]));
            q[k] = jr == 0 ? eq0[k] : (jr == 1 ? eq1[k] : (jr == 2 ? eq2[k] : eq3[k]));
        }
    }
    float wk[8], v = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) { wk[k] = fmaxf(fmaf(-gl, q[k], fmaf(-gh, q[k], p[k])), 0.f); v += wk[k]; }
    const int l_star = pick_lane((double)v, tau3, tau4);
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
            run += (double)wk[k];
            if (wk[k] > 0.f) last_pos = k;
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

// Pass 1 for one row of one tile.  The tile's e go to the register array DST (ISREG, a literal) or to
// shared-memory slot SLOT.  O / SET / SUM / SX / BX: the thread's running reference for this row (an
// integer-valued float), whether it is set, sum of e, sum of e x and largest exponent.  A chunk whose
// largest exponent would exceed 60 moves the reference up and rescales what the thread has stored so
// far by an exact power of two (rare: it takes logits 60 T / log2(e) above the first chunk's maximum):
// the NSM_DONE shared-memory tiles of this row, and the register tiles named in RESCALE_REGS (a
// statement list using the factor f_).  Register tiles are separate named arrays and every index is a
// literal, so that they stay in registers.
#define SPECV_SCALE8(A, F)                                                                                   \
    do { _Pragma("unroll") for (int k_ = 0; k_ < 8; ++k_) A[k_] *= (F); } while (0)
#define SPECV_P1_ROW(Z, DST, SLOT, ISREG, ROWOFF, NSM_DONE, RESCALE_REGS, O, SET, SUM, SX, BX)               \
    do {                                                                                                     \
        const float zm_ = max8(Z);                                                                           \
        if (!(SET) && zm_ > -CUDART_INF_F) {                                                                 \
            (O) = fminf(fmaxf(ceilf(zm_ * s_hi), -1.0e9f), 1.0e9f);                                          \
            (SET) = true;                                                                                    \
        }                                                                                                    \
        const float xm_ = fmaf(zm_, s_lo, fmaf(zm_, s_hi, -(O)));                                            \
        if (xm_ > 60.f && xm_ < CUDART_INF_F) {                                                              \
            const float kf_ = fminf(ceilf(xm_), 1.0e9f);                                                     \
            const float f_ = pow2i(-(int)fminf(kf_, 200.f));                                                 \
            RESCALE_REGS                                                                                     \
            for (int j_ = 0; j_ < (NSM_DONE); ++j_) {                                                        \
                float4 *d_ = es + (size_t)(j_ * 4 + (ROWOFF)) * NCONS + tid;                                 \
                scale_f4(d_, f_); scale_f4(d_ + NCONS, f_);                                                  \
            }                                                                                                \
            if (FEAT) { (SX) = f_ * fmaf(-kf_, (SUM), (SX)); (BX) -= kf_; }                                  \
            (SUM) *= f_;                                                                                     \
            (O) += kf_;                                                                                      \
        }                                                                                                    \
        if (ISREG) {                                                                                         \
            (SUM) += exp_chunk<FEAT>(Z, s_hi, s_lo, (O), DST, (SX));                                         \
        } else {                                                                                             \
            float e8_[8];                                                                                    \
            (SUM) += exp_chunk<FEAT>(Z, s_hi, s_lo, (O), e8_, (SX));                                         \
            float4 *d_ = es + (size_t)((SLOT) * 4 + (ROWOFF)) * NCONS + tid;                                 \
            d_[0] = make_float4(e8_[0], e8_[1], e8_[2], e8_[3]);                                             \
            d_[NCONS] = make_float4(e8_[4], e8_[5], e8_[6], e8_[7]);                                         \
        }                                                                                                    \
        if (FEAT) (BX) = fmaxf((BX), fmaf(zm_, s_lo, fmaf(zm_, s_hi, -(O))));                                \
    } while (0)

// ------------------------------------------------------------------------------------------------
// writing the outputs of one sequence: run by the whole warp whose lane made the last arrival
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ void finalize_sequence(const VParams &P, int b)
{
    const int lane = threadIdx.x & 31;
    const int N = P.N;
    const int *parent = P.parent + (long long)b * P.topo_stride;
    const int *token = P.token + (long long)b * N;
    const NodeRec *rec = P.rec + (long long)b * N;
    const float *ua = P.u_accept + (long long)b * N;
    int status = 0;
    for (int i = lane; i < N; i += 32) status = max(status, __ldcg(&rec[i].status));
    status = __reduce_max_sync(0xffffffffu, status);
    int acc = -1, len = 0;
    if (!status) {
        if (N <= FAST_N) {
            const int par = lane < N ? __ldg(parent + lane) : -2;
            if (P.mode == MODE_SPECINFER) {
                const int nx = lane < N ? __ldcg(&rec[lane].next_child) : -1;
                acc = 0;
                for (int hop = 0; hop < N; ++hop) {
                    const int n = __shfl_sync(0xffffffffu, nx, acc);
                    if (n < 0 || n >= N) break;
                    acc = n;
                }
            } else {
                // depth-first post-order; the first node with u < w_fin (the root always) is accepted
                const bool hit = lane < N && (lane == 0 || (double)__ldg(ua + lane) < __ldcg(&rec[lane].thr));
                int cur = 0;
                for (int guard = 0; guard < 4 * N + 4 && acc < 0; ++guard) {
                    for (;;) {
                        const unsigned m = __ballot_sync(0xffffffffu, par == cur);
                        if (!m) break;
                        cur = __ffs(m) - 1;
                    }
                    for (;;) {
                        const int h = __shfl_sync(0xffffffffu, (int)hit, cur);
                        if (cur == 0 || h) { acc = cur; break; }
                        const int p = __shfl_sync(0xffffffffu, par, cur);
                        const unsigned m = __ballot_sync(0xffffffffu, par == p) & ~((2u << cur) - 1u);
                        if (m) { cur = __ffs(m) - 1; break; }
                        cur = p;
                    }
                }
            }
            if (acc >= 0)
                for (int x = acc; x > 0 && len <= N; x = __shfl_sync(0xffffffffu, par, x)) ++len;
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
    int bonus = acc >= 0 ? __ldcg(&rec[acc].bonus) : -1;
    if (acc >= 0 && bonus < 0 && !status) status = SPEC_DEV_NONFINITE;
    if (status) { acc = -1; len = -1; bonus = -1; }
    int *ot = P.out.out_tokens + (long long)b * N;
    for (int i = lane; i < N; i += 32) ot[i] = -1;
    __syncwarp();
    if (lane == 0) {
        P.out.accepted_node[b] = acc;
        P.out.accept_len[b] = len;
        P.out.bonus_token[b] = bonus;
        P.out.status[b] = status;
        if (acc >= 0) {
            ot[len] = bonus;
            int i = len;
            for (int x = acc; x != 0 && i > 0; x = parent[x]) ot[--i] = token[x];
        }
    }
    if (P.out.node_thr)
        for (int i = lane; i < N; i += 32) P.out.node_thr[(long long)b * N + i] = (float)__ldcg(&rec[i].thr);
    if (P.out.node_w_in && P.mode == MODE_TRAVERSAL)
        for (int i = lane; i < N; i += 32) P.out.node_w_in[(long long)b * N + i] = (float)__ldcg(&rec[i].w_in);
    if (P.out.margin) {
        float *mg = P.out.margin + (long long)b * (N + 1);
        for (int i = lane; i < N; i += 32)
            mg[i] = i == 0 ? CUDART_NAN_F : (float)fabs((double)ua[i] - __ldcg(&rec[i].thr));
        if (lane == 0) mg[N] = acc >= 0 ? __ldcg(&rec[acc].bonus_margin) : CUDART_NAN_F;
    }
}

// `count` arrivals of a node at its sequence, made by lane 0 of a converged warp; the warp that makes
// the last of the 2N arrivals writes the sequence's outputs.
__device__ __forceinline__ void arrive_sequence(const VParams &P, int b, unsigned count)
{
    int last = 0;
    if ((threadIdx.x & 31) == 0) {
        __threadfence();
        const unsigned prev = atomicAdd(P.done + b, count);
        last = (prev + count == 2u * (unsigned)P.N) ? 1 : 0;
        if (last) __threadfence();
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) finalize_sequence(P, b);
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
template <int DT, int NW, bool FEAT>
__global__ void __launch_bounds__((NW + 1) * 32, NW <= 7 ? 2 : 1) spec_verify_kernel(const VParams P)
{
    constexpr int NCONS = NW * 32;
    constexpr int TILE = NCONS * 8;
    constexpr int ESZ = DT == SPEC_BF16 ? 2 : 4;
    constexpr int ROWB = TILE * ESZ;        // bytes of one row's tile
    constexpr int STAGE = 2 * ROWB;
    constexpr int NP = FEAT ? 10 : 6;       // doubles a warp sends in the first exchange
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    Hdr &S = *reinterpret_cast<Hdr *>(dyn_smem);
    double *xchg = reinterpret_cast<double *>(dyn_smem + P.off_x);   // [parity 2][rank C][warp NW][NP]
    float4 *es = reinterpret_cast<float4 *>(dyn_smem + P.off_es);    // [slot][p lo, p hi, q lo, q hi][NCONS]
    unsigned char *ring = dyn_smem + P.off_ring;
    const int C = P.C, NS = P.NS;
    const unsigned rank = cluster_ctarank();
    const int cid = blockIdx.x / C, NC = gridDim.x / C;
    const long long total = (long long)P.B * P.N;
    const long long tok0 = (long long)rank * P.slice_len;
    const int n_slice = (int)max(0ll, min((long long)P.slice_len, (long long)P.V - tok0));
    const int ntiles = (n_slice + TILE - 1) / TILE;
    const int nsm = max(ntiles - RT, 0);      // the first nsm tiles of the slice keep their e in shared memory,
    const int nrg = ntiles - nsm;             // the last nrg (<= RT) in registers
    const bool trav = P.mode == MODE_TRAVERSAL;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&S.full[s], 1); mbar_init(&S.empty[s], NW); }
        mbar_init(&S.xbar[0], 1);
        mbar_init(&S.xbar[1], 1);
        S.poison = 0;
        mbar_fence_init();
    }
    __syncthreads();
    cluster_sync_all();        // every CTA of the cluster runs and has its barriers initialised

    if (warp == NW) {
        // ======================= producer warp: fills the ring, node after node =======================
        int g = 0;
        bool ok = true;
        for (long long id = cid; id < total && ok; id += NC) {
            const int a = (int)(id / P.B), b = (int)(id % P.B);
            const bool hq = warp_has_children(P.parent + (long long)b * P.topo_stride, P.N, a, lane);
            const long long row = (long long)b * P.seq_stride + (long long)a * P.node_stride + tok0;
            const unsigned char *src_p = (const unsigned char *)P.zp + row * ESZ;
            const unsigned char *src_q = (const unsigned char *)P.zq + row * ESZ;
            const bool aligned = ((((uintptr_t)src_p) | ((uintptr_t)src_q)) & 15) == 0;
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
        if (!ok && lane == 0) {
            // gave up: wait (bounded) for the copies still in flight before leaving
            for (int k = 1; k <= NS && k <= g; ++k) {
                const int gg = g - k;
                mbar_wait(&S.full[gg % NS], (uint32_t)((gg / NS) & 1));
            }
        }
    } else {
        // ================================ consumer warps ================================================
        WarpArea &W = S.wa[warp];
        const bool scribe = rank == 0 && warp == 0;     // the one warp that writes the node's record
        int stage = 0;          // ring position (same sequence as the producer's) and its phase
        uint32_t phase = 0;
        int xn = 0;             // exchanges done
        const bool has_cut = P.cut != nullptr;

// take the next tile from the ring: raw chunks of this thread, then hand the stage back
#define SPECV_NEXT_TILE(TILE_INDEX)                                                                          \
        if (!poisoned && !mbar_wait(&S.full[stage], phase)) { S.poison = 1; poisoned = true; }               \
        {                                                                                                    \
            const unsigned char *sp_ = ring + (size_t)stage * STAGE + (size_t)tid * 8 * ESZ;                 \
            raw_p = read_raw<DT>(sp_);                                                                       \
            if (hq) raw_q = read_raw<DT>(sp_ + ROWB);                                                        \
        }                                                                                                    \
        __syncwarp();                                                                                        \
        if (lane == 0) mbar_arrive(&S.empty[stage]);                                                         \
        if (++stage == NS) { stage = 0; phase ^= 1u; }                                                       \
        const int nvalid = poisoned ? 0 : n_slice - ((TILE_INDEX) * TILE + tid * 8);

        for (long long id = cid; id < total; id += NC) {
            const int a = (int)(id / P.B), b = (int)(id % P.B);
            const int *parent = P.parent + (long long)b * P.topo_stride;
            const double s_d = 1.4426950408889634 / (double)(P.T_seq ? __ldg(P.T_seq + b) : P.T);
            // s = s_hi + s_lo with s_lo > 0, so that a logit of -inf gives the exponent -inf and not NaN
            float s_hi = (float)s_d;
            if ((double)s_hi > s_d) s_hi = __uint_as_float(__float_as_uint(s_hi) - 1u);
            float s_lo = (float)(s_d - (double)s_hi);
            if (!(s_lo > 0.f)) s_lo = 1.0e-30f;
            const long long ci = ((long long)b * P.N + a) * 2;
            const float cut_p = has_cut ? __ldg(P.cut + ci) : -CUDART_INF_F;
            const float cut_q = has_cut ? __ldg(P.cut + ci + 1) : -CUDART_INF_F;
            const bool hq = warp_has_children(parent, P.N, a, lane);

            // ---- pass 1: logits -> e, per-thread sums --------------------------------------------------
            float ep0[8], ep1[8], ep2[8], ep3[8], eq0[8], eq1[8], eq2[8], eq3[8];
            float op_f = 0.f, oq_f = 0.f;        // the thread's reference per row (integer-valued)
            bool set_p = false, set_q = false;
            float Sp_t = 0.f, Sq_t = 0.f, SXp_t = 0.f, SXq_t = 0.f;
            float bxp = -CUDART_INF_F, bxq = -CUDART_INF_F;      // FEAT: largest exponent seen, relative to the reference
            bool poisoned = *(volatile int *)&S.poison != 0;
            {
                RawChunk<DT> raw_p, raw_q;
                float z[8];
                float dummy[8];
                for (int i = 0; i < nsm; ++i) {
                    SPECV_NEXT_TILE(i)
                    unpack_chunk<DT>(raw_p, z);
                    mask_chunk(z, nvalid, has_cut, cut_p);
                    SPECV_P1_ROW(z, dummy, i, false, 0, i, , op_f, set_p, Sp_t, SXp_t, bxp);
                    if (hq) {
                        unpack_chunk<DT>(raw_q, z);
                        mask_chunk(z, nvalid, has_cut, cut_q);
                        SPECV_P1_ROW(z, dummy, i, false, 2, i, , oq_f, set_q, Sq_t, SXq_t, bxq);
                    }
                }
// one register tile: J its number, EP / EQ its arrays, RP / RQ the statements rescaling the earlier ones
#define SPECV_REG_TILE(J, EP, EQ, RP, RQ)                                                                    \
                if ((J) < nrg) {                                                                             \
                    SPECV_NEXT_TILE(nsm + (J))                                                               \
                    unpack_chunk<DT>(raw_p, z);                                                              \
                    mask_chunk(z, nvalid, has_cut, cut_p);                                                   \
                    SPECV_P1_ROW(z, EP, 0, true, 0, nsm, RP, op_f, set_p, Sp_t, SXp_t, bxp);                 \
                    if (hq) {                                                                                \
                        unpack_chunk<DT>(raw_q, z);                                                          \
                        mask_chunk(z, nvalid, has_cut, cut_q);                                               \
                        SPECV_P1_ROW(z, EQ, 0, true, 2, nsm, RQ, oq_f, set_q, Sq_t, SXq_t, bxq);             \
                    } else {                                                                                 \
                        _Pragma("unroll") for (int k = 0; k < 8; ++k) EQ[k] = 0.f;                           \
                    }                                                                                        \
                } else {                                                                                     \
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) { EP[k] = 0.f; EQ[k] = 0.f; }              \
                }
                SPECV_REG_TILE(0, ep0, eq0, , )
                SPECV_REG_TILE(1, ep1, eq1, SPECV_SCALE8(ep0, f_);, SPECV_SCALE8(eq0, f_);)
                SPECV_REG_TILE(2, ep2, eq2, SPECV_SCALE8(ep0, f_); SPECV_SCALE8(ep1, f_);, SPECV_SCALE8(eq0, f_); SPECV_SCALE8(eq1, f_);)
                SPECV_REG_TILE(3, ep3, eq3, SPECV_SCALE8(ep0, f_); SPECV_SCALE8(ep1, f_); SPECV_SCALE8(ep2, f_);,
                               SPECV_SCALE8(eq0, f_); SPECV_SCALE8(eq1, f_); SPECV_SCALE8(eq2, f_);)
#undef SPECV_REG_TILE
            }
            const int op_t = set_p ? (int)op_f : OMIN, oq_t = set_q ? (int)oq_f : OMIN;

            // ---- first exchange: every warp sends (reference, sum) of both rows to every CTA ---------------
            const int par1 = xn & 1;
            {
                const int Ow_p = __reduce_max_sync(0xffffffffu, op_t), Ow_q = __reduce_max_sync(0xffffffffu, oq_t);
                const double fp = (double)pow2i(max(op_t - Ow_p, -127)), fq = (double)pow2i(max(oq_t - Ow_q, -127));
                double pay[NP];
                pay[0] = (double)Ow_p; pay[1] = warp_sum((double)Sp_t * fp);
                pay[2] = (double)Ow_q; pay[3] = warp_sum((double)Sq_t * fq);
                pay[4] = 1.0; pay[5] = 0.0;
                if (FEAT) {
                    pay[6] = warp_sum(fp * ((double)SXp_t + (double)max(op_t - Ow_p, -100000) * (double)Sp_t));
                    pay[7] = warp_sum(fq * ((double)SXq_t + (double)max(oq_t - Ow_q, -100000) * (double)Sq_t));
                    double v_bp = set_p ? (double)op_f + (double)bxp : -1.0e300;
                    double v_bq = set_q ? (double)oq_f + (double)bxq : -1.0e300;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        v_bp = fmax(v_bp, __shfl_xor_sync(0xffffffffu, v_bp, o));
                        v_bq = fmax(v_bq, __shfl_xor_sync(0xffffffffu, v_bq, o));
                    }
                    pay[8] = v_bp; pay[9] = v_bq;
                }
                // Traversal: the weight handed down by the parent (polled by the scribe warp, bounded)
                if (scribe && trav && a > 0) {
                    unsigned long long bits = W_PENDING;
                    if (lane == 0) {
                        const int pa = __ldg(parent + a);
                        if (pa >= 0 && pa < a) {
                            volatile unsigned long long *slot = P.w_pub + (long long)b * P.N + a;
                            const long long t0 = clock64();
                            for (;;) {
                                bits = *slot;
                                if (bits != W_PENDING || clock64() - t0 > WAIT_CYCLES || *(volatile int *)&S.poison) break;
                                __nanosleep(64);
                            }
                            __threadfence();
                        } else {
                            bits = 0ull;        // a node with a bad parent index is reported below; nobody publishes for it
                        }
                    }
                    bits = __shfl_sync(0xffffffffu, bits, 0);
                    if (bits == W_PENDING) { pay[4] = 0.0; pay[5] = 1.0; }
                    else pay[4] = __longlong_as_double((long long)bits);
                }
                if (poisoned || *(volatile int *)&S.poison) pay[5] = 1.0;
                double *mine = xchg + ((size_t)(par1 * C + rank) * NW + warp) * NP;
                if (warp == 0 && lane == 0) mbar_arrive_expect_tx(&S.xbar[par1], (uint32_t)(C * NW * NP * 8));
                if (lane < C) {
#pragma unroll
                    for (int v = 0; v < NP; ++v) st_async_f64(mine + v, &S.xbar[par1], (uint32_t)lane, pay[v]);
                }
            }

            // ---- while the exchange is in flight: children of a, validation, their tokens' exponents --------
            int kc = 0, err = 0;
            {
                const int *token = P.token + (long long)b * P.N;
                if (lane == 0) {
                    const int pa = __ldg(parent + a);
                    if (a == 0 ? (pa != -1) : (pa < 0 || pa >= a)) err = SPEC_DEV_TOPOLOGY;
                    if (a > 0) {
                        const int x = __ldg(token + a);
                        if (x < 0 || x >= P.V) err = SPEC_DEV_TOKEN;
                    }
                }
                for (int c0 = a + 1; c0 < P.N; c0 += 32) {
                    const int c = c0 + lane;
                    const bool is = c < P.N && __ldg(parent + c) == a;
                    const unsigned bal = __ballot_sync(0xffffffffu, is);
                    if (is) {
                        const int pos = kc + __popc(bal & ((1u << lane) - 1u));
                        if (pos < KMAX) {
                            const int x = __ldg(token + c);
                            W.child[pos] = c;
                            W.cpn[pos] = x;
                            W.cu[pos] = __ldg(P.u_accept + (long long)b * P.N + c);
                            if (x < 0 || x >= P.V) err = SPEC_DEV_TOKEN;
                        }
                    }
                    kc += __popc(bal);
                }
                if (kc > KMAX) err = SPEC_DEV_TOPOLOGY;
                err = __reduce_max_sync(0xffffffffu, err);
                __syncwarp();
                const int j = lane & 15;
                const bool mine = !err && j < kc;
                const int xt = mine ? W.cpn[j] : 0;
                __syncwarp();
                if (mine) {
                    const long long rowb = (long long)b * P.seq_stride + (long long)a * P.node_stride;
                    const float z = load_logit(lane < 16 ? P.zp : P.zq, DT, rowb + xt);
                    const double xd = (double)z * s_d;
                    double m = 0.0;
                    int n = 0;
                    if (fabs(xd) < 1.0e9) {
                        const double nd = rint(xd);
                        n = (int)nd;
                        m = (z >= (lane < 16 ? cut_p : cut_q)) ? exp2_frac(xd - nd) : 0.0;
                    } else if (!(xd < 0.0)) {
                        m = CUDART_NAN;          // +inf or NaN: the row is reported as not finite anyway
                    }
                    if (lane < 16) { W.cpm[j] = m; W.cpn[j] = n; }
                    else { W.cqm[j] = m; W.cqn[j] = n; }
                }
            }

            // ---- the exchanged values: lane r merges the NW warps of rank r, then the ranks are merged ----
            double E_r;          // lane r: rank r's total of the current U
            {
                if (!*(volatile int *)&S.poison && !mbar_wait_cluster(&S.xbar[par1], (uint32_t)((xn >> 1) & 1))) S.poison = 1;
                ++xn;
                int Op_r = OMIN, Oq_r = OMIN;
                double Sp_r = 0.0, Sq_r = 0.0, Xp_r = 0.0, Xq_r = 0.0, bp_r = -1.0e300, bq_r = -1.0e300, fl_r = 0.0;
                if (lane < C) {
                    const double *src = xchg + (size_t)(par1 * C + lane) * NW * NP;
#pragma unroll
                    for (int w = 0; w < NW; ++w) {
                        Op_r = max(Op_r, (int)src[w * NP]);
                        Oq_r = max(Oq_r, (int)src[w * NP + 2]);
                    }
#pragma unroll
                    for (int w = 0; w < NW; ++w) {
                        const int dp = (int)src[w * NP] - Op_r, dq = (int)src[w * NP + 2] - Oq_r;
                        const double f0 = pow2d(dp), f1 = pow2d(dq);
                        Sp_r = fma(src[w * NP + 1], f0, Sp_r);
                        Sq_r = fma(src[w * NP + 3], f1, Sq_r);
                        fl_r += src[w * NP + 5];
                        if (FEAT) {
                            Xp_r += f0 * (src[w * NP + 6] + (double)max(dp, -100000) * src[w * NP + 1]);
                            Xq_r += f1 * (src[w * NP + 7] + (double)max(dq, -100000) * src[w * NP + 3]);
                            bp_r = fmax(bp_r, src[w * NP + 8]);
                            bq_r = fmax(bq_r, src[w * NP + 9]);
                        }
                    }
                }
                const int O_p = __reduce_max_sync(0xffffffffu, Op_r), O_q = __reduce_max_sync(0xffffffffu, Oq_r);
                const double zp_r = Sp_r * pow2d(Op_r - O_p), zq_r = Sq_r * pow2d(Oq_r - O_q);
                const double Z_p = warp_sum(zp_r), Z_q = warp_sum(zq_r);
                const double w_in = xchg[(size_t)(par1 * C) * NW * NP + 4];
                if (warp_sum(fl_r) != 0.0 || *(volatile int *)&S.poison) err = SPEC_DEV_TIMEOUT;
                const bool bad_p = !(Z_p > 0.0) || !(Z_p < CUDART_INF);
                const bool bad_q = hq && (!(Z_q > 0.0) || !(Z_q < CUDART_INF));
                if ((bad_p || bad_q) && !err) err = SPEC_DEV_NONFINITE;
                if (FEAT && P.features) {
                    const double X_p = warp_sum(pow2d(Op_r - O_p) * (Xp_r + (double)max(Op_r - O_p, -100000) * Sp_r));
                    const double X_q = warp_sum(pow2d(Oq_r - O_q) * (Xq_r + (double)max(Oq_r - O_q, -100000) * Sq_r));
                    double b_p = bp_r, b_q = bq_r;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        b_p = fmax(b_p, __shfl_xor_sync(0xffffffffu, b_p, o));
                        b_q = fmax(b_q, __shfl_xor_sync(0xffffffffu, b_q, o));
                    }
                    if (scribe && lane == 0) {
                        // H = ln Z - (ln 2 / Z) sum e x, with e = 2^x relative to the row reference
                        float *f = P.features + ((long long)b * P.N + a) * 4;
                        f[0] = bad_p ? CUDART_NAN_F : (float)(log(Z_p) - 0.6931471805599453 * X_p / Z_p);
                        f[2] = bad_p ? CUDART_NAN_F : (float)(exp2(b_p - (double)O_p) / Z_p);
                        f[1] = (hq && !bad_q) ? (float)(log(Z_q) - 0.6931471805599453 * X_q / Z_q) : 0.f;
                        f[3] = (hq && !bad_q) ? (float)(exp2(b_q - (double)O_q) / Z_q) : 0.f;
                    }
                }
                const bool live = !err && w_in > 0.0;
                const double invZp = err ? 0.0 : __drcp_rn(Z_p), invZq = (err || !hq) ? 0.0 : __drcp_rn(Z_q);
                const double A = live ? w_in * invZp : 0.0;
                E_r = A * zp_r;
                if (lane == 0) {
                    W.c = 0.0; W.E = err ? 0.0 : w_in; W.G = 1.0; W.g_commit = 0.0;
                    W.A = A; W.w_in = w_in; W.invZp = invZp; W.invZq = invZq;
                    W.Rg = (live && hq) ? Z_p * invZq * (w_in == 1.0 ? 1.0 : __drcp_rn(w_in)) : 0.0;
                    W.Z_p = Z_p; W.Z_q = Z_q; W.O_p = O_p; W.O_q = O_q;
                }
                __syncwarp();
            }

            // the thread's scale factors, exact powers of two: phi = 2^(o_p - O_p) converts its sums to the
            // row's units, rho = 2^((o_q - O_q) - (o_p - O_p)) its draft e to the units of its target e
            const int kphi = max(min(op_t - W.O_p, 0), -127), kq = max(min(oq_t - W.O_q, 0), -127);
            const float phi_t = pow2i(kphi), rho_t = pow2i(min(kq - kphi, 100));

            // ---- sibling loop: the same scalar recursion in every warp of the cluster ------------------------
            bool dead = !(W.A > 0.0);
            int acc = -1;
            const int kce = min(kc, KMAX);
            if (err && scribe && lane == 0) {
                // nothing below a faulty node is evaluated: every child gets weight / threshold 0
                NodeRec *rec = P.rec + (long long)b * P.N;
                for (int c = a + 1; c < P.N; ++c)
                    if (__ldg(parent + c) == a) {
                        if (trav) {
                            rec[c].w_in = 0.0;
                            __threadfence();
                            *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + c) = 0ull;
                        } else {
                            rec[c].thr = 0.0;
                        }
                    }
            }
            for (int j = 0; j < kce && !err; ++j) {
                const double st_c = W.c, st_E = W.E, st_G = W.G, w_in = W.w_in;
                const double Pp = W.cpm[j] * pow2d(W.cpn[j] - W.O_p) * W.invZp;
                const double Pq = W.cqm[j] * pow2d(W.cqn[j] - W.O_q) * W.invZq;
                const double Ux = w_in * Pp - st_c * Pq;
                const double denom = trav ? st_G : st_E;
                const bool zero = dead || !(Ux > 0.0), one = !zero && !(Pq > 0.0);
                if (scribe) {
                    const double thr = zero ? 0.0 : (one ? 1.0 : fmin(1.0, Ux / (denom * Pq)));
                    if (lane == 0) {
                        NodeRec *rec = P.rec + (long long)b * P.N;
                        const int cj = W.child[j];
                        if (trav) {
                            rec[cj].w_in = thr;
                            __threadfence();
                            *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + cj) =
                                (unsigned long long)__double_as_longlong(thr);
                        } else {
                            rec[cj].thr = thr;
                        }
                    }
                }
                if (!trav && acc < 0 && !zero && (one || (double)W.cu[j] * denom * Pq < Ux)) {
                    acc = W.child[j];
                    if (!P.all_thr) {
                        if (scribe && lane == 0)
                            for (int jj = j + 1; jj < kce; ++jj) P.rec[(long long)b * P.N + W.child[jj]].thr = CUDART_NAN;
                        break;
                    }
                }
                if (dead) continue;          // weight 0: the remaining children need no pass
                // residual step after rejecting child j: c' = c + G; one pass + one exchange
                const double g = (st_c + st_G) * W.Rg;
                float g_hi, g_lo;
                split_float(g, g_hi, g_lo);
                g_hi *= rho_t; g_lo *= rho_t;
                float tot = 0.f;
                for (int i = 0; i < nsm; ++i) {
                    float p[8], q[8];
                    const float4 *d = es + (size_t)(i * 4) * NCONS + tid;
                    load_e8(d, NCONS, p);
                    load_e8(d + 2 * NCONS, NCONS, q);
                    tot += residual_chunk(p, q, g_hi, g_lo);
                }
                tot += (residual_chunk(ep0, eq0, g_hi, g_lo) + residual_chunk(ep1, eq1, g_hi, g_lo)) +
                       (residual_chunk(ep2, eq2, g_hi, g_lo) + residual_chunk(ep3, eq3, g_hi, g_lo));
                const double wsum = W.A * warp_sum((double)(tot * phi_t));
                const int par = xn & 1;
                if (warp == 0 && lane == 0) mbar_arrive_expect_tx(&S.xbar[par], (uint32_t)(C * NW * 8));
                if (lane < C) st_async_f64(xchg + ((size_t)(par * C + rank) * NW + warp) * NP, &S.xbar[par], (uint32_t)lane, wsum);
                if (!*(volatile int *)&S.poison && !mbar_wait_cluster(&S.xbar[par], (uint32_t)((xn >> 1) & 1))) S.poison = 1;
                ++xn;
                double y = 0.0;
                if (lane < C) {
                    const double *src = xchg + (size_t)(par * C + lane) * NW * NP;
#pragma unroll
                    for (int w = 0; w < NW; ++w) y += src[(size_t)w * NP];
                }
                const double En = warp_sum(y);
                if (*(volatile int *)&S.poison) { err = SPEC_DEV_TIMEOUT; break; }
                __syncwarp();
                if (En > 0.0) {
                    if (lane == 0) {
                        W.c = st_c + st_G; W.E = En; W.G = En + st_G - st_E;
                        W.g_commit = g;
                    }
                    E_r = y;
                } else if (!(st_E >= st_G)) {
                    dead = true;       // S = 0 with w < 1: the weight drops to 0 (Traversal only)
                    if (lane == 0) W.E = 0.0;
                }
                // else S = 0 with w = 1 (P equals q up to rounding): the state stays
                __syncwarp();
            }

            // ---- the node's outcome -----------------------------------------------------------------------------
            const double w_fin = (dead || err) ? 0.0 : W.E / W.G;
            bool want_bonus;
            if (trav) want_bonus = (a == 0) || ((double)__ldg(P.u_accept + (long long)b * P.N + a) < w_fin);
            else want_bonus = acc < 0;
            if (dead || err) want_bonus = false;
            int owner = -1;
            double tau = 0.0, E_tot = 0.0;
            if (want_bonus) {
                E_tot = warp_sum(lane < C ? E_r : 0.0);
                const double target = (double)__ldg(P.u_bonus + (long long)b * P.N + a) * E_tot;
                owner = pick_lane(lane < C ? E_r : 0.0, target, tau);
            }
            if (scribe) {
                if (lane == 0) {
                    NodeRec &R = P.rec[(long long)b * P.N + a];
                    R.O_p = (double)W.O_p; R.Z_p = W.Z_p; R.O_q = (double)W.O_q; R.Z_q = W.Z_q;
                    R.c_fin = W.c; R.E_fin = (dead || err) ? 0.0 : W.E;
                    R.cut_p = cut_p; R.cut_q = cut_q;
                    R.next_child = acc;
                    R.status = err;
                    if (trav) { R.thr = (a == 0) ? 1.0 : w_fin; if (a == 0) R.w_in = 1.0; }
                    else { R.w_in = 1.0; if (a == 0) R.thr = 1.0; }
                    if (owner < 0) { R.bonus = -1; R.bonus_margin = 0.f; }
                }
                arrive_sequence(P, b, owner < 0 ? 2u : 1u);
            }

            // ---- bonus token: inverse CDF over the owner CTA's slice -----------------------------------------
            if (owner == (int)rank) {
                float gh_c, gl_c;                     // coefficient of the committed state, in this thread's units
                split_float(W.g_commit, gh_c, gl_c);
                gh_c *= rho_t; gl_c *= rho_t;
                const double invA = 1.0 / W.A;
                const double tau_rel = tau * invA, tot_rel = E_tot * invA;       // in units of e relative to O_p
                // per-tile totals of every warp
                for (int i = 0; i < nsm; ++i) {
                    float p[8], q[8];
                    const float4 *d = es + (size_t)(i * 4) * NCONS + tid;
                    load_e8(d, NCONS, p);
                    load_e8(d + 2 * NCONS, NCONS, q);
                    const double r = warp_sum((double)(residual_chunk(p, q, gh_c, gl_c) * phi_t));
                    if (lane == 0) S.wtile[warp][i] = r;
                }
                {
                    const double r0 = warp_sum((double)(residual_chunk(ep0, eq0, gh_c, gl_c) * phi_t));
                    const double r1 = warp_sum((double)(residual_chunk(ep1, eq1, gh_c, gl_c) * phi_t));
                    const double r2 = warp_sum((double)(residual_chunk(ep2, eq2, gh_c, gl_c) * phi_t));
                    const double r3 = warp_sum((double)(residual_chunk(ep3, eq3, gh_c, gl_c) * phi_t));
                    if (lane == 0) {
                        S.wtile[warp][nsm] = r0; S.wtile[warp][nsm + 1] = r1;
                        S.wtile[warp][nsm + 2] = r2; S.wtile[warp][nsm + 3] = r3;
                    }
                }
                bar_sync(1, NCONS);
                // tile, then warp inside the tile, then lane inside the warp, then token inside the chunk
                double Ti = 0.0;
                if (lane < nsm + RT)
                    for (int w = 0; w < NW; ++w) Ti += S.wtile[w][lane];
                double tau2, tau3, tau4;
                const int i_star = pick_lane(Ti, tau_rel, tau2);
                const double Ww = (i_star >= 0 && lane < NW) ? S.wtile[lane][i_star] : 0.0;
                const int w_star = i_star >= 0 ? pick_lane(Ww, tau2, tau3) : -1;
                bar_sync(1, NCONS);          // wtile may be rewritten by the next node only after everyone has read it
                if (w_star < 0) {
                    if (warp == 0) {
                        if (lane == 0) { NodeRec &R = P.rec[(long long)b * P.N + a]; R.bonus = -1; R.bonus_margin = 0.f; }
                        arrive_sequence(P, b, 1u);
                    }
                } else if (warp == w_star) {
                    float p[8], q[8];
                    if (i_star < nsm) {
                        const float4 *d = es + (size_t)(i_star * 4) * NCONS + tid;
                        load_e8(d, NCONS, p);
                        load_e8(d + 2 * NCONS, NCONS, q);
                    } else {
                        const int jr = i_star - nsm;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            p[k] = jr == 0 ? ep0[k] : (jr == 1 ? ep1[k] : (jr == 2 ? ep2[k] : ep3[k]));
                            q[k] = jr == 0 ? eq0[k] : (jr == 1 ? eq1[k] : (jr == 2 ? eq2[k] : eq3[k]));
                        }
                    }
                    float wk[8], v = 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) { wk[k] = fmaxf(fmaf(-gl_c, q[k], fmaf(-gh_c, q[k], p[k])), 0.f); v += wk[k]; }
                    const int l_star = pick_lane((double)(v * phi_t), tau3, tau4);
                    if (lane == l_star) {
                        const double phi = (double)phi_t;
                        const double tau_c = phi > 0.0 ? tau4 / phi : CUDART_INF;
                        double run = 0.0, dlo = 0.0, dhi = 0.0;
                        int found = -1, last_pos = -1;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const double before = run;
                            run += (double)wk[k];
                            if (wk[k] > 0.f) last_pos = k;
                            if (found < 0 && run > tau_c) { found = k; dlo = tau_c - before; dhi = run - tau_c; }
                        }
                        if (found < 0) { found = last_pos; dlo = 0.0; dhi = 0.0; }
                        NodeRec &R = P.rec[(long long)b * P.N + a];
                        R.bonus = found >= 0 ? (int)(tok0 + (long long)i_star * TILE + tid * 8 + found) : -1;
                        R.bonus_margin = (float)(fmin(dlo, dhi) * phi / tot_rel);
                    } else if (l_star < 0 && lane == 0) {
                        NodeRec &R = P.rec[(long long)b * P.N + a];
                        R.bonus = -1;
                        R.bonus_margin = 0.f;
                    }
                    __syncwarp();
                    arrive_sequence(P, b, 1u);
                }
            }
        }
#undef SPECV_NEXT_TILE
    }
    __syncthreads();
    cluster_sync_all();        // nobody leaves while a peer may still write to its shared memory
}

}  // namespace specv
