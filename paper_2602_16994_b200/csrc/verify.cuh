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
// After j rejected children the unnormalised target law of a node is
//     U_j(t) = (w_in P0(t) - c_j q(t))+ ,   c_0 = 0,  c_{j+1} = c_j + G_j,
//     E_j = sum_t U_j(t),  G_{j+1} = E_{j+1} + G_j - E_j   (G_0 = 1, E_0 = w_in).
// SpecInfer has w_in = 1, G_j = E_j: U_j / E_j is the residual after j updates P <- norm((P - q)+)
// and child j is accepted with min(1, U_j(x) / (E_j q(x))).  In Traversal Verification E_j / G_j is
// the node's weight after j rejected subtrees (w <- S / (S + 1 - w), P <- (wP - q)+ / S without the
// renormalisation) and child j is handed min(1, U_j(x) / (G_j q(x))).  One sibling step is one pass
// over the resident e computing sum (e_p - g e_q)+ plus one scalar exchange through distributed
// shared memory.
//
// Exchanges.  Every consumer warp of every CTA of the cluster sends its partial sum straight into
// the shared memory of all CTAs (st.async, which counts the bytes on the receiver's mbarrier); every
// warp waits on its own CTA's mbarrier and reduces all partials itself, in one fixed order, so all
// warps of the cluster hold bit-identical totals and take identical decisions without any CTA-wide
// barrier.
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
// A residual step whose mass is below this fraction of the mass before it is treated as S = 0: with
// fp32 exponentials, P = q (for instance two one-token nuclei on the same token) leaves a residual of
// about 1e-14 instead of exactly nothing.
constexpr double RESIDUAL_FLOOR = 1.0e-10;
constexpr double WEIGHT_SNAP = 1.0e-6;      // Traversal: a handed-down weight this close to 1 is 1

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
    const float *u_accept, *u_bonus;
    NodeRec *rec;
    unsigned long long *w_pub;   // [B*N] weight handed to a node by its parent (Traversal), W_PENDING until known
    unsigned int *done;          // [B] arrivals per sequence (two per node); the last one writes the outputs
    SpecOut out;
};

// per consumer warp: the children of the current node and the scalar state of its recursion
struct __align__(16) WarpArea {
    double cpm[KMAX], cqm[KMAX];   // final probabilities of the children's tokens under p and q
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

// sum over one chunk of (e_p - g e_q)+, g = gh + gl (two tokens per fused multiply-add)
__device__ __forceinline__ float residual_chunk(const float (&p)[8], const float (&q)[8], float gh, float gl)
{
    const unsigned long long ngh2 = pack_f32x2(-gh, -gh), ngl2 = pack_f32x2(-gl, -gl);
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < 8; k += 2) {
        const unsigned long long q2 = pack_f32x2(q[k], q[k + 1]);
        float r0, r1;
        unpack_f32x2(fma_f32x2(ngl2, q2, fma_f32x2(ngh2, q2, pack_f32x2(p[k], p[k + 1]))), r0, r1);
        acc += fmaxf(r0, 0.f) + fmaxf(r1, 0.f);
    }
    return acc;
}

// Inverse-CDF search over one CTA's resident residual (e_p - g e_q)+, run by all consumer warps of
// the CTA that owns the target (tau_rel, in units of e).  Token order is (tile, warp, lane, position
// in the chunk): the tile, then the warp inside the tile, then the lane, then the token.  The per-tile
// totals of a warp are reduced together, so that the shuffles of the ten tiles overlap; warp 0 alone
// picks tile and warp.
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
    float r[TMAX];
#pragma unroll
    for (int i = 0; i < SMT; ++i) {
        r[i] = 0.f;
        if (i < nsm) {
            float p[8], q[8];
            const float4 *d = es + (size_t)(i * 4) * NCONS + tid;
            load_e8(d, NCONS, p);
            load_e8(d + 2 * NCONS, NCONS, q);
            r[i] = residual_chunk(p, q, gh, gl);
        }
    }
    r[SMT + 0] = residual_chunk(ep0, eq0, gh, gl);
    r[SMT + 1] = residual_chunk(ep1, eq1, gh, gl);
    r[SMT + 2] = residual_chunk(ep2, eq2, gh, gl);
    r[SMT + 3] = residual_chunk(ep3, eq3, gh, gl);
    // a warp's total of one tile: 256 tokens, summed in fp32 like the chunks themselves; every level
    // above works in fp64 on these stored values, so the levels agree with each other exactly
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int i = 0; i < TMAX; ++i) r[i] += __shfl_xor_sync(0xffffffffu, r[i], o);
    }
#pragma unroll
    for (int i = 0; i < TMAX; ++i)
        if (lane == i) wtile[warp][i] = (double)r[i];
    bar_sync(1, NCONS);
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
    bar_sync(1, NCONS);
    const int s_star = (int)wtile[NW][0], w_star = (int)wtile[NW][1];
    const double tau3 = wtile[NW][2];
    double tau4;
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
        // release: the node's record (written by this warp, ordered before by __syncwarp where another
        // lane wrote it) is visible to whoever sees the count; acquire: the last arrival sees all records
        unsigned prev;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(prev) : "l"(P.done + b), "r"(count) : "memory");
        last = (prev + count == 2u * (unsigned)P.N) ? 1 : 0;
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) finalize_sequence(P, b);
}

}  // namespace specv
