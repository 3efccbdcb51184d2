// libspecverify: batched draft-tree verification for sm_100a.
//
// One thread-block cluster owns one tree node.  The node's target row (and its draft row when it
// has children) is brought on chip once with bulk asynchronous copies (cp.async.bulk completing on
// an mbarrier), each CTA of the cluster keeping a contiguous vocabulary slice.  The slice is turned
// in place into fp32 exponentials e = exp((z - m)/T); everything the verification rules need
// afterwards is a function of those two resident arrays:
//
//     after j rejected children the (unnormalised) target law of the node is
//         U_j(t) = (w_in * P0(t) - c_j * q(t))+ ,     c_0 = 0,  c_{j+1} = c_j + G_j,
//     with E_j = sum_t U_j(t) and G_{j+1} = E_{j+1} + G_j - E_j (G_0 = 1, E_0 = w_in).
//
// For SpecInfer (Algorithm 4) w_in = 1, so G_j = E_j and U_j / E_j is the residual after j updates
// P <- norm((P - q)+); child j is accepted with min(1, U_j(x)/(E_j q(x))).  For Traversal
// Verification w_j = E_j / G_j is the node's weight after j rejected subtrees (the block
// verification step w <- S/(S + 1 - w), P <- (wP - q)+/S written without renormalising), child j is
// handed min(1, U_j(x)/(G_j q(x))).  Each sibling step is therefore one pass over shared memory
// computing sum (e_p - gamma e_q)+ and one scalar exchange through distributed shared memory; no
// HBM traffic.  The bonus token is an inverse-CDF search over the resident slice.
//
// Scalars that decide something (ratios, weights, normalisers) are kept in fp64; vocabulary-wide
// elementwise work is fp32 with fp64 accumulation.
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "specverify.h"

namespace cg = cooperative_groups;

namespace {

constexpr int NT = 512;              // threads per CTA
constexpr int NWARP = NT / 32;
constexpr int KMAX = SPEC_MAX_CHILDREN;
constexpr int CMAX = 16;             // CTAs per cluster (16 needs the non-portable attribute)
constexpr int NX = 10;               // doubles per CTA per exchange
constexpr uint32_t BULK_CHUNK = 16384;
constexpr int SPIN_MBAR = 1 << 22;   // bounded waits: give up, flag the sequence, carry on
constexpr int SPIN_FLAG = 1 << 21;
constexpr unsigned long long W_PENDING = 0xFFFFFFFFFFFFFFFFull;

enum Mode { MODE_SPECINFER = 0, MODE_TRAVERSAL = 1 };

struct __align__(16) NodeRec {
    double m_p, Z_p, m_q, Z_q;   // row max of z (global over the cluster) and sum of kept e
    double c_fin, E_fin, w_in;   // final state: U = (w_in P0 - c_fin q)+, E_fin = sum U
    double thr;                  // threshold the node is tested with (written by its parent in
                                 // SpecInfer mode, by itself in Traversal mode)
    float cut_p, cut_q;          // smallest kept logit value (-inf: nothing cut)
    float bonus_margin;
    int next_child;              // SpecInfer: accepted child or -1
    int bonus;                   // speculative bonus token of this node or -1
    int status;
    int pad[2];
};

struct KParams {
    int B, N, V, dtype, mode, SL, all_thr;
    const void *zp, *zq;
    long long seq_stride, node_stride, topo_stride;
    const int *parent, *token;
    float T;
    const float *T_seq;
    int top_k;
    float top_p;
    const float *u_accept, *u_bonus;
    NodeRec *rec;
    unsigned long long *w_pub;
    float *features;
};

// ------------------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok)
                 : "r"(smem_u32(bar)), "r"(parity)
                 : "memory");
    return ok != 0;
}
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_down_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ float load_logit(const void *base, int dtype, long long idx)
{
    if (dtype == SPEC_F32) return __ldg((const float *)base + idx);
    return __uint_as_float((uint32_t)__ldg((const unsigned short *)base + idx) << 16);
}

// exp2((z - m) * s) with s = s_hi + s_lo: the product is formed in two parts so that the rounding of
// the exponent (|x| up to ~100) does not cost relative accuracy in e.
__device__ __forceinline__ float exp_scaled(float z, float m, float s_hi, float s_lo, float &x_out)
{
    float d = z - m;
    float x = d * s_hi;
    float lo = fmaf(d, s_lo, fmaf(d, s_hi, -x));
    x_out = x;
    if (!(x > -150.f)) { x_out = 0.f; return 0.f; }
    float e = ex2_approx(x);
    return fmaf(e, lo * 0.6931471805599453f, e);
}

// ------------------------------------------------------------------------------------------------
// shared state of one CTA
// ------------------------------------------------------------------------------------------------
struct Shared {
    double warp_part[NWARP][NX];
    double xchg[2][CMAX][NX];
    double scale_p[CMAX], scale_q[CMAX];   // exp((m_r - m)/T) per cluster rank
    double child_ep[KMAX], child_eq[KMAX]; // exp((z[x] - m)/T) of the children's tokens, fp64
    double ctl_d[4];
    float child_u[KMAX];
    int child[KMAX], child_tok[KMAX];
    int ctl_i[4];
    int kc, err;
    uint64_t mbar;
};

// Thread 0 holds v[0..nv); copies them into slot [parity][my_rank] of every CTA of the cluster, then
// the cluster barrier makes all slots visible everywhere.
__device__ __forceinline__ void cluster_allgather(cg::cluster_group &cluster, Shared &S, int parity,
                                                  const double *v, int nv)
{
    if (threadIdx.x == 0) {
        unsigned C = cluster.num_blocks(), me = cluster.block_rank();
        for (unsigned r = 0; r < C; ++r) {
            double *dst = cluster.map_shared_rank(&S.xchg[parity][me][0], r);
            for (int i = 0; i < nv; ++i) dst[i] = v[i];
        }
    }
    cluster.sync();
}

// block-wide sum of nv doubles per thread; result valid in thread 0.  Uses S.warp_part; the caller
// must pass a block or cluster barrier before the next use.
template <int NV>
__device__ __forceinline__ void block_sum(Shared &S, double (&v)[NV])
{
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = warp_sum(v[i]);
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < NV; ++i) S.warp_part[w][i] = v[i];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            double t = 0.0;
            for (int k = 0; k < NWARP; ++k) t += S.warp_part[k][i];
            v[i] = t;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// row staging: global -> shared (raw dtype), placed so that the in-place widening to fp32 is safe
// ------------------------------------------------------------------------------------------------
// region: SL floats.  fp32 raw data sits at the start; bf16 raw data in the upper half.
__device__ __forceinline__ unsigned char *raw_ptr(float *region, int SL, int dtype)
{
    return (unsigned char *)region + (dtype == SPEC_BF16 ? 2 * (size_t)SL : 0);
}

// Issue the copy of `n` elements starting at element `g0` of the row at `row` into `region`.
// Thread 0 enqueues bulk copies for the 16-byte aligned body; everything else (a misaligned row,
// the last partial 16 bytes) is fetched with ordinary loads by all threads.
// Returns the number of bytes that will complete on the mbarrier (valid in thread 0).
__device__ __forceinline__ uint32_t stage_row(float *region, int SL, int dtype, const void *row,
                                              long long g0, int n, uint64_t *bar, bool count_only)
{
    const int esz = dtype == SPEC_BF16 ? 2 : 4;
    const unsigned char *src = (const unsigned char *)row + g0 * esz;
    unsigned char *dst = raw_ptr(region, SL, dtype);
    bool aligned = (((uintptr_t)src) & 15) == 0;
    uint32_t body = aligned ? (((uint32_t)n * esz) & ~15u) : 0u;
    if (count_only) return body;
    if (threadIdx.x == 0) {
        for (uint32_t off = 0; off < body; off += BULK_CHUNK) {
            uint32_t sz = body - off < BULK_CHUNK ? body - off : BULK_CHUNK;
            bulk_g2s(dst + off, src + off, sz, bar);
        }
    }
    int first = body / esz;               // elements not covered by the bulk copies
    if (dtype == SPEC_BF16) {
        const unsigned short *s = (const unsigned short *)src;
        unsigned short *d = (unsigned short *)dst;
        for (int i = first + threadIdx.x; i < n; i += NT) d[i] = __ldg(s + i);
    } else {
        const float *s = (const float *)src;
        float *d = (float *)dst;
        for (int i = first + threadIdx.x; i < n; i += NT) d[i] = __ldg(s + i);
    }
    return body;
}

// max over the raw slice (ignoring NaN, which is reported through `nan`)
__device__ __forceinline__ float raw_max(const float *region, int SL, int dtype, int n, bool &nan)
{
    float m = -CUDART_INF_F;
    bool bad = false;
    const unsigned char *raw = raw_ptr(const_cast<float *>(region), SL, dtype);
    if (dtype == SPEC_BF16) {
        const uint4 *v = (const uint4 *)raw;
        int nv = n >> 3;
        for (int i = threadIdx.x; i < nv; i += NT) {
            uint4 q = v[i];
            uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float a = bf16_lo(w[k]), b = bf16_hi(w[k]);
                bad |= (a != a) | (b != b);
                m = fmaxf(m, fmaxf(a, b));
            }
        }
        const unsigned short *h = (const unsigned short *)raw;
        for (int i = (nv << 3) + threadIdx.x; i < n; i += NT) {
            float a = __uint_as_float((uint32_t)h[i] << 16);
            bad |= (a != a);
            m = fmaxf(m, a);
        }
    } else {
        const float4 *v = (const float4 *)raw;
        int nv = n >> 2;
        for (int i = threadIdx.x; i < nv; i += NT) {
            float4 q = v[i];
            bad |= (q.x != q.x) | (q.y != q.y) | (q.z != q.z) | (q.w != q.w);
            m = fmaxf(m, fmaxf(fmaxf(q.x, q.y), fmaxf(q.z, q.w)));
        }
        const float *h = (const float *)raw;
        for (int i = (nv << 2) + threadIdx.x; i < n; i += NT) {
            float a = h[i];
            bad |= (a != a);
            m = fmaxf(m, a);
        }
    }
    nan = bad;
    return m;
}

// In-place widening raw -> e = exp((z - m)/T) for z >= cut (0 otherwise, and 0 in the padding up to
// SL).  Accumulates sum e and sum e*log2(e).  bf16: a step reads 8 values per thread, a block
// barrier, then writes 8 floats; step s writes bytes [16384 s, 16384 (s+1)) of the region while the
// unread raw data starts at 2 SL + 8192 (s+1) >= 16384 (s+1) as long as a later step exists.
__device__ __forceinline__ void widen_exp(float *region, int SL, int dtype, int n, float m, float cut,
                                          float s_hi, float s_lo, double &sum_e, double &sum_ex)
{
    double acc_e = 0.0, acc_x = 0.0;
    if (dtype == SPEC_BF16) {
        const unsigned char *raw = raw_ptr(region, SL, dtype);
        int steps = (SL + NT * 8 - 1) / (NT * 8);
        for (int s = 0; s < steps; ++s) {
            int t0 = (s * NT + threadIdx.x) * 8;
            bool act = t0 < SL;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (act) q = *(const uint4 *)(raw + (size_t)t0 * 2);
            __syncthreads();
            if (act) {
                uint32_t w[4] = {q.x, q.y, q.z, q.w};
                float e[8];
                float pe = 0.f, px = 0.f;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    float z = (k & 1) ? bf16_hi(w[k >> 1]) : bf16_lo(w[k >> 1]);
                    bool keep = (t0 + k < n) && (z >= cut);
                    float x;
                    float v = exp_scaled(keep ? z : -CUDART_INF_F, m, s_hi, s_lo, x);
                    e[k] = v;
                    pe += v;
                    px = fmaf(v, x, px);
                }
                acc_e += (double)pe;
                acc_x += (double)px;
                float4 *o = (float4 *)(region + t0);
                o[0] = make_float4(e[0], e[1], e[2], e[3]);
                o[1] = make_float4(e[4], e[5], e[6], e[7]);
            }
        }
    } else {
        int nv = SL >> 2;
        float4 *v = (float4 *)region;
        for (int i = threadIdx.x; i < nv; i += NT) {
            float4 q = v[i];
            float zz[4] = {q.x, q.y, q.z, q.w};
            float e[4];
            float pe = 0.f, px = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float x;
                bool keep = ((i * 4 + k) < n) && (zz[k] >= cut);
                float val = exp_scaled(keep ? zz[k] : -CUDART_INF_F, m, s_hi, s_lo, x);
                e[k] = val;
                pe += val;
                px = fmaf(val, x, px);
            }
            acc_e += (double)pe;
            acc_x += (double)px;
            v[i] = make_float4(e[0], e[1], e[2], e[3]);
        }
    }
    sum_e = acc_e;
    sum_ex = acc_x;
}

// sum over the slice of (ep - gamma * eq)+ ; gamma = g_hi + g_lo
__device__ __forceinline__ double pass_residual_sum(const float *ep, const float *eq, int SL, float g_hi, float g_lo)
{
    const float4 *a = (const float4 *)ep, *b = (const float4 *)eq;
    int nv = SL >> 2;
    double acc = 0.0;
    for (int i = threadIdx.x; i < nv; i += NT) {
        float4 p = a[i], q = b[i];
        float s0 = fmaxf(fmaf(-g_lo, q.x, fmaf(-g_hi, q.x, p.x)), 0.f);
        float s1 = fmaxf(fmaf(-g_lo, q.y, fmaf(-g_hi, q.y, p.y)), 0.f);
        float s2 = fmaxf(fmaf(-g_lo, q.z, fmaf(-g_hi, q.z, p.z)), 0.f);
        float s3 = fmaxf(fmaf(-g_lo, q.w, fmaf(-g_hi, q.w, p.w)), 0.f);
        acc += (double)((s0 + s1) + (s2 + s3));
    }
    return acc;
}

// Inverse CDF inside one slice.  Weights w_t = (ep[t] - gamma eq[t])+ (eq may be NULL: w = ep).
// Each thread owns a contiguous run of float4 groups (an odd count, so that the 128-bit shared loads
// of a warp fall in distinct bank groups), sums it in fp64, a block scan finds the owning thread,
// which walks its run again.  Returns the local token index (block-uniform), or the last
// positive-weight token if tau is not below the slice total, or -1 if the slice holds no weight.
__device__ __forceinline__ int slice_inverse_cdf(Shared &S, const float *ep, const float *eq, int SL,
                                                 float g_hi, float g_lo, double tau, double &dist_lo,
                                                 double &dist_hi)
{
    const int nv = SL >> 2;
    int L4 = (nv + NT - 1) / NT;
    L4 |= 1;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int i0 = threadIdx.x * L4, i1 = min(i0 + L4, nv);
    const float4 *a = (const float4 *)ep, *b = (const float4 *)eq;
    double seg = 0.0;
    int last_pos = -1;
    for (int i = i0; i < i1; ++i) {
        float4 p = a[i];
        float v[4] = {p.x, p.y, p.z, p.w};
        if (eq) {
            float4 q = b[i];
            v[0] = fmaxf(fmaf(-g_lo, q.x, fmaf(-g_hi, q.x, p.x)), 0.f);
            v[1] = fmaxf(fmaf(-g_lo, q.y, fmaf(-g_hi, q.y, p.y)), 0.f);
            v[2] = fmaxf(fmaf(-g_lo, q.z, fmaf(-g_hi, q.z, p.z)), 0.f);
            v[3] = fmaxf(fmaf(-g_lo, q.w, fmaf(-g_hi, q.w, p.w)), 0.f);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            seg += (double)v[k];
            if (v[k] > 0.f) last_pos = i * 4 + k;
        }
    }
    // block-wide exclusive scan of seg
    double inc = seg;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();                    // warp_part / ctl may still be read from the previous phase
    if (lane == 31) S.warp_part[w][0] = inc;
    if (threadIdx.x == 0) { S.ctl_i[2] = -1; S.ctl_i[3] = -1; }
    __syncthreads();
    double base = 0.0, total = 0.0;
    for (int k = 0; k < NWARP; ++k) {
        double t = S.warp_part[k][0];
        if (k < w) base += t;
        total += t;
    }
    double excl = base + inc - seg, incl = base + inc;
    if (seg > 0.0 && excl <= tau && tau < incl) {
        double run = excl;
        int found = -1;
        double before = excl;
        for (int i = i0; i < i1 && found < 0; ++i) {
            float4 p = a[i];
            float v[4] = {p.x, p.y, p.z, p.w};
            if (eq) {
                float4 q = b[i];
                v[0] = fmaxf(fmaf(-g_lo, q.x, fmaf(-g_hi, q.x, p.x)), 0.f);
                v[1] = fmaxf(fmaf(-g_lo, q.y, fmaf(-g_hi, q.y, p.y)), 0.f);
                v[2] = fmaxf(fmaf(-g_lo, q.z, fmaf(-g_hi, q.z, p.z)), 0.f);
                v[3] = fmaxf(fmaf(-g_lo, q.w, fmaf(-g_hi, q.w, p.w)), 0.f);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (found < 0) {
                    before = run;
                    run += (double)v[k];
                    if (run > tau) found = i * 4 + k;
                }
            }
        }
        if (found < 0) found = last_pos;   // cannot happen: incl is this very sum
        S.ctl_i[2] = found;
        S.ctl_d[2] = tau - before;
        S.ctl_d[3] = run - tau;
    }
    // fallback: last positive-weight token of the slice
    if (last_pos >= 0) atomicMax(&S.ctl_i[3], last_pos);
    __syncthreads();
    int tok = S.ctl_i[2];
    if (tok >= 0) { dist_lo = S.ctl_d[2]; dist_hi = S.ctl_d[3]; }
    else { tok = S.ctl_i[3]; dist_lo = 0.0; dist_hi = 0.0; }
    (void)total;
    return tok;
}

__device__ __forceinline__ void split_float(double g, float &hi, float &lo)
{
    hi = (float)g;
    lo = (float)(g - (double)hi);
}

// ------------------------------------------------------------------------------------------------
// the node kernel (SpecInfer / Traversal)
// ------------------------------------------------------------------------------------------------
extern __shared__ __align__(128) unsigned char dyn_smem[];

__global__ void __launch_bounds__(NT, 1) spec_node_kernel(const KParams P)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int cid = blockIdx.x / C;
    const int a = cid / P.B, b = cid % P.B;     // node-major: parents are scheduled before children
    const int tid = threadIdx.x;
    const int SL = P.SL;
    __shared__ Shared S;
    cluster.barrier_arrive();            // peers must be running before their shared memory is written

    float *ep = (float *)dyn_smem;
    float *eq = ep + SL;
    const long long tok0 = (long long)rank * SL;
    const int n = (int)max(0ll, min((long long)SL, (long long)P.V - tok0));
    const int *parent = P.parent + (long long)b * P.topo_stride;
    const int *token = P.token + (long long)b * P.N;
    NodeRec *rec = P.rec + (long long)b * P.N;
    const double T = (double)(P.T_seq ? __ldg(P.T_seq + b) : P.T);
    int parity = 0;

    // ---- topology: children of a (warp 0), validation -------------------------------------------
    if (tid < 32) {
        int err = 0, kc = 0;
        if (tid == 0) {
            int pa = __ldg(parent + a);
            if (a == 0 ? (pa != -1) : (pa < 0 || pa >= a)) err = SPEC_DEV_TOPOLOGY;
            if (a > 0) {
                int x = __ldg(token + a);
                if (x < 0 || x >= P.V) err = SPEC_DEV_TOKEN;
            }
        }
        for (int c0 = a + 1; c0 < P.N; c0 += 32) {
            int c = c0 + tid;
            bool is = c < P.N && __ldg(parent + c) == a;
            unsigned bal = __ballot_sync(0xffffffffu, is);
            if (is) {
                int pos = kc + __popc(bal & ((1u << tid) - 1u));
                if (pos < KMAX) {
                    int x = __ldg(token + c);
                    S.child[pos] = c;
                    S.child_tok[pos] = x;
                    S.child_u[pos] = __ldg(P.u_accept + (long long)b * P.N + c);
                    if (x < 0 || x >= P.V) err = SPEC_DEV_TOKEN;
                }
            }
            kc += __popc(bal);
        }
        if (kc > KMAX) err = SPEC_DEV_TOPOLOGY;
        err = __reduce_max_sync(0xffffffffu, err);
        if (tid == 0) {
            S.kc = err ? 0 : kc;
            S.err = err;
            mbar_init(&S.mbar, 1);
        }
    }
    __syncthreads();
    const int kc = S.kc;
    const bool has_q = kc > 0;
    int err = S.err;

    // ---- stage the rows -------------------------------------------------------------------------
    const void *row_p = (const unsigned char *)P.zp +
                        ((long long)b * P.seq_stride + (long long)a * P.node_stride) * (P.dtype == SPEC_BF16 ? 2 : 4);
    const void *row_q = (const unsigned char *)P.zq +
                        ((long long)b * P.seq_stride + (long long)a * P.node_stride) * (P.dtype == SPEC_BF16 ? 2 : 4);
    uint32_t tx = stage_row(ep, SL, P.dtype, row_p, tok0, n, &S.mbar, true);
    if (has_q) tx += stage_row(eq, SL, P.dtype, row_q, tok0, n, &S.mbar, true);
    if (tid == 0 && tx) mbar_expect_tx(&S.mbar, tx);
    stage_row(ep, SL, P.dtype, row_p, tok0, n, &S.mbar, false);
    if (has_q) stage_row(eq, SL, P.dtype, row_q, tok0, n, &S.mbar, false);
    if (tx) {
        int spins = 0;
        while (!mbar_try_wait(&S.mbar, 0)) {
            if (++spins > SPIN_MBAR) { err = SPEC_DEV_TIMEOUT; break; }
        }
        if (err == SPEC_DEV_TIMEOUT) {          // wait once more for the copies in flight, bounded
            spins = 0;
            while (!mbar_try_wait(&S.mbar, 0) && ++spins < SPIN_MBAR) {}
        }
    }
    __syncthreads();

    // ---- local max, widening to exponentials ------------------------------------------------------
    bool nan_p = false, nan_q = false;
    float mp = raw_max(ep, SL, P.dtype, n, nan_p);
    float mq = has_q ? raw_max(eq, SL, P.dtype, n, nan_q) : -CUDART_INF_F;
    mp = warp_max(mp);
    mq = warp_max(mq);
    if ((tid & 31) == 0) { S.warp_part[tid >> 5][0] = (double)mp; S.warp_part[tid >> 5][1] = (double)mq; }
    int any_nan = __syncthreads_or((int)(nan_p | nan_q));
    mp = -CUDART_INF_F; mq = -CUDART_INF_F;
    for (int k = 0; k < NWARP; ++k) {
        mp = fmaxf(mp, (float)S.warp_part[k][0]);
        mq = fmaxf(mq, (float)S.warp_part[k][1]);
    }
    __syncthreads();
    float s_hi, s_lo;
    split_float(1.4426950408889634 / T, s_hi, s_lo);
    const float ref_p = (mp > -CUDART_INF_F && mp < CUDART_INF_F) ? mp : 0.f;   // empty / all -inf slice: e = 0
    const float ref_q = (mq > -CUDART_INF_F && mq < CUDART_INF_F) ? mq : 0.f;
    double v[NX];
#pragma unroll
    for (int i = 0; i < NX; ++i) v[i] = 0.0;
    widen_exp(ep, SL, P.dtype, n, ref_p, -CUDART_INF_F, s_hi, s_lo, v[1], v[2]);
    if (has_q) widen_exp(eq, SL, P.dtype, n, ref_q, -CUDART_INF_F, s_hi, s_lo, v[4], v[5]);
    {
        double red[4] = {v[1], v[2], v[4], v[5]};
        block_sum<4>(S, red);
        v[1] = red[0]; v[2] = red[1]; v[4] = red[2]; v[5] = red[3];
    }
    v[0] = (double)mp; v[3] = (double)mq; v[6] = any_nan ? 1.0 : 0.0;
    v[7] = 1.0;   // w_in
    v[8] = 0.0;   // timeout flag of the wait below

    // ---- Traversal: weight handed down by the parent (rank 0 waits, bounded) -----------------------
    if (P.mode == MODE_TRAVERSAL && a > 0 && rank == 0 && tid == 0) {
        volatile unsigned long long *slot = P.w_pub + (long long)b * P.N + a;
        unsigned long long bits = W_PENDING;
        for (int spins = 0; spins < SPIN_FLAG; ++spins) {
            bits = *slot;
            if (bits != W_PENDING) break;
            __nanosleep(64);
        }
        if (bits == W_PENDING) { v[7] = 0.0; v[8] = 1.0; }
        else { __threadfence(); v[7] = __longlong_as_double((long long)bits); }
    }

    // ---- exchange 1: per-slice max / sums (+ w_in from rank 0) -----------------------------------
    cluster.barrier_wait();
    cluster_allgather(cluster, S, parity, v, NX);
    double (*X)[NX] = S.xchg[parity];
    parity ^= 1;
    double m_p = -CUDART_INF, m_q = -CUDART_INF;
    bool bad = false;
    for (int r = 0; r < C; ++r) {
        m_p = fmax(m_p, X[r][0]);
        m_q = fmax(m_q, X[r][3]);
        bad |= X[r][6] != 0.0;
    }
    const double w_in = X[0][7];
    if (X[0][8] != 0.0) err = SPEC_DEV_TIMEOUT;
    if (bad || !(m_p > -CUDART_INF && m_p < CUDART_INF)) err = err ? err : SPEC_DEV_NONFINITE;
    if (has_q && !(m_q > -CUDART_INF && m_q < CUDART_INF)) err = err ? err : SPEC_DEV_NONFINITE;
    if (tid < C) {
        double mr = X[tid][0];
        S.scale_p[tid] = (mr > -CUDART_INF && m_p < CUDART_INF) ? exp((mr - m_p) / T) : 0.0;
    } else if (tid >= 32 && tid < 32 + C) {
        double mr = X[tid - 32][3];
        S.scale_q[tid - 32] = (has_q && mr > -CUDART_INF && m_q < CUDART_INF) ? exp((mr - m_q) / T) : 0.0;
    } else if (tid >= 64 && tid < 64 + kc) {
        int j = tid - 64;
        long long x = S.child_tok[j];
        double zpx = (double)load_logit(row_p, P.dtype, x), zqx = (double)load_logit(row_q, P.dtype, x);
        S.child_ep[j] = exp((zpx - m_p) / T);
        S.child_eq[j] = exp((zqx - m_q) / T);
    }
    __syncthreads();
    double Z_p = 0.0, Z_q = 0.0, XL_p = 0.0, XL_q = 0.0;   // XL: sum over tokens of p * ln p pieces
    for (int r = 0; r < C; ++r) {
        double sp = S.scale_p[r], sq = S.scale_q[r];
        Z_p += sp * X[r][1];
        Z_q += sq * X[r][4];
    }
    if (P.features && rank == 0 && tid == 0) {
        // H = -sum p ln p with p = e s_r / Z and ln e = ln2 * x
        double hp = 0.0, hq = 0.0;
        for (int r = 0; r < C; ++r) {
            double sp = S.scale_p[r], sq = S.scale_q[r];
            if (sp > 0.0) hp -= (sp / Z_p) * (0.6931471805599453 * X[r][2] + (log(sp) - log(Z_p)) * X[r][1]);
            if (has_q && sq > 0.0) hq -= (sq / Z_q) * (0.6931471805599453 * X[r][5] + (log(sq) - log(Z_q)) * X[r][4]);
        }
        float *f = P.features + ((long long)b * P.N + a) * 4;
        f[0] = (float)hp;
        f[1] = has_q ? (float)hq : 0.f;
        f[2] = (float)(1.0 / Z_p);
        f[3] = has_q ? (float)(1.0 / Z_q) : 0.f;
    }
    (void)XL_p; (void)XL_q;

    // ---- sibling loop: thread 0 of every CTA runs the same scalar recursion ------------------------
    // state: U = (w_in P0 - c q)+, E = sum U, G as in the header comment; part[r] = slice totals of U
    double c = 0.0, E = w_in, G = 1.0;
    double part[CMAX];
    const double A = (Z_p > 0.0) ? w_in / Z_p : 0.0;        // U = A * s_p[r] * ep - (c/Z_q) * s_q[r] * eq
    for (int r = 0; r < CMAX; ++r) part[r] = (r < C) ? A * S.scale_p[r] * X[r][1] : 0.0;
    const double a_me = A * S.scale_p[rank];
    const double bq_me = (has_q && Z_q > 0.0) ? S.scale_q[rank] / Z_q : 0.0;
    int accepted_child = -1;
    bool dead = !(w_in > 0.0);           // Traversal: weight 0 reaches nothing below
    const bool trav = P.mode == MODE_TRAVERSAL;
    double gamma_me = 0.0;

    for (int j = 0; j < kc; ++j) {
        // decision for child j from the current state (thread 0), then the next residual coefficient
        if (tid == 0) {
            const double Pp = S.child_ep[j] / Z_p, Pq = S.child_eq[j] / Z_q;
            double Ux = w_in * Pp - c * Pq;
            double thr;
            const double denom = trav ? G : E;
            if (dead || !(Ux > 0.0)) thr = 0.0;
            else if (!(Pq > 0.0)) thr = 1.0;
            else thr = fmin(1.0, Ux / (denom * Pq));
            const int cj = S.child[j];
            int stop = 0;
            if (trav) {
                if (rank == 0) {
                    rec[cj].w_in = thr;
                    __threadfence();
                    *(volatile unsigned long long *)(P.w_pub + (long long)b * P.N + cj) =
                        (unsigned long long)__double_as_longlong(thr);
                }
            } else {
                if (rank == 0) rec[cj].thr = thr;
                if (accepted_child < 0 && (double)S.child_u[j] < thr) {
                    accepted_child = cj;
                    if (!P.all_thr) stop = 1;
                }
            }
            S.ctl_i[0] = stop;
            // residual step after rejecting child j: c' = c + G
            double g = 0.0;
            int do_pass = (!dead && !stop) ? 1 : 0;
            if (do_pass) {
                double cn = c + G;
                g = (a_me > 0.0) ? (cn * bq_me) / a_me : 0.0;
                S.ctl_d[0] = g;
            }
            S.ctl_i[1] = do_pass;
        }
        __syncthreads();
        const int stop = S.ctl_i[0], do_pass = S.ctl_i[1];
        if (stop) {
            if (tid == 0 && rank == 0)
                for (int jj = j + 1; jj < kc; ++jj) rec[S.child[jj]].thr = CUDART_NAN;
            break;
        }
        if (do_pass) {
            const double g = S.ctl_d[0];
            float g_hi, g_lo;
            split_float(g, g_hi, g_lo);
            double sum[1] = {(a_me > 0.0) ? pass_residual_sum(ep, eq, SL, g_hi, g_lo) : 0.0};
            block_sum<1>(S, sum);
            double mine = a_me * sum[0];
            cluster_allgather(cluster, S, parity, &mine, 1);
            if (tid == 0) {
                double (*Y)[NX] = S.xchg[parity];
                double En = 0.0;
                for (int r = 0; r < C; ++r) En += Y[r][0];
                if (En > 0.0) {
                    double Gn = En + G - E;
                    c = c + G;
                    E = En;
                    G = Gn;
                    gamma_me = g;
                    for (int r = 0; r < C; ++r) part[r] = Y[r][0];
                } else if (!(E >= G)) {
                    dead = true;      // S = 0 with w < 1: weight drops to 0 (Traversal only)
                    E = 0.0;
                }
                // else: S = 0 with w = 1 (P == q up to rounding): state unchanged
            }
            parity ^= 1;
        }
    }

    // ---- final state, bonus draw -----------------------------------------------------------------------
    if (tid == 0) {
        const double w_fin = dead ? 0.0 : E / G;
        int want_bonus;
        if (trav) want_bonus = (a == 0) || ((double)__ldg(P.u_accept + (long long)b * P.N + a) < w_fin);
        else want_bonus = accepted_child < 0;
        if (dead) want_bonus = 0;        // weight 0: the node is never accepted
        int owner = -1;
        double tau = 0.0, tot = 0.0;
        if (want_bonus) {
            for (int r = 0; r < C; ++r) tot += part[r];
            double target = (double)__ldg(P.u_bonus + (long long)b * P.N + a) * tot;
            double pre = 0.0;
            int last_pos = -1;
            for (int r = 0; r < C; ++r) {
                if (part[r] > 0.0) last_pos = r;
                if (owner < 0 && pre + part[r] > target) { owner = r; tau = target - pre; }
                if (owner < 0) pre += part[r];
            }
            if (owner < 0) { owner = last_pos; tau = CUDART_INF; }   // rounding: take the last token with weight
        }
        S.ctl_i[0] = owner;
        S.ctl_d[0] = (owner == rank && a_me > 0.0) ? tau / a_me : 0.0;
        S.ctl_d[1] = gamma_me;
        if (rank == 0) {
            NodeRec &R = rec[a];
            R.m_p = m_p; R.Z_p = Z_p; R.m_q = m_q; R.Z_q = Z_q;
            R.c_fin = c; R.E_fin = dead ? 0.0 : E;
            R.cut_p = -CUDART_INF_F; R.cut_q = -CUDART_INF_F;
            R.next_child = accepted_child;
            R.status = err;
            if (trav) { R.thr = (a == 0) ? 1.0 : w_fin; if (a == 0) R.w_in = 1.0; }
            else { R.w_in = 1.0; if (a == 0) R.thr = 1.0; }
            if (owner < 0) { R.bonus = -1; R.bonus_margin = 0.f; }
        }
        S.ctl_d[2] = tot;
    }
    __syncthreads();
    const int owner = S.ctl_i[0];
    if (owner == rank) {
        const double tauF = S.ctl_d[0], g = S.ctl_d[1], tot = S.ctl_d[2];
        float g_hi, g_lo;
        split_float(g, g_hi, g_lo);
        double dlo = 0.0, dhi = 0.0;
        int t = slice_inverse_cdf(S, ep, (has_q && g != 0.0) ? eq : nullptr, SL, g_hi, g_lo, tauF, dlo, dhi);
        if (tid == 0) {
            NodeRec &R = rec[a];
            R.bonus = t >= 0 ? (int)(tok0 + t) : -1;
            R.bonus_margin = (float)(fmin(dlo, dhi) * a_me / tot);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// finalize: one thread per sequence walks the per-node records
// ------------------------------------------------------------------------------------------------
struct FParams {
    int B, N, mode;
    const int *parent, *token;
    long long topo_stride;
    const float *u_accept;
    const NodeRec *rec;
    SpecOut out;
};

__device__ __forceinline__ int first_child(const int *parent, int N, int a)
{
    for (int c = a + 1; c < N; ++c)
        if (parent[c] == a) return c;
    return -1;
}
__device__ __forceinline__ int next_sibling(const int *parent, int N, int c)
{
    int p = parent[c];
    for (int d = c + 1; d < N; ++d)
        if (parent[d] == p) return d;
    return -1;
}

__global__ void spec_finalize_kernel(const FParams P)
{
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= P.B) return;
    const int N = P.N;
    const int *parent = P.parent + (long long)b * P.topo_stride;
    const int *token = P.token + (long long)b * N;
    const NodeRec *rec = P.rec + (long long)b * N;
    const float *ua = P.u_accept + (long long)b * N;
    int status = 0;
    for (int i = 0; i < N; ++i) status = max(status, rec[i].status);
    int acc = -1;
    if (!status) {
        if (P.mode == MODE_SPECINFER) {
            acc = 0;
            for (int hop = 0; hop < N; ++hop) {
                int nx = rec[acc].next_child;
                if (nx < 0) break;
                acc = nx;
            }
        } else {
            // depth-first post-order; the first node with u < w_fin (the root always) is accepted
            int cur = 0;
            for (int guard = 0; guard < 4 * N + 4 && acc < 0; ++guard) {
                int fc;
                while ((fc = first_child(parent, N, cur)) >= 0) cur = fc;     // descend to a leaf
                for (;;) {
                    if (cur == 0 || (double)ua[cur] < rec[cur].thr) { acc = cur; break; }
                    int sib = next_sibling(parent, N, cur);
                    if (sib >= 0) { cur = sib; break; }
                    cur = parent[cur];
                }
            }
            if (acc < 0) status = SPEC_DEV_TOPOLOGY;
        }
    }
    int len = 0;
    if (acc >= 0)
        for (int x = acc; x != 0; x = parent[x]) ++len;
    int bonus = acc >= 0 ? rec[acc].bonus : -1;
    if (acc >= 0 && bonus < 0 && !status) status = SPEC_DEV_NONFINITE;
    if (status) { acc = -1; len = -1; bonus = -1; }
    P.out.accepted_node[b] = acc;
    P.out.accept_len[b] = len;
    P.out.bonus_token[b] = bonus;
    P.out.status[b] = status;
    int *ot = P.out.out_tokens + (long long)b * N;
    for (int i = 0; i < N; ++i) ot[i] = -1;
    if (acc >= 0) {
        ot[len] = bonus;
        int i = len;
        for (int x = acc; x != 0; x = parent[x]) ot[--i] = token[x];
    }
    if (P.out.node_thr)
        for (int i = 0; i < N; ++i) P.out.node_thr[(long long)b * N + i] = (float)rec[i].thr;
    if (P.out.node_w_in && P.mode == MODE_TRAVERSAL)
        for (int i = 0; i < N; ++i) P.out.node_w_in[(long long)b * N + i] = (float)rec[i].w_in;
    if (P.out.margin) {
        float *mg = P.out.margin + (long long)b * (N + 1);
        mg[0] = CUDART_NAN_F;
        for (int i = 1; i < N; ++i) mg[i] = (float)fabs((double)ua[i] - rec[i].thr);
        mg[N] = acc >= 0 ? rec[acc].bonus_margin : CUDART_NAN_F;
    }
}

// ------------------------------------------------------------------------------------------------
// residual output: the law the bonus was drawn from, for the accepted node of each sequence
// ------------------------------------------------------------------------------------------------
struct RParams {
    int B, N, V, dtype;
    const void *zp, *zq;
    long long seq_stride, node_stride;
    float T;
    const float *T_seq;
    const NodeRec *rec;
    const int *accepted;
    float *residual;
};

__global__ void spec_residual_kernel(const RParams P)
{
    const int b = blockIdx.y;
    const int acc = P.accepted[b];
    float *out = P.residual + (long long)b * P.V;
    if (acc < 0) {
        for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < P.V; t += gridDim.x * blockDim.x) out[t] = 0.f;
        return;
    }
    const NodeRec R = P.rec[(long long)b * P.N + acc];
    const double T = (double)(P.T_seq ? P.T_seq[b] : P.T);
    const long long row = (long long)b * P.seq_stride + (long long)acc * P.node_stride;
    const bool use_q = R.c_fin != 0.0;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < P.V; t += gridDim.x * blockDim.x) {
        float zp = load_logit(P.zp, P.dtype, row + t);
        double u = (zp >= R.cut_p) ? R.w_in * exp(((double)zp - R.m_p) / T) / R.Z_p : 0.0;
        if (use_q) {
            float zq = load_logit(P.zq, P.dtype, row + t);
            if (zq >= R.cut_q) u -= R.c_fin * exp(((double)zq - R.m_q) / T) / R.Z_q;
        }
        out[t] = (float)(u > 0.0 ? u / R.E_fin : 0.0);
    }
}

// ------------------------------------------------------------------------------------------------
// spec_tree_probs: materialise the sampling distribution of every row
// ------------------------------------------------------------------------------------------------
struct TParams {
    int rows, N, V, dtype, SL;
    const void *z;
    long long seq_stride, node_stride;
    float T;
    const float *T_seq;
    float *probs, *stats;
};

__global__ void __launch_bounds__(NT, 1) spec_probs_kernel(const TParams P)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int row_id = blockIdx.x / C;
    const int b = row_id / P.N, a = row_id % P.N;
    const int tid = threadIdx.x;
    const int SL = P.SL;
    __shared__ Shared S;
    float *ep = (float *)dyn_smem;
    const long long tok0 = (long long)rank * SL;
    const int n = (int)max(0ll, min((long long)SL, (long long)P.V - tok0));
    const double T = (double)(P.T_seq ? __ldg(P.T_seq + b) : P.T);
    if (tid == 0) mbar_init(&S.mbar, 1);
    __syncthreads();
    const void *row = (const unsigned char *)P.z +
                      ((long long)b * P.seq_stride + (long long)a * P.node_stride) * (P.dtype == SPEC_BF16 ? 2 : 4);
    uint32_t tx = stage_row(ep, SL, P.dtype, row, tok0, n, &S.mbar, true);
    if (tid == 0 && tx) mbar_expect_tx(&S.mbar, tx);
    stage_row(ep, SL, P.dtype, row, tok0, n, &S.mbar, false);
    if (tx) {
        int spins = 0;
        while (!mbar_try_wait(&S.mbar, 0) && ++spins < SPIN_MBAR) {}
    }
    __syncthreads();
    bool nan = false;
    float m = warp_max(raw_max(ep, SL, P.dtype, n, nan));
    if ((tid & 31) == 0) S.warp_part[tid >> 5][0] = (double)m;
    int any_nan = __syncthreads_or((int)nan);
    m = -CUDART_INF_F;
    for (int k = 0; k < NWARP; ++k) m = fmaxf(m, (float)S.warp_part[k][0]);
    __syncthreads();
    float s_hi, s_lo;
    split_float(1.4426950408889634 / T, s_hi, s_lo);
    const float ref = (m > -CUDART_INF_F && m < CUDART_INF_F) ? m : 0.f;
    double v[NX];
#pragma unroll
    for (int i = 0; i < NX; ++i) v[i] = 0.0;
    widen_exp(ep, SL, P.dtype, n, ref, -CUDART_INF_F, s_hi, s_lo, v[1], v[2]);
    {
        double red[2] = {v[1], v[2]};
        block_sum<2>(S, red);
        v[1] = red[0]; v[2] = red[1];
    }
    v[0] = (double)m; v[6] = any_nan ? 1.0 : 0.0;
    cluster.sync();                      // peers must be running before their shared memory is written
    cluster_allgather(cluster, S, 0, v, NX);
    double (*X)[NX] = S.xchg[0];
    double mg = -CUDART_INF;
    bool bad = false;
    for (int r = 0; r < C; ++r) { mg = fmax(mg, X[r][0]); bad |= X[r][6] != 0.0; }
    bad |= !(mg > -CUDART_INF && mg < CUDART_INF);
    if (tid < C) {
        double mr = X[tid][0];
        S.scale_p[tid] = (!bad && mr > -CUDART_INF) ? exp((mr - mg) / T) : 0.0;
    }
    __syncthreads();
    double Z = 0.0;
    for (int r = 0; r < C; ++r) Z += S.scale_p[r] * X[r][1];
    const float mul = bad ? 0.f : (float)(S.scale_p[rank] / Z);
    if (P.probs) {
        float *out = P.probs + (long long)row_id * P.V + tok0;
        for (int i = tid; i < n; i += NT) out[i] = ep[i] * mul;
    }
    if (P.stats && rank == 0 && tid == 0) {
        float *st = P.stats + (long long)row_id * 6;
        if (bad) {
            for (int i = 0; i < 6; ++i) st[i] = CUDART_NAN_F;
        } else {
            double h = 0.0;
            for (int r = 0; r < C; ++r) {
                double sp = S.scale_p[r];
                if (sp > 0.0) h -= (sp / Z) * (0.6931471805599453 * X[r][2] + (log(sp) - log(Z)) * X[r][1]);
            }
            st[0] = (float)(mg / T); st[1] = (float)Z; st[2] = (float)P.V;
            st[3] = (float)h; st[4] = (float)(1.0 / Z); st[5] = -CUDART_INF_F;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// spec_sample_bonus: inverse CDF over rows of fp32 weights
// ------------------------------------------------------------------------------------------------
struct BParams {
    int R, V, SL;
    const float *w, *u;
    int *token;
    float *margin;
};

__global__ void __launch_bounds__(NT, 1) spec_bonus_kernel(const BParams P)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int r_id = blockIdx.x / C;
    const int tid = threadIdx.x;
    const int SL = P.SL;
    __shared__ Shared S;
    float *ep = (float *)dyn_smem;
    const long long tok0 = (long long)rank * SL;
    const int n = (int)max(0ll, min((long long)SL, (long long)P.V - tok0));
    if (tid == 0) mbar_init(&S.mbar, 1);
    __syncthreads();
    const float *row = P.w + (long long)r_id * P.V;
    uint32_t tx = stage_row(ep, SL, SPEC_F32, row, tok0, n, &S.mbar, true);
    if (tid == 0 && tx) mbar_expect_tx(&S.mbar, tx);
    stage_row(ep, SL, SPEC_F32, row, tok0, n, &S.mbar, false);
    if (tx) {
        int spins = 0;
        while (!mbar_try_wait(&S.mbar, 0) && ++spins < SPIN_MBAR) {}
    }
    for (int i = n + tid; i < SL; i += NT) ep[i] = 0.f;     // padding carries no weight
    __syncthreads();
    // slice total in the same order the search will use is not required: the search rescans
    double acc = 0.0;
    {
        const float4 *a4 = (const float4 *)ep;
        for (int i = tid; i < (SL >> 2); i += NT) {
            float4 p = a4[i];
            acc += (double)((p.x + p.y) + (p.z + p.w));
        }
    }
    double red[1] = {acc};
    block_sum<1>(S, red);
    cluster.sync();                      // peers must be running before their shared memory is written
    cluster_allgather(cluster, S, 0, red, 1);
    double (*X)[NX] = S.xchg[0];
    double tot = 0.0;
    for (int r = 0; r < C; ++r) tot += X[r][0];
    const double target = (double)__ldg(P.u + r_id) * tot;
    int owner = -1, last_pos = -1;
    double pre = 0.0, tau = 0.0;
    for (int r = 0; r < C; ++r) {
        if (X[r][0] > 0.0) last_pos = r;
        if (owner < 0 && pre + X[r][0] > target) { owner = r; tau = target - pre; }
        if (owner < 0) pre += X[r][0];
    }
    if (owner < 0) { owner = last_pos; tau = CUDART_INF; }
    if (owner < 0) {
        if (rank == 0 && tid == 0) { P.token[r_id] = -1; if (P.margin) P.margin[r_id] = 0.f; }
        return;
    }
    if (owner == rank) {
        double dlo = 0.0, dhi = 0.0;
        int t = slice_inverse_cdf(S, ep, nullptr, SL, 0.f, 0.f, tau, dlo, dhi);
        if (tid == 0) {
            P.token[r_id] = t >= 0 ? (int)(tok0 + t) : -1;
            if (P.margin) P.margin[r_id] = (float)(fmin(dlo, dhi) / tot);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct Plan {
    int C, SL, smem;
};

constexpr int SMEM_BUDGET = 227 * 1024 - (int)sizeof(Shared) - 1024;

bool make_plan(int V, int bytes_per_token, Plan *p)
{
    for (int C = 1; C <= CMAX; C <<= 1) {
        long long sl = ((long long)V + C - 1) / C;
        sl = (sl + 63) / 64 * 64;
        long long need = sl * bytes_per_token;
        if (need <= SMEM_BUDGET) {
            p->C = C; p->SL = (int)sl; p->smem = (int)need;
            return true;
        }
    }
    return false;
}

int check_in(const SpecIn *in, bool need_tree)
{
    if (!in) return SPEC_ERR_NULL;
    if (in->B <= 0 || in->N <= 0 || in->V <= 0 || in->N > SPEC_MAX_NODES) return SPEC_ERR_SHAPE;
    if ((long long)in->B * in->N > (1ll << 24)) return SPEC_ERR_SHAPE;
    if (in->logits_dtype != SPEC_F32 && in->logits_dtype != SPEC_BF16) return SPEC_ERR_DTYPE;
    if (in->node_stride < in->V || in->seq_stride < 0) return SPEC_ERR_SHAPE;
    if (in->topo_seq_stride != 0 && in->topo_seq_stride < in->N) return SPEC_ERR_SHAPE;
    if (!(in->temperature > 0.f) || !(in->temperature < 3.0e38f)) {
        if (!in->temperature_per_seq) return SPEC_ERR_PARAM;
    }
    if (in->top_k < 0 || !(in->top_p > 0.f) || in->top_p > 1.f) return SPEC_ERR_PARAM;
    if (need_tree) {
        if (!in->target_logits || !in->draft_logits || !in->parent || !in->token || !in->u_accept || !in->u_bonus)
            return SPEC_ERR_NULL;
    }
    return SPEC_OK;
}

int64_t workspace_need(const SpecIn *in)
{
    int64_t nodes = (int64_t)in->B * in->N;
    int64_t rec = (nodes * (int64_t)sizeof(NodeRec) + 255) / 256 * 256;
    int64_t pub = (nodes * 8 + 255) / 256 * 256;
    return rec + pub;
}

template <typename K>
int launch_clustered(K kernel, int clusters, const Plan &pl, cudaStream_t st, void *params_ptr)
{
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem);
    if (e != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    if (pl.C > 8) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_UNSUPPORTED; }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)clusters * pl.C, 1, 1);
    cfg.blockDim = dim3(NT, 1, 1);
    cfg.dynamicSmemBytes = (size_t)pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = pl.C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    void *args[1] = {params_ptr};
    e = cudaLaunchKernelExC(&cfg, (const void *)kernel, args);
    if (e != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    return SPEC_OK;
}

int verify_common(const SpecIn *in, const SpecOut *out, void *ws, int64_t ws_bytes, void *stream, int mode)
{
    int rc = check_in(in, true);
    if (rc) return rc;
    if (!out || !out->accepted_node || !out->accept_len || !out->out_tokens || !out->bonus_token || !out->status)
        return SPEC_ERR_NULL;
    if (in->top_k > 0 && in->top_k < in->V) return SPEC_ERR_UNSUPPORTED;
    if (in->top_p < 1.f) return SPEC_ERR_UNSUPPORTED;
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < workspace_need(in)) return SPEC_ERR_WORKSPACE;
    Plan pl;
    if (!make_plan(in->V, 8, &pl)) return SPEC_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t nodes = (int64_t)in->B * in->N;
    NodeRec *rec = (NodeRec *)ws;
    unsigned long long *pub =
        (unsigned long long *)((unsigned char *)ws + (nodes * (int64_t)sizeof(NodeRec) + 255) / 256 * 256);
    if (mode == MODE_TRAVERSAL) {
        if (cudaMemsetAsync(pub, 0xFF, (size_t)nodes * 8, st) != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    }
    KParams kp = {};
    kp.B = in->B; kp.N = in->N; kp.V = in->V; kp.dtype = in->logits_dtype; kp.mode = mode; kp.SL = pl.SL;
    kp.all_thr = (out->node_thr != nullptr || out->margin != nullptr) ? 1 : 0;
    kp.zp = in->target_logits; kp.zq = in->draft_logits;
    kp.seq_stride = in->seq_stride; kp.node_stride = in->node_stride; kp.topo_stride = in->topo_seq_stride;
    kp.parent = in->parent; kp.token = in->token;
    kp.T = in->temperature; kp.T_seq = in->temperature_per_seq; kp.top_k = in->top_k; kp.top_p = in->top_p;
    kp.u_accept = in->u_accept; kp.u_bonus = in->u_bonus;
    kp.rec = rec; kp.w_pub = pub; kp.features = out->node_features;
    rc = launch_clustered(spec_node_kernel, (int)nodes, pl, st, &kp);
    if (rc) return rc;
    FParams fp = {};
    fp.B = in->B; fp.N = in->N; fp.mode = mode; fp.parent = in->parent; fp.token = in->token;
    fp.topo_stride = in->topo_seq_stride; fp.u_accept = in->u_accept; fp.rec = rec; fp.out = *out;
    spec_finalize_kernel<<<(in->B + 63) / 64, 64, 0, st>>>(fp);
    if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    if (out->residual) {
        RParams rp = {};
        rp.B = in->B; rp.N = in->N; rp.V = in->V; rp.dtype = in->logits_dtype;
        rp.zp = in->target_logits; rp.zq = in->draft_logits;
        rp.seq_stride = in->seq_stride; rp.node_stride = in->node_stride;
        rp.T = in->temperature; rp.T_seq = in->temperature_per_seq;
        rp.rec = rec; rp.accepted = out->accepted_node; rp.residual = out->residual;
        int gx = (in->V + 255) / 256;
        if (gx > 296) gx = 296;
        spec_residual_kernel<<<dim3(gx, in->B), 256, 0, st>>>(rp);
        if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    }
    return SPEC_OK;
}


// ------------------------------------------------------------------------------------------------
// host-buffer entry point: staging layout inside the caller's device buffer
// ------------------------------------------------------------------------------------------------
struct HostLayout {
    int64_t zp, zq, parent, token, ua, ub, acc, len, toks, bonus, status, ws, total;
    int64_t logit_bytes, parent_bytes, bn4, b4;
};

inline int64_t up256(int64_t x) { return (x + 255) / 256 * 256; }

HostLayout host_layout(const SpecIn *in)
{
    HostLayout L = {};
    const int64_t esz = in->logits_dtype == SPEC_BF16 ? 2 : 4;
    L.logit_bytes = (int64_t)in->B * in->N * in->V * esz;
    L.parent_bytes = (in->topo_seq_stride ? (int64_t)in->B : 1) * in->N * 4;
    L.bn4 = (int64_t)in->B * in->N * 4;
    L.b4 = (int64_t)in->B * 4;
    int64_t o = 0;
    L.zp = o; o += up256(L.logit_bytes);
    L.zq = o; o += up256(L.logit_bytes);
    L.parent = o; o += up256(L.parent_bytes);
    L.token = o; o += up256(L.bn4);
    L.ua = o; o += up256(L.bn4);
    L.ub = o; o += up256(L.bn4);
    L.acc = o; o += up256(L.b4);
    L.len = o; o += up256(L.b4);
    L.toks = o; o += up256(L.bn4);
    L.bonus = o; o += up256(L.b4);
    L.status = o; o += up256(L.b4);
    L.ws = o; o += up256(workspace_need(in));
    L.total = o;
    return L;
}

}  // namespace

extern "C" {

int32_t spec_workspace_bytes(const SpecIn *in, int64_t *bytes)
{
    if (!in || !bytes) return SPEC_ERR_NULL;
    if (in->B <= 0 || in->N <= 0 || in->N > SPEC_MAX_NODES || (long long)in->B * in->N > (1ll << 24))
        return SPEC_ERR_SHAPE;
    *bytes = workspace_need(in);
    return SPEC_OK;
}

int32_t spec_query_plan(int32_t V, int32_t logits_dtype, int32_t *cluster_size, int32_t *slice_len,
                        int32_t *smem_bytes, int32_t *threads)
{
    if (V <= 0) return SPEC_ERR_SHAPE;
    if (logits_dtype != SPEC_F32 && logits_dtype != SPEC_BF16) return SPEC_ERR_DTYPE;
    Plan pl;
    if (!make_plan(V, 8, &pl)) return SPEC_ERR_UNSUPPORTED;
    if (cluster_size) *cluster_size = pl.C;
    if (slice_len) *slice_len = pl.SL;
    if (smem_bytes) *smem_bytes = pl.smem;
    if (threads) *threads = NT;
    return SPEC_OK;
}

int32_t spec_verify_specinfer(const SpecIn *in, const SpecOut *out, void *ws, int64_t ws_bytes, void *stream)
{
    return verify_common(in, out, ws, ws_bytes, stream, MODE_SPECINFER);
}

int32_t spec_verify_traversal(const SpecIn *in, const SpecOut *out, void *ws, int64_t ws_bytes, void *stream)
{
    return verify_common(in, out, ws, ws_bytes, stream, MODE_TRAVERSAL);
}

int32_t spec_tree_probs(const SpecIn *in, int32_t which, float *probs, float *row_stats, void *ws,
                        int64_t ws_bytes, void *stream)
{
    (void)ws; (void)ws_bytes;
    int rc = check_in(in, false);
    if (rc) return rc;
    if (which != 0 && which != 1) return SPEC_ERR_PARAM;
    const void *z = which ? in->draft_logits : in->target_logits;
    if (!z || (!probs && !row_stats)) return SPEC_ERR_NULL;
    if (in->top_k > 0 && in->top_k < in->V) return SPEC_ERR_UNSUPPORTED;
    if (in->top_p < 1.f) return SPEC_ERR_UNSUPPORTED;
    Plan pl;
    if (!make_plan(in->V, 4, &pl)) return SPEC_ERR_UNSUPPORTED;
    TParams tp = {};
    tp.rows = in->B * in->N; tp.N = in->N; tp.V = in->V; tp.dtype = in->logits_dtype; tp.SL = pl.SL;
    tp.z = z; tp.seq_stride = in->seq_stride; tp.node_stride = in->node_stride;
    tp.T = in->temperature; tp.T_seq = in->temperature_per_seq; tp.probs = probs; tp.stats = row_stats;
    return launch_clustered(spec_probs_kernel, tp.rows, pl, (cudaStream_t)stream, &tp);
}

int32_t spec_sample_bonus(const float *weights, int32_t R, int32_t V, const float *u, int32_t *token,
                          float *margin, void *ws, int64_t ws_bytes, void *stream)
{
    (void)ws; (void)ws_bytes;
    if (!weights || !u || !token) return SPEC_ERR_NULL;
    if (R <= 0 || V <= 0) return SPEC_ERR_SHAPE;
    Plan pl;
    if (!make_plan(V, 4, &pl)) return SPEC_ERR_UNSUPPORTED;
    BParams bp = {R, V, pl.SL, weights, u, token, margin};
    return launch_clustered(spec_bonus_kernel, R, pl, (cudaStream_t)stream, &bp);
}


int32_t spec_host_staging_bytes(const SpecIn *in, int64_t *bytes)
{
    if (!in || !bytes) return SPEC_ERR_NULL;
    int rc = check_in(in, false);
    if (rc) return rc;
    *bytes = host_layout(in).total;
    return SPEC_OK;
}

int32_t spec_verify_host(const SpecIn *in, const SpecOut *out, int32_t algorithm, void *dev_buf,
                         int64_t dev_bytes, void *stream)
{
    int rc = check_in(in, true);
    if (rc) return rc;
    if (!out || !out->accepted_node || !out->accept_len || !out->out_tokens || !out->bonus_token || !out->status)
        return SPEC_ERR_NULL;
    if (out->residual || out->node_thr || out->node_w_in || out->node_features || out->margin)
        return SPEC_ERR_UNSUPPORTED;
    if (algorithm != 0 && algorithm != 1) return SPEC_ERR_PARAM;
    if (in->temperature_per_seq) return SPEC_ERR_UNSUPPORTED;
    if (in->node_stride != in->V || in->seq_stride != (int64_t)in->N * in->V) return SPEC_ERR_SHAPE;
    if (in->topo_seq_stride != 0 && in->topo_seq_stride != in->N) return SPEC_ERR_SHAPE;
    const HostLayout L = host_layout(in);
    if (!dev_buf || ((uintptr_t)dev_buf & 255) || dev_bytes < L.total) return SPEC_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char *d = (unsigned char *)dev_buf;
    bool ok = true;
    ok &= cudaMemcpyAsync(d + L.zp, in->target_logits, (size_t)L.logit_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + L.zq, in->draft_logits, (size_t)L.logit_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + L.parent, in->parent, (size_t)L.parent_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + L.token, in->token, (size_t)L.bn4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + L.ua, in->u_accept, (size_t)L.bn4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + L.ub, in->u_bonus, (size_t)L.bn4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    SpecIn din = *in;
    din.target_logits = d + L.zp; din.draft_logits = d + L.zq;
    din.parent = (const int32_t *)(d + L.parent); din.token = (const int32_t *)(d + L.token);
    din.u_accept = (const float *)(d + L.ua); din.u_bonus = (const float *)(d + L.ub);
    SpecOut dout = {};
    dout.accepted_node = (int32_t *)(d + L.acc); dout.accept_len = (int32_t *)(d + L.len);
    dout.out_tokens = (int32_t *)(d + L.toks); dout.bonus_token = (int32_t *)(d + L.bonus);
    dout.status = (int32_t *)(d + L.status);
    rc = verify_common(&din, &dout, d + L.ws, L.total - L.ws, stream, algorithm == 0 ? MODE_SPECINFER : MODE_TRAVERSAL);
    if (rc) return rc;
    ok &= cudaMemcpyAsync(out->accepted_node, dout.accepted_node, (size_t)L.b4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(out->accept_len, dout.accept_len, (size_t)L.b4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(out->out_tokens, dout.out_tokens, (size_t)L.bn4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(out->bonus_token, dout.bonus_token, (size_t)L.b4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(out->status, dout.status, (size_t)L.b4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (!ok || cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    return SPEC_OK;
}

}  // extern "C"
