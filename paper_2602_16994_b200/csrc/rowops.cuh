// Row kernels of libspecverify: materialised sampling distributions (spec_tree_probs) and the
// stand-alone inverse-CDF draw (spec_sample_bonus).  One cluster per row; each CTA stages its
// vocabulary slice with bulk asynchronous copies and the CTAs combine through distributed shared
// memory.  These are utility entry points; the verification path proper is verify.cuh.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace specv {
namespace rowops {
namespace cg = cooperative_groups;

constexpr int NT = 512;              // threads per CTA
constexpr int NWARP = NT / 32;
constexpr int CMAX = 16;             // CTAs per cluster (16 needs the non-portable attribute)
constexpr int NX = 10;               // doubles per CTA per exchange
constexpr uint32_t BULK_CHUNK = 16384;

__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) { mbar_arrive_expect_tx(bar, bytes); }
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_down_sync(0xffffffffu, v, o));
    return v;
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
    double ctl_d[4];
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
                                          float s_hi, float s_lo, double &sum_e, double &sum_ex, int &kept)
{
    double acc_e = 0.0, acc_x = 0.0;
    int nk = 0;
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
                    nk += keep ? 1 : 0;
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
                nk += keep ? 1 : 0;
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
    kept = nk;
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
    const float *cut;        // optional [rows*2] smallest kept logit (target, draft) of every row
    int which;
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
    if (tid == 0) { mbar_init(&S.mbar, 1); mbar_fence_init(); }
    __syncthreads();
    const void *row = (const unsigned char *)P.z +
                      ((long long)b * P.seq_stride + (long long)a * P.node_stride) * (P.dtype == SPEC_BF16 ? 2 : 4);
    uint32_t tx = stage_row(ep, SL, P.dtype, row, tok0, n, &S.mbar, true);
    if (tid == 0 && tx) mbar_expect_tx(&S.mbar, tx);
    stage_row(ep, SL, P.dtype, row, tok0, n, &S.mbar, false);
    bool gave_up = false;
    if (tx) gave_up = !mbar_wait(&S.mbar, 0);
    __syncthreads();
    bool nan = gave_up;          // a copy that was given up on: the row comes out as a non-finite one
    bool nan2 = false;
    float m = warp_max(raw_max(ep, SL, P.dtype, n, nan2));
    nan = nan || nan2;
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
    const float cutv = P.cut ? __ldg(P.cut + (long long)row_id * 2 + P.which) : -CUDART_INF_F;
    int kept = 0;
    widen_exp(ep, SL, P.dtype, n, ref, cutv, s_hi, s_lo, v[1], v[2], kept);
    {
        double red[3] = {v[1], v[2], (double)kept};
        block_sum<3>(S, red);
        v[1] = red[0]; v[2] = red[1]; v[3] = red[2];
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
            double nkept = 0.0;
            for (int r = 0; r < C; ++r) nkept += X[r][3];
            st[0] = (float)(mg / T); st[1] = (float)Z; st[2] = (float)nkept;
            st[3] = (float)h; st[4] = (float)(1.0 / Z); st[5] = cutv;
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
    if (tid == 0) { mbar_init(&S.mbar, 1); mbar_fence_init(); }
    __syncthreads();
    const float *row = P.w + (long long)r_id * P.V;
    uint32_t tx = stage_row(ep, SL, SPEC_F32, row, tok0, n, &S.mbar, true);
    if (tid == 0 && tx) mbar_expect_tx(&S.mbar, tx);
    stage_row(ep, SL, SPEC_F32, row, tok0, n, &S.mbar, false);
    int gave_up = 0;
    if (tx) gave_up = mbar_wait(&S.mbar, 0) ? 0 : 1;
    for (int i = n + tid; i < SL; i += NT) ep[i] = 0.f;     // padding carries no weight
    // a copy that was given up on: the slice counts as empty (its bytes may still be on their way)
    if (__syncthreads_or(gave_up))
        for (int i = tid; i < SL; i += NT) ep[i] = 0.f;
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


}  // namespace rowops
}  // namespace specv
