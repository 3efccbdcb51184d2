// Streaming row statistics (no truncation): every logit row the verifiers may touch is read once from
// HBM, straight into registers, and reduced to per-slice partial sums of the row's softmax normaliser.
// No residency, no clusters: one CTA per (row, slice of 8192 tokens), 32 logits per thread loaded with
// four 16-byte loads before any arithmetic, so a whole SM keeps more than 100 KB of loads in flight.
//
// A thread turns its logits into e = 2^(z s - o) (s = log2(e)/T, o = ceil of its own largest z s, an
// integer, so partial sums combine by exact powers of two) and the CTA writes, for its slice,
//     O = largest o, S = sum e 2^(o - O), X = sum e x 2^(o - O) with x = z s - O, the largest exponent.
// The walk kernel merges the slices of a row when it needs the row's normaliser.
#pragma once
#include "common.cuh"

namespace specv {

// one slice of one row (stream kernel) or a whole row (row-statistics kernel, one slice per row)
struct __align__(16) RowPart {
    double S;          // sum over kept tokens of 2^(z s - O)
    double X;          // sum over kept tokens of e x, x = z s - O
    int O;             // reference (integer); ROWPART_EMPTY when the slice has no finite logit
    float xmax;        // largest exponent relative to O
    float cut;         // smallest kept logit of the row (-inf: nothing cut)
    int bad;           // 1: NaN or +inf seen; -1: row not read (draft row of a node without children)
};
constexpr int ROWPART_EMPTY = -(1 << 30);

namespace stream {

constexpr int NT = 256;
constexpr int PER = 32;                  // logits per thread
constexpr int SLICE = NT * PER;          // logits per CTA

struct SParams {
    int B, N, V, NSL;
    const void *zp, *zq;
    long long seq_stride, node_stride, topo_stride;
    const int *parent;
    float T;
    const float *T_seq;
    RowPart *part;           // [B*N*2][NSL]
};

template <int DT>
__global__ void __launch_bounds__(NT, 4) spec_row_partial_kernel(const SParams P)
{
    constexpr int ESZ = DT == SPEC_BF16 ? 2 : 4;
    __shared__ double sS[NT / 32], sX[NT / 32], sB[NT / 32];
    __shared__ int sO[NT / 32], sBad[NT / 32];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const long long id = blockIdx.x;
    const int j = (int)(id % P.NSL);
    const long long row2 = id / P.NSL;
    const int which = (int)(row2 & 1);
    const long long row = row2 >> 1;
    const int b = (int)(row / P.N), a = (int)(row % P.N);
    RowPart *out = P.part + row2 * P.NSL + j;
    if (which == 1) {
        // a draft row is read only for nodes that have children
        const int *parent = P.parent + (long long)b * P.topo_stride;
        bool any = false;
        for (int c = a + 1 + tid; c < P.N; c += NT) any |= __ldg(parent + c) == a;
        if (!__syncthreads_or((int)any)) {
            if (tid == 0) { RowPart r = {}; r.O = ROWPART_EMPTY; r.cut = -CUDART_INF_F; r.bad = -1; *out = r; }
            return;
        }
    }
    const int tok0 = j * SLICE;
    const int n = min(SLICE, P.V - tok0);
    const unsigned char *src = (const unsigned char *)(which ? P.zq : P.zp) +
                               ((long long)b * P.seq_stride + (long long)a * P.node_stride + tok0) * ESZ;
    const bool aligned = (((uintptr_t)src) & 15) == 0;

    // ---- 32 logits per thread: chunk c of the thread is tokens (tid + c NT) * 8 ... + 8 -----------------------
    float z[PER];
#pragma unroll
    for (int c = 0; c < PER / 8; ++c) {
        const int t0 = (tid + c * NT) * 8;
        if (aligned && t0 + 8 <= n) {
            if (DT == SPEC_BF16) {
                const uint4 r = __ldg(reinterpret_cast<const uint4 *>(src) + (tid + c * NT));
                z[c * 8 + 0] = bf16_lo(r.x); z[c * 8 + 1] = bf16_hi(r.x); z[c * 8 + 2] = bf16_lo(r.y); z[c * 8 + 3] = bf16_hi(r.y);
                z[c * 8 + 4] = bf16_lo(r.z); z[c * 8 + 5] = bf16_hi(r.z); z[c * 8 + 6] = bf16_lo(r.w); z[c * 8 + 7] = bf16_hi(r.w);
            } else {
                const float4 r0 = __ldg(reinterpret_cast<const float4 *>(src) + 2 * (tid + c * NT));
                const float4 r1 = __ldg(reinterpret_cast<const float4 *>(src) + 2 * (tid + c * NT) + 1);
                z[c * 8 + 0] = r0.x; z[c * 8 + 1] = r0.y; z[c * 8 + 2] = r0.z; z[c * 8 + 3] = r0.w;
                z[c * 8 + 4] = r1.x; z[c * 8 + 5] = r1.y; z[c * 8 + 6] = r1.z; z[c * 8 + 7] = r1.w;
            }
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k)
                z[c * 8 + k] = (t0 + k < n) ? load_logit(src, DT, t0 + k) : -CUDART_INF_F;
        }
    }
    const double s_d = 1.4426950408889634 / (double)(P.T_seq ? __ldg(P.T_seq + b) : P.T);
    float s_hi = (float)s_d;
    if ((double)s_hi > s_d) s_hi = __uint_as_float(__float_as_uint(s_hi) - 1u);
    float s_lo = (float)(s_d - (double)s_hi);
    if (!(s_lo > 0.f)) s_lo = 1.0e-30f;

    float zm = -CUDART_INF_F;
    int bad = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        bad |= (z[k] != z[k]) || (z[k] == CUDART_INF_F);
        zm = fmaxf(zm, z[k]);
    }
    const bool any = zm > -CUDART_INF_F;
    const float of = any ? fminf(fmaxf(ceilf(zm * s_hi), -1.0e9f), 1.0e9f) : 0.f;
    const int o_t = any ? (int)of : ROWPART_EMPTY;
    float sum[4] = {0.f, 0.f, 0.f, 0.f}, sx[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        const float x = fmaxf(fmaf(z[k], s_lo, fmaf(z[k], s_hi, -of)), -200.f);
        const float e = ex2_approx(x);
        sum[k & 3] += e;
        sx[k & 3] = fmaf(e, x, sx[k & 3]);
    }
    const float S_t = (sum[0] + sum[1]) + (sum[2] + sum[3]);
    const float X_t = (sx[0] + sx[1]) + (sx[2] + sx[3]);
    const float xm_t = fmaf(zm, s_lo, fmaf(zm, s_hi, -of));

    // ---- warp, then CTA: merge (reference, sums) pairs by exact powers of two ------------------------------------
    const int O_w = __reduce_max_sync(0xffffffffu, o_t);
    const int d = max(o_t - O_w, -100000);
    const double f = (double)pow2i(max(d, -127));
    const double Sw = warp_sum((double)S_t * f);
    const double Xw = warp_sum(f * ((double)X_t + (double)d * (double)S_t));
    double best = any ? (double)o_t + (double)xm_t : -1.0e300;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = fmax(best, __shfl_xor_sync(0xffffffffu, best, o));
    bad = __any_sync(0xffffffffu, bad);
    if (lane == 0) { sS[w] = Sw; sX[w] = Xw; sB[w] = best; sO[w] = O_w; sBad[w] = bad; }
    __syncthreads();
    if (tid == 0) {
        int O = ROWPART_EMPTY, bd = 0;
        double bst = -1.0e300;
        for (int k = 0; k < NT / 32; ++k) { O = max(O, sO[k]); bd |= sBad[k]; bst = fmax(bst, sB[k]); }
        double S = 0.0, X = 0.0;
        for (int k = 0; k < NT / 32; ++k) {
            const int dk = max(sO[k] - O, -100000);
            const double fk = pow2d(dk);
            S += sS[k] * fk;
            X += fk * (sX[k] + (double)dk * sS[k]);
        }
        RowPart r;
        r.S = S; r.X = X; r.O = O; r.xmax = O > ROWPART_EMPTY ? (float)(bst - (double)O) : 0.f;
        r.cut = -CUDART_INF_F; r.bad = bd;
        *out = r;
    }
}

// Selector features of every node from the row statistics: entropy (nats) and largest probability of
// the target and draft sampling distributions.  One warp per node.
struct FParams {
    long long nodes;
    int NSL;
    const RowPart *part;
    float *features;         // [nodes][4]: H_p, H_q, top1_p, top1_q (q entries 0 for nodes without children)
};

__global__ void spec_features_kernel(const FParams P)
{
    const long long node = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (node >= P.nodes) return;
    float f[4] = {0.f, 0.f, 0.f, 0.f};
    for (int which = 0; which < 2; ++which) {
        const RowPart *p = P.part + (node * 2 + which) * P.NSL;
        int O = ROWPART_EMPTY, bad = 0, unread = 0;
        for (int j = lane; j < P.NSL; j += 32) { O = max(O, p[j].O); bad |= p[j].bad == 1; unread |= p[j].bad == -1; }
        O = __reduce_max_sync(0xffffffffu, O);
        bad = __any_sync(0xffffffffu, bad);
        unread = __any_sync(0xffffffffu, unread);
        double S = 0.0, X = 0.0, best = -1.0e300;
        for (int j = lane; j < P.NSL; j += 32) {
            if (p[j].O > ROWPART_EMPTY) {
                const int d = max(p[j].O - O, -100000);
                const double fk = pow2d(d);
                S += p[j].S * fk;
                X += fk * (p[j].X + (double)d * p[j].S);
                best = fmax(best, (double)p[j].O + (double)p[j].xmax);
            }
        }
        S = warp_sum(S);
        X = warp_sum(X);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = fmax(best, __shfl_xor_sync(0xffffffffu, best, o));
        if (unread) continue;
        if (bad || !(S > 0.0) || !(S < CUDART_INF)) { f[which] = CUDART_NAN_F; f[2 + which] = CUDART_NAN_F; continue; }
        f[which] = (float)(log(S) - 0.6931471805599453 * X / S);
        f[2 + which] = (float)(exp2(best - (double)O) / S);
    }
    if (lane == 0) {
        float *o = P.features + node * 4;
        o[0] = f[0]; o[1] = f[1]; o[2] = f[2]; o[3] = f[3];
    }
}

}  // namespace stream
}  // namespace specv
