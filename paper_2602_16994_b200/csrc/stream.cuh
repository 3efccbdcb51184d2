// Streaming row statistics (no truncation): every logit row the verifiers may touch is read once from
// HBM, straight into registers, and reduced to per-slice partial sums of the row's softmax normaliser.
// No residency, no clusters: a CTA streams a row (or a part of it) in slices of 8192 logits, 32 per thread,
// the asynchronous copies of the next slices in flight while the current one is exponentiated.
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
constexpr int ROW_TIMEOUT = 3;          // RowPart::bad of a row whose copy into shared memory was given up on

namespace stream {

constexpr int NT = 256;
constexpr int PER = 32;                  // logits per thread
constexpr int SLICE = NT * PER;          // logits per CTA

struct SParams {
    int B, N, V, NSL;        // NSL: parts a row is split into (more CTAs than rows)
    const void *zp, *zq;
    long long seq_stride, node_stride, topo_stride;
    const int *parent;
    float T;
    const float *T_seq;
    RowPart *part;           // [B*N*2][NSL]
    // optional (every-node verification follows): the per-node weight slots and the per-sequence accepted-node
    // slots are set to pending, the arrival counters and the item counter to zero here, which saves the memset
    // nodes of a call
    unsigned long long *w_pub;   // [B*N]
    unsigned int *done;          // [B]
    int *fin;                    // [B] set to -1 (no accepted node selected yet)
    unsigned int *best;          // [B] set to all-ones (no acceptance known yet)
    unsigned long long *order;   // [B*N] set to 0 (post-order table not computed yet)
    unsigned int *ticket;        // [1] item counter of the every-node kernel
};

// depth of the per-thread staging ring and its size
template <int DT> struct Ring {
    static constexpr int NV = DT == SPEC_BF16 ? 1 : 2;         // 16-byte units per chunk of 8 logits
    static constexpr int UNITS = (PER / 8) * NV;               // 16-byte units per thread and slice
    static constexpr int DEPTH = DT == SPEC_BF16 ? 5 : 3;
    static constexpr int BYTES = DEPTH * UNITS * NT * 16;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// One CTA per (row, part of the row).  The part's slices of 8192 logits are streamed one after the
// other; every thread stages its own 32 logits of the next DEPTH - 1 slices in shared memory with
// asynchronous 16-byte copies (a thread reads back only what it copied itself, so the ring needs no
// barrier) and keeps a running (reference, sum) pair, rescaled by an exact power of two when a later
// slice raises its reference.  The CTA reduces once per part.
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));     // a NaN operand yields the other one
    return d;
}

// FEAT: also accumulate X (needed only by the entropy features).  Without it a NaN or +inf logit is
// found from the sum itself (such a logit makes its e, and so the thread's sum, non-finite), which
// keeps comparisons out of the inner loop.
template <int DT, bool FEAT>
__global__ void __launch_bounds__(NT, 2) spec_row_partial_kernel(const SParams P)
{
    constexpr int ESZ = DT == SPEC_BF16 ? 2 : 4;
    constexpr int NV = Ring<DT>::NV, UNITS = Ring<DT>::UNITS, DEPTH = Ring<DT>::DEPTH;
    __shared__ double sS[NT / 32], sX[NT / 32], sB[NT / 32];
    __shared__ int sO[NT / 32], sBad[NT / 32];
    uint4 *ring = reinterpret_cast<uint4 *>(dyn_smem);            // [DEPTH][UNITS][NT]
    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const long long items = 2ll * P.B * P.N * P.NSL;
    const int slices_row = (P.V + SLICE - 1) / SLICE;
    const int slices_part = (slices_row + P.NSL - 1) / P.NSL;
    grid_launch_dependents();     // a dependent verifier's CTAs may take the places of CTAs that have finished

    for (long long id = blockIdx.x; id < items; id += gridDim.x) {
        const int h = (int)(id % P.NSL);
        const long long row2 = id / P.NSL;
        const int which = (int)(row2 & 1);
        const long long row = row2 >> 1;
        const int b = (int)(row / P.N), a = (int)(row % P.N);
        RowPart *out = P.part + row2 * P.NSL + h;
        if (P.w_pub && which == 0 && h == 0 && tid == 0) {
            P.w_pub[row] = W_PENDING;
            P.order[row] = 0ull;
            if (a == 0) { P.done[b] = 0u; P.fin[b] = -1; P.best[b] = 0xFFFFFFFFu; }
            if (row == 0) *P.ticket = 0u;
        }
        if (which == 1) {
            // a draft row is read only for nodes that have children (every warp finds out by itself)
            const int *parent = P.parent + (long long)b * P.topo_stride;
            bool any = false;
            for (int c0 = a + 1; c0 < P.N && !any; c0 += 32) {
                const int c = c0 + lane;
                any = __any_sync(0xffffffffu, c < P.N && __ldg(parent + c) == a);
            }
            if (!any) {
                if (tid == 0) { RowPart r = {}; r.O = ROWPART_EMPTY; r.cut = -CUDART_INF_F; r.bad = -1; *out = r; }
                continue;
            }
        }
        const unsigned char *rowp = (const unsigned char *)(which ? P.zq : P.zp) +
                                    ((long long)b * P.seq_stride + (long long)a * P.node_stride) * ESZ;
        const bool aligned = (((uintptr_t)rowp) & 15) == 0;
        const int s_begin = h * slices_part, s_end = min(slices_row, s_begin + slices_part);
        const double s_d = 1.4426950408889634 / (double)(P.T_seq ? __ldg(P.T_seq + b) : P.T);
        float s_hi = (float)s_d;
        if ((double)s_hi > s_d) s_hi = __uint_as_float(__float_as_uint(s_hi) - 1u);
        float s_lo = (float)(s_d - (double)s_hi);
        if (!(s_lo > 0.f)) s_lo = 1.0e-30f;

        // the thread's running state
        float of = 0.f, S_t = 0.f, X_t = 0.f, xm_t = -CUDART_INF_F;
        bool set = false;
        int bad = 0;

        // a slice's maximum moves the thread's reference up by an exact power of two
        auto new_reference = [&](float zm) {
            bad |= zm == CUDART_INF_F;
            if (zm > -CUDART_INF_F) {
                const float onew = fminf(fmaxf(ceilf(zm * s_hi), -1.0e9f), 1.0e9f);
                if (!set) { of = onew; set = true; }
                else if (onew > of) {
                    const float dlt = of - onew;
                    const float f = pow2i((int)fmaxf(dlt, -127.f));
                    X_t = f * fmaf(dlt, S_t, X_t);
                    S_t *= f;
                    xm_t += dlt;
                    of = onew;
                }
                if (FEAT) xm_t = fmaxf(xm_t, fmaf(zm, s_lo, fmaf(zm, s_hi, -of)));
            }
        };
        // 8 logits into the sums
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f, b0 = 0.f, b1 = 0.f;
        auto add8 = [&](const float (&z)[8]) {
            if (FEAT) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float x = fmaxf(fmaf(z[k], s_lo, fmaf(z[k], s_hi, -of)), -200.f);
                    bad |= z[k] != z[k];
                    const float e = ex2_approx(x);
                    if (k & 1) { a1 += e; b1 = fmaf(e, x, b1); } else { a0 += e; b0 = fmaf(e, x, b0); }
                }
            } else {
                // two logits per instruction: the exponents z s - of and the running sums as fp32 pairs
                // (each half is the same IEEE operation as the scalar form)
                const unsigned long long sh2 = pack_f32x2(s_hi, s_hi), sl2 = pack_f32x2(s_lo, s_lo), no2 = pack_f32x2(-of, -of);
                unsigned long long acc01 = pack_f32x2(a0, a1), acc23 = pack_f32x2(a2, a3);
#pragma unroll
                for (int k = 0; k < 8; k += 2) {
                    const unsigned long long z2 = pack_f32x2(z[k], z[k + 1]);
                    const unsigned long long x2 = fma_f32x2(z2, sl2, fma_f32x2(z2, sh2, no2));
                    float x0, x1;
                    unpack_f32x2(x2, x0, x1);
                    const unsigned long long e2 = pack_f32x2(ex2_approx(x0), ex2_approx(x1));
                    if (k & 2) acc23 = add_f32x2(acc23, e2); else acc01 = add_f32x2(acc01, e2);
                }
                unpack_f32x2(acc01, a0, a1);
                unpack_f32x2(acc23, a2, a3);
            }
        };
        auto flush = [&]() {
            S_t += (a0 + a1) + (a2 + a3);
            X_t += b0 + b1;
            a0 = a1 = a2 = a3 = b0 = b1 = 0.f;
        };

        // ---- whole slices of an aligned row go through the ring ------------------------------------------------
        const int tok_end = min(P.V, s_end * SLICE);                       // first token past this part
        const int nfull = aligned ? max(0, (tok_end - s_begin * SLICE) / SLICE) : 0;
        {
            const unsigned char *src = rowp + (size_t)s_begin * SLICE * ESZ + (size_t)tid * 16 * NV;
            const uint32_t dst0 = ring_s + (uint32_t)tid * 16u;
            int isl = 0, ist = 0, cst = 0;
            auto issue = [&]() {
                if (isl < nfull) {
#pragma unroll
                    for (int c = 0; c < PER / 8; ++c)
#pragma unroll
                        for (int k = 0; k < NV; ++k)
                            cp_async16(dst0 + (uint32_t)((ist * UNITS + c * NV + k) * NT) * 16u, src + (size_t)c * NT * 16 * NV + k * 16, 16);
                    src += (size_t)SLICE * ESZ;
                    ++isl;
                    ist = ist + 1 == DEPTH ? 0 : ist + 1;
                }
                cp_async_commit();
            };
#pragma unroll
            for (int k = 0; k < DEPTH - 1; ++k) issue();
            // ---- the ragged end of the part (and every slice of a misaligned row) by plain loads, while the ring fills
            for (int t_base = (s_begin + nfull) * SLICE; t_base < tok_end; t_base += SLICE) {
                const int n = min(SLICE, tok_end - t_base);
                const unsigned char *src = rowp + (size_t)t_base * ESZ;
                float z[PER];
#pragma unroll
                for (int c = 0; c < PER / 8; ++c) {
                    const int t0 = (tid + c * NT) * 8;
                    if (aligned && t0 + 8 <= n) {
                        const uint4 *s4 = reinterpret_cast<const uint4 *>(src) + (size_t)(tid + c * NT) * NV;
                        if (DT == SPEC_BF16) {
                            const uint4 r = __ldg(s4);
                            z[c * 8 + 0] = bf16_lo(r.x); z[c * 8 + 1] = bf16_hi(r.x); z[c * 8 + 2] = bf16_lo(r.y); z[c * 8 + 3] = bf16_hi(r.y);
                            z[c * 8 + 4] = bf16_lo(r.z); z[c * 8 + 5] = bf16_hi(r.z); z[c * 8 + 6] = bf16_lo(r.w); z[c * 8 + 7] = bf16_hi(r.w);
                        } else {
                            const uint4 r0 = __ldg(s4), r1 = __ldg(s4 + NV - 1);
                            z[c * 8 + 0] = __uint_as_float(r0.x); z[c * 8 + 1] = __uint_as_float(r0.y); z[c * 8 + 2] = __uint_as_float(r0.z); z[c * 8 + 3] = __uint_as_float(r0.w);
                            z[c * 8 + 4] = __uint_as_float(r1.x); z[c * 8 + 5] = __uint_as_float(r1.y); z[c * 8 + 6] = __uint_as_float(r1.z); z[c * 8 + 7] = __uint_as_float(r1.w);
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < 8; ++k) z[c * 8 + k] = (t0 + k < n) ? load_logit(src, DT, t0 + k) : -CUDART_INF_F;
                    }
                }
                float zm = -CUDART_INF_F;
#pragma unroll
                for (int k = 0; k < PER; ++k) zm = fmaxf(zm, z[k]);
                new_reference(zm);
#pragma unroll
                for (int c = 0; c < PER / 8; ++c) {
                    float z8[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) z8[k] = z[c * 8 + k];
                    add8(z8);
                }
                flush();
            }
            for (int sl = 0; sl < nfull; ++sl) {
                cp_async_wait<DEPTH - 2>();
                const uint4 *st = ring + (size_t)cst * UNITS * NT + tid;
                uint4 raw[UNITS];
#pragma unroll
                for (int u = 0; u < UNITS; ++u) raw[u] = st[u * NT];
                cst = cst + 1 == DEPTH ? 0 : cst + 1;
                issue();                                  // the stage read in the previous iteration is free again
                float zm;
                if (DT == SPEC_BF16) {
                    uint32_t m2 = 0xFF80FF80u;            // the slice maximum on packed pairs
#pragma unroll
                    for (int u = 0; u < UNITS; ++u)
                        m2 = max_bf16x2(m2, max_bf16x2(max_bf16x2(raw[u].x, raw[u].y), max_bf16x2(raw[u].z, raw[u].w)));
                    zm = fmaxf(bf16_lo(m2), bf16_hi(m2));
                } else {
                    zm = -CUDART_INF_F;
#pragma unroll
                    for (int u = 0; u < UNITS; ++u)
                        zm = fmaxf(zm, fmaxf(fmaxf(__uint_as_float(raw[u].x), __uint_as_float(raw[u].y)),
                                             fmaxf(__uint_as_float(raw[u].z), __uint_as_float(raw[u].w))));
                }
                new_reference(zm);
#pragma unroll
                for (int c = 0; c < PER / 8; ++c) {
                    float z[8];
                    if (DT == SPEC_BF16) {
                        const uint4 r = raw[c];
                        z[0] = bf16_lo(r.x); z[1] = bf16_hi(r.x); z[2] = bf16_lo(r.y); z[3] = bf16_hi(r.y);
                        z[4] = bf16_lo(r.z); z[5] = bf16_hi(r.z); z[6] = bf16_lo(r.w); z[7] = bf16_hi(r.w);
                    } else {
                        const uint4 r0 = raw[c * NV], r1 = raw[c * NV + NV - 1];
                        z[0] = __uint_as_float(r0.x); z[1] = __uint_as_float(r0.y); z[2] = __uint_as_float(r0.z); z[3] = __uint_as_float(r0.w);
                        z[4] = __uint_as_float(r1.x); z[5] = __uint_as_float(r1.y); z[6] = __uint_as_float(r1.z); z[7] = __uint_as_float(r1.w);
                    }
                    add8(z);
                }
                flush();
            }
            cp_async_wait<0>();
        }
        // a NaN logit leaves a NaN in the sum; +inf was seen in the maximum
        bad |= !(fabsf(S_t) <= 3.0e38f);
        const int o_t = set ? (int)of : ROWPART_EMPTY;

        // ---- warp, then CTA: merge (reference, sums) pairs by exact powers of two --------------------------------
        const int O_w = __reduce_max_sync(0xffffffffu, o_t);
        const int d = max(o_t - O_w, -100000);
        const double f = (double)pow2i(max(d, -127));
        const double Sw = warp_sum((double)S_t * f);
        double Xw = 0.0, best = -1.0e300;
        if (FEAT) {
            Xw = warp_sum(f * ((double)X_t + (double)d * (double)S_t));
            best = set ? (double)o_t + (double)xm_t : -1.0e300;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best = fmax(best, __shfl_xor_sync(0xffffffffu, best, o));
        }
        bad = __any_sync(0xffffffffu, bad);
        __syncthreads();             // the previous item's partials have been read
        if (lane == 0) { sS[w] = Sw; sX[w] = Xw; sB[w] = best; sO[w] = O_w; sBad[w] = bad; }
        __syncthreads();
        if (w == 0) {
            // the warps' partials, one per lane
            const bool has = lane < NT / 32;
            const int Ok = has ? sO[lane] : ROWPART_EMPTY;
            const int O = __reduce_max_sync(0xffffffffu, Ok);
            const int dk = max(Ok - O, -100000);
            const double fk = pow2d(dk), Sk = has ? sS[lane] : 0.0;
            double S = Sk * fk, X = has ? fk * (sX[lane] + (double)dk * Sk) : 0.0, bst = has ? sB[lane] : -1.0e300;
#pragma unroll
            for (int o = (NT / 64); o > 0; o >>= 1) {
                S += __shfl_xor_sync(0xffffffffu, S, o);
                X += __shfl_xor_sync(0xffffffffu, X, o);
                bst = fmax(bst, __shfl_xor_sync(0xffffffffu, bst, o));
            }
            const int bd = __any_sync(0xffffffffu, has && sBad[lane]);
            if (lane == 0) {
                RowPart r;
                r.S = S; r.X = X; r.O = O; r.xmax = (FEAT && O > ROWPART_EMPTY) ? (float)(bst - (double)O) : 0.f;
                r.cut = -CUDART_INF_F; r.bad = bd;
                *out = r;
            }
        }
    }
}

// Merge the slices of every row into one record (slice 0 of the merged array): one warp per row.
struct MParams {
    long long rows2;
    int NSL;
    const RowPart *part;     // [rows2][NSL]
    RowPart *merged;         // [rows2]
};

__global__ void spec_row_merge_kernel(const MParams P)
{
    const long long r2 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (r2 >= P.rows2) return;
    const RowPart *p = P.part + r2 * P.NSL;
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
    if (lane == 0) {
        RowPart r;
        r.S = S; r.X = X; r.O = O; r.xmax = O > ROWPART_EMPTY ? (float)(best - (double)O) : 0.f;
        r.cut = -CUDART_INF_F;
        r.bad = unread ? -1 : ((bad || !(S > 0.0) || !(S < CUDART_INF)) ? 1 : 0);
        P.merged[r2] = r;
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
