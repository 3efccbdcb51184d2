// Row statistics for truncated sampling distributions (top-k / top-p; rules in cut.cuh), fast path.
//
// The nucleus of a row is a few dozen to a few hundred tokens out of 10^5, so the selection need not
// see the vocabulary: one CTA per row reads the row twice -- from HBM for the maximum (and every
// thread's own maximum), then from L2 to collect the CANDIDATES, the tokens at or above a bound that
// is known to lie below the cut, into a list of keys in shared memory -- and runs the radix selection
// (counts for top-k, fixed-point masses for top-p, exactly the arithmetic of rowstat.cuh) on that
// list.  The kept tokens are among the candidates, so the normaliser, the entropy sum and the kept
// count come from the list as well.
//   top-k        bound = the k-th largest of the per-thread maxima (each is a logit of the row, so at
//                least k logits lie at or above it);
//   top-p alone  bound = 14 octaves below the row maximum; the total mass is summed exactly over the
//                whole row in the second read.
// A row whose candidates overflow the list, whose k exceeds what the thread maxima can bound, or whose
// nucleus reaches below the bound is left to the general kernel of rowstat.cuh: it is marked
// (RowPart::bad = ROW_TODO), its id appended to a list in the workspace, and that kernel, launched
// afterwards, takes only the listed rows.
#pragma once
#include "rowstat.cuh"

namespace specv {
namespace trunc {

constexpr int NT = 512;
constexpr int NW = NT / 32;
constexpr int NB = cut::NB;
constexpr int PER = NB / NT;
constexpr int CAP = 4096;            // candidate list capacity
constexpr int ROW_TODO = 2;          // RowPart::bad of a row left to the general kernel
constexpr float WINDOW_OCTAVES = 14.f;

struct __align__(16) Shared {
    unsigned long long hist[NB];
    unsigned long long warp_tot[NW];
    double red[NW][4];
    uint32_t keys[CAP];
    uint32_t tmax[NT];               // keys of the per-thread maxima
    int count;                       // candidates appended (may exceed CAP: overflow)
    int sel_bin, found;
    unsigned long long sel_above;
};

// First bin from the top at which above + running sum reaches target; -1 when the total stays below.
// Same rule as rowstat's cluster-wide selection, for one CTA.
__device__ __forceinline__ int select_bin(Shared &S, double above, double target, unsigned long long &sum_above)
{
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    __syncthreads();                         // the histogram is complete
    unsigned long long loc[PER], lsum = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        loc[k] = S.hist[NB - 1 - (tid * PER + k)];
        lsum += loc[k];
    }
    unsigned long long incl = lsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) S.warp_tot[w] = incl;
    if (tid == 0) { S.found = 0; S.sel_bin = -1; S.sel_above = 0; }
    __syncthreads();
    unsigned long long base = 0;
    for (int k = 0; k < w; ++k) base += S.warp_tot[k];
    unsigned long long run = base + incl - lsum;
    if (above + (double)run < target && above + (double)(run + lsum) >= target) {
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            if (above + (double)run < target && above + (double)(run + loc[k]) >= target) {
                S.sel_bin = NB - 1 - (tid * PER + k);
                S.sel_above = run;
                S.found = 1;
            }
            run += loc[k];
        }
    }
    __syncthreads();
    sum_above = S.sel_above;
    const int r = S.found ? S.sel_bin : -1;
    __syncthreads();
    return r;
}

// Radix selection over `n` keys in shared memory.  MASS false: the key of the need-th largest element
// (need counts elements); MASS true: the key at which the cumulative fixed-point mass of the elements
// with key >= key_min, taken in descending key order, first reaches `need`.  Returns false when the
// elements do not reach `need` at all.
template <int DT, bool MASS>
__device__ __forceinline__ bool select_key(Shared &S, const uint32_t *keys, int n, double need, uint32_t key_min,
                                           float m, float sf, uint32_t &key_out)
{
    constexpr int LEVELS = DT == SPEC_BF16 ? 2 : 3;
    const int tid = threadIdx.x;
    uint32_t prefix = 0, pmask = 0;
    double above = 0.0;
#pragma unroll 1
    for (int lv = 0; lv < LEVELS; ++lv) {
        const int sh = lv == 0 ? 21 : (DT == SPEC_BF16 ? 16 : (lv == 1 ? 10 : 0));
        const uint32_t bm = (1u << (lv == 0 ? 11 : (DT == SPEC_BF16 ? 5 : (lv == 1 ? 11 : 10)))) - 1u;
        for (int i = tid; i < NB; i += NT) S.hist[i] = 0;
        __syncthreads();
        for (int i0 = 0; i0 < n; i0 += NT) {
            const int i = i0 + tid;
            const uint32_t k = i < n ? keys[i] : 0u;
            const bool in = i < n && k >= key_min && (k & pmask) == prefix;
            if (MASS) {
                const float z = cut::value_of(k);
                rowstat::hist_mass(S.hist, in, (int)((k >> sh) & bm),
                                   in ? (unsigned long long)((double)ex2_approx((z - m) * sf) * cut::FIX) : 0ull);
            } else {
                rowstat::hist_count(S.hist, in, (int)((k >> sh) & bm));
            }
        }
        unsigned long long sum_above;
        const int bin = select_bin(S, above, need, sum_above);
        if (bin < 0) return false;
        above += (double)sum_above;
        prefix |= (uint32_t)bin << sh;
        pmask |= bm << sh;
    }
    key_out = prefix;
    if (DT == SPEC_BF16 && !(key_out & 0x80000000u)) key_out |= 0xFFFFu;     // the low half of a bf16 key
    return true;
}

// Visit every logit of a row in global memory, 8 per thread and step when the row is 16-byte aligned.
// Trip counts are the same for all lanes of a warp; OKVAR tells whether the lane's chunk exists.
// BODY sees the chunk as float z8[8] (beyond the row: -inf).
#define SPECV_FOR_CHUNKS(OKVAR, BODY)                                                                        \
    do {                                                                                                     \
        const int nchunk_ = (P.V + 7) >> 3;                                                                  \
        for (int c0_ = 0; c0_ < nchunk_; c0_ += NT) {                                                        \
            const int ci_ = c0_ + tid;                                                                       \
            const bool OKVAR = ci_ < nchunk_;                                                                \
            float z8[8];                                                                                     \
            if (OKVAR && aligned && ci_ * 8 + 8 <= P.V) {                                                    \
                if (DT == SPEC_BF16) {                                                                       \
                    const uint4 r_ = __ldg(reinterpret_cast<const uint4 *>(src) + ci_);                      \
                    z8[0] = bf16_lo(r_.x); z8[1] = bf16_hi(r_.x); z8[2] = bf16_lo(r_.y); z8[3] = bf16_hi(r_.y); \
                    z8[4] = bf16_lo(r_.z); z8[5] = bf16_hi(r_.z); z8[6] = bf16_lo(r_.w); z8[7] = bf16_hi(r_.w); \
                } else {                                                                                     \
                    const float4 a_ = __ldg(reinterpret_cast<const float4 *>(src) + 2 * ci_);                \
                    const float4 b_ = __ldg(reinterpret_cast<const float4 *>(src) + 2 * ci_ + 1);            \
                    z8[0] = a_.x; z8[1] = a_.y; z8[2] = a_.z; z8[3] = a_.w;                                  \
                    z8[4] = b_.x; z8[5] = b_.y; z8[6] = b_.z; z8[7] = b_.w;                                  \
                }                                                                                            \
            } else {                                                                                         \
                _Pragma("unroll") for (int k_ = 0; k_ < 8; ++k_)                                             \
                    z8[k_] = (OKVAR && ci_ * 8 + k_ < P.V) ? load_logit(src, DT, (long long)ci_ * 8 + k_) : -CUDART_INF_F; \
            }                                                                                                \
            BODY                                                                                             \
        }                                                                                                    \
    } while (0)

template <int DT>
__global__ void __launch_bounds__(NT, 2) spec_row_trunc_kernel(const rowstat::RParams P)
{
    constexpr int ESZ = DT == SPEC_BF16 ? 2 : 4;
    __shared__ Shared S;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const long long items = 2ll * P.B * P.N;
    const bool use_k = P.top_k > 0 && P.top_k < P.V, use_p = P.top_p < 1.f;

    for (long long id = blockIdx.x; id < items; id += gridDim.x) {
        const long long row = id >> 1;
        const int which = (int)(id & 1);
        const int b = (int)(row / P.N), a = (int)(row % P.N);
        RowPart *out = P.part + row * 2 + which;
        __syncthreads();                               // the previous row's shared state is no longer read
        if (which == 1) {
            bool any = false;
            if (P.parent) {
                const int *parent = P.parent + (long long)b * P.topo_stride;
                for (int c = a + 1 + tid; c < P.N; c += NT) any |= __ldg(parent + c) == a;
            }
            if (!__syncthreads_or((int)any)) {        // a draft row is read only for nodes with children
                if (tid == 0) {
                    RowPart r = {};
                    r.cut = -CUDART_INF_F; r.O = ROWPART_EMPTY; r.bad = -1;
                    *out = r;
                    P.cut[row * 2 + 1] = -CUDART_INF_F;
                }
                continue;
            }
        }
        const unsigned char *src = (const unsigned char *)(which ? P.zq : P.zp) +
                                   ((long long)b * P.seq_stride + (long long)a * P.node_stride) * ESZ;
        const bool aligned = (((uintptr_t)src) & 15) == 0;
        const float Tf = P.T_seq ? __ldg(P.T_seq + b) : P.T;
        const float sf = 1.4426950408889634f / Tf;
        const double s_d = 1.4426950408889634 / (double)Tf;

        // ---- first read (HBM): the row maximum, every thread's own maximum, NaN / +inf ------------------
        float mt = -CUDART_INF_F;
        int bad = 0;
        SPECV_FOR_CHUNKS(ok, {
            float m8 = z8[0];
#pragma unroll
            for (int k = 0; k < 8; ++k) { bad |= (z8[k] != z8[k]) || (z8[k] == CUDART_INF_F); m8 = fmaxf(m8, z8[k]); }
            mt = fmaxf(mt, m8);
        });
        float m;
        {
            float wm = mt;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
            if (lane == 0) S.red[w][0] = (double)wm;
            S.tmax[tid] = cut::key_of(mt);
            if (tid == 0) S.count = 0;
            bad = __syncthreads_or(bad);
            double mm = -CUDART_INF;
            for (int k = 0; k < NW; ++k) mm = fmax(mm, S.red[k][0]);
            m = (float)mm;
            bad = bad || !(mm > -CUDART_INF);
        }
        if (bad) {
            if (tid == 0) {
                RowPart r = {};
                r.cut = -CUDART_INF_F; r.O = ROWPART_EMPTY; r.bad = 1;
                *out = r;
                P.cut[row * 2 + which] = -CUDART_INF_F;
            }
            continue;
        }

        // ---- the bound below which no kept token lies ----------------------------------------------------------
        bool todo = false;
        uint32_t key_lo = 0u;
        if (use_k) {
            // the k-th largest of the per-thread maxima (threads without a finite logit hold key_of(-inf))
            if (P.top_k <= NT / 4) todo = !select_key<DT, false>(S, S.tmax, NT, (double)P.top_k, 0u, m, sf, key_lo);
            else todo = true;
        } else {
            key_lo = cut::key_of(m - WINDOW_OCTAVES / sf);
        }
        const float z_lo = cut::value_of(key_lo);

        // ---- second read (L2): the candidates; for top-p alone also the exact mass of the whole row ------------
        unsigned long long tot_fix = 0;
        if (!todo) {
            const bool want_total = use_p && !use_k;
            unsigned long long part = 0;
            SPECV_FOR_CHUNKS(ok, {
                float m8 = z8[0];
#pragma unroll
                for (int k = 1; k < 8; ++k) m8 = fmaxf(m8, z8[k]);
                if (want_total) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (z8[k] > -CUDART_INF_F) part += (unsigned long long)((double)ex2_approx((z8[k] - m) * sf) * cut::FIX);
                }
                if (__any_sync(0xffffffffu, ok && m8 >= z_lo)) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const bool in = ok && z8[k] >= z_lo;
                        const unsigned bal = __ballot_sync(0xffffffffu, in);
                        if (bal) {
                            int base = 0;
                            if (lane == 0) base = atomicAdd(&S.count, __popc(bal));
                            base = __shfl_sync(0xffffffffu, base, 0);
                            const int pos = base + __popc(bal & ((1u << lane) - 1u));
                            if (in && pos < CAP) S.keys[pos] = cut::key_of(z8[k]);
                        }
                    }
                }
            });
            if (want_total) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                if (lane == 0) S.warp_tot[w] = part;
            }
            __syncthreads();
            if (want_total)
                for (int k = 0; k < NW; ++k) tot_fix += S.warp_tot[k];
            if (S.count > CAP) todo = true;
            __syncthreads();
        }
        const int n_c = todo ? 0 : S.count;

        // ---- selection on the list ---------------------------------------------------------------------------------
        uint32_t key_cut = 0u;
        if (!todo && use_k) {
            // at least k logits lie at or above the bound, so the k-th largest is in the list
            todo = !select_key<DT, false>(S, S.keys, n_c, (double)P.top_k, 0u, m, sf, key_cut);
        }
        if (!todo && use_p) {
            const uint32_t key_k = key_cut;              // the set: key >= key_k (0: the whole row)
            if (use_k) {
                // the set's mass, exactly: its tokens are all in the list
                unsigned long long part = 0;
                for (int i = tid; i < n_c; i += NT) {
                    const uint32_t k = S.keys[i];
                    if (k >= key_k) part += (unsigned long long)((double)ex2_approx((cut::value_of(k) - m) * sf) * cut::FIX);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                __syncthreads();
                if (lane == 0) S.warp_tot[w] = part;
                __syncthreads();
                tot_fix = 0;
                for (int k = 0; k < NW; ++k) tot_fix += S.warp_tot[k];
                __syncthreads();
            }
            const double target = (double)P.top_p * (double)tot_fix;
            uint32_t key_p = 0u;
            if (select_key<DT, true>(S, S.keys, n_c, target, key_k, m, sf, key_p)) key_cut = key_p;
            else if (!use_k) todo = true;                // the nucleus reaches below the window
            // with top-k: the set itself does not reach the target (rounding): the whole set is kept
        }
        if (todo || key_cut == 0u) {
            // left to the general kernel (key_cut = 0 would mean that nothing is cut, which the rules
            // above never produce from a list)
            if (tid == 0) {
                RowPart r = {};
                r.cut = -CUDART_INF_F; r.O = ROWPART_EMPTY; r.bad = ROW_TODO;
                *out = r;
                const int pos = atomicAdd(P.todo, 1);
                P.todo[1 + pos] = (int)id;
            }
            continue;
        }
        const float cutv = cut::value_of(key_cut);

        // ---- normaliser, entropy sum over the kept tokens: they are all in the list -------------------------
        const double Od = ceil((double)m * s_d);
        const float of = (float)fmin(fmax(Od, -1.0e9), 1.0e9);
        float s_hi = (float)s_d;
        if ((double)s_hi > s_d) s_hi = __uint_as_float(__float_as_uint(s_hi) - 1u);
        float s_lo = (float)(s_d - (double)s_hi);
        if (!(s_lo > 0.f)) s_lo = 1.0e-30f;
        double v[4] = {0.0, 0.0, 0.0, 0.0};
        for (int i = tid; i < n_c; i += NT) {
            const uint32_t k = S.keys[i];
            if (k >= key_cut) {
                const float z = cut::value_of(k);
                const float x = fmaxf(fmaf(z, s_lo, fmaf(z, s_hi, -of)), -200.f);
                const float e = ex2_approx(x);
                v[0] += (double)e;
                v[1] += (double)e * (double)x;
                v[2] += 1.0;
            }
        }
#pragma unroll
        for (int k = 0; k < 3; ++k) v[k] = warp_sum(v[k]);
        __syncthreads();
        if (lane == 0) { S.red[w][0] = v[0]; S.red[w][1] = v[1]; S.red[w][2] = v[2]; }
        __syncthreads();
        if (tid == 0) {
            double Z = 0.0, X = 0.0;
            for (int k = 0; k < NW; ++k) { Z += S.red[k][0]; X += S.red[k][1]; }
            RowPart r;
            r.S = Z; r.X = X; r.O = (int)of; r.cut = cutv;
            r.xmax = (float)((double)m * s_d - (double)of);
            r.bad = 0;
            *out = r;
            P.cut[row * 2 + which] = cutv;
        }
    }
}
#undef SPECV_FOR_CHUNKS

}  // namespace trunc
}  // namespace specv
