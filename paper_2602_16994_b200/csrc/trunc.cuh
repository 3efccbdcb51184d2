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
//   top-p alone  bound = 14 octaves below the row maximum; the mass of the whole row, which fixes the
//                target, is summed in the first read (fp32 sums of 8, fp64 above).
// bf16 rows need no list: a bf16 logit has 16 significant key bits, the candidates' values are at most
// 2048 consecutive keys below the maximum's, and a histogram of counts over those values is enough
// for both rules and for the kept sums.
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

// e 2^44 truncated to an integer, for e = 2^x in [0, 2): integer arithmetic on the bits of the float
// (the same value as casting the exact product (double)e * 2^44 to an unsigned integer)
__device__ __forceinline__ unsigned long long fix44(float e)
{
    const uint32_t u = __float_as_uint(e);
    const int ex = (int)(u >> 23) & 0xFF;
    if (ex == 0) return 0ull;                                    // zero (subnormals are flushed by ex2.approx.ftz)
    const unsigned long long mant = (unsigned long long)((u & 0x7FFFFFu) | 0x800000u);
    const int sh = ex - 127 - 23 + 44;                           // e = mant 2^(ex - 127 - 23)
    return sh >= 0 ? mant << sh : (sh > -64 ? mant >> (-sh) : 0ull);
}

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

// Thread t holds PER consecutive bins in loc (bin t * PER + k).  First bin at which the running sum
// reaches target, -1 when the total stays below; with frac >= 0 the target is frac times the total.
// sum_before: the sum of the bins before the one found; total: the sum of all bins.
__device__ __forceinline__ int scan_find(Shared &S, const unsigned long long (&loc)[PER], double target, double frac,
                                         unsigned long long &sum_before, unsigned long long &total)
{
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    unsigned long long lsum = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) lsum += loc[k];
    unsigned long long incl = lsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) S.warp_tot[w] = incl;
    if (tid == 0) { S.found = 0; S.sel_bin = -1; S.sel_above = 0; }
    __syncthreads();
    unsigned long long base = 0, tot = 0;
    for (int k = 0; k < NW; ++k) { if (k < w) base += S.warp_tot[k]; tot += S.warp_tot[k]; }
    if (frac >= 0.0) target = frac * (double)tot;
    unsigned long long run = base + incl - lsum;
    if ((double)run < target && (double)(run + lsum) >= target) {
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            if ((double)run < target && (double)(run + loc[k]) >= target) {
                S.sel_bin = tid * PER + k;
                S.sel_above = run;
                S.found = 1;
            }
            run += loc[k];
        }
    }
    __syncthreads();
    sum_before = S.sel_above;
    total = tot;
    return S.found ? S.sel_bin : -1;
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
                                   in ? fix44(ex2_approx((z - m) * sf)) : 0ull);
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

// Visit every logit of a row in global memory in chunks of 8 (16-byte loads where the row is 16-byte
// aligned and the chunk lies inside it).  Four chunks per thread and step, all their loads issued before
// any is used.  Trip counts are the same for all lanes of a warp; OKVAR tells whether the lane's chunk
// exists.  BODY sees the chunk as float z8[8] (beyond the row: -inf).
#define SPECV_FOR_CHUNKS(OKVAR, BODY)                                                                        \
    do {                                                                                                     \
        constexpr int UN_ = (DT == SPEC_BF16 && !TOTAL) ? 4 : 2;                                                                               \
        constexpr int NV_ = DT == SPEC_BF16 ? 1 : 2;                                                         \
        const int nchunk_ = (P.V + 7) >> 3;                                                                  \
        for (int c0_ = 0; c0_ < nchunk_; c0_ += NT * UN_) {                                                  \
            uint4 raw_[UN_ * NV_];                                                                           \
            _Pragma("unroll") for (int u_ = 0; u_ < UN_; ++u_) {                                             \
                const int ci_ = c0_ + u_ * NT + tid;                                                         \
                if (aligned && ci_ * 8 + 8 <= P.V) {                                                         \
                    _Pragma("unroll") for (int v_ = 0; v_ < NV_; ++v_)                                       \
                        raw_[u_ * NV_ + v_] = __ldg(reinterpret_cast<const uint4 *>(src) + (size_t)ci_ * NV_ + v_); \
                }                                                                                            \
            }                                                                                                \
            _Pragma("unroll") for (int u_ = 0; u_ < UN_; ++u_) {                                             \
                const int ci_ = c0_ + u_ * NT + tid;                                                         \
                const bool OKVAR = ci_ < nchunk_;                                                            \
                float z8[8];                                                                                 \
                if (aligned && ci_ * 8 + 8 <= P.V) {                                                         \
                    if (DT == SPEC_BF16) {                                                                   \
                        const uint4 r_ = raw_[u_ * NV_];                                                     \
                        z8[0] = bf16_lo(r_.x); z8[1] = bf16_hi(r_.x); z8[2] = bf16_lo(r_.y); z8[3] = bf16_hi(r_.y); \
                        z8[4] = bf16_lo(r_.z); z8[5] = bf16_hi(r_.z); z8[6] = bf16_lo(r_.w); z8[7] = bf16_hi(r_.w); \
                    } else {                                                                                 \
                        const uint4 a_ = raw_[u_ * NV_], b_ = raw_[u_ * NV_ + NV_ - 1];                      \
                        z8[0] = __uint_as_float(a_.x); z8[1] = __uint_as_float(a_.y); z8[2] = __uint_as_float(a_.z); z8[3] = __uint_as_float(a_.w); \
                        z8[4] = __uint_as_float(b_.x); z8[5] = __uint_as_float(b_.y); z8[6] = __uint_as_float(b_.z); z8[7] = __uint_as_float(b_.w); \
                    }                                                                                        \
                } else {                                                                                     \
                    _Pragma("unroll") for (int k_ = 0; k_ < 8; ++k_)                                         \
                        z8[k_] = (OKVAR && ci_ * 8 + k_ < P.V) ? load_logit(src, DT, (long long)ci_ * 8 + k_) : -CUDART_INF_F; \
                }                                                                                            \
                BODY                                                                                         \
            }                                                                                                \
        }                                                                                                    \
    } while (0)

// TOTAL: top-p without top-k (the first read also sums the mass of the whole row)
template <int DT, bool TOTAL>
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

        float s_hi = (float)s_d;
        if ((double)s_hi > s_d) s_hi = __uint_as_float(__float_as_uint(s_hi) - 1u);
        float s_lo = (float)(s_d - (double)s_hi);
        if (!(s_lo > 0.f)) s_lo = 1.0e-30f;
        constexpr bool want_total = TOTAL;

        // ---- first read (HBM): the row maximum, every thread's own maximum, NaN / +inf; for top-p alone
        // also the mass of the whole row, as in the streaming statistics kernel: a running integer
        // reference per thread, fp32 sums of 8, fp64 above (the total fixes the target, top_p times it,
        // to about 1e-7 relative; the candidates' own masses stay exact)
        float mt = -CUDART_INF_F;
        int bad = 0;
        float of_t = 0.f;
        double Sd = 0.0;
        bool set = false;
        SPECV_FOR_CHUNKS(ok, {
            float m8 = z8[0];
#pragma unroll
            for (int k = 0; k < 8; ++k) { bad |= (z8[k] != z8[k]) || (z8[k] == CUDART_INF_F); m8 = fmaxf(m8, z8[k]); }
            mt = fmaxf(mt, m8);
            if (want_total && m8 > -CUDART_INF_F && m8 < CUDART_INF_F) {
                const float onew = fminf(fmaxf(ceilf(m8 * s_hi), -1.0e9f), 1.0e9f);
                if (!set) { of_t = onew; set = true; }
                else if (onew > of_t) { Sd *= (double)pow2i((int)fmaxf(of_t - onew, -127.f)); of_t = onew; }
                float s8 = 0.f;
#pragma unroll
                for (int k = 0; k < 8; ++k) s8 += ex2_approx(fmaf(z8[k], s_lo, fmaf(z8[k], s_hi, -of_t)));
                Sd += (double)s8;
            }
        });
        float m;
        double total_rel_m = 0.0;          // sum over the row of 2^((z - m) s)
        {
            float wm = mt;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
            const int o_t = set ? (int)of_t : ROWPART_EMPTY;
            const int O_w = __reduce_max_sync(0xffffffffu, o_t);
            const double Sw = want_total ? warp_sum(Sd * (double)pow2i(max(o_t - O_w, -127))) : 0.0;
            if (lane == 0) { S.red[w][0] = (double)wm; S.red[w][1] = Sw; S.red[w][2] = (double)O_w; }
            S.tmax[tid] = cut::key_of(mt);
            if (tid == 0) S.count = 0;
            bad = __syncthreads_or(bad);
            double mm = -CUDART_INF, Om = (double)ROWPART_EMPTY;
            for (int k = 0; k < NW; ++k) { mm = fmax(mm, S.red[k][0]); Om = fmax(Om, S.red[k][2]); }
            m = (float)mm;
            bad = bad || !(mm > -CUDART_INF);
            if (want_total && !bad) {
                double St = 0.0;
                for (int k = 0; k < NW; ++k) St += S.red[k][1] * pow2d(max((int)(S.red[k][2] - Om), -1000));
                // from units of 2^Om to units of the row maximum: 2^(Om - m s), Om - m s in [0, 1]
                const double d = Om - (double)m * s_d;
                total_rel_m = St * 1.4142135623730951 * exp2_frac(fmin(fmax(d, 0.0), 1.0) - 0.5);
            }
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

        const double Od = ceil((double)m * s_d);
        const float of = (float)fmin(fmax(Od, -1.0e9), 1.0e9);
        if (DT == SPEC_BF16) {
            // ---- bf16 rows: a histogram over logit VALUES.  A bf16 logit has 16 significant key bits, and
            // the candidates lie within a few octaves of the maximum, so their values fall into at most NB
            // consecutive keys counted down from the maximum's: bin d = key16(max) - key16(z).  Counts per
            // value are all the selection needs (the mass of a bin is its count times the mass of its
            // value), and every number of candidates fits.
            uint32_t *cnt = reinterpret_cast<uint32_t *>(S.hist);
            const int k16m = (int)(cut::key_of(m) >> 16);
            auto value_of_bin = [&](int d) -> float {
                uint32_t key = (uint32_t)(k16m - d) << 16;
                if (!(key & 0x80000000u)) key |= 0xFFFFu;
                return cut::value_of(key);
            };
            bool todo = false;
            int d_lo = 0;
            unsigned long long loc[PER], before, total;
            if (use_k) {
                // bound: the k-th largest of the per-thread maxima
                for (int i = tid; i < NB; i += NT) cnt[i] = 0;
                __syncthreads();
                {
                    const int d = k16m - (int)(S.tmax[tid] >> 16);
                    if (d >= 0 && d < NB) atomicAdd(&cnt[d], 1u);
                }
                __syncthreads();
#pragma unroll
                for (int k = 0; k < PER; ++k) loc[k] = cnt[tid * PER + k];
                d_lo = scan_find(S, loc, (double)P.top_k, -1.0, before, total);
                if (d_lo < 0) todo = true;
                __syncthreads();
            } else {
                d_lo = k16m - (int)(cut::key_of(m - WINDOW_OCTAVES / sf) >> 16);
                if (d_lo < 0 || d_lo >= NB) todo = true;
            }
            int d_cut = -1;
            if (!todo) {
                const float z_lo = value_of_bin(d_lo);
                for (int i = tid; i < NB; i += NT) cnt[i] = 0;
                __syncthreads();
                // ---- second read (L2 where the row is still there): count the candidates by value ------------
                SPECV_FOR_CHUNKS(ok, {
                    float m8 = z8[0];
#pragma unroll
                    for (int k = 1; k < 8; ++k) m8 = fmaxf(m8, z8[k]);
                    if (ok && m8 >= z_lo) {
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            if (z8[k] >= z_lo) atomicAdd(&cnt[k16m - (int)(cut::key_of(z8[k]) >> 16)], 1u);
                    }
                });
                __syncthreads();
                unsigned long long c[PER], ms[PER];
#pragma unroll
                for (int k = 0; k < PER; ++k) {
                    const int d = tid * PER + k;
                    c[k] = d <= d_lo ? (unsigned long long)cnt[d] : 0ull;
                    ms[k] = c[k] ? c[k] * fix44(ex2_approx((value_of_bin(d) - m) * sf)) : 0ull;
                }
                int d_k = d_lo;                 // the set: bins 0 .. d_k
                if (use_k) {
                    d_k = scan_find(S, c, (double)P.top_k, -1.0, before, total);
                    if (d_k < 0) todo = true;
                }
                d_cut = d_k;
                if (!todo && use_p) {
#pragma unroll
                    for (int k = 0; k < PER; ++k) loc[k] = (tid * PER + k) <= d_k ? ms[k] : 0ull;
                    const int d_p = use_k ? scan_find(S, loc, 0.0, (double)P.top_p, before, total)
                                          : scan_find(S, loc, (double)P.top_p * total_rel_m * cut::FIX, -1.0, before, total);
                    if (d_p >= 0) d_cut = d_p;
                    else if (!use_k) todo = true;        // the nucleus reaches below the window
                    // with top-k: the set itself does not reach the target (rounding): the whole set is kept
                }
                if (!todo) {
                    double v[2] = {0.0, 0.0};
#pragma unroll
                    for (int k = 0; k < PER; ++k) {
                        const int d = tid * PER + k;
                        if (d <= d_cut && c[k]) {
                            const float z = value_of_bin(d);
                            const float x = fmaxf(fmaf(z, s_lo, fmaf(z, s_hi, -of)), -200.f);
                            const double e = (double)ex2_approx(x) * (double)c[k];
                            v[0] += e;
                            v[1] += e * (double)x;
                        }
                    }
                    v[0] = warp_sum(v[0]);
                    v[1] = warp_sum(v[1]);
                    __syncthreads();
                    if (lane == 0) { S.red[w][0] = v[0]; S.red[w][1] = v[1]; }
                    __syncthreads();
                    if (tid == 0) {
                        double Z = 0.0, X = 0.0;
                        for (int k = 0; k < NW; ++k) { Z += S.red[k][0]; X += S.red[k][1]; }
                        const float cutv = value_of_bin(d_cut);
                        RowPart r;
                        r.S = Z; r.X = X; r.O = (int)of; r.cut = cutv;
                        r.xmax = (float)((double)m * s_d - (double)of);
                        r.bad = 0;
                        *out = r;
                        P.cut[row * 2 + which] = cutv;
                    }
                }
            }
            if (todo && tid == 0) {
                RowPart r = {};
                r.cut = -CUDART_INF_F; r.O = ROWPART_EMPTY; r.bad = ROW_TODO;
                *out = r;
                const int pos = atomicAdd(P.todo, 1);
                P.todo[1 + pos] = (int)id;
            }
            continue;
        }

        // ---- fp32 rows: candidates in a list, radix selection on the list --------------------------------------
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

        // ---- second read (L2 where the row is still there): the candidates --------------------------------------
        unsigned long long tot_fix = 0;
        if (!todo) {
            SPECV_FOR_CHUNKS(ok, {
                float m8 = z8[0];
#pragma unroll
                for (int k = 1; k < 8; ++k) m8 = fmaxf(m8, z8[k]);
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
            __syncthreads();
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
                    if (k >= key_k) part += fix44(ex2_approx((cut::value_of(k) - m) * sf));
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
            const double target = (double)P.top_p * (use_k ? (double)tot_fix : total_rel_m * cut::FIX);
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
