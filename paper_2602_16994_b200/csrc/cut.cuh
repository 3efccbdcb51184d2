// Row cut values for top-k / top-p truncation (the paper's experimental setup names temperature and
// nucleus sampling; top-k is an addition of the workloads).  One CTA per logit row finds the smallest
// kept logit VALUE of the row:
//   top-k: the k-th largest logit value (ties at that value are all kept);
//   top-p: within the top-k set, tokens of equal logit form a group; groups in descending order; the
//          cut is the value of the first group at which the cumulative mass reaches top_p times the
//          mass of the set.
// Both are radix selections on an order-preserving integer image of the logit (sign-flipped bits,
// -0 folded into +0), 11 bits per level from the top, so equal logits can never be separated and the
// answer does not depend on token order.  Counts are integers; masses are accumulated as 64-bit fixed
// point (2^44 per unit of e = exp((z - max)/T)), so every sum is exact and order-free.  The row is
// swept once per level from global memory (it stays in L2 between sweeps).
#pragma once
#include "common.cuh"

namespace specv {
namespace cut {

constexpr int NT = 512;
constexpr int NBITS = 11;
constexpr int NB = 1 << NBITS;          // bins per level
constexpr int PER = NB / NT;            // bins per thread in the scan
constexpr double FIX = 17592186044416.0;   // 2^44

struct CParams {
    int B, N, V, dtype, top_k;
    float top_p;
    const void *zp, *zq;
    long long seq_stride, node_stride, topo_stride;
    const int *parent;
    float T;
    const float *T_seq;
    float *cut;              // [B*N*2]
    int only_target;         // 1: compute slot 0 of every pair only (no tree given)
};

__device__ __forceinline__ uint32_t key_of(float z)
{
    uint32_t u = __float_as_uint(z);
    if (u == 0x80000000u) u = 0u;                       // -0 and +0 are one value
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float value_of(uint32_t key)
{
    const uint32_t u = (key & 0x80000000u) ? (key & 0x7FFFFFFFu) : ~key;
    return __uint_as_float(u);
}

struct Shared {
    unsigned long long hist[NB];
    unsigned long long warp_tot[NT / 32];
    float warp_max[NT / 32];
    int sel_bin, found;
    unsigned long long sel_above;
};

// Descending scan of hist: the first bin (from the top) at which above + running sum reaches `target`.
// Returns the bin (or -1 when the total stays below the target) and the sum strictly above it.
__device__ __forceinline__ int select_bin(Shared &S, double above, double target, unsigned long long &sum_above)
{
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    unsigned long long loc[PER], lsum = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) { loc[k] = S.hist[NB - 1 - (tid * PER + k)]; lsum += loc[k]; }
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
    unsigned long long run = base + incl - lsum;       // sum of the bins above this thread's
    if (above + (double)run < target && above + (double)(run + lsum) >= target) {
        // the crossing lies in this thread's bins: exactly one of them satisfies the test
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
    return S.found ? S.sel_bin : -1;
}

template <int DT>
__global__ void __launch_bounds__(NT) spec_row_cut_kernel(const CParams P)
{
    __shared__ Shared S;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int row = blockIdx.x >> 1, which = blockIdx.x & 1;
    const int b = row / P.N, a = row % P.N;
    float *out = P.cut + (long long)row * 2 + which;
    if (which == 1 && P.only_target) {
        if (tid == 0) *out = -CUDART_INF_F;
        return;
    }
    if (which == 1) {
        // a draft row is read only for nodes that have children
        const int *parent = P.parent + (long long)b * P.topo_stride;
        bool any = false;
        for (int c = a + 1 + tid; c < P.N; c += NT) any |= __ldg(parent + c) == a;
        if (!__syncthreads_or((int)any)) {
            if (tid == 0) *out = -CUDART_INF_F;
            return;
        }
    }
    const long long base = (long long)b * P.seq_stride + (long long)a * P.node_stride;
    const void *z = which ? P.zq : P.zp;
    const int V = P.V;
    const bool use_k = P.top_k > 0 && P.top_k < V, use_p = P.top_p < 1.f;
    const float s = 1.4426950408889634f / (P.T_seq ? __ldg(P.T_seq + b) : P.T);

    // row maximum (masses are relative to it)
    float m = -CUDART_INF_F;
    if (use_p) {
        for (int t = tid; t < V; t += NT) m = fmaxf(m, load_logit(z, DT, base + t));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) S.warp_max[w] = m;
        __syncthreads();
        m = -CUDART_INF_F;
        for (int k = 0; k < NT / 32; ++k) m = fmaxf(m, S.warp_max[k]);
        __syncthreads();
    }
    constexpr int LEVELS = DT == SPEC_BF16 ? 2 : 3;
    const int shifts[3] = {21, DT == SPEC_BF16 ? 16 : 10, 0};
    const int widths[3] = {11, DT == SPEC_BF16 ? 5 : 11, 10};

    uint32_t key_k = 0;          // smallest kept key after top-k (0: everything)
    if (use_k) {
        uint32_t prefix = 0, pmask = 0;
        double need = (double)P.top_k;
        bool all = false;
        for (int lv = 0; lv < LEVELS && !all; ++lv) {
            for (int i = tid; i < NB; i += NT) S.hist[i] = 0;
            __syncthreads();
            const int sh = shifts[lv];
            const uint32_t bm = (1u << widths[lv]) - 1u;
            for (int t = tid; t < V; t += NT) {
                const uint32_t k = key_of(load_logit(z, DT, base + t));
                if ((k & pmask) == prefix) atomicAdd(&S.hist[(k >> sh) & bm], 1ull);
            }
            __syncthreads();
            unsigned long long above;
            const int bin = select_bin(S, 0.0, need, above);
            if (bin < 0) { all = true; break; }
            need -= (double)above;
            prefix |= (uint32_t)bin << sh;
            pmask |= bm << sh;
            __syncthreads();
        }
        key_k = all ? 0u : prefix;
        if (DT == SPEC_BF16 && key_k && !(key_k & 0x80000000u)) key_k |= 0xFFFFu;   // the exact image of a negative bf16
    }
    uint32_t key_cut = key_k;
    if (use_p) {
        uint32_t prefix = 0, pmask = 0;
        double above_mass = 0.0, target = 0.0;
        bool all = false;
        for (int lv = 0; lv < LEVELS && !all; ++lv) {
            for (int i = tid; i < NB; i += NT) S.hist[i] = 0;
            __syncthreads();
            const int sh = shifts[lv];
            const uint32_t bm = (1u << widths[lv]) - 1u;
            for (int t = tid; t < V; t += NT) {
                const float zv = load_logit(z, DT, base + t);
                const uint32_t k = key_of(zv);
                if (k >= key_k && (k & pmask) == prefix) {
                    const float e = ex2_approx((zv - m) * s);
                    atomicAdd(&S.hist[(k >> sh) & bm], (unsigned long long)((double)e * FIX));
                }
            }
            __syncthreads();
            if (lv == 0) {
                // total mass of the top-k set: sum of all bins (exact, order-free)
                unsigned long long part = 0;
                for (int i = tid; i < NB; i += NT) part += S.hist[i];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                if (lane == 0) S.warp_tot[w] = part;
                __syncthreads();
                unsigned long long tot = 0;
                for (int k = 0; k < NT / 32; ++k) tot += S.warp_tot[k];
                target = (double)P.top_p * (double)tot;
                __syncthreads();
            }
            unsigned long long above;
            const int bin = select_bin(S, above_mass, target, above);
            if (bin < 0) { all = true; break; }       // rounding kept the total below the target: keep the whole set
            above_mass += (double)above;
            prefix |= (uint32_t)bin << sh;
            pmask |= bm << sh;
            __syncthreads();
        }
        if (!all) {
            key_cut = prefix;
            if (DT == SPEC_BF16 && !(key_cut & 0x80000000u)) key_cut |= 0xFFFFu;
        }
    }
    if (tid == 0) *out = key_cut == 0u ? -CUDART_INF_F : value_of(key_cut);
}

}  // namespace cut
}  // namespace specv
