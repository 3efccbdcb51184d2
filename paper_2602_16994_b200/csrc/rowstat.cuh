// Row statistics in one read of the logits: for every row the verifiers will touch, the sampling
// distribution's cut (top-k / top-p; see cut.cuh for the rules), its integer reference O = ceil(max z s),
// the normaliser Z = sum over kept tokens of 2^(z s - O), the kept count, and (for the selector features)
// sum e x and the largest exponent.  s = log2(e) / T.
//
// One thread-block cluster per row, clusters persistent over the row list.  Each CTA brings its slice of
// the row into shared memory with one bulk asynchronous copy and keeps the RAW logits there, so the
// radix-selection levels (counts for top-k, fixed-point masses for top-p) and the final sum all sweep
// shared memory: HBM is read once.  Histograms are per CTA; after a cluster barrier every thread adds
// up its bins over the CTAs through distributed shared memory, so all CTAs select the same bin.
//
// Shared-memory atomics on a handful of hot bins serialise, so the histograms only ever see
// candidates: for top-k the tokens at or above the k-th largest of the per-thread maxima (a lower
// bound of the k-th largest logit, found by the same radix selection over one value per thread); for
// top-p the tokens within 20 octaves of the row maximum, while the total mass is summed exactly in
// registers (if the nucleus boundary is not among the candidates the level is redone over all tokens).
#pragma once
#include "common.cuh"
#include "cut.cuh"
#include "stream.cuh"

namespace specv {
namespace rowstat {

constexpr int NT = 512;
constexpr int NW = NT / 32;
constexpr int NB = cut::NB;
constexpr int PER = NB / NT;
constexpr int CMAXR = 16;

struct RParams {
    int B, N, V, C, dtype, top_k;
    int slice_len;             // tokens per CTA slice (multiple of 8)
    float top_p;
    const void *zp, *zq;
    long long seq_stride, node_stride, topo_stride;
    const int *parent;         // NULL: every row of `zp` only (spec_tree_probs)
    float T;
    const float *T_seq;
    RowPart *part;             // [B*N*2]: the row's statistics as one slice
    float *cut;                // [B*N*2] smallest kept logit of every row (for spec_tree_probs)
    int *todo;                 // [1 + B*N*2]: count, then the ids of the rows the fast path (trunc.cuh) left over
    int only_todo;             // 1: take only the rows listed in todo
};

struct __align__(16) Shared {
    unsigned long long hist[NB];
    unsigned long long warp_tot[NW];
    double xv[2][CMAXR][4];    // cluster exchanges (double buffered)
    double red[NW][4];
    uint64_t mbar;
    int sel_bin, found;
    unsigned long long sel_above;
};

__device__ __forceinline__ void cluster_barrier()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned long long ld_remote_u64(const unsigned long long *local_addr, uint32_t rank)
{
    unsigned long long v;
    asm volatile("{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %1, %2;\n\tld.shared::cluster.u64 %0, [ra];\n\t}"
                 : "=l"(v)
                 : "r"(smem_u32(local_addr)), "r"(rank)
                 : "memory");
    return v;
}
__device__ __forceinline__ void st_remote_f64_plain(double *local_addr, uint32_t rank, double v)
{
    asm volatile("{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %0, %1;\n\tst.shared::cluster.f64 [ra], %2;\n\t}" ::"r"(
                     smem_u32(local_addr)),
                 "r"(rank), "d"(v)
                 : "memory");
}

// all-gather of up to 4 doubles per CTA; returns with S.xv[par][r][*] filled for every rank r
__device__ __forceinline__ void cluster_allgather4(Shared &S, int par, int C, uint32_t rank, const double (&v)[4])
{
    if (threadIdx.x < (unsigned)(C * 4)) {
        const int peer = threadIdx.x >> 2, k = threadIdx.x & 3;
        st_remote_f64_plain(&S.xv[par][rank][k], (uint32_t)peer, v[k]);
    }
    cluster_barrier();
}

// block-wide sum of 4 doubles; result in every thread
__device__ __forceinline__ void block_sum4(Shared &S, double (&v)[4])
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < 4; ++k) v[k] = warp_sum(v[k]);
    __syncthreads();
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) S.red[w][k] = v[k];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        double t = 0.0;
        for (int i = 0; i < NW; ++i) t += S.red[i][k];
        v[k] = t;
    }
}

// Sum the per-CTA histograms over the cluster (every thread its PER bins), then find the first bin from
// the top at which above + running sum reaches target.  Same answer in every CTA.  Returns -1 when the
// total stays below the target.  With frac >= 0 the target is first set to frac times the sum of all bins.
__device__ __forceinline__ int cluster_select_bin(Shared &S, int C, double above, double &target, double frac,
                                                  unsigned long long &sum_above)
{
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    cluster_barrier();                       // every CTA's histogram is complete
    unsigned long long loc[PER], lsum = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        const int bin = NB - 1 - (tid * PER + k);
        unsigned long long t = 0;
        for (int r = 0; r < C; ++r) t += ld_remote_u64(&S.hist[bin], (uint32_t)r);
        loc[k] = t;
        lsum += t;
    }
    cluster_barrier();                       // everyone has read: the histograms may be cleared
    unsigned long long incl = lsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) S.warp_tot[w] = incl;
    if (tid == 0) { S.found = 0; S.sel_bin = -1; S.sel_above = 0; }
    __syncthreads();
    unsigned long long base = 0, tot = 0;
    for (int k = 0; k < NW; ++k) { if (k < w) base += S.warp_tot[k]; tot += S.warp_tot[k]; }
    if (frac >= 0.0) target = frac * (double)tot;
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

// Warp-collective additions to a histogram: lanes that hit the same bin are combined first, so a hot bin
// costs one shared-memory atomic per warp and not one per token.  Every lane of the warp must call these
// (pred says whether the lane takes part).
__device__ __forceinline__ void hist_count(unsigned long long *hist, bool pred, int bin)
{
    const int lane = threadIdx.x & 31;
    unsigned active = __ballot_sync(0xffffffffu, pred);
    while (active) {
        const int leader = __ffs(active) - 1;
        const int lb = __shfl_sync(0xffffffffu, bin, leader);
        const unsigned same = __ballot_sync(0xffffffffu, pred && bin == lb);
        if (lane == leader) atomicAdd(&hist[lb], (unsigned long long)__popc(same));
        active &= ~same;
    }
}
__device__ __forceinline__ void hist_mass(unsigned long long *hist, bool pred, int bin, unsigned long long val)
{
    const int lane = threadIdx.x & 31;
    unsigned active = __ballot_sync(0xffffffffu, pred);
    while (active) {
        const int leader = __ffs(active) - 1;
        const int lb = __shfl_sync(0xffffffffu, bin, leader);
        const bool mine = pred && bin == lb;
        const unsigned same = __ballot_sync(0xffffffffu, mine);
        unsigned long long v = mine ? val : 0ull;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == leader) atomicAdd(&hist[lb], v);
        active &= ~same;
    }
}

// Visit every logit of the slice, 8 per thread and step (16-byte loads for bf16, 32-byte for fp32), the
// ragged end one by one.  Trip counts are the same for all lanes of a warp: OKVAR tells whether the lane
// holds a real token (ZVAR is -inf otherwise), so BODY may use warp-collective operations.
#define SPECV_FOR_TOKENS(ZVAR, OKVAR, BODY)                                                                  \
    do {                                                                                                     \
        const int n8_ = n >> 3;                                                                              \
        for (int b8_ = 0; b8_ < n8_; b8_ += NT) {                                                            \
            const int i8_ = b8_ + tid;                                                                       \
            const bool OKVAR = i8_ < n8_;                                                                    \
            float zz_[8];                                                                                    \
            if (OKVAR) {                                                                                     \
                if (DT == SPEC_BF16) {                                                                       \
                    const uint4 r_ = reinterpret_cast<const uint4 *>(raw)[i8_];                              \
                    zz_[0] = bf16_lo(r_.x); zz_[1] = bf16_hi(r_.x); zz_[2] = bf16_lo(r_.y); zz_[3] = bf16_hi(r_.y); \
                    zz_[4] = bf16_lo(r_.z); zz_[5] = bf16_hi(r_.z); zz_[6] = bf16_lo(r_.w); zz_[7] = bf16_hi(r_.w); \
                } else {                                                                                     \
                    const float4 a_ = reinterpret_cast<const float4 *>(raw)[2 * i8_];                        \
                    const float4 b_ = reinterpret_cast<const float4 *>(raw)[2 * i8_ + 1];                    \
                    zz_[0] = a_.x; zz_[1] = a_.y; zz_[2] = a_.z; zz_[3] = a_.w;                              \
                    zz_[4] = b_.x; zz_[5] = b_.y; zz_[6] = b_.z; zz_[7] = b_.w;                              \
                }                                                                                            \
            } else {                                                                                         \
                _Pragma("unroll") for (int k_ = 0; k_ < 8; ++k_) zz_[k_] = -CUDART_INF_F;                    \
            }                                                                                                \
            _Pragma("unroll") for (int k_ = 0; k_ < 8; ++k_) { const float ZVAR = zz_[k_]; BODY }            \
        }                                                                                                    \
        for (int bt_ = n8_ << 3; bt_ < n; bt_ += NT) {                                                       \
            const int i_ = bt_ + tid;                                                                        \
            const bool OKVAR = i_ < n;                                                                       \
            const float ZVAR = !OKVAR ? -CUDART_INF_F                                                        \
                               : (DT == SPEC_BF16                                                            \
                                      ? __uint_as_float((uint32_t)((const unsigned short *)raw)[i_] << 16)   \
                                      : ((const float *)raw)[i_]);                                           \
            BODY                                                                                             \
        }                                                                                                    \
    } while (0)

template <int DT>
__global__ void __launch_bounds__(NT, 2) spec_row_stat_kernel(const RParams P)
{
    constexpr int ESZ = DT == SPEC_BF16 ? 2 : 4;
    constexpr int LEVELS = DT == SPEC_BF16 ? 2 : 3;
    __shared__ Shared S;
    unsigned char *raw = dyn_smem;                // this CTA's slice of the row, as it sits in HBM
    const int tid = threadIdx.x;
    const int C = P.C;
    const uint32_t rank = cluster_ctarank();
    const int cid = blockIdx.x / C, NC = gridDim.x / C;
    const long long tok0 = (long long)rank * P.slice_len;
    const int n = (int)max(0ll, min((long long)P.slice_len, (long long)P.V - tok0));
    const long long items = 2ll * P.B * P.N;
    const bool use_k = P.top_k > 0 && P.top_k < P.V, use_p = P.top_p < 1.f;
    if (tid == 0) { mbar_init(&S.mbar, 1); mbar_fence_init(); }
    __syncthreads();
    cluster_barrier();
    uint32_t phase = 0;
    int xpar = 0;

// level parameters: 11 bits from the top, then 5 (bf16: 16 significant key bits) or 11 + 10 (fp32)
#define SPECV_LEVEL_SHIFT(LV) ((LV) == 0 ? 21 : (DT == SPEC_BF16 ? 16 : ((LV) == 1 ? 10 : 0)))
#define SPECV_LEVEL_MASK(LV) ((1u << ((LV) == 0 ? 11 : (DT == SPEC_BF16 ? 5 : ((LV) == 1 ? 11 : 10)))) - 1u)

    const long long n_items = P.only_todo ? (long long)__ldcg(P.todo) : items;
    for (long long it = cid; it < n_items; it += NC) {
        const long long id = P.only_todo ? (long long)__ldcg(P.todo + 1 + it) : it;
        const long long row = id >> 1;
        const int which = (int)(id & 1);
        const int b = (int)(row / P.N), a = (int)(row % P.N);
        RowPart *out = P.part + row * 2 + which;
        if (which == 1) {
            bool any = false;
            if (P.parent) {
                const int *parent = P.parent + (long long)b * P.topo_stride;
                for (int c = a + 1 + tid; c < P.N; c += NT) any |= __ldg(parent + c) == a;
            }
            if (!__syncthreads_or((int)any)) {        // a draft row is read only for nodes with children
                if (rank == 0 && tid == 0) {
                    RowPart r = {};
                    r.cut = -CUDART_INF_F; r.O = ROWPART_EMPTY; r.bad = -1;        // row not read
                    *out = r;
                    P.cut[row * 2 + 1] = -CUDART_INF_F;
                }
                continue;
            }
        }
        const unsigned char *src = (const unsigned char *)(which ? P.zq : P.zp) +
                                   ((long long)b * P.seq_stride + (long long)a * P.node_stride + tok0) * ESZ;
        // ---- the slice: one bulk copy for the 16-byte aligned body, plain loads for the rest -----------
        {
            const bool aligned = (((uintptr_t)src) & 15) == 0;
            const uint32_t body = aligned ? (((uint32_t)n * ESZ) & ~15u) : 0u;
            if (tid == 0 && body) {
                mbar_arrive_expect_tx(&S.mbar, body);
                bulk_g2s(raw, src, body, &S.mbar);
            }
            if (ESZ == 2) {
                for (int e = (int)(body / 2) + tid; e < n; e += NT) ((unsigned short *)raw)[e] = __ldg((const unsigned short *)src + e);
            } else {
                for (int e = (int)(body / 4) + tid; e < n; e += NT) ((float *)raw)[e] = __ldg((const float *)src + e);
            }
            int gave_up = 0;
            if (body) {
                gave_up = mbar_wait(&S.mbar, phase) ? 0 : 1;
                phase ^= 1u;
            }
            // a copy that was given up on: the row is reported, not used (the decision is cluster-wide)
            gave_up = __syncthreads_or(gave_up);
            {
                double v[4] = {(double)gave_up, 0.0, 0.0, 0.0};
                cluster_allgather4(S, xpar, C, rank, v);
                gave_up = 0;
                for (int r = 0; r < C; ++r) gave_up |= S.xv[xpar][r][0] != 0.0;
                xpar ^= 1;
            }
            if (gave_up) {
                if (rank == 0 && tid == 0) {
                    RowPart r = {};
                    r.cut = -CUDART_INF_F; r.O = ROWPART_EMPTY; r.bad = ROW_TIMEOUT;
                    *out = r;
                    P.cut[row * 2 + which] = -CUDART_INF_F;
                }
                __syncthreads();
                continue;
            }
        }
        const float Tf = P.T_seq ? __ldg(P.T_seq + b) : P.T;
        const float sf = 1.4426950408889634f / Tf;
        const double s_d = 1.4426950408889634 / (double)Tf;

        // ---- row maximum (and the thread's own maximum), NaN / +inf ------------------------------------------
        float mt = -CUDART_INF_F;
        int bad = 0;
        SPECV_FOR_TOKENS(z, ok, { if (ok) { bad |= (z != z) || (z == CUDART_INF_F); mt = fmaxf(mt, z); } });
        float m;
        {
            double v[4] = {0.0, 0.0, 0.0, 0.0};
            float wm = mt;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
            __syncthreads();
            if ((tid & 31) == 0) S.red[tid >> 5][0] = (double)wm;
            bad = __syncthreads_or(bad);
            double mm = -CUDART_INF;
            for (int k = 0; k < NW; ++k) mm = fmax(mm, S.red[k][0]);
            v[0] = mm; v[1] = (double)bad;
            cluster_allgather4(S, xpar, C, rank, v);
            double M = -CUDART_INF, bd = 0.0;
            for (int r = 0; r < C; ++r) { M = fmax(M, S.xv[xpar][r][0]); bd += S.xv[xpar][r][1]; }
            xpar ^= 1;
            m = (float)M;
            bad = bd != 0.0 || !(M > -CUDART_INF);
        }
        uint32_t key_cut = 0u;
        if (!bad && (use_k || use_p)) {
            // ---- top-k: the k-th largest logit value -------------------------------------------------------
            uint32_t key_k = 0u;
            if (use_k) {
                // a lower bound first: the k-th largest of the per-thread maxima (needs k of them)
                float lower = -CUDART_INF_F;
                if (P.top_k <= (C * NT) / 4) {
                    uint32_t prefix = 0, pmask = 0;
                    double need = (double)P.top_k;
                    bool all = false;
#pragma unroll 1
                    for (int lv = 0; lv < LEVELS && !all; ++lv) {
                        const int sh = SPECV_LEVEL_SHIFT(lv);
                        const uint32_t bm = SPECV_LEVEL_MASK(lv);
                        for (int i = tid; i < NB; i += NT) S.hist[i] = 0;
                        __syncthreads();
                        {
                            const uint32_t k = cut::key_of(mt);
                            hist_count(S.hist, mt > -CUDART_INF_F && (k & pmask) == prefix, (int)((k >> sh) & bm));
                        }
                        unsigned long long above;
                        const int bin = cluster_select_bin(S, C, 0.0, need, -1.0, above);
                        if (bin < 0) { all = true; break; }
                        need -= (double)above;
                        prefix |= (uint32_t)bin << sh;
                        pmask |= bm << sh;
                    }
                    if (!all) {
                        if (DT == SPEC_BF16 && !(prefix & 0x80000000u)) prefix |= 0xFFFFu;
                        lower = cut::value_of(prefix);
                    }
                }
                uint32_t prefix = 0, pmask = 0;
                double need = (double)P.top_k;
                bool all = false;
#pragma unroll 1
                for (int lv = 0; lv < LEVELS && !all; ++lv) {
                    const int sh = SPECV_LEVEL_SHIFT(lv);
                    const uint32_t bm = SPECV_LEVEL_MASK(lv);
                    for (int i = tid; i < NB; i += NT) S.hist[i] = 0;
                    __syncthreads();
                    SPECV_FOR_TOKENS(z, ok, {
                        const uint32_t k = cut::key_of(z);
                        hist_count(S.hist, ok && z >= lower && (k & pmask) == prefix, (int)((k >> sh) & bm));
                    });
                    unsigned long long above;
                    const int bin = cluster_select_bin(S, C, 0.0, need, -1.0, above);
                    if (bin < 0) { all = true; break; }
                    need -= (double)above;
                    prefix |= (uint32_t)bin << sh;
                    pmask |= bm << sh;
                }
                key_k = all ? 0u : prefix;
                if (DT == SPEC_BF16 && key_k && !(key_k & 0x80000000u)) key_k |= 0xFFFFu;
            }
            key_cut = key_k;
            // ---- top-p: the first value group at which the mass reaches top_p of the set's ---------------------
            if (use_p) {
                const float zk = key_k == 0u ? -CUDART_INF_F : cut::value_of(key_k);      // the top-k set: z >= zk
                // total mass of the set, exactly (fixed point, integer sums)
                unsigned long long tot_fix;
                {
                    unsigned long long part = 0;
                    SPECV_FOR_TOKENS(z, ok, {
                        if (ok && z >= zk) part += (unsigned long long)((double)ex2_approx((z - m) * sf) * cut::FIX);
                    });
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                    __syncthreads();
                    if ((tid & 31) == 0) S.warp_tot[tid >> 5] = part;
                    __syncthreads();
                    unsigned long long cta = 0;
                    for (int k = 0; k < NW; ++k) cta += S.warp_tot[k];
                    // exact in a double pair: high and low 32 bits travel separately
                    double v[4] = {(double)(cta >> 32), (double)(cta & 0xFFFFFFFFull), 0.0, 0.0};
                    cluster_allgather4(S, xpar, C, rank, v);
                    tot_fix = 0;
                    for (int r = 0; r < C; ++r)
                        tot_fix += ((unsigned long long)S.xv[xpar][r][0] << 32) + (unsigned long long)S.xv[xpar][r][1];
                    xpar ^= 1;
                }
                double target = (double)P.top_p * (double)tot_fix;
                // candidates: within 20 octaves of the maximum; everything if the boundary is not among them
                float zc = fmaxf(zk, m - 20.f / sf);
#pragma unroll 1
                for (int attempt = 0; attempt < 2; ++attempt) {
                    uint32_t prefix = 0, pmask = 0;
                    double above_mass = 0.0;
                    bool all = false;
#pragma unroll 1
                    for (int lv = 0; lv < LEVELS && !all; ++lv) {
                        const int sh = SPECV_LEVEL_SHIFT(lv);
                        const uint32_t bm = SPECV_LEVEL_MASK(lv);
                        for (int i = tid; i < NB; i += NT) S.hist[i] = 0;
                        __syncthreads();
                        SPECV_FOR_TOKENS(z, ok, {
                            const uint32_t k = cut::key_of(z);
                            const bool in = ok && z >= zc && (k & pmask) == prefix;
                            if (__any_sync(0xffffffffu, in))
                                hist_mass(S.hist, in, (int)((k >> sh) & bm),
                                          in ? (unsigned long long)((double)ex2_approx((z - m) * sf) * cut::FIX) : 0ull);
                        });
                        unsigned long long above;
                        const int bin = cluster_select_bin(S, C, above_mass, target, -1.0, above);
                        if (bin < 0) { all = true; break; }
                        above_mass += (double)above;
                        prefix |= (uint32_t)bin << sh;
                        pmask |= bm << sh;
                    }
                    if (!all) {
                        key_cut = prefix;
                        if (DT == SPEC_BF16 && !(key_cut & 0x80000000u)) key_cut |= 0xFFFFu;
                        break;
                    }
                    // the candidates did not reach the target: once more over the whole set; if even that
                    // stays below (rounding), the whole set is kept
                    if (zc <= zk) break;
                    zc = zk;
                }
            }
        }
        const float cutv = key_cut == 0u ? -CUDART_INF_F : cut::value_of(key_cut);

        // ---- normaliser, entropy sum, kept count over the kept tokens ---------------------------------------
        const double Od = bad ? 0.0 : ceil((double)m * s_d);
        const float of = (float)fmin(fmax(Od, -1.0e9), 1.0e9);
        float s_hi = (float)s_d;
        if ((double)s_hi > s_d) s_hi = __uint_as_float(__float_as_uint(s_hi) - 1u);
        float s_lo = (float)(s_d - (double)s_hi);
        if (!(s_lo > 0.f)) s_lo = 1.0e-30f;
        double acc_e = 0.0, acc_x = 0.0;
        int kept = 0;
        if (!bad) {
            const int n8 = n >> 3;
            (void)n8;
            float pe = 0.f, px = 0.f;
            int cnt = 0;
            SPECV_FOR_TOKENS(z, ok, {
                if (ok && z >= cutv) {
                    const float x = fmaxf(fmaf(z, s_lo, fmaf(z, s_hi, -of)), -200.f);
                    const float e = ex2_approx(x);
                    pe += e;
                    px = fmaf(e, x, px);
                    ++kept;
                }
                if (++cnt == 64) { acc_e += (double)pe; acc_x += (double)px; pe = 0.f; px = 0.f; cnt = 0; }
            });
            acc_e += (double)pe;
            acc_x += (double)px;
        }
        {
            double v[4] = {acc_e, acc_x, (double)kept, 0.0};
            block_sum4(S, v);
            cluster_allgather4(S, xpar, C, rank, v);
            double Z = 0.0, X = 0.0, K = 0.0;
            for (int r = 0; r < C; ++r) { Z += S.xv[xpar][r][0]; X += S.xv[xpar][r][1]; K += S.xv[xpar][r][2]; }
            xpar ^= 1;
            if (rank == 0 && tid == 0) {
                RowPart r;
                r.S = Z; r.X = X; r.O = bad ? ROWPART_EMPTY : (int)of; r.cut = cutv;
                r.xmax = bad ? 0.f : (float)((double)m * s_d - (double)of);
                r.bad = bad ? 1 : 0;
                (void)K;
                *out = r;
                P.cut[row * 2 + which] = cutv;
            }
        }
        __syncthreads();         // the slice is overwritten by the next row's copy
    }
#undef SPECV_LEVEL_SHIFT
#undef SPECV_LEVEL_MASK
    cluster_barrier();           // nobody leaves while a peer may still read its shared memory
}

}  // namespace rowstat
}  // namespace specv
