// libspecverify: batched draft-tree verification for sm_100a -- host side of the C ABI.
//
// Kernels: stream.cuh (row statistics, the one pass over HBM), rowstat.cuh (the same for top-k / top-p
// rows), walk.cuh (SpecInfer along the accepted path), tree.cuh (every node: Traversal Verification,
// diagnostic outputs), rowops.cuh (materialised row distributions, stand-alone inverse CDF), and the
// residual kernel below.  This file validates
// arguments, chooses the launch plan and enqueues; it never allocates and, except for the
// host-buffer entry point, never synchronises.
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "analysis.cuh"
#include "common.cuh"
#include "cut.cuh"
#include "rowops.cuh"
#include "rowstat.cuh"
#include "tree.cuh"
#include "trunc.cuh"
#include "specverify.h"
#include "verify.cuh"
#include "walk.cuh"

namespace specv {
namespace {

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
    const double *gseq;        // [B*N][KMAX] step coefficients of every node
    const int *accepted;
    float *residual;
};

// The accepted node's final law, token by token: the recursion of verify.cuh replayed in fp64 with the
// node's recorded coefficients, u <- (g_j u - e_q)+ from u = e_p, divided by the recorded total.
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
    const double *g = P.gseq + ((long long)b * P.N + acc) * KMAX;
    const double s = 1.4426950408889634 / (double)(P.T_seq ? P.T_seq[b] : P.T);
    const long long row = (long long)b * P.seq_stride + (long long)acc * P.node_stride;
    const int nsteps = R.nsteps;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < P.V; t += gridDim.x * blockDim.x) {
        double u = 0.0;
        if (nsteps == STATE_IS_Q) {
            const float zq = load_logit(P.zq, P.dtype, row + t);
            if (zq >= R.cut_q) u = exp2((double)zq * s - R.O_q);
        } else {
            const float zp = load_logit(P.zp, P.dtype, row + t);
            if (zp >= R.cut_p) u = exp2((double)zp * s - R.O_p);
            if (nsteps > 0) {
                const float zq = load_logit(P.zq, P.dtype, row + t);
                const double eq = zq >= R.cut_q ? exp2((double)zq * s - R.O_q) : 0.0;
                for (int j = 0; j < nsteps; ++j) u = fmax(fma(g[j], u, -eq), 0.0);
            }
        }
        out[t] = (float)(R.kappa > 0.0 ? u / R.kappa : 0.0);
    }
}

// ------------------------------------------------------------------------------------------------
// launch plans
// ------------------------------------------------------------------------------------------------
struct VPlan {
    int C, NW, slice_len, NS, nsm, off_x, off_list, off_es, off_ring, smem;
    int whole_sm;       // one CTA per SM: the kernel variant without a register limit may be used
};

constexpr int SMEM_1CTA = 227 * 1024;          // opt-in limit per CTA
constexpr int SMEM_2CTA = 113 * 1024;          // so that two CTAs share an SM

inline int up(int x, int m) { return (x + m - 1) / m * m; }

// Launch shape of the cluster kernels (walk, tree).  Smallest cluster whose slices fit on chip: seven
// consumer warps + the producer warp (256 threads, two CTAs per SM, 128 registers each) while a slice
// fits in TMAX tiles of 1792 tokens, fifteen consumer warps (one CTA per SM) above that.
// Dynamic shared memory: header | exchange slots [2][C][NW][2] doubles | exact lists [NW] | resident e
// of the tiles that do not fit in registers | ring stages.
bool make_vplan(int V, int dtype, VPlan *p, int hdr_bytes = (int)sizeof(Hdr), bool whole_sm = false, int want_c = 0,
                int want_nw = 0)
{
    const int esz = dtype == SPEC_BF16 ? 2 : 4;
    for (int pass = 0; pass < 2; ++pass) {
        const int NW = pass == 0 ? 7 : 15;
        if (want_nw && NW != want_nw) continue;
        const int tile = NW * 32 * 8;
        const int budget = (NW == 7 && !whole_sm) ? SMEM_2CTA : SMEM_1CTA;
        for (int C = 1; C <= CMAX; C <<= 1) {
            if (want_c && C != want_c) continue;
            const int slice = up((V + C - 1) / C, 8);
            const int tiles = (slice + tile - 1) / tile;
            if (tiles > TMAX) continue;
            if (pass == 0 && C > 8 && !want_c) continue;   // prefer one CTA per SM over a non-portable cluster
            const int off_x = up(hdr_bytes, 128);
            const int off_list = off_x + up(2 * C * NW * 2 * 8, 128);
            const int off_es = off_list + up(NW * (int)sizeof(WarpList), 128);
            const int stage = 2 * tile * esz;
            const int nsm = tiles > RT ? tiles - RT : 0;
            if (nsm > SMT) continue;
            const int es_bytes = nsm * tile * 8;
            const int off_ring = off_es + es_bytes;
            int ns = (budget - off_ring) / stage;
            if (ns > NSMAX) ns = NSMAX;
            if (ns > 2 * tiles) ns = 2 * tiles;
            if (ns < 2) continue;
            p->C = C; p->NW = NW; p->slice_len = slice; p->NS = ns; p->nsm = nsm; p->whole_sm = 0;
            p->off_x = off_x; p->off_list = off_list; p->off_es = off_es; p->off_ring = off_ring;
            p->smem = off_ring + ns * stage;
            return true;
        }
    }
    return false;
}

struct RowPlan {
    int C, SL, smem;
};
constexpr int ROW_SMEM_BUDGET = 227 * 1024 - (int)sizeof(rowops::Shared) - 1024;

bool make_row_plan(int V, int bytes_per_token, RowPlan *p)
{
    for (int C = 1; C <= rowops::CMAX; C <<= 1) {
        long long sl = ((long long)V + C - 1) / C;
        sl = (sl + 63) / 64 * 64;
        long long need = sl * bytes_per_token;
        if (need <= ROW_SMEM_BUDGET) {
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

inline int64_t up256(int64_t x) { return (x + 255) / 256 * 256; }

// workspace layout: node records | published weights + arrival counters (cleared per call) | row cuts
struct WsLayout {
    int64_t rec, pub, fin, best, done, ticket, order, cut, todo, stat, gseq, total;
};
constexpr int MAX_PARTS = 4;      // parts a row may be split into by the streaming statistics kernel
WsLayout ws_layout(const SpecIn *in, int slices = MAX_PARTS)   // slices = 0: one record per row only
{
    WsLayout L;
    const int64_t nodes = (int64_t)in->B * in->N;
    int64_t o = 0;
    L.rec = o; o += up256(nodes * (int64_t)sizeof(NodeRec));
    // set to all-ones per call: published weights, accepted nodes, earliest known acceptance; set to zero:
    // arrival counters, item counter, post-order table
    L.pub = o; o += nodes * 8;
    L.fin = o; o += (int64_t)in->B * 4;
    L.best = o; o += (int64_t)in->B * 4;
    L.done = o; o += (int64_t)in->B * 4;
    L.ticket = o; o += 4;
    o = (o + 7) / 8 * 8;
    L.order = o; o += nodes * 8;
    o = up256(o);
    L.cut = o; o += up256(nodes * 8);
    L.todo = o; o += up256(4 + nodes * 8);          // count, then ids of the rows left to the general top-k / top-p kernel
    L.stat = o; o += up256(nodes * 2 * (slices + 1) * (int64_t)sizeof(RowPart));      // one record per row, then the parts
    L.gseq = o; o += up256(nodes * KMAX * 8);       // step coefficients of every node
    L.total = o;
    return L;
}

// kernels enqueued by the library in this process (benchmarks report it)
std::atomic<long long> g_kernel_launches{0};

template <typename K>
int launch_clustered(K kernel, int ctas, int C, int threads, int smem, cudaStream_t st, void *params_ptr,
                     bool dependent = false)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas, 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // dependent: the kernel waits by itself (grid_dependency_wait) for the kernel before it in the stream, so
    // its CTAs may be placed, and run their set-up, while that kernel's last CTAs still work
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    void *args[1] = {params_ptr};
    cudaError_t e = cudaLaunchKernelExC(&cfg, (const void *)kernel, args);
    if (e != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
    return SPEC_OK;
}

std::mutex g_cache_mutex;

int sm_count()
{
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 148; }
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { cudaGetLastError(); n = 148; }
        cached[dev] = n;
    }
    return cached[dev];
}

// Kernel attributes are set once per (device, kernel): the largest dynamic shared memory asked for
// so far and the permission for clusters above 8 CTAs.  Later calls only launch.
template <typename K>
int prepare_kernel(K kernel, int C, int smem)
{
    struct Entry { const void *k; int dev, smem, big; };
    static Entry cache[256];
    static int used = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    Entry *ent = nullptr;
    for (int i = 0; i < used; ++i)
        if (cache[i].k == (const void *)kernel && cache[i].dev == dev) ent = &cache[i];
    if (!ent) {
        if (used >= 256) return SPEC_ERR_CUDA;
        ent = &cache[used++];
        *ent = Entry{(const void *)kernel, dev, -1, 0};
    }
    if (smem > ent->smem) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
        ent->smem = smem;
    }
    if (C > 8 && !ent->big) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_UNSUPPORTED; }
        ent->big = 1;
    }
    return SPEC_OK;
}

// number of clusters of this shape that can be resident at once (cached per device / kernel / shape)
template <typename K>
int resident_clusters(K kernel, int C, int threads, int smem)
{
    struct Entry { const void *k; int dev, C, smem, n; };
    static Entry cache[256];
    static int used = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    for (int i = 0; i < used; ++i)
        if (cache[i].k == (const void *)kernel && cache[i].dev == dev && cache[i].C == C && cache[i].smem == smem)
            return cache[i].n;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(C * 1024), 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, (const void *)kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
    if (used < 256) cache[used++] = Entry{(const void *)kernel, dev, C, smem, n};
    return n;
}

template <int DT, int NW, bool AN>
int launch_tree(const VPlan &pl, TParams &tp, cudaStream_t st)
{
    auto kernel = spec_tree_kernel<DT, NW, AN>;
    int rc = prepare_kernel(kernel, pl.C, pl.smem);
    if (rc) return rc;
    const int threads = (NW + 1) * 32;
    int nc = resident_clusters(kernel, pl.C, threads, pl.smem);
    if (nc <= 0) return SPEC_ERR_UNSUPPORTED;
    const long long items = (long long)tp.v.B * tp.v.N + tp.v.B;
    if (nc > items) nc = (int)items;
    return launch_clustered(kernel, nc * pl.C, pl.C, threads, pl.smem, st, &tp);
}

// row statistics (cut, reference, normaliser) of every row the verifiers read, or of every row of `z`
// when no tree is given
int launch_rowstat(const SpecIn *in, const void *zp, const void *zq, const int *parent, unsigned char *ws,
                   const WsLayout &L, cudaStream_t st)
{
    const int esz = in->logits_dtype == SPEC_BF16 ? 2 : 4;
    const int budget = 113 * 1024 - (int)sizeof(rowstat::Shared) - 2048;
    int C = 1;
    while (C <= rowstat::CMAXR && (long long)up((in->V + C - 1) / C, 8) * esz > budget) C <<= 1;
    if (C > rowstat::CMAXR) return SPEC_ERR_UNSUPPORTED;
    rowstat::RParams rp = {};
    rp.B = in->B; rp.N = in->N; rp.V = in->V; rp.C = C; rp.dtype = in->logits_dtype;
    rp.top_k = in->top_k; rp.top_p = in->top_p; rp.slice_len = up((in->V + C - 1) / C, 8);
    rp.zp = zp; rp.zq = zq; rp.seq_stride = in->seq_stride; rp.node_stride = in->node_stride;
    rp.topo_stride = in->topo_seq_stride; rp.parent = parent; rp.T = in->temperature; rp.T_seq = in->temperature_per_seq;
    rp.part = (RowPart *)(ws + L.stat); rp.cut = (float *)(ws + L.cut);
    rp.todo = (int *)(ws + L.todo); rp.only_todo = 0;
    const int smem = up(rp.slice_len * esz, 128);
    const long long items = 2ll * in->B * in->N;
    int rc, nc;
    // fast path first: one CTA per row, selection on a candidate list; the rows it cannot settle are
    // listed in the workspace and taken by the general kernel afterwards
    if (cudaMemsetAsync(rp.todo, 0, 4, st) != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    {
        const long long want = 2ll * sm_count();
        const unsigned grid = (unsigned)(items < want ? items : want);
        const bool total = in->top_p < 1.f && !(in->top_k > 0 && in->top_k < in->V);
        if (in->logits_dtype == SPEC_BF16) {
            if (total) trunc::spec_row_trunc_kernel<SPEC_BF16, true><<<grid, trunc::NT, 0, st>>>(rp);
            else trunc::spec_row_trunc_kernel<SPEC_BF16, false><<<grid, trunc::NT, 0, st>>>(rp);
        } else {
            if (total) trunc::spec_row_trunc_kernel<SPEC_F32, true><<<grid, trunc::NT, 0, st>>>(rp);
            else trunc::spec_row_trunc_kernel<SPEC_F32, false><<<grid, trunc::NT, 0, st>>>(rp);
        }
        if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
        g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
    }
    rp.only_todo = 1;
    if (in->logits_dtype == SPEC_BF16) {
        auto k = rowstat::spec_row_stat_kernel<SPEC_BF16>;
        if ((rc = prepare_kernel(k, C, smem))) return rc;
        nc = resident_clusters(k, C, rowstat::NT, smem);
        if (nc <= 0) return SPEC_ERR_UNSUPPORTED;
        if (nc > items) nc = (int)items;
        return launch_clustered(k, nc * C, C, rowstat::NT, smem, st, &rp);
    }
    auto k = rowstat::spec_row_stat_kernel<SPEC_F32>;
    if ((rc = prepare_kernel(k, C, smem))) return rc;
    nc = resident_clusters(k, C, rowstat::NT, smem);
    if (nc <= 0) return SPEC_ERR_UNSUPPORTED;
    if (nc > items) nc = (int)items;
    return launch_clustered(k, nc * C, C, rowstat::NT, smem, st, &rp);
}

// SpecInfer without diagnostic outputs: row statistics of every row, then one walk per sequence
template <int DT, int NW, int MINB, bool OT = false>
int launch_walk(const VPlan &pl, WParams &wp, cudaStream_t st)
{
    auto kernel = spec_walk_kernel<DT, NW, MINB, OT>;
    int rc = prepare_kernel(kernel, pl.C, pl.smem);
    if (rc) return rc;
    const int threads = (NW + 1) * 32;
    int nc = resident_clusters(kernel, pl.C, threads, pl.smem);
    if (nc <= 0) return SPEC_ERR_UNSUPPORTED;
    if (nc > wp.B) nc = wp.B;
    return launch_clustered(kernel, nc * pl.C, pl.C, threads, pl.smem, st, &wp, true);
}

// Statistics of every row the verifiers read (reference, normaliser, cut; one record per row at the
// start of the statistics region), and the entropy features when asked for.  `parts`: the streaming
// kernel may split rows into parts (needs the parts region of the workspace).
int row_statistics(const SpecIn *in, const SpecOut *out, unsigned char *w, const WsLayout &L, bool trunc, bool parts,
                   cudaStream_t st, bool init_nodes = false)
{
    int rc;
    int NSL = 1;
    RowPart *part = (RowPart *)(w + L.stat);
    if (trunc) {
        if (init_nodes &&
            (cudaMemsetAsync(w + L.pub, 0xFF, (size_t)(L.done - L.pub), st) != cudaSuccess ||
             cudaMemsetAsync(w + L.done, 0, (size_t)(L.order - L.done) + (size_t)in->B * in->N * 8, st) != cudaSuccess)) {
            cudaGetLastError();
            return SPEC_ERR_CUDA;
        }
        rc = launch_rowstat(in, in->target_logits, in->draft_logits, in->parent, w, L, st);
        if (rc) return rc;
    } else {
        // rows are split into parts only when there are fewer rows than resident CTAs
        const long long rows2 = 2ll * in->B * in->N;
        const int slices_row = (in->V + stream::SLICE - 1) / stream::SLICE;
        NSL = 1;
        while (parts && NSL < MAX_PARTS && NSL < slices_row && rows2 * NSL < 2 * sm_count()) NSL *= 2;
        stream::SParams sp = {};
        sp.B = in->B; sp.N = in->N; sp.V = in->V; sp.NSL = NSL;
        sp.zp = in->target_logits; sp.zq = in->draft_logits;
        sp.seq_stride = in->seq_stride; sp.node_stride = in->node_stride; sp.topo_stride = in->topo_seq_stride;
        sp.parent = in->parent; sp.T = in->temperature; sp.T_seq = in->temperature_per_seq; sp.part = part;
        // parts go to the second half of the statistics region, the merged rows to its start; a row
        // in one part is final as written.  One CTA per item: those of unread rows retire at once.
        RowPart *parts = part + 2ll * in->B * in->N;
        sp.part = NSL > 1 ? parts : part;
        if (init_nodes) {
            sp.w_pub = (unsigned long long *)(w + L.pub); sp.done = (unsigned int *)(w + L.done);
            sp.fin = (int *)(w + L.fin); sp.ticket = (unsigned int *)(w + L.ticket);
            sp.best = (unsigned int *)(w + L.best); sp.order = (unsigned long long *)(w + L.order);
        }
        const long long items = 2ll * in->B * in->N * NSL;
        const unsigned grid = (unsigned)(items < (1ll << 20) ? items : (1ll << 20));
        int prc;
        const bool feat = out->node_features != nullptr;
#define SPECV_STREAM(DTV, FT)                                                                                     \
    do {                                                                                                          \
        if ((prc = prepare_kernel(stream::spec_row_partial_kernel<DTV, FT>, 1, stream::Ring<DTV>::BYTES))) return prc; \
        stream::spec_row_partial_kernel<DTV, FT><<<grid, stream::NT, stream::Ring<DTV>::BYTES, st>>>(sp);         \
        g_kernel_launches.fetch_add(1, std::memory_order_relaxed);                                               \
    } while (0)
        if (in->logits_dtype == SPEC_BF16) { if (feat) SPECV_STREAM(SPEC_BF16, true); else SPECV_STREAM(SPEC_BF16, false); }
        else { if (feat) SPECV_STREAM(SPEC_F32, true); else SPECV_STREAM(SPEC_F32, false); }
#undef SPECV_STREAM
        if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
        if (NSL > 1) {
            stream::MParams mp = {2ll * in->B * in->N, NSL, parts, part};
            stream::spec_row_merge_kernel<<<(unsigned)((mp.rows2 * 32 + 255) / 256), 256, 0, st>>>(mp);
            g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
            if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
        }
        NSL = 1;
    }
    if (out->node_features) {
        stream::FParams fp = {(long long)in->B * in->N, NSL, part, out->node_features};
        const unsigned grid = (unsigned)(((long long)in->B * in->N * 32 + 255) / 256);
        stream::spec_features_kernel<<<grid, 256, 0, st>>>(fp);
        g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    }
    return SPEC_OK;
}

int verify_walk(const SpecIn *in, const SpecOut *out, unsigned char *w, const WsLayout &L, const VPlan &pl,
                bool trunc, bool parts, cudaStream_t st, int solver = -1)
{
    int rc = row_statistics(in, out, w, L, trunc, parts, st);
    if (rc) return rc;
    const int NSL = 1;
    RowPart *part = (RowPart *)(w + L.stat);
    WParams wp = {};
    wp.B = in->B; wp.N = in->N; wp.V = in->V; wp.C = pl.C; wp.NSL = NSL;
    wp.slice_len = pl.slice_len; wp.NS = pl.NS; wp.nsm = pl.nsm; wp.off_x = pl.off_x; wp.off_list = pl.off_list; wp.off_es = pl.off_es;
    wp.off_ring = pl.off_ring;
    wp.zp = in->target_logits; wp.zq = in->draft_logits;
    wp.seq_stride = in->seq_stride; wp.node_stride = in->node_stride; wp.topo_stride = in->topo_seq_stride;
    wp.parent = in->parent; wp.token = in->token; wp.T = in->temperature; wp.T_seq = in->temperature_per_seq;
    wp.part = part; wp.u_accept = in->u_accept; wp.u_bonus = in->u_bonus; wp.out = *out;
    const bool bf = in->logits_dtype == SPEC_BF16;
    if (solver >= 0) {
        // the walk with another OTLP solver (Algorithms 1-3): its own instantiation, two CTAs per SM
        wp.solver = solver;
        if (pl.NW == 7) return bf ? launch_walk<SPEC_BF16, 7, 2, true>(pl, wp, st) : launch_walk<SPEC_F32, 7, 2, true>(pl, wp, st);
        return bf ? launch_walk<SPEC_BF16, 15, 1, true>(pl, wp, st) : launch_walk<SPEC_F32, 15, 1, true>(pl, wp, st);
    }
    if (pl.NW == 7 && pl.whole_sm) return bf ? launch_walk<SPEC_BF16, 7, 1>(pl, wp, st) : launch_walk<SPEC_F32, 7, 1>(pl, wp, st);
    if (pl.NW == 7) return bf ? launch_walk<SPEC_BF16, 7, 2>(pl, wp, st) : launch_walk<SPEC_F32, 7, 2>(pl, wp, st);
    return bf ? launch_walk<SPEC_BF16, 15, 1>(pl, wp, st) : launch_walk<SPEC_F32, 15, 1>(pl, wp, st);
}

void fill_tparams(const SpecIn *in, const SpecOut *out, unsigned char *w, const WsLayout &L, const VPlan &pl, int mode,
                  TParams &tp)
{
    VParams &vp = tp.v;
    vp.B = in->B; vp.N = in->N; vp.V = in->V; vp.C = pl.C; vp.mode = mode;
    vp.all_thr = (out->node_thr != nullptr || out->margin != nullptr) ? 1 : 0;
    vp.slice_len = pl.slice_len; vp.NS = pl.NS; vp.nsm = pl.nsm;
    vp.off_x = pl.off_x; vp.off_list = pl.off_list; vp.off_es = pl.off_es; vp.off_ring = pl.off_ring;
    vp.zp = in->target_logits; vp.zq = in->draft_logits;
    vp.seq_stride = in->seq_stride; vp.node_stride = in->node_stride; vp.topo_stride = in->topo_seq_stride;
    vp.parent = in->parent; vp.token = in->token;
    vp.T = in->temperature; vp.T_seq = in->temperature_per_seq;
    vp.u_accept = in->u_accept; vp.u_bonus = in->u_bonus;
    vp.rec = (NodeRec *)(w + L.rec);
    vp.w_pub = (unsigned long long *)(w + L.pub);
    vp.done = (unsigned int *)(w + L.done);
    vp.fin = (int *)(w + L.fin);
    vp.best = (unsigned int *)(w + L.best);
    vp.order = (unsigned long long *)(w + L.order);
    // Traversal without per-node diagnostics: subtrees that come after a known acceptance in the traversal
    // order are not evaluated
    vp.prune = (mode == MODE_TRAVERSAL && !out->node_thr && !out->node_w_in && !out->margin) ? 1 : 0;
    vp.out = *out;
    tp.part = (const RowPart *)(w + L.stat);
    tp.gseq = (double *)(w + L.gseq);
    tp.ticket = (unsigned int *)(w + L.ticket);
}

int launch_tree_any(const SpecIn *in, const VPlan &pl, TParams &tp, bool analysis, cudaStream_t st)
{
    const bool bf = in->logits_dtype == SPEC_BF16;
    if (analysis) {
        if (pl.NW == 7) return bf ? launch_tree<SPEC_BF16, 7, true>(pl, tp, st) : launch_tree<SPEC_F32, 7, true>(pl, tp, st);
        return bf ? launch_tree<SPEC_BF16, 15, true>(pl, tp, st) : launch_tree<SPEC_F32, 15, true>(pl, tp, st);
    }
    if (pl.NW == 7) return bf ? launch_tree<SPEC_BF16, 7, false>(pl, tp, st) : launch_tree<SPEC_F32, 7, false>(pl, tp, st);
    return bf ? launch_tree<SPEC_BF16, 15, false>(pl, tp, st) : launch_tree<SPEC_F32, 15, false>(pl, tp, st);
}

int verify_common(const SpecIn *in, const SpecOut *out, void *ws, int64_t ws_bytes, void *stream, int mode,
                  bool parts = true)
{
    int rc = check_in(in, true);
    if (rc) return rc;
    if (!out || !out->accepted_node || !out->accept_len || !out->out_tokens || !out->bonus_token || !out->status)
        return SPEC_ERR_NULL;
    const bool trunc = (in->top_k > 0 && in->top_k < in->V) || in->top_p < 1.f;
    const WsLayout L = ws_layout(in, parts ? MAX_PARTS : 0);
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < L.total) return SPEC_ERR_WORKSPACE;
    VPlan pl;
    if (!make_vplan(in->V, in->logits_dtype, &pl)) return SPEC_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char *w = (unsigned char *)ws;
    const bool diagnostics = out->residual || out->node_thr || out->node_w_in || out->margin;
    if (mode == MODE_SPECINFER && !diagnostics && in->N <= NWALK) {
        // the walk keeps one cluster per sequence busy: when all of them fit on the chip with one CTA
        // per SM, each CTA may use the whole SM's shared memory for its ring and twice the registers
        VPlan wpl;
        if (!make_vplan(in->V, in->logits_dtype, &wpl, (int)sizeof(WHdr), false)) return SPEC_ERR_UNSUPPORTED;
        if ((long long)in->B * wpl.C <= sm_count()) {
            VPlan big;
            if (make_vplan(in->V, in->logits_dtype, &big, (int)sizeof(WHdr), true, wpl.C, wpl.NW)) { wpl = big; wpl.whole_sm = 1; }
        }
        return verify_walk(in, out, w, L, wpl, trunc, parts, st);
    }
    // every node of every sequence on chip once, on top of the row statistics (which also set the
    // published-weight slots to pending and the arrival counters to zero)
    rc = row_statistics(in, out, w, L, trunc, parts, st, true);
    if (rc) return rc;
    TParams tp = {};
    fill_tparams(in, out, w, L, pl, mode, tp);
    VParams &vp = tp.v;
    rc = launch_tree_any(in, pl, tp, false, st);
    if (rc) return rc;
    if (out->residual) {
        RParams rp = {};
        rp.B = in->B; rp.N = in->N; rp.V = in->V; rp.dtype = in->logits_dtype;
        rp.zp = in->target_logits; rp.zq = in->draft_logits;
        rp.seq_stride = in->seq_stride; rp.node_stride = in->node_stride;
        rp.T = in->temperature; rp.T_seq = in->temperature_per_seq;
        rp.rec = vp.rec; rp.gseq = tp.gseq; rp.accepted = out->accepted_node; rp.residual = out->residual;
        int gx = (in->V + 255) / 256;
        if (gx > 296) gx = 296;
        spec_residual_kernel<<<dim3(gx, in->B), 256, 0, st>>>(rp);
        g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
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
    L.ws = o; o += up256(ws_layout(in).total);
    L.total = o;
    return L;
}

// ------------------------------------------------------------------------------------------------
// scratch that lives inside the library image, for spec_verify_specinfer_static
// ------------------------------------------------------------------------------------------------
constexpr int64_t STATIC_WS_BYTES = SPEC_STATIC_WS_BYTES;
static __device__ __align__(256) unsigned char g_static_ws[STATIC_WS_BYTES];

// Device address of g_static_ws on the current device.  In host code the array's name is only a
// handle for the runtime, never a device pointer, so the address is asked for once per device (with
// that device current) and remembered.
int static_ws_address(void **ptr)
{
    static void *addr[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) { cudaGetLastError(); return SPEC_ERR_CUDA; }
        addr[dev] = p;
    }
    *ptr = addr[dev];
    return SPEC_OK;
}

}  // namespace
}  // namespace specv

using namespace specv;

extern "C" {

int32_t spec_workspace_bytes(const SpecIn *in, int64_t *bytes)
{
    if (!in || !bytes) return SPEC_ERR_NULL;
    if (in->B <= 0 || in->N <= 0 || in->N > SPEC_MAX_NODES || (long long)in->B * in->N > (1ll << 24))
        return SPEC_ERR_SHAPE;
    *bytes = ws_layout(in).total;
    return SPEC_OK;
}

int32_t spec_query_plan(int32_t V, int32_t logits_dtype, int32_t *cluster_size, int32_t *slice_len,
                        int32_t *smem_bytes, int32_t *threads)
{
    if (V <= 0) return SPEC_ERR_SHAPE;
    if (logits_dtype != SPEC_F32 && logits_dtype != SPEC_BF16) return SPEC_ERR_DTYPE;
    VPlan pl;
    if (!make_vplan(V, logits_dtype, &pl)) return SPEC_ERR_UNSUPPORTED;
    if (cluster_size) *cluster_size = pl.C;
    if (slice_len) *slice_len = pl.slice_len;
    if (smem_bytes) *smem_bytes = pl.smem;
    if (threads) *threads = (pl.NW + 1) * 32;
    return SPEC_OK;
}

int64_t spec_kernel_launches(void) { return (int64_t)g_kernel_launches.load(std::memory_order_relaxed); }

int32_t spec_test_hooks(int64_t wait_cycles, int32_t hold_slot)
{
    const long long wc = wait_cycles > 0 ? (long long)wait_cycles : WAIT_CYCLES_DEFAULT;
    const int hs = hold_slot;
    if (cudaMemcpyToSymbol(c_wait_cycles, &wc, sizeof(wc)) != cudaSuccess ||
        cudaMemcpyToSymbol(c_hold_slot, &hs, sizeof(hs)) != cudaSuccess) {
        cudaGetLastError();
        return SPEC_ERR_CUDA;
    }
    return SPEC_OK;
}

int32_t spec_row_statistics(const SpecIn *in, void *ws, int64_t ws_bytes, void *stream)
{
    int rc = check_in(in, true);
    if (rc) return rc;
    const bool trunc = (in->top_k > 0 && in->top_k < in->V) || in->top_p < 1.f;
    const WsLayout L = ws_layout(in);
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < L.total) return SPEC_ERR_WORKSPACE;
    SpecOut none = {};
    return row_statistics(in, &none, (unsigned char *)ws, L, trunc, true, (cudaStream_t)stream, true);
}

int32_t spec_verify_specinfer(const SpecIn *in, const SpecOut *out, void *ws, int64_t ws_bytes, void *stream)
{
    return verify_common(in, out, ws, ws_bytes, stream, MODE_SPECINFER);
}

int32_t spec_verify_traversal(const SpecIn *in, const SpecOut *out, void *ws, int64_t ws_bytes, void *stream)
{
    return verify_common(in, out, ws, ws_bytes, stream, MODE_TRAVERSAL);
}

int32_t spec_verify_otlp(const SpecIn *in, const SpecOut *out, int32_t solver, void *ws, int64_t ws_bytes, void *stream)
{
    int rc = check_in(in, true);
    if (rc) return rc;
    if (!out || !out->accepted_node || !out->accept_len || !out->out_tokens || !out->bonus_token || !out->status)
        return SPEC_ERR_NULL;
    if (solver < 0 || solver > 2) return SPEC_ERR_PARAM;
    if (out->residual || out->node_thr || out->node_w_in || out->margin || out->node_features || in->N > NWALK)
        return SPEC_ERR_UNSUPPORTED;
    const bool trunc = (in->top_k > 0 && in->top_k < in->V) || in->top_p < 1.f;
    const WsLayout L = ws_layout(in);
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < L.total) return SPEC_ERR_WORKSPACE;
    VPlan wpl;
    if (!make_vplan(in->V, in->logits_dtype, &wpl, (int)sizeof(WHdr), false)) return SPEC_ERR_UNSUPPORTED;
    return verify_walk(in, out, (unsigned char *)ws, L, wpl, trunc, true, (cudaStream_t)stream, solver);
}

int32_t spec_verify_specinfer_static(const SpecIn *in, const SpecOut *out, void *stream)
{
    int rc = check_in(in, true);
    if (rc) return rc;
    if ((int64_t)in->B * in->N > SPEC_STATIC_MAX_NODES || ws_layout(in, 0).total > STATIC_WS_BYTES) return SPEC_ERR_WORKSPACE;
    void *ws = nullptr;
    rc = static_ws_address(&ws);
    if (rc) return rc;
    return verify_common(in, out, ws, STATIC_WS_BYTES, stream, MODE_SPECINFER, false);
}

// analysis workspace: the verifiers' layout | per-node scalars | scratch for the decision outputs nobody reads
struct AnLayout {
    int64_t an, acc, len, toks, bonus, status, total;
};
static AnLayout an_layout(const SpecIn *in)
{
    AnLayout A;
    const int64_t nodes = (int64_t)in->B * in->N;
    int64_t o = up256(ws_layout(in).total);
    A.an = o; o += up256(nodes * (int64_t)sizeof(AnRec));
    A.acc = o; o += up256((int64_t)in->B * 4);
    A.len = o; o += up256((int64_t)in->B * 4);
    A.toks = o; o += up256(nodes * 4);
    A.bonus = o; o += up256((int64_t)in->B * 4);
    A.status = o; o += up256((int64_t)in->B * 4);
    A.total = o;
    return A;
}

int32_t spec_analysis_workspace_bytes(const SpecIn *in, int64_t *bytes)
{
    if (!in || !bytes) return SPEC_ERR_NULL;
    if (in->B <= 0 || in->N <= 0 || in->N > SPEC_MAX_NODES || (long long)in->B * in->N > (1ll << 24))
        return SPEC_ERR_SHAPE;
    *bytes = an_layout(in).total;
    return SPEC_OK;
}

int32_t spec_tree_analysis(const SpecIn *in, const SpecAnalysisOut *out, void *ws, int64_t ws_bytes, void *stream)
{
    int rc = check_in(in, true);
    if (rc) return rc;
    if (!out || !out->acceptance || !out->divergence || !out->branch || !out->reach || !out->block_eff) return SPEC_ERR_NULL;
    const bool trunc = (in->top_k > 0 && in->top_k < in->V) || in->top_p < 1.f;
    const WsLayout L = ws_layout(in);
    const AnLayout A = an_layout(in);
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < A.total) return SPEC_ERR_WORKSPACE;
    VPlan pl;
    if (!make_vplan(in->V, in->logits_dtype, &pl)) return SPEC_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char *w = (unsigned char *)ws;
    const int64_t nodes = (int64_t)in->B * in->N;
    // outputs start as NaN (all-ones), the per-node scalars as "no children"
    bool ok = true;
    ok &= cudaMemsetAsync(out->acceptance, 0xFF, (size_t)nodes * 16, st) == cudaSuccess;
    ok &= cudaMemsetAsync(out->divergence, 0xFF, (size_t)nodes * 12, st) == cudaSuccess;
    ok &= cudaMemsetAsync(out->branch, 0xFF, (size_t)nodes * 4 * analysis::NSOLVER, st) == cudaSuccess;
    ok &= cudaMemsetAsync(w + A.an, 0, (size_t)nodes * sizeof(AnRec), st) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    SpecOut so = {};
    so.accepted_node = (int32_t *)(w + A.acc); so.accept_len = (int32_t *)(w + A.len);
    so.out_tokens = (int32_t *)(w + A.toks); so.bonus_token = (int32_t *)(w + A.bonus);
    so.status = (int32_t *)(w + A.status);
    rc = row_statistics(in, &so, w, L, trunc, true, st, true);
    if (rc) return rc;
    TParams tp = {};
    fill_tparams(in, &so, w, L, pl, MODE_SPECINFER, tp);
    tp.v.all_thr = 1;
    tp.an = (AnRec *)(w + A.an); tp.an_acc = out->acceptance; tp.an_div = out->divergence;
    rc = launch_tree_any(in, pl, tp, true, st);
    if (rc) return rc;
    analysis::BParams bp = {in->B, in->N, in->parent, in->token, in->topo_seq_stride, tp.an, out->acceptance, out->branch};
    analysis::spec_branch_kernel<<<(unsigned)((nodes + 3) / 4), 128, 0, st>>>(bp);
    g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
    analysis::RParams rp = {in->B, in->N, in->parent, in->topo_seq_stride, out->branch, out->reach, out->block_eff};
    analysis::spec_reach_kernel<<<(unsigned)((analysis::NSOLVER * in->B + 127) / 128), 128, 0, st>>>(rp);
    g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
    if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    return SPEC_OK;
}

int32_t spec_latency_model(const double *t_q, const double *t_p, int32_t n_len, int32_t ctx, const int32_t *actions,
                           int32_t n_actions, double *T_hat, void *stream)
{
    if (!t_q || !t_p || !actions || !T_hat) return SPEC_ERR_NULL;
    if (n_len <= 0 || n_actions <= 0 || ctx < 0) return SPEC_ERR_SHAPE;
    analysis::LParams lp = {t_q, t_p, n_len, ctx, n_actions, actions, T_hat};
    analysis::spec_latency_kernel<<<(unsigned)((n_actions + 127) / 128), 128, 0, (cudaStream_t)stream>>>(lp);
    g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
    if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    return SPEC_OK;
}

int32_t spec_tree_probs(const SpecIn *in, int32_t which, float *probs, float *row_stats, void *ws,
                        int64_t ws_bytes, void *stream)
{
    int rc = check_in(in, false);
    if (rc) return rc;
    if (which != 0 && which != 1) return SPEC_ERR_PARAM;
    const void *z = which ? in->draft_logits : in->target_logits;
    if (!z || (!probs && !row_stats)) return SPEC_ERR_NULL;
    const bool trunc = (in->top_k > 0 && in->top_k < in->V) || in->top_p < 1.f;
    const float *cutp = nullptr;
    if (trunc) {
        // the cuts of every row of the chosen side go to slot 0 of every pair in the workspace
        const WsLayout L = ws_layout(in);
        if (!ws || ((uintptr_t)ws & 255) || ws_bytes < L.total) return SPEC_ERR_WORKSPACE;
        rc = launch_rowstat(in, z, z, nullptr, (unsigned char *)ws, L, (cudaStream_t)stream);
        if (rc) return rc;
        cutp = (const float *)((unsigned char *)ws + L.cut);
    }
    RowPlan pl;
    if (!make_row_plan(in->V, 4, &pl)) return SPEC_ERR_UNSUPPORTED;
    rowops::TParams tp = {};
    tp.rows = in->B * in->N; tp.N = in->N; tp.V = in->V; tp.dtype = in->logits_dtype; tp.SL = pl.SL;
    tp.z = z; tp.seq_stride = in->seq_stride; tp.node_stride = in->node_stride;
    tp.T = in->temperature; tp.T_seq = in->temperature_per_seq; tp.probs = probs; tp.stats = row_stats;
    tp.cut = cutp; tp.which = 0;
    rc = prepare_kernel(rowops::spec_probs_kernel, pl.C, pl.smem);
    if (rc) return rc;
    return launch_clustered(rowops::spec_probs_kernel, tp.rows * pl.C, pl.C, rowops::NT, pl.smem, (cudaStream_t)stream, &tp);
}

int32_t spec_sample_bonus(const float *weights, int32_t R, int32_t V, const float *u, int32_t *token,
                          float *margin, void *ws, int64_t ws_bytes, void *stream)
{
    (void)ws; (void)ws_bytes;
    if (!weights || !u || !token) return SPEC_ERR_NULL;
    if (R <= 0 || V <= 0) return SPEC_ERR_SHAPE;
    RowPlan pl;
    if (!make_row_plan(V, 4, &pl)) return SPEC_ERR_UNSUPPORTED;
    rowops::BParams bp = {R, V, pl.SL, weights, u, token, margin};
    int rc = prepare_kernel(rowops::spec_bonus_kernel, pl.C, pl.smem);
    if (rc) return rc;
    return launch_clustered(rowops::spec_bonus_kernel, R * pl.C, pl.C, rowops::NT, pl.smem, (cudaStream_t)stream, &bp);
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
