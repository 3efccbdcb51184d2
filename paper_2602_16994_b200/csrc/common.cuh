// Shared device helpers of libspecverify (sm_100a): mbarrier / bulk-copy / cluster PTX wrappers,
// bounded waits, exact power-of-two scaling and small warp utilities.
#pragma once
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "specverify.h"

namespace specv {

constexpr int KMAX = SPEC_MAX_CHILDREN;
// Every on-device wait gives up after this many clock cycles (about 2 s).  A variable and not a constant so
// that a test can shorten it (spec_test_hooks) and watch a wait run out without waiting for seconds.
constexpr long long WAIT_CYCLES_DEFAULT = 4000000000ll;
__constant__ long long c_wait_cycles = WAIT_CYCLES_DEFAULT;
// Test hook: index b * N + node of a published-weight slot that the every-node kernel leaves pending (-1: none)
__constant__ int c_hold_slot = -1;
#define WAIT_CYCLES c_wait_cycles
constexpr unsigned long long W_PENDING = 0xFFFFFFFFFFFFFFFFull;

extern __shared__ __align__(128) unsigned char dyn_smem[];

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier ----------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t *bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded waits: false when the limit ran out (the caller flags the error and carries on).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > WAIT_CYCLES) return false;
    return true;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity)
{
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait_cluster(bar, parity))
        if (clock64() - t0 > WAIT_CYCLES) return false;
    return true;
}

// ---- programmatic dependent launch: a kernel launched with the stream-serialisation attribute may start
// while the kernel before it still runs; it waits here before touching anything that kernel writes (a
// no-op for a kernel launched without the attribute).  The earlier kernel lets its dependents be scheduled
// with the second call; its memory is visible to them only after the wait.
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void grid_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---- bulk asynchronous copy global -> shared, completing on an mbarrier (no multicast) -----------
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// ---- cluster -----------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// remote store of 8 bytes that counts on the receiver's mbarrier (same offsets in CTA `rank`)
__device__ __forceinline__ void st_async_f64(double *slot, uint64_t *bar, uint32_t rank, double v)
{
    asm volatile(
        "{\n\t.reg .b32 ra, rb;\n\tmapa.shared::cluster.u32 ra, %0, %2;\n\tmapa.shared::cluster.u32 rb, %1, %2;\n\t"
        "st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b64 [ra], %3, [rb];\n\t}" ::"r"(smem_u32(slot)),
        "r"(smem_u32(bar)), "r"(rank), "l"(__double_as_longlong(v))
        : "memory");
}
// named barrier for a subset of the CTA's warps
__device__ __forceinline__ void bar_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// ---- arithmetic --------------------------------------------------------------------------------
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^k for an integer k: exact; k <= -127 gives 0, k is clamped at 127
__device__ __forceinline__ float pow2i(int k)
{
    k = max(-127, min(127, k));
    return __int_as_float((k + 127) << 23);
}
// 2^k as a double, k clamped to the normal range (k <= -1023 gives 0)
__device__ __forceinline__ double pow2d(int k)
{
    k = min(k, 1023);
    return k < -1022 ? 0.0 : __hiloint2double((k + 1023) << 20, 0);
}
// 2^f for |f| <= 0.5 to about 1e-15 (Taylor series of exp(f ln 2), degree 13)
__device__ __forceinline__ double exp2_frac(double f)
{
    const double t = f * 0.6931471805599453094;
    double p = 1.0 / 6227020800.0;
    p = fma(p, t, 1.0 / 479001600.0); p = fma(p, t, 1.0 / 39916800.0); p = fma(p, t, 1.0 / 3628800.0);
    p = fma(p, t, 1.0 / 362880.0); p = fma(p, t, 1.0 / 40320.0); p = fma(p, t, 1.0 / 5040.0);
    p = fma(p, t, 1.0 / 720.0); p = fma(p, t, 1.0 / 120.0); p = fma(p, t, 1.0 / 24.0);
    p = fma(p, t, 1.0 / 6.0); p = fma(p, t, 0.5); p = fma(p, t, 1.0); p = fma(p, t, 1.0);
    return p;
}
// fp32 pairs in one 64-bit register: packed fused multiply-add and add (sm_100)
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c)
{
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b)
{
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ void split_float(double g, float &hi, float &lo)
{
    hi = (float)g;
    lo = (float)(g - (double)hi);
}
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// The cluster kernels run long stretches of code once per node or sequence; there the time goes into
// fetching instructions, not executing them, so their helpers exist once (not inlined) and are warm
// in the instruction cache after the first call.
__device__ __noinline__ double warp_sum_once(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __noinline__ double exp2_frac_once(double f) { return exp2_frac(f); }
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float load_logit(const void *base, int dtype, long long idx)
{
    if (dtype == SPEC_F32) return __ldg((const float *)base + idx);
    return __uint_as_float((uint32_t)__ldg((const unsigned short *)base + idx) << 16);
}

// ---- per-node record in the workspace --------------------------------------------------------------
struct __align__(16) NodeRec {
    double O_p, Z_p, O_q, Z_q;   // row reference (log2 units, an integer) and sum of kept 2^(z s - O)
    double kappa;                // total of the node's final state u (see verify.cuh)
    double w_in;                 // Traversal: weight handed down by the parent
    double thr;                  // threshold the node is tested with
    float cut_p, cut_q;          // smallest kept logit value (-inf: nothing cut)
    float bonus_margin;
    int next_child;              // SpecInfer: accepted child or -1
    int bonus;                   // bonus token this node would emit, or -1
    int status;
    int nsteps;                  // sibling steps its final state went through; STATE_IS_Q: the state equals q
    int pad;
};
constexpr int STATE_IS_Q = -1;

}  // namespace specv
