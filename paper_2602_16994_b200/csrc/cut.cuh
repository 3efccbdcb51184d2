// Row cut values for top-k / top-p truncation (the paper's experimental setup names temperature and
// nucleus sampling; top-k is an addition of the workloads): constants and the key transform; the
// selection itself runs inside the row-statistics kernels (trunc.cuh: the fast path on candidates;
// rowstat.cuh: the general kernel for the rows the fast path leaves over).  The cut of a row is the
// smallest kept logit VALUE:
//   top-k: the k-th largest logit value (ties at that value are all kept);
//   top-p: within the top-k set, tokens of equal logit form a group; groups in descending order; the
//          cut is the value of the first group at which the cumulative mass reaches top_p times the
//          mass of the set.
// Both are radix selections on an order-preserving integer image of the logit (sign-flipped bits,
// -0 folded into +0), 11 bits per level from the top, so equal logits can never be separated and the
// answer does not depend on token order.  Counts are integers; masses are accumulated as 64-bit fixed
// point (2^44 per unit of e = exp((z - max)/T)), so every sum is exact and order-free.  (One exception:
// for top-p without top-k the fast path sums the mass of the whole row, which only fixes the target,
// in floating point to about 1e-7 relative; the masses of the candidates stay exact.)
#pragma once
#include "common.cuh"

namespace specv {
namespace cut {

constexpr int NBITS = 11;
constexpr int NB = 1 << NBITS;          // bins per level
constexpr double FIX = 17592186044416.0;   // 2^44

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

}  // namespace cut
}  // namespace specv
