// Fixed-order float sums over the rows of a bucket, shared by the codec variants whose scale or
// reconstruction values are sums (L2 norm, class means): the per-row values are the leaves of a
// balanced binary tree of adjacent pairs, the leaf count padded with zeros to a power of two.
// Adding +0 is exact, so evaluating more (all-zero) leaves or levels than the padded tree has
// does not change the result.
#pragma once

#include "mqg_common.cuh"

namespace mqg {

// Five tree levels inside a warp: lane l holds the sum of rows (l & ~(2d - 1)) .. + 2d - 1 after
// the step with distance d.  Both partners compute the same sum (addition commutes bit for bit).
__device__ __forceinline__ float warp_tree(float a, uint32_t levels_end)
{
    for (uint32_t d = 1; d < levels_end; d <<= 1)
        a = __fadd_rn(a, __shfl_xor_sync(0xFFFFFFFFu, a, d));
    return a;
}

// Tree over `count` <= 8 values v[first .. first + count) padded with zeros to eight leaves.
__device__ __forceinline__ float tree8(const float* v, uint32_t first, uint32_t count)
{
    float x[8];
#pragma unroll
    for (uint32_t i = 0; i < 8; ++i) x[i] = i < count ? v[first + i] : 0.0f;
    return __fadd_rn(__fadd_rn(__fadd_rn(x[0], x[1]), __fadd_rn(x[2], x[3])),
                     __fadd_rn(__fadd_rn(x[4], x[5]), __fadd_rn(x[6], x[7])));
}

// The bucket's sum from the per-row values of a 256-thread tile that holds whole buckets of `rpb` rows
// (thread t owns row t of the tile; threads without a row pass 0).  Every thread of the CTA must
// call it.  s_part: kMaxTileRows floats of shared memory, free for reuse after the call's last
// barrier only.
__device__ __forceinline__ float bucket_tree_sum(float a, uint32_t rpb, float* s_part)
{
    const uint32_t t = threadIdx.x;
    if ((rpb & (rpb - 1)) == 0 && rpb <= 32) return warp_tree(a, rpb);
    if (rpb % 32 == 0) {
        a = warp_tree(a, 32);
        if ((t & 31) == 0) s_part[t >> 5] = a;
        __syncthreads();
        const uint32_t wpb = rpb / 32;
        const uint32_t first = (t / rpb) * wpb;
        return first + wpb <= kMaxTileRows / 32 ? tree8(s_part, first, wpb) : 0.0f;
    }
    // any other shape: one tree level per barrier pair, in place
    s_part[t] = a;
    __syncthreads();
    const uint32_t b0 = (t / rpb) * rpb, j = t - b0;
    for (uint32_t d = 1; d < rpb; d <<= 1) {
        const bool node = (j & (2 * d - 1)) == 0;
        float v = 0.0f;
        if (node) {
            v = s_part[t];
            if (j + d < rpb && t + d < (uint32_t)kMaxTileRows) v = __fadd_rn(v, s_part[t + d]);
        }
        __syncthreads();
        if (node) s_part[t] = v;
        __syncthreads();
    }
    return b0 < (uint32_t)kMaxTileRows ? s_part[b0] : 0.0f;
}

}  // namespace mqg
