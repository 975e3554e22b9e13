// fp64 building blocks for tensors of at most 64 elements: the pair operator applied by one warp
// to two vectors in shared memory, and the whole tree by one warp (the single-launch kernel uses
// that; the kernel in adasum_short.cu spreads the pairs of a level over the warps of a block).
#pragma once

#include <stdint.h>

namespace adasum {

constexpr int kShortSlotElems = 64;       // doubles per leaf slot = the longest short tensor

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1)
        v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

// a <- Adasum(a, b) for vectors of len <= 64 doubles in shared memory, by one warp.
__device__ __forceinline__ void pair_in_place(double* a, const double* b, int len, int lane)
{
    const double a0 = lane < len ? a[lane] : 0.0, a1 = lane + 32 < len ? a[lane + 32] : 0.0;
    const double b0 = lane < len ? b[lane] : 0.0, b1 = lane + 32 < len ? b[lane + 32] : 0.0;
    const double dot = warp_sum(a0 * b0 + a1 * b1);
    const double na = warp_sum(a0 * a0 + a1 * a1);
    const double nb = warp_sum(b0 * b0 + b1 * b1);
    // Algorithm 1, "Apply Adasum"; an operand with zero squared norm keeps coefficient 1
    const double ca = na == 0.0 ? 1.0 : 1.0 - dot / (2.0 * na);
    const double cb = nb == 0.0 ? 1.0 : 1.0 - dot / (2.0 * nb);
    if (lane < len)
        a[lane] = ca * a0 + cb * b0;
    if (lane + 32 < len)
        a[lane + 32] = ca * a1 + cb * b1;
}


// The tree over slot[0 .. n) (each kShortSlotElems doubles) by ONE warp; the result ends in slot[0].
// order: 0 bottom-up pairs with carry, 1 sequential, 2 top-down halves.
__device__ __forceinline__ void warp_tree_in_place(double* slot, int n, int len, int order)
{
    const int lane = threadIdx.x & 31;
    if (order == 1) {
        for (int k = 1; k < n; ++k) {
            pair_in_place(slot, slot + k * kShortSlotElems, len, lane);
            __syncwarp();
        }
    } else if (order == 2) {
        int max_depth = 0;
        while ((1 << max_depth) < n)
            ++max_depth;
        for (int depth = max_depth - 1; depth >= 0; --depth) {
            for (int j = 0; j < (1 << depth); ++j) {
                int lo = 0, hi = n;
                bool alive = true;
                for (int t = 0; t < depth && alive; ++t) {
                    if (hi - lo < 2) {
                        alive = false;
                    } else {
                        const int m = lo + (hi - lo) / 2;
                        if ((j >> (depth - 1 - t)) & 1)
                            lo = m;
                        else
                            hi = m;
                    }
                }
                if (alive && hi - lo >= 2) {
                    pair_in_place(slot + lo * kShortSlotElems, slot + (lo + (hi - lo) / 2) * kShortSlotElems, len, lane);
                    __syncwarp();
                }
            }
        }
    } else {
        for (int w = 1; w < n; w *= 2)
            for (int left = 0; left + w < n; left += 2 * w) {
                pair_in_place(slot + left * kShortSlotElems, slot + (left + w) * kShortSlotElems, len, lane);
                __syncwarp();
            }
    }
}

}  // namespace adasum
