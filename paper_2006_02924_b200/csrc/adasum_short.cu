// Tensors of at most kShortTensorElems elements, reduced in fp64 from the loads to the store.
//
// The result of the tree is sum_i w_i g_i with weights that can be large and of both signs while
// the sum is small (a one-element tensor whose workers disagree in sign); the streaming kernels'
// fp32 products, weights and sums then lose what cancels.  Section 4.4.1 accumulates in double for
// this reason.  For long tensors the cancellation averages out and fp32 partial sums over a few
// thousand elements are enough; for tensors this short the whole tree costs next to nothing in
// fp64, so they are taken out of the streaming kernels' segment tables and handled here, with the
// operator applied literally: dot product and squared norms of a pair, the two coefficients, the
// combination, level after level (Section 3.4; Algorithm 1's order).
//
// One block per short tensor.  The leaves are converted to fp64 in shared memory,
// kShortChunkLeaves at a time (a chunk of 2^k adjacent leaves is a complete sub-tree); a warp
// handles one pair: each lane holds two elements of either operand, the three sums are
// butterfly-reduced in fp64 (every lane ends with the same bits), the combination is written over
// the left operand.  Slots: at width w the operands of the level sit at the multiples of w, and an
// operand without a right sibling simply stays where it is (the carry rule for odd counts).
#include "adasum_internal.h"

namespace adasum {
namespace {

static_assert(kShortTensorElems == kShortSlotElems, "a leaf slot holds the longest short tensor");
constexpr int kShortThreads = 256;
constexpr int kShortWarps = kShortThreads / 32;
constexpr int kShortMaxChunks = kMaxOperandsPerLaunch / kShortChunkLeaves;

template <typename T>
__device__ __forceinline__ double short_load(const void* p, const void* start, int64_t e)
{
    const T* src = static_cast<const T*>(p);
    if (start != nullptr)
        return (double)delta_one(src, static_cast<const T*>(start), e);
    return (double)Element<T>::one(src + e);
}
template <>
__device__ __forceinline__ double short_load<double>(const void* p, const void*, int64_t e)
{
    return static_cast<const double*>(p)[e];
}

// The tree over slot[0 .. n) (each kShortTensorElems doubles); the result ends in slot[0].
// Called by the whole block; ends with a block barrier.
__device__ void tree_in_place(double* slot, int n, int len, int order)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (order == 1) {
        // sequential recursion: x = g_0, then x = Adasum(x, g_k)
        if (warp == 0) {
            for (int k = 1; k < n; ++k) {
                pair_in_place(slot, slot + k * kShortTensorElems, len, lane);
                __syncwarp();
            }
        }
        __syncthreads();
    } else if (order == 2) {
        // top-down halves: the node over [lo, hi) combines [lo, mid) and [mid, hi), mid = lo + (hi - lo) / 2;
        // deepest nodes first; node j of a depth is found by walking down from the root along j's bits
        int max_depth = 0;
        while ((1 << max_depth) < n)
            ++max_depth;
        for (int depth = max_depth - 1; depth >= 0; --depth) {
            for (int j = warp; j < (1 << depth); j += kShortWarps) {
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
                    const int mid = lo + (hi - lo) / 2;
                    pair_in_place(slot + lo * kShortTensorElems, slot + mid * kShortTensorElems, len, lane);
                }
            }
            __syncthreads();
        }
    } else {
        for (int w = 1; w < n; w *= 2) {
            for (int left = 2 * w * warp; left + w < n; left += 2 * w * kShortWarps)
                pair_in_place(slot + left * kShortTensorElems, slot + (left + w) * kShortTensorElems, len, lane);
            __syncthreads();
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kShortThreads)
short_tensor_kernel(const __grid_constant__ OperandTable ops, int operands, ShortArgs a)
{
    __shared__ double slot[kShortChunkLeaves * kShortTensorElems];      // 32 KB
    __shared__ double chunk_result[kShortMaxChunks * kShortTensorElems];
    __shared__ double leaf_norm[kShortChunkLeaves];
    const ShortTensor st = a.table[blockIdx.x];
    const int len = st.len;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = (operands + kShortChunkLeaves - 1) / kShortChunkLeaves;
    const bool want_sums = a.leaf_sum_in == nullptr && (a.orthogonality != nullptr || a.leaf_sum_out != nullptr);
    const int64_t first_elem = a.leaf_sum_in != nullptr ? st.packed : st.begin;
    double leaf_sum = 0.0;        // thread 0

    for (int c = 0; c < chunks; ++c) {
        const int first = c * kShortChunkLeaves;
        const int n = min(kShortChunkLeaves, operands - first);
        for (int idx = threadIdx.x; idx < n * len; idx += kShortThreads) {
            const int i = idx / len, e = idx - i * len;
            double x = short_load<T>(ops.ptr[first + i], a.start, first_elem + e);
            if (a.leaf_scales != nullptr)      // the buffer holds scale x gradient (Section 4.4.1)
                x /= (double)a.leaf_scales[(int64_t)(a.worker_base + first + i) * a.num_tensors + st.tensor];
            slot[i * kShortTensorElems + e] = x;
        }
        __syncthreads();
        if (want_sums) {
            for (int i = warp; i < n; i += kShortWarps) {
                const double x0 = lane < len ? slot[i * kShortTensorElems + lane] : 0.0;
                const double x1 = lane + 32 < len ? slot[i * kShortTensorElems + lane + 32] : 0.0;
                const double s = warp_sum(x0 * x0 + x1 * x1);
                if (lane == 0)
                    leaf_norm[i] = s;
            }
            __syncthreads();
            if (threadIdx.x == 0)
                for (int i = 0; i < n; ++i)
                    leaf_sum += leaf_norm[i];
        }
        tree_in_place(slot, n, len, chunks > 1 ? 0 : a.order);
        if (threadIdx.x < len)
            chunk_result[c * kShortTensorElems + threadIdx.x] = slot[threadIdx.x];
        __syncthreads();
    }
    if (chunks > 1)
        tree_in_place(chunk_result, chunks, len, 0);

    // the sum of the leaves' squared norms, when the leaves were earlier launches' sub-trees
    if (threadIdx.x == 0 && a.leaf_sum_in != nullptr)
        for (int j = 0; j < a.leaf_sum_launches; ++j)
            leaf_sum += a.leaf_sum_in[(int64_t)j * a.leaf_sum_stride + blockIdx.x];

    if (a.out == nullptr) {
        if (threadIdx.x < len)
            a.vec_out[st.packed + threadIdx.x] = chunk_result[threadIdx.x];
        if (threadIdx.x == 0 && a.leaf_sum_out != nullptr)
            a.leaf_sum_out[blockIdx.x] = leaf_sum;
        return;
    }
    if (a.orthogonality != nullptr && warp == 0) {
        const double r0 = lane < len ? chunk_result[lane] : 0.0, r1 = lane + 32 < len ? chunk_result[lane + 32] : 0.0;
        const double norm = warp_sum(r0 * r0 + r1 * r1);
        if (lane == 0)       // Section 3.6; NaN when every leaf is zero
            a.orthogonality[st.tensor] = leaf_sum == 0.0 ? __int_as_float(0x7fc00000) : (float)(norm / leaf_sum);
    }
    if (threadIdx.x < len) {
        double y = chunk_result[threadIdx.x];
        const int64_t e = st.begin + threadIdx.x;
        if (a.base != nullptr)
            y += (double)load_as_float(a.base, a.base_dtype, e);
        store_from_float(a.out, a.out_dtype, e, (float)y);
    }
}

}  // namespace

cudaError_t launch_short_tensors(int dtype, const OperandTable& ops, int operands, int num_short,
                                 const ShortArgs& args, cudaStream_t stream)
{
    if (num_short <= 0)
        return cudaSuccess;
    if (operands < 1 || operands > kMaxOperandsPerLaunch)
        return cudaErrorInvalidValue;
    const dim3 grid((unsigned)num_short), block(kShortThreads);
    switch (dtype) {
    case 0: short_tensor_kernel<float><<<grid, block, 0, stream>>>(ops, operands, args); break;
    case 1: short_tensor_kernel<__half><<<grid, block, 0, stream>>>(ops, operands, args); break;
    case 2: short_tensor_kernel<__nv_bfloat16><<<grid, block, 0, stream>>>(ops, operands, args); break;
    case 3: short_tensor_kernel<double><<<grid, block, 0, stream>>>(ops, operands, args); break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace adasum
