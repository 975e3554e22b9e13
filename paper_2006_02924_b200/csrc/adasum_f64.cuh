// Device kernels for fp64 gradient buffers.
//
// The paper's implementation offers the operator for fp16, fp32 and fp64 tensors (Section 4.4).  An
// fp64 caller expects fp64 results, so nothing here is narrower than a double: products and sums on
// the fp64 pipes, partial Gram matrices, leaf weights, intermediates and (unless fp32 is asked for)
// the output are doubles.  Same structure as the fp32 family: a level handles groups of R = 2 or 4
// adjacent operands (a complete sub-tree of Algorithm 1's binary tree): pass 1 forms each group's
// Gram matrix per tensor, the last block of a (tensor, group) adds the per-segment matrices in a
// fixed order and runs the tree on the Gram matrix, pass 2 writes the weighted sums.
#pragma once

#include "adasum_kernels.cuh"

namespace adasum {

struct FinishArgsF64 {
    const int32_t* seg_first;   // [2 t], [2 t + 1]: first and one-past-last segment of tensor t
    int* counters;              // [tensor][group], zero on entry and on exit
    double* weights;            // [tensor][group][R]
    TreeOptions tree;
};

// grid = (segments, groups in this launch); block = kThreads.
// partials[(segment * groups_total + group_base + blockIdx.y) * E + entry], doubles.
// start != nullptr: the rows are (operand - start) (the delta form of Section 4.1).
template <int R, bool VEC>
__global__ void __launch_bounds__(kThreads)
gram_partial_f64_kernel(const __grid_constant__ OperandTable ops, int operands,
                        const Segment* __restrict__ segments, double* __restrict__ partials,
                        int groups_total, int group_base, FinishArgsF64 fin, const double* __restrict__ start)
{
    constexpr int E = gram_entries(R);
    const Segment seg = segments[blockIdx.x];
    const int first = blockIdx.y * R;
    const int members = min(R, operands - first);
    const int group = group_base + blockIdx.y;

    const double* src[R];
#pragma unroll
    for (int i = 0; i < R; ++i)
        src[i] = static_cast<const double*>(ops.ptr[first + (i < members ? i : 0)]);

    double acc[E];
#pragma unroll
    for (int k = 0; k < E; ++k)
        acc[k] = 0.0;
    auto accumulate = [&](const double (&col)[R]) {
        int idx = 0;
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int j = i; j < R; ++j)
                acc[idx] = fma(col[i], col[j], acc[idx]), ++idx;
    };

    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    int64_t body_begin, body_end;
    split_segment<2, VEC>(begin, end, body_begin, body_end);
    for (int64_t v = body_begin + (int64_t)threadIdx.x * 2; v < body_end; v += (int64_t)kThreads * 2) {
        double2 x[R];
        const double2 s = start != nullptr ? *reinterpret_cast<const double2*>(start + v) : make_double2(0.0, 0.0);
#pragma unroll
        for (int i = 0; i < R; ++i)
            x[i] = i < members ? __ldg(reinterpret_cast<const double2*>(src[i] + v)) : s;
        double col[R];
#pragma unroll
        for (int i = 0; i < R; ++i)
            col[i] = x[i].x - s.x;
        accumulate(col);
#pragma unroll
        for (int i = 0; i < R; ++i)
            col[i] = x[i].y - s.y;
        accumulate(col);
    }
    for (int pass = 0; pass < 2; ++pass) {       // scalar head [begin, body_begin) and tail [body_end, end)
        const int64_t lo = pass == 0 ? begin : body_end;
        const int64_t hi = pass == 0 ? body_begin : end;
        for (int64_t e = lo + threadIdx.x; e < hi; e += kThreads) {
            const double s = start != nullptr ? start[e] : 0.0;
            double col[R];
#pragma unroll
            for (int i = 0; i < R; ++i)
                col[i] = i < members ? __ldg(src[i] + e) - s : 0.0;
            accumulate(col);
        }
    }

    // block reduction: warp shuffles, then the warps' sums in warp order
    __shared__ double warp_sums[kWarps][E];
    __shared__ double gram[E];
    __shared__ int is_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < E; ++k) {
        double sum = acc[k];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1)
            sum += __shfl_xor_sync(0xffffffffu, sum, d);
        if (lane == 0)
            warp_sums[warp][k] = sum;
    }
    __syncthreads();
    double* dst = partials + ((int64_t)blockIdx.x * groups_total + group) * E;
    for (int k = threadIdx.x; k < E; k += kThreads) {
        double sum = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w)
            sum += warp_sums[w][k];
        dst[k] = sum;
    }

    // the block that hands in the tensor's last partial matrix adds them all up (segment order)
    __threadfence();
    __syncthreads();
    const int s0 = fin.seg_first[2 * seg.tensor], s1 = fin.seg_first[2 * seg.tensor + 1];
    if (threadIdx.x == 0) {
        int* counter = fin.counters + (int64_t)seg.tensor * groups_total + group;
        const int ticket = atomicAdd(counter, 1);
        is_last = ticket == s1 - s0 - 1;
        if (is_last)
            *counter = 0;
    }
    __syncthreads();
    if (!is_last)
        return;
    __threadfence();
    constexpr int Q = kThreads / E;
    __shared__ double slice_sum[Q * E];
    {
        const int q = threadIdx.x / E, kk = threadIdx.x - q * E;
        if (q < Q) {
            const double* srcp = partials + (int64_t)group * E + kk;
            const int64_t stride = (int64_t)groups_total * E;
            double sum = 0.0;
#pragma unroll 4
            for (int sg = s0 + q; sg < s1; sg += Q)
                sum += __ldcg(srcp + sg * stride);
            slice_sum[q * E + kk] = sum;
        }
    }
    __syncthreads();
    if (threadIdx.x < E) {
        double sum = slice_sum[threadIdx.x];
        for (int qq = 1; qq < Q; ++qq)
            sum += slice_sum[qq * E + threadIdx.x];
        gram[threadIdx.x] = sum;
    }
    __syncthreads();
    tree_weights_from_gram<R, double>(gram, members, fin.weights + ((int64_t)seg.tensor * groups_total + group) * R,
                                      fin.tree, seg.tensor, group);
}

// grid = (segments, groups in this launch); block = kThreads.
// dst_base + (group_base + blockIdx.y) * dst_stride elements is the group's output buffer: doubles,
// or, for a last level with out_f32 set, floats.  base (last level of the delta form) is added.
template <int R, bool VEC>
__global__ void __launch_bounds__(kThreads)
weighted_sum_f64_kernel(const __grid_constant__ OperandTable ops, int operands,
                        const Segment* __restrict__ segments, const double* __restrict__ weights,
                        int groups_total, int group_base, void* dst_base, int64_t dst_stride,
                        const double* start, const double* base, int out_f32)
{
    const Segment seg = segments[gridDim.x - 1 - blockIdx.x];      // last to first: what pass 1 left in the L2
    const int first = blockIdx.y * R;
    const int members = min(R, operands - first);
    const int group = group_base + blockIdx.y;
    double w[R];
    const double* src[R];
#pragma unroll
    for (int i = 0; i < R; ++i) {
        w[i] = i < members ? weights[((int64_t)seg.tensor * groups_total + group) * R + i] : 0.0;
        src[i] = static_cast<const double*>(ops.ptr[first + (i < members ? i : 0)]);
    }
    double* dst64 = static_cast<double*>(dst_base) + (int64_t)group * dst_stride;
    float* dst32 = static_cast<float*>(dst_base) + (int64_t)group * dst_stride;

    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    int64_t body_begin, body_end;
    split_segment<2, VEC>(begin, end, body_begin, body_end);
    for (int64_t v = body_begin + (int64_t)threadIdx.x * 2; v < body_end; v += (int64_t)kThreads * 2) {
        // plain loads for start / base: out may be the same buffer (each element is read by the thread that writes it)
        const double2 s = start != nullptr ? *reinterpret_cast<const double2*>(start + v) : make_double2(0.0, 0.0);
        double2 y = make_double2(0.0, 0.0);
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (i < members) {
                const double2 x = __ldg(reinterpret_cast<const double2*>(src[i] + v));
                y.x = fma(w[i], x.x - s.x, y.x);
                y.y = fma(w[i], x.y - s.y, y.y);
            }
        }
        if (base != nullptr) {
            const double2 bb = *reinterpret_cast<const double2*>(base + v);
            y.x += bb.x;
            y.y += bb.y;
        }
        if (out_f32)
            *reinterpret_cast<float2*>(dst32 + v) = make_float2((float)y.x, (float)y.y);
        else
            *reinterpret_cast<double2*>(dst64 + v) = y;
    }
    for (int pass = 0; pass < 2; ++pass) {
        const int64_t lo = pass == 0 ? begin : body_end;
        const int64_t hi = pass == 0 ? body_begin : end;
        for (int64_t e = lo + threadIdx.x; e < hi; e += kThreads) {
            const double s = start != nullptr ? start[e] : 0.0;
            double y = 0.0;
#pragma unroll
            for (int i = 0; i < R; ++i)
                if (i < members)
                    y = fma(w[i], __ldg(src[i] + e) - s, y);
            if (base != nullptr)
                y += base[e];
            if (out_f32)
                dst32[e] = (float)y;
            else
                dst64[e] = y;
        }
    }
}

// n_workers = 1: the result is the input (start + (input - start) with a start).
__global__ void __launch_bounds__(kThreads)
convert_f64_kernel(const double* src, void* dst, int64_t n, const double* start, int out_f32)
{
    for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < n; e += (int64_t)gridDim.x * kThreads) {
        const double y = start != nullptr ? start[e] + (src[e] - start[e]) : src[e];
        if (out_f32)
            static_cast<float*>(dst)[e] = (float)y;
        else
            static_cast<double*>(dst)[e] = y;
    }
}

}  // namespace adasum
