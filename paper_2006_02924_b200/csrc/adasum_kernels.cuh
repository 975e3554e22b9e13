// Device kernels of the N-way Adasum combine for sm_100a.
//
// One "level" of the reduction handles groups of R adjacent operands (R = 2, 4, 8 or 16).  A group
// is a complete sub-tree of the paper's binary tree (Section 3.4; Algorithm 1 pairs neighbours at
// distance 1, 2, 4, ...), and every node of that sub-tree is a linear combination of the group's
// leaves.  So a level is three kernels:
//
//   gram_partial   stream the operands once; per (segment, group) the R x R Gram matrix
//                  G_ij = sum_e x_i[e] x_j[e] of the segment's elements, fp32, upper triangle.
//                  For R = 2 these are Algorithm 1's three scalars [a.b, a.a, b.b].
//   tree_weights   per (tensor, group): add the segments' partial matrices in fp64 in a fixed
//                  order, then run the binary tree on the Gram matrix alone to get the R leaf
//                  weights (the "Apply Adasum" coefficients, composed down the sub-tree).
//   weighted_sum   stream the operands a second time; out = sum_i weight_i x_i.
//
// The kernels never wait on one another and use no floating-point atomics, so results are
// deterministic and there is nothing that can spin.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace adasum {

constexpr int kThreads = 256;               // threads per block of the streaming kernels
constexpr int kWarps = kThreads / 32;
constexpr int kMaxOperandsPerLaunch = 256;  // operand pointers carried in one kernel argument
constexpr int kMaxRadix = 16;

// A contiguous run of elements of one tensor inside the fused buffers.
struct Segment {
    int64_t begin;   // first element (index into every worker's buffer)
    int32_t len;     // number of elements, > 0
    int32_t tensor;  // which tensor the run belongs to
};

struct OperandTable {
    const void* ptr[kMaxOperandsPerLaunch];
};

__host__ __device__ constexpr int gram_entries(int radix) { return radix * (radix + 1) / 2; }

// Row-major position of (i, j), i <= j, in the packed upper triangle of an R x R matrix.
__host__ __device__ constexpr int gram_index(int radix, int i, int j)
{
    return i * radix - (i * (i - 1)) / 2 + (j - i);
}

// ---- element access -------------------------------------------------------------------------

__device__ __forceinline__ uint4 load_streaming_16B(const void* p)
{
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
        : "l"(p));
    return v;
}

template <typename T>
struct Element;

template <>
struct Element<float> {
    static constexpr int kVec = 4;
    static __device__ __forceinline__ float one(const float* p) { return __ldg(p); }
    static __device__ __forceinline__ void vec(const float* p, float (&x)[kVec])
    {
        uint4 v = load_streaming_16B(p);
        x[0] = __uint_as_float(v.x);
        x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z);
        x[3] = __uint_as_float(v.w);
    }
};

template <>
struct Element<__half> {
    static constexpr int kVec = 8;
    static __device__ __forceinline__ float one(const __half* p) { return __half2float(__ldg(p)); }
    static __device__ __forceinline__ void vec(const __half* p, float (&x)[kVec])
    {
        uint4 v = load_streaming_16B(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __half2 h = *reinterpret_cast<const __half2*>(&w[i]);
            float2 f = __half22float2(h);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
};

template <>
struct Element<__nv_bfloat16> {
    static constexpr int kVec = 8;
    static __device__ __forceinline__ float one(const __nv_bfloat16* p)
    {
        return __bfloat162float(__ldg(p));
    }
    static __device__ __forceinline__ void vec(const __nv_bfloat16* p, float (&x)[kVec])
    {
        uint4 v = load_streaming_16B(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {            // a bf16 is the upper half of an fp32
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

// Split a segment [begin, end) into a scalar head, a 16-byte-aligned vector body and a scalar
// tail.  Without VEC (some buffer is not 16-byte aligned) everything is "tail".
template <int V, bool VEC>
__device__ __forceinline__ void split_segment(int64_t begin, int64_t end, int64_t& body_begin,
                                              int64_t& body_end)
{
    if (VEC) {
        int64_t up = (begin + V - 1) / V * V;
        body_begin = up < end ? up : end;
        int64_t down = end / V * V;
        body_end = down > body_begin ? down : body_begin;
    } else {
        body_begin = begin;
        body_end = begin;
    }
}

// ---- pass 1: partial Gram matrices -------------------------------------------------------------

template <int R>
__device__ __forceinline__ void gram_accumulate(const float (&x)[R], float (&acc)[gram_entries(R)])
{
    int idx = 0;
#pragma unroll
    for (int i = 0; i < R; ++i) {
#pragma unroll
        for (int j = i; j < R; ++j) {
            acc[idx] = fmaf(x[i], x[j], acc[idx]);
            ++idx;
        }
    }
}

// grid = (segments, groups in this launch); block = kThreads.
// partials[(segment * groups_total + group_base + blockIdx.y) * E + entry]
template <typename T, int R, bool VEC>
__global__ void __launch_bounds__(kThreads)
gram_partial_kernel(const __grid_constant__ OperandTable ops, int operands,
                    const Segment* __restrict__ segments, float* __restrict__ partials,
                    int groups_total, int group_base)
{
    constexpr int E = gram_entries(R);
    constexpr int V = Element<T>::kVec;
    const Segment seg = segments[blockIdx.x];
    const int first = blockIdx.y * R;
    const int members = min(R, operands - first);

    const T* src[R];
#pragma unroll
    for (int i = 0; i < R; ++i)
        src[i] = static_cast<const T*>(ops.ptr[first + (i < members ? i : 0)]);

    float acc[E];
#pragma unroll
    for (int k = 0; k < E; ++k)
        acc[k] = 0.0f;

    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    int64_t body_begin, body_end;
    split_segment<V, VEC>(begin, end, body_begin, body_end);

    for (int64_t v = body_begin + (int64_t)threadIdx.x * V; v < body_end; v += (int64_t)kThreads * V) {
        float x[R][V];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (i < members) {
                Element<T>::vec(src[i] + v, x[i]);
            } else {
#pragma unroll
                for (int j = 0; j < V; ++j)
                    x[i][j] = 0.0f;
            }
        }
#pragma unroll
        for (int j = 0; j < V; ++j) {
            float col[R];
#pragma unroll
            for (int i = 0; i < R; ++i)
                col[i] = x[i][j];
            gram_accumulate<R>(col, acc);
        }
    }
    // scalar head [begin, body_begin) and tail [body_end, end)
    for (int pass = 0; pass < 2; ++pass) {
        const int64_t lo = pass == 0 ? begin : body_end;
        const int64_t hi = pass == 0 ? body_begin : end;
        for (int64_t e = lo + threadIdx.x; e < hi; e += kThreads) {
            float col[R];
#pragma unroll
            for (int i = 0; i < R; ++i)
                col[i] = i < members ? Element<T>::one(src[i] + e) : 0.0f;
            gram_accumulate<R>(col, acc);
        }
    }

    // block reduction: warp shuffles, then the warps' sums in warp order
    __shared__ float warp_sums[kWarps][E];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < E; ++k) {
        float s = acc[k];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1)
            s += __shfl_xor_sync(0xffffffffu, s, d);
        if (lane == 0)
            warp_sums[warp][k] = s;
    }
    __syncthreads();
    float* dst = partials + ((int64_t)blockIdx.x * groups_total + group_base + blockIdx.y) * E;
    for (int k = threadIdx.x; k < E; k += kThreads) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w)
            s += warp_sums[w][k];
        dst[k] = s;
    }
}

// ---- coefficients: the binary tree evaluated on a Gram matrix ---------------------------------

// Algorithm 1, "Apply Adasum": x' = a (1 - v1 / 2 v2) + b (1 - v1 / 2 v3) with
// v = [a.b, a.a, b.b].  An operand with zero squared norm keeps coefficient 1.
__device__ __forceinline__ void pair_coefficients(double dot, double norm_a, double norm_b,
                                                  double& coef_a, double& coef_b)
{
    coef_a = norm_a == 0.0 ? 1.0 : 1.0 - dot / (2.0 * norm_a);
    coef_b = norm_b == 0.0 ? 1.0 : 1.0 - dot / (2.0 * norm_b);
}

// Leaf weights of the sub-tree over `members` leaves whose Gram matrix is `gram` (packed upper
// triangle, row length R).  Bottom-up: blocks of width 1, 2, 4, ...; the block [L, L+w) is
// paired with [L+w, L+2w); a block without a right sibling is carried unchanged.  The squared
// norm of a parent follows from its children: |ca a + cb b|^2 = ca^2 |a|^2 + cb^2 |b|^2 + 2 ca cb a.b.
template <int R>
__device__ void tree_weights_from_gram(const double* gram, int members, double* weight,
                                       double* root_norm)
{
    double norm[R];
    for (int i = 0; i < members; ++i) {
        weight[i] = 1.0;
        norm[i] = gram[gram_index(R, i, i)];
    }
    for (int w = 1; w < members; w *= 2) {
        for (int left = 0; left + w < members; left += 2 * w) {
            const int mid = left + w;
            const int right_end = min(left + 2 * w, members);
            double dot = 0.0;
            for (int i = left; i < mid; ++i) {
                double row = 0.0;
                for (int k = mid; k < right_end; ++k)
                    row += weight[k] * gram[gram_index(R, i, k)];
                dot += weight[i] * row;
            }
            double ca, cb;
            pair_coefficients(dot, norm[left], norm[mid], ca, cb);
            for (int i = left; i < mid; ++i)
                weight[i] *= ca;
            for (int k = mid; k < right_end; ++k)
                weight[k] *= cb;
            norm[left] = ca * ca * norm[left] + cb * cb * norm[mid] + 2.0 * ca * cb * dot;
        }
    }
    *root_norm = norm[0];
}

// grid = (tensors, groups); block = kThreads.
// Sums the tensor's per-segment partial matrices in fp64 (fixed order), then thread 0 runs the
// tree.  weights[(tensor * groups + group) * R + i] = weight of leaf i (fp32).
template <int R>
__global__ void __launch_bounds__(kThreads)
tree_weights_kernel(const float* __restrict__ partials, const int32_t* __restrict__ seg_first,
                    int operands, float* __restrict__ weights)
{
    constexpr int E = gram_entries(R);
    constexpr int Q = kThreads / E > 0 ? kThreads / E : 1;   // segment slices summed in parallel
    const int tensor = blockIdx.x, group = blockIdx.y, groups = gridDim.y;
    const int members = min(R, operands - group * R);
    const int s0 = seg_first[tensor], s1 = seg_first[tensor + 1];

    __shared__ double slice_sum[Q][E];
    __shared__ double gram[E];
    for (int idx = threadIdx.x; idx < Q * E; idx += kThreads) {
        const int q = idx / E, k = idx - q * E;
        double s = 0.0;
        for (int seg = s0 + q; seg < s1; seg += Q)
            s += (double)partials[((int64_t)seg * groups + group) * E + k];
        slice_sum[q][k] = s;
    }
    __syncthreads();
    for (int k = threadIdx.x; k < E; k += kThreads) {
        double s = 0.0;
        for (int q = 0; q < Q; ++q)
            s += slice_sum[q][k];
        gram[k] = s;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double weight[R], root_norm;
        tree_weights_from_gram<R>(gram, members, weight, &root_norm);
        float* dst = weights + ((int64_t)tensor * groups + group) * R;
        for (int i = 0; i < R; ++i)
            dst[i] = i < members ? (float)weight[i] : 0.0f;
    }
}

// ---- pass 2: weighted sum ---------------------------------------------------------------------

// grid = (segments, groups in this launch); block = kThreads.
// dst_base + (group_base + blockIdx.y) * dst_stride is the group's output buffer (fp32).
template <typename T, int R, bool VEC>
__global__ void __launch_bounds__(kThreads)
weighted_sum_kernel(const __grid_constant__ OperandTable ops, int operands,
                    const Segment* __restrict__ segments, const float* __restrict__ weights,
                    int groups_total, int group_base, float* __restrict__ dst_base,
                    int64_t dst_stride)
{
    constexpr int V = Element<T>::kVec;
    const Segment seg = segments[blockIdx.x];
    const int first = blockIdx.y * R;
    const int members = min(R, operands - first);
    const int group = group_base + blockIdx.y;

    const T* src[R];
    float w[R];
    const float* wsrc = weights + ((int64_t)seg.tensor * groups_total + group) * R;
#pragma unroll
    for (int i = 0; i < R; ++i) {
        src[i] = static_cast<const T*>(ops.ptr[first + (i < members ? i : 0)]);
        w[i] = i < members ? __ldg(wsrc + i) : 0.0f;
    }
    float* dst = dst_base + (int64_t)group * dst_stride;

    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    int64_t body_begin, body_end;
    split_segment<V, VEC>(begin, end, body_begin, body_end);

    for (int64_t v = body_begin + (int64_t)threadIdx.x * V; v < body_end; v += (int64_t)kThreads * V) {
        float x[R][V];
#pragma unroll
        for (int i = 0; i < R; ++i)
            if (i < members)
                Element<T>::vec(src[i] + v, x[i]);
        float y[V];
#pragma unroll
        for (int j = 0; j < V; ++j)
            y[j] = 0.0f;
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (i < members) {
#pragma unroll
                for (int j = 0; j < V; ++j)
                    y[j] = fmaf(w[i], x[i][j], y[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < V; j += 4)
            *reinterpret_cast<float4*>(dst + v + j) = make_float4(y[j], y[j + 1], y[j + 2], y[j + 3]);
    }
    for (int pass = 0; pass < 2; ++pass) {
        const int64_t lo = pass == 0 ? begin : body_end;
        const int64_t hi = pass == 0 ? body_begin : end;
        for (int64_t e = lo + threadIdx.x; e < hi; e += kThreads) {
            float y = 0.0f;
#pragma unroll
            for (int i = 0; i < R; ++i)
                if (i < members)
                    y = fmaf(w[i], Element<T>::one(src[i] + e), y);
            dst[e] = y;
        }
    }
}

// n_workers = 1: the result is the input, converted to fp32.
template <typename T>
__global__ void __launch_bounds__(kThreads)
convert_kernel(const T* __restrict__ src, float* __restrict__ dst, int64_t n)
{
    for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < n;
         e += (int64_t)gridDim.x * kThreads)
        dst[e] = Element<T>::one(src + e);
}

}  // namespace adasum
