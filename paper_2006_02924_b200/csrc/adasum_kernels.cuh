// Device kernels of the N-way Adasum combine for sm_100a.
//
// One "level" of the reduction handles groups of R adjacent operands (R = 2 ... 64).  A group
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
// The Gram matrix of a group is a dense contraction X X^T (R x P times P x R).  For R <= 8 it is
// cheap enough for the fp32 pipes (gram_partial_kernel); for R >= 8 it runs on the tensor cores
// (gram_partial_mma_kernel; gram_partial_tc64_kernel for 64 fp16 / bf16 rows): fp16 / bf16 products
// are exact in the fp32 accumulator, fp32 inputs are split into two tf32 terms (three products).
//
// Two more kernels merge neighbouring steps: fused_small_kernel (both passes of a small input in
// one cooperative launch) and wsum_gram_kernel (pass 2 of a level with pass 1 of the next).
// Tensors of at most 64 elements are not streamed at all: they are reduced in fp64 with the
// operator applied literally (adasum_short.cu; one warp each inside fused_small_kernel).
//
// No kernel waits on another kernel and none uses floating-point atomics, so results are
// deterministic.  The only waits are inside a launch: the grid barrier of the cooperative
// fused_small_kernel, and the bounded mbarrier waits between the copying warps and the tensor
// core in gram_partial_tc64_kernel.
#pragma once

#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "adasum_short.cuh"

namespace adasum {

constexpr int kThreads = 256;               // threads per block of the streaming kernels
constexpr int kWarps = kThreads / 32;
constexpr int kMaxOperandsPerLaunch = 256;  // operand pointers carried in one kernel argument
constexpr int kMaxRadix = 64;
constexpr int ADASUM_DEVICE_TIMEOUT = 7;    // value of ADASUM_ERR_TIMEOUT, written to a status word by a kernel

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

// Read-once data (pass 2): bypass L1 and mark the lines evict-first in L2.
__device__ __forceinline__ uint4 load_streaming_16B(const void* p)
{
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
        : "l"(p));
    return v;
}

// Data that pass 2 will read again (pass 1): ordinary L2 policy, so that the last part of the
// operands is still resident when pass 2 starts from the end.
__device__ __forceinline__ uint4 load_keep_16B(const void* p)
{
    uint4 v;
    asm("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
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
        uint4 v = load_keep_16B(p);
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
        uint4 v = load_keep_16B(p);
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
        uint4 v = load_keep_16B(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {            // a bf16 is the upper half of an fp32
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

// 16 bytes of T as floats.
template <typename T>
__device__ __forceinline__ void decode_vector(const uint4& v, float (&x)[Element<T>::kVec]);
template <>
__device__ __forceinline__ void decode_vector<float>(const uint4& v, float (&x)[4])
{
    x[0] = __uint_as_float(v.x);
    x[1] = __uint_as_float(v.y);
    x[2] = __uint_as_float(v.z);
    x[3] = __uint_as_float(v.w);
}
template <>
__device__ __forceinline__ void decode_vector<__half>(const uint4& v, float (&x)[8])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
    }
}
template <>
__device__ __forceinline__ void decode_vector<__nv_bfloat16>(const uint4& v, float (&x)[8])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

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

// ---- the "optimizer delta" form and the output format -------------------------------------------
//
// Section 4.1 (the figure that wraps an optimizer): every worker takes a local optimizer step from
// the common parameters `start`, the operator combines the effective gradients current_i - start,
// and the combination is added back to `start`.  With DELTA the first level's operands are read as
// (ptr[i] - start), the difference rounded once to the operands' own type T (what
// `current - start` gives in a framework); `base` is added to the last level's result; the last
// level may store fp16 / bf16 instead of fp32.
struct PassExtras {
    const void* start;    // DELTA kernels: subtracted from every operand of this level (type T)
    const void* base;     // last level: result = base + sum (nullptr: nothing added)
    int base_dtype;       // 0 fp32, 1 fp16, 2 bf16
    int out_dtype;        // type of the level's destination: 0 fp32 (always, except a last level), 1 fp16, 2 bf16
};

// Data that the same thread may overwrite later in the same kernel (out == start): a plain load.
__device__ __forceinline__ uint4 load_plain_16B(const void* p) { return *reinterpret_cast<const uint4*>(p); }

// c - s on the packed words of a 16-byte vector, in T, round to nearest even.
template <typename T>
__device__ __forceinline__ uint4 delta_words(const uint4& c, const uint4& s);
template <>
__device__ __forceinline__ uint4 delta_words<float>(const uint4& c, const uint4& s)
{
    return make_uint4(__float_as_uint(__fsub_rn(__uint_as_float(c.x), __uint_as_float(s.x))),
                      __float_as_uint(__fsub_rn(__uint_as_float(c.y), __uint_as_float(s.y))),
                      __float_as_uint(__fsub_rn(__uint_as_float(c.z), __uint_as_float(s.z))),
                      __float_as_uint(__fsub_rn(__uint_as_float(c.w), __uint_as_float(s.w))));
}
template <>
__device__ __forceinline__ uint4 delta_words<__half>(const uint4& c, const uint4& s)
{
    const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, sw[4] = {s.x, s.y, s.z, s.w};
    uint32_t d[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __half2 r = __hsub2(*reinterpret_cast<const __half2*>(&cw[i]), *reinterpret_cast<const __half2*>(&sw[i]));
        d[i] = *reinterpret_cast<const uint32_t*>(&r);
    }
    return make_uint4(d[0], d[1], d[2], d[3]);
}
template <>
__device__ __forceinline__ uint4 delta_words<__nv_bfloat16>(const uint4& c, const uint4& s)
{
    const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, sw[4] = {s.x, s.y, s.z, s.w};
    uint32_t d[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 r = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&cw[i]),
                                         *reinterpret_cast<const __nv_bfloat162*>(&sw[i]));
        d[i] = *reinterpret_cast<const uint32_t*>(&r);
    }
    return make_uint4(d[0], d[1], d[2], d[3]);
}
// One element: c - s in T, as a float.
__device__ __forceinline__ float delta_one(const float* c, const float* s, int64_t e) { return __fsub_rn(c[e], s[e]); }
__device__ __forceinline__ float delta_one(const __half* c, const __half* s, int64_t e)
{
    return __half2float(__hsub(c[e], s[e]));
}
__device__ __forceinline__ float delta_one(const __nv_bfloat16* c, const __nv_bfloat16* s, int64_t e)
{
    return __bfloat162float(__hsub(c[e], s[e]));
}

// Element e of a buffer of the given dtype code, as a float (plain load).
__device__ __forceinline__ float load_as_float(const void* p, int dtype, int64_t e)
{
    if (dtype == 0)
        return static_cast<const float*>(p)[e];
    if (dtype == 1)
        return __half2float(static_cast<const __half*>(p)[e]);
    return __bfloat162float(static_cast<const __nv_bfloat16*>(p)[e]);
}
__device__ __forceinline__ void store_from_float(void* p, int dtype, int64_t e, float y)
{
    if (dtype == 0)
        static_cast<float*>(p)[e] = y;
    else if (dtype == 1)
        static_cast<__half*>(p)[e] = __float2half_rn(y);
    else
        static_cast<__nv_bfloat16*>(p)[e] = __float2bfloat16_rn(y);
}
// N = 4 or 8 consecutive elements starting at element e (e a multiple of N, buffer 16-byte aligned).
template <int N>
__device__ __forceinline__ void add_vector_as_float(const void* p, int dtype, int64_t e, float (&y)[N])
{
    if (dtype == 0) {
#pragma unroll
        for (int j = 0; j < N; j += 4) {
            const float4 b = *reinterpret_cast<const float4*>(static_cast<const float*>(p) + e + j);
            y[j] += b.x; y[j + 1] += b.y; y[j + 2] += b.z; y[j + 3] += b.w;
        }
    } else {
        uint32_t w[N / 2];
        if constexpr (N == 8) {
            const uint4 b = *reinterpret_cast<const uint4*>(static_cast<const unsigned short*>(p) + e);
            w[0] = b.x; w[1] = b.y; w[2] = b.z; w[3] = b.w;
        } else {
            const uint2 b = *reinterpret_cast<const uint2*>(static_cast<const unsigned short*>(p) + e);
            w[0] = b.x; w[1] = b.y;
        }
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            if (dtype == 1) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
                y[2 * i] += f.x; y[2 * i + 1] += f.y;
            } else {
                y[2 * i] += __uint_as_float(w[i] << 16);
                y[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
            }
        }
    }
}
template <int N>
__device__ __forceinline__ void store_vector_from_float(void* p, int dtype, int64_t e, const float (&y)[N])
{
    if (dtype == 0) {
#pragma unroll
        for (int j = 0; j < N; j += 4)
            *reinterpret_cast<float4*>(static_cast<float*>(p) + e + j) = make_float4(y[j], y[j + 1], y[j + 2], y[j + 3]);
    } else {
        uint32_t w[N / 2];
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            if (dtype == 1) {
                const __half2 h = __floats2half2_rn(y[2 * i], y[2 * i + 1]);
                w[i] = *reinterpret_cast<const uint32_t*>(&h);
            } else {
                const __nv_bfloat162 h = __floats2bfloat162_rn(y[2 * i], y[2 * i + 1]);
                w[i] = *reinterpret_cast<const uint32_t*>(&h);
            }
        }
        if constexpr (N == 8)
            *reinterpret_cast<uint4*>(static_cast<unsigned short*>(p) + e) = make_uint4(w[0], w[1], w[2], w[3]);
        else
            *reinterpret_cast<uint2*>(static_cast<unsigned short*>(p) + e) = make_uint2(w[0], w[1]);
    }
}

// ---- finishing a group inside pass 1 -----------------------------------------------------------
//
// The block that writes the LAST per-segment partial matrix of a (tensor, group) also adds up all
// of that tensor's partials and derives the leaf weights, so no separate launch
// (and no idle GPU while a small kernel runs) separates pass 1 from pass 2.  "Last" is decided by
// an integer ticket counter per (tensor, group); the sums themselves are taken in segment order,
// so the result does not depend on which block happens to be last.  The counter is returned to
// zero by that block.  counters == nullptr switches the mechanism off (the caller then launches
// gram_finish_kernel).
// What the coefficient step produces besides the leaf weights.
struct TreeOptions {
    int linear;               // 1: the sequential recursion Adasum(Adasum(g[0..n]), g[n+1]) of Section 3.4
                              //    instead of the binary tree; 2: the binary tree split by halves
                              //    from the top instead of paired bottom-up (single-level plans only)
    int level_is_first;       // this level's operands are the workers' gradients
    int level_is_last;        // this level's single group produces the result
    int groups_first;         // number of groups of the first level
    double* leaf_norm_sums;   // [tensor][groups_first]: sum of the leaves' squared norms, or nullptr
    float* orthogonality;     // [tensor]: |result|^2 / sum_i |g_i|^2 (Section 3.6), or nullptr
    // Dynamic scaling (Section 4.4.1): worker w's buffer holds leaf_scales[w * num_tensors + t] times
    // its gradient for tensor t; nullptr: the buffers hold the gradients themselves.  Read by the
    // first level only.
    const float* leaf_scales;
    int num_tensors;
};

struct FinishArgs {
    const int32_t* seg_first;   // [2 t], [2 t + 1]: first and one-past-last segment of tensor t
    int* counters;              // [tensor][group], zero on entry
    float* weights;             // [tensor][group][R]
    TreeOptions tree;
    int selftest_timeout;       // gram_partial_tc64_kernel only: leave the last tile unmultiplied and wait briefly,
                                // so that the epilogue's bounded wait runs out (test of the status path)
    // Tensors of more than kSegmentsPerGroup segments are finished in two steps (nullptr: in one):
    // the block that hands in the last partial of a run of kSegmentsPerGroup segments adds that
    // run's partials, and the block that hands in the tensor's last run sum adds the run sums.
    const int32_t* group_first; // [tensor]: number of the tensor's first run
    int* group_counters;        // [run][group], zero on entry
    double* group_sums;         // [run][group][E]
};

constexpr int kSegmentsPerGroup = 16;

template <int R>
__device__ void add_partials_in_block(const float* partials, int seg_begin, int seg_end, int group, int groups_total,
                                      double* gram);
template <int R, typename W = float>
__device__ void tree_weights_from_gram(const double* gram, int members, W* __restrict__ dst, const TreeOptions& opt,
                                       int tensor, int group);

// Called by every thread of the block after its partial matrix (number seg_index) has been written.
template <int R>
__device__ __forceinline__ void finish_if_last(const FinishArgs& fin, const float* partials, int tensor, int group,
                                               int groups_total, int members, int seg_index)
{
    if (fin.counters == nullptr)
        return;
    constexpr int E = gram_entries(R);
    __shared__ int is_last;
    __shared__ double gram[E];
    const int s0 = fin.seg_first[2 * tensor], s1 = fin.seg_first[2 * tensor + 1];
    const bool in_runs = fin.group_sums != nullptr && s1 - s0 > kSegmentsPerGroup;
    const int runs = (s1 - s0 + kSegmentsPerGroup - 1) / kSegmentsPerGroup;
    const double* run_sums = nullptr;
    if (in_runs) {
        const int run = (seg_index - s0) / kSegmentsPerGroup;
        const int run_begin = s0 + run * kSegmentsPerGroup;
        const int run_end = min(run_begin + kSegmentsPerGroup, s1);
        const int64_t first_slot = (int64_t)fin.group_first[tensor] * groups_total + group;
        const int64_t slot = first_slot + (int64_t)run * groups_total;
        run_sums = fin.group_sums + first_slot * E;
        __threadfence();                   // this block's partial is visible device-wide ...
        __syncthreads();
        if (threadIdx.x == 0) {
            const int ticket = atomicAdd(fin.group_counters + slot, 1);      // ... before its ticket is drawn
            is_last = ticket == run_end - run_begin - 1;
            if (is_last)
                fin.group_counters[slot] = 0;
        }
        __syncthreads();
        if (!is_last)
            return;
        __threadfence();
        add_partials_in_block<R>(partials, run_begin, run_end, group, groups_total, gram);
        double* run_sum = fin.group_sums + slot * E;
        for (int k = threadIdx.x; k < E; k += (int)blockDim.x)
            run_sum[k] = gram[k];
    }
    __threadfence();                       // this block's partial (or run sum) is visible device-wide ...
    __syncthreads();
    if (threadIdx.x == 0) {
        int* counter = fin.counters + (int64_t)tensor * groups_total + group;
        const int ticket = atomicAdd(counter, 1);      // ... before its ticket is drawn
        is_last = ticket == (in_runs ? runs : s1 - s0) - 1;
        if (is_last)
            *counter = 0;                  // ready for the next level / the next call
    }
    __syncthreads();
    if (!is_last)
        return;
    __threadfence();
    if (in_runs) {
        // the run sums, in run order
        const int64_t stride = (int64_t)groups_total * E;
        for (int k = threadIdx.x; k < E; k += (int)blockDim.x) {
            double sum = 0.0;
#pragma unroll 8
            for (int r = 0; r < runs; ++r)
                sum += __ldcg(run_sums + r * stride + k);
            gram[k] = sum;
        }
        __syncthreads();
    } else {
        add_partials_in_block<R>(partials, s0, s1, group, groups_total, gram);
    }
    tree_weights_from_gram<R>(gram, members, fin.weights + ((int64_t)tensor * groups_total + group) * R, fin.tree,
                              tensor, group);
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

// The Gram matrix of one segment of the group whose first operand is ops.ptr[first], computed by
// the whole block on the fp32 pipes and written to dst[0 .. E).
// With DELTA the rows are (operand - start), rounded to T.
template <typename T, int R, bool VEC, bool DELTA = false, int UNROLL = 1>
__device__ __forceinline__ void gram_of_segment(const OperandTable& ops, int first, int members,
                                                const Segment& seg, float* __restrict__ dst,
                                                const T* start = nullptr)
{
    constexpr int E = gram_entries(R);
    constexpr int V = Element<T>::kVec;

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

    // UNROLL > 1 (the single-launch kernel, whose blocks are few and bound by latency): that many
    // independent vectors per thread in flight
#pragma unroll(UNROLL)
    for (int64_t v = body_begin + (int64_t)threadIdx.x * V; v < body_end; v += (int64_t)kThreads * V) {
        float x[R][V];
        uint4 sraw = make_uint4(0u, 0u, 0u, 0u);
        if constexpr (DELTA)
            sraw = load_plain_16B(start + v);
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (i < members) {
                if constexpr (DELTA)
                    decode_vector<T>(delta_words<T>(load_keep_16B(src[i] + v), sraw), x[i]);
                else
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
            for (int i = 0; i < R; ++i) {
                if constexpr (DELTA)
                    col[i] = i < members ? delta_one(src[i], start, e) : 0.0f;
                else
                    col[i] = i < members ? Element<T>::one(src[i] + e) : 0.0f;
            }
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
    for (int k = threadIdx.x; k < E; k += kThreads) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w)
            s += warp_sums[w][k];
        dst[k] = s;
    }
}

// grid = (segments, groups in this launch); block = kThreads.
// partials[(segment * groups_total + group_base + blockIdx.y) * E + entry]
template <typename T, int R, bool VEC, bool DELTA = false>
__global__ void __launch_bounds__(kThreads)
gram_partial_kernel(const __grid_constant__ OperandTable ops, int operands,
                    const Segment* __restrict__ segments, float* __restrict__ partials,
                    int groups_total, int group_base, FinishArgs fin, const void* start)
{
    constexpr int E = gram_entries(R);
    const Segment seg = segments[blockIdx.x];
    const int first = blockIdx.y * R;
    const int members = min(R, operands - first);
    gram_of_segment<T, R, VEC, DELTA>(ops, first, members, seg,
                                      partials + ((int64_t)blockIdx.x * groups_total + group_base + blockIdx.y) * E,
                                      static_cast<const T*>(start));
    finish_if_last<R>(fin, partials, seg.tensor, group_base + blockIdx.y, groups_total, members, (int)blockIdx.x);
}

// ---- asynchronous copies into shared memory ----------------------------------------------------

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// ---- pass 1 on the tensor cores ----------------------------------------------------------------
//
// G = X X^T with X the R x (segment length) matrix of a group's rows.  A thread block streams the
// segment in tiles of 32 KB (R rows of 32 KB / R contiguous bytes, fully coalesced 512-byte warp
// accesses, cp.async, several tiles in flight).  Warp w multiplies chunks w * DEPTH ... of each
// tile (a chunk is 64 bytes of every row).  Lane (g, t) = (lane / 4, lane % 4) reads, for every
// block of 8 rows, the 16 bytes of row 8 rb + g at chunk offset 16 t: those four words are exactly
// the lane's share of the A fragment (rows g and g + 8 of a 16-row block) and of the B fragment
// (column g of an 8-column block) of mma.sync m16n8k8 (tf32) / m16n8k16 (fp16, bf16), because both
// operands of X X^T are the same rows and the order of the K index inside a chunk is free as long
// as A and B agree.
//
// fp16 / bf16 products are exact in the fp32 accumulator.  fp32 inputs are split x = hi + lo with
// hi the nearest tf32: G = H + C + C^T with H = Xhi Xhi^T (upper blocks only) and C = Xhi Xlo^T
// (all blocks; lo lo^T, about 2^-22 relative, is dropped).  The tensor core's own accumulation is
// not correctly rounded, so for fp32 inputs its chains are kept to one tile and the tile results
// are added with ordinary rounded adds.

template <int R>
__host__ __device__ constexpr int mma_upper_blocks()     // 16 x 8 blocks that touch the upper triangle
{
    int n = 0;
    for (int mb = 0; mb < (R + 15) / 16; ++mb)     // R = 8: half a row block, rows 8..15 are zero
        n += R / 8 - 2 * mb;
    return n;
}
template <int R>
__host__ __device__ constexpr int mma_all_blocks() { return ((R + 15) / 16) * (R / 8); }

// Index of block (mb, nb), nb >= 2 mb, in the upper-block numbering.
template <int R>
__host__ __device__ constexpr int mma_upper_index(int mb, int nb)
{
    int n = 0;
    for (int m = 0; m < mb; ++m)
        n += R / 8 - 2 * m;
    return n + nb - 2 * mb;
}

// Where element (r, c) of a 16 x 8 accumulator block lives: register (0..3) * 32 + lane.
__host__ __device__ constexpr int mma_fragment_slot(int r, int c)
{
    return (((r >= 8 ? 2 : 0) + (c & 1)) * 32) + (r % 8) * 4 + c / 2;
}

#define ADASUM_MMA_ASM(shape, types)                                                                   \
    asm volatile("mma.sync.aligned." shape ".row.col.f32." types ".f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, " \
                 "{%8,%9}, {%0,%1,%2,%3};"                                                             \
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])                                      \
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1))

template <typename T>
__device__ __forceinline__ void mma_step(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1);
template <>
__device__ __forceinline__ void mma_step<float>(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                uint32_t a3, uint32_t b0, uint32_t b1)
{
    ADASUM_MMA_ASM("m16n8k8", "tf32.tf32");
}
template <>
__device__ __forceinline__ void mma_step<__half>(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                 uint32_t a3, uint32_t b0, uint32_t b1)
{
    ADASUM_MMA_ASM("m16n8k16", "f16.f16");
}
template <>
__device__ __forceinline__ void mma_step<__nv_bfloat16>(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                        uint32_t a3, uint32_t b0, uint32_t b1)
{
    ADASUM_MMA_ASM("m16n8k16", "bf16.bf16");
}
#undef ADASUM_MMA_ASM

// The 16 bytes of `row` that start at element e0, as four words, with every element outside
// [begin, end) replaced by zero.  Used for the ragged ends of a segment and for unaligned buffers.
template <typename T>
__device__ __forceinline__ uint4 load_masked_words(const T* row, int64_t e0, int64_t begin, int64_t end);
template <>
__device__ __forceinline__ uint4 load_masked_words<float>(const float* row, int64_t e0, int64_t begin, int64_t end)
{
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int64_t e = e0 + j;
        w[j] = (e >= begin && e < end) ? __float_as_uint(__ldg(row + e)) : 0u;
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}
template <typename T16>
__device__ __forceinline__ uint4 load_masked_words16(const T16* row, int64_t e0, int64_t begin, int64_t end)
{
    const unsigned short* bits = reinterpret_cast<const unsigned short*>(row);
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int64_t e = e0 + 2 * j;
        const uint32_t lo = (e >= begin && e < end) ? (uint32_t)__ldg(bits + e) : 0u;
        const uint32_t hi = (e + 1 >= begin && e + 1 < end) ? (uint32_t)__ldg(bits + e + 1) : 0u;
        w[j] = lo | (hi << 16);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}
template <>
__device__ __forceinline__ uint4 load_masked_words<__half>(const __half* row, int64_t e0, int64_t begin, int64_t end)
{
    return load_masked_words16(row, e0, begin, end);
}
template <>
__device__ __forceinline__ uint4 load_masked_words<__nv_bfloat16>(const __nv_bfloat16* row, int64_t e0,
                                                                   int64_t begin, int64_t end)
{
    return load_masked_words16(row, e0, begin, end);
}

__device__ __forceinline__ void cp_async_16B_shared(uint32_t smem_addr, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void store_shared_16B(uint32_t smem_addr, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(smem_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
__device__ __forceinline__ uint4 load_shared_16B(uint32_t smem_addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(smem_addr)
                 : "memory");
    return v;
}

template <typename T, int R>
__host__ __device__ constexpr int mma_depth() { return 64 / R > 0 ? 64 / R : 1; }   // chunks per warp per tile
template <typename T, int R>
__host__ __device__ constexpr int mma_min_blocks()
{
    return (R >= 64 || (R >= 32 && sizeof(T) == 4)) ? 1 : 2;
}
// Tiles kept in shared memory: 3 where two blocks share an SM, 6 for the register-heavy kernels
// that run one block per SM.
template <typename T, int R>
__host__ __device__ constexpr int mma_stages() { return mma_min_blocks<T, R>() == 1 ? 6 : 3; }
constexpr int kMmaTileBytes = 32 * 1024;
// With DELTA every stage carries one more row: the same columns of `start`.
template <typename T, int R, bool DELTA = false>
__host__ __device__ constexpr size_t mma_smem_bytes()
{
    return (size_t)mma_stages<T, R>() * (kMmaTileBytes + (DELTA ? kMmaTileBytes / R : 0));
}

// Sizes of the tensor-core Gram pass that its pieces below share.
template <typename T, int R, bool DELTA>
struct MmaShape {
    static constexpr int V = Element<T>::kVec;          // elements per 16-byte vector
    static constexpr int RB = R / 8;                    // blocks of 8 rows
    static constexpr int MB = (R + 15) / 16;            // blocks of 16 rows (R = 8: the upper half is zero)
    static constexpr int RBP = 2 * MB;                  // row blocks the fragments are indexed with
    static constexpr int UBLK = mma_upper_blocks<R>();
    static constexpr bool SPLIT = sizeof(T) == 4;
    static constexpr int CBLK = SPLIT ? mma_all_blocks<R>() : 0;
    static constexpr int CDIM = SPLIT ? CBLK : 1;
    static constexpr int DEPTH = mma_depth<T, R>();
    static constexpr int STAGES = mma_stages<T, R>();
    static constexpr int ROW_BYTES = kMmaTileBytes / R;
    static constexpr int STAGE_BYTES = kMmaTileBytes + (DELTA ? ROW_BYTES : 0);
    static constexpr int PIECES_PER_ROW = ROW_BYTES / 16;
    static constexpr int TILE_ELEMS = PIECES_PER_ROW * V;               // elements of one row in a tile
    static constexpr int PIECES = kMmaTileBytes / 16 / kThreads;        // 16-byte pieces a thread copies per tile
    static constexpr int ROWS_PER_PASS = kThreads / PIECES_PER_ROW;     // piece i of a thread is in row row0 + i * this
    static constexpr int SLOTS = (UBLK + CBLK) * 128;                   // accumulator words of a warp
    static constexpr int SLAB_BYTES = kWarps * SLOTS * (int)sizeof(float);
    static_assert(DEPTH * kWarps * 64 == ROW_BYTES, "a tile row is split evenly among the warps");
    static_assert(PIECES_PER_ROW % 32 == 0 && kThreads % PIECES_PER_ROW == 0, "a warp copies within one row");
    static_assert(SLAB_BYTES <= STAGES * STAGE_BYTES, "the stages hold the fragments");
};

// Copy side of the tensor-core Gram pass: piece i of this thread is (row0 + i * ROWS_PER_PASS, col0)
// of every tile.
//
// Shared-memory layout of a tile: row-major, 64-byte chunk index XOR (row & 1), so that the
// fragment reads of a quarter warp (two rows, four 16-byte pieces each) fall into distinct banks.
//
// DELTA: the rows are (operand - start), rounded to T.  The tile gets one more row, unswizzled,
// with the same columns of `start`; a lane subtracts its 16 bytes of it from every fragment it
// loads.  Rows beyond the group's members are copies of `start`, so that they come out as zero.
template <typename T, int R, bool VEC, bool DELTA>
struct MmaCopier {
    using S = MmaShape<T, R, DELTA>;
    const T* src[S::PIECES];     // row pointer + this thread's column; rows beyond the members alias row 0
    const T* start_src;          // DELTA: threads of row0 == 0 copy it
    uint32_t smem_base;
    int row0, col0, members;
    bool full_group;

    __device__ __forceinline__ void init(const OperandTable& ops, int first, int members_, const void* start_ptr,
                                         uint32_t smem_base_)
    {
        smem_base = smem_base_;
        members = members_;
        row0 = threadIdx.x / S::PIECES_PER_ROW;
        col0 = threadIdx.x % S::PIECES_PER_ROW;
#pragma unroll
        for (int i = 0; i < S::PIECES; ++i) {
            const int row = row0 + i * S::ROWS_PER_PASS;
            src[i] = static_cast<const T*>(ops.ptr[first + (row < members ? row : 0)]) + col0 * S::V;
            if (DELTA && row >= members)
                src[i] = static_cast<const T*>(start_ptr) + col0 * S::V;
        }
        start_src = static_cast<const T*>(start_ptr) + col0 * S::V;
        full_group = members == R || DELTA;
    }
    // byte offset of piece i inside a tile (the swizzle depends on the row's parity)
    __device__ __forceinline__ uint32_t piece_offset(int i) const
    {
        const int row = row0 + i * S::ROWS_PER_PASS;
        return row * S::ROW_BYTES + (((col0 >> 2) ^ (row & 1)) << 6) + ((col0 & 3) << 4);
    }
    // Starts the copy of the tile whose first element is tile_elem0 into `stage` (elements outside
    // [begin, end) become zero).  The caller commits the copy group.
    __device__ __forceinline__ void issue(int64_t begin, int64_t end, int64_t tile_elem0, int stage) const
    {
        const uint32_t dst = smem_base + stage * S::STAGE_BYTES;
        if (VEC && full_group && tile_elem0 >= begin && tile_elem0 + S::TILE_ELEMS <= end) {
#pragma unroll
            for (int i = 0; i < S::PIECES; ++i)
                cp_async_16B_shared(dst + piece_offset(i), src[i] + tile_elem0);
            if (DELTA && row0 == 0)
                cp_async_16B_shared(dst + kMmaTileBytes + (col0 << 4), start_src + tile_elem0);
        } else {
            // ragged tile, partial group or unaligned buffers: test every piece
            const int64_t e0 = tile_elem0 + (int64_t)col0 * S::V;
            const bool whole = VEC && e0 >= begin && e0 + S::V <= end;
#pragma unroll
            for (int i = 0; i < S::PIECES; ++i) {
                const uint32_t slot = dst + piece_offset(i);
                if (!DELTA && row0 + i * S::ROWS_PER_PASS >= members)
                    store_shared_16B(slot, make_uint4(0u, 0u, 0u, 0u));
                else if (whole)
                    cp_async_16B_shared(slot, src[i] + tile_elem0);
                else
                    store_shared_16B(slot, load_masked_words<T>(src[i] - col0 * S::V, e0, begin, end));
            }
            if (DELTA && row0 == 0) {
                if (whole)
                    cp_async_16B_shared(dst + kMmaTileBytes + (col0 << 4), start_src + tile_elem0);
                else
                    store_shared_16B(dst + kMmaTileBytes + (col0 << 4),
                                     load_masked_words<T>(start_src - col0 * S::V, e0, begin, end));
            }
        }
    }
};

// Multiply side: adds the products of the tile in `stage` to the warp's accumulators.  `acc` are
// the accumulators themselves for 16-bit inputs and the rounded sums of H for fp32, `acc_c` the
// rounded sums of C (fp32 only).
template <typename T, int R, bool DELTA>
__device__ __forceinline__ void mma_multiply_tile(uint32_t stage_addr, int warp, int g, int t,
                                                  float (&acc)[MmaShape<T, R, DELTA>::UBLK][4],
                                                  float (&acc_c)[MmaShape<T, R, DELTA>::CDIM][4])
{
    using S = MmaShape<T, R, DELTA>;
    constexpr int RB = S::RB, MB = S::MB, RBP = S::RBP, UBLK = S::UBLK, CBLK = S::CBLK, DEPTH = S::DEPTH;
    constexpr int ROW_BYTES = S::ROW_BYTES;
    const uint32_t src_stage = stage_addr + g * ROW_BYTES + (t << 4);
    const uint32_t start_stage = stage_addr + kMmaTileBytes + (t << 4);
    uint32_t chunk_off[DEPTH];
#pragma unroll
    for (int d = 0; d < DEPTH; ++d)
        chunk_off[d] = ((warp * DEPTH + d) ^ (g & 1)) << 6;

    if constexpr (!S::SPLIT) {
#pragma unroll
        for (int d = 0; d < DEPTH; ++d) {
            uint32_t w[RBP][4];
            uint4 sv = make_uint4(0u, 0u, 0u, 0u);
            if constexpr (DELTA)
                sv = load_shared_16B(start_stage + ((warp * DEPTH + d) << 6));
#pragma unroll
            for (int rb = 0; rb < RBP; ++rb) {
                uint4 v = rb < RB ? load_shared_16B(src_stage + chunk_off[d] + rb * 8 * ROW_BYTES)
                                  : make_uint4(0u, 0u, 0u, 0u);
                if (DELTA && rb < RB)
                    v = delta_words<T>(v, sv);
                w[rb][0] = v.x; w[rb][1] = v.y; w[rb][2] = v.z; w[rb][3] = v.w;
            }
#pragma unroll
            for (int step = 0; step < 2; ++step) {
#pragma unroll
                for (int mb = 0; mb < MB; ++mb)
#pragma unroll
                    for (int nb = 2 * mb; nb < RB; ++nb)
                        mma_step<T>(acc[mma_upper_index<R>(mb, nb)], w[2 * mb][2 * step], w[2 * mb + 1][2 * step],
                                    w[2 * mb][2 * step + 1], w[2 * mb + 1][2 * step + 1], w[nb][2 * step],
                                    w[nb][2 * step + 1]);
            }
        }
    } else {
        float tile_h[UBLK][4], tile_c[S::CDIM][4];
#pragma unroll
        for (int b = 0; b < UBLK; ++b)
#pragma unroll
            for (int r = 0; r < 4; ++r)
                tile_h[b][r] = 0.0f;
#pragma unroll
        for (int b = 0; b < CBLK; ++b)
#pragma unroll
            for (int r = 0; r < 4; ++r)
                tile_c[b][r] = 0.0f;
#pragma unroll
        for (int d = 0; d < DEPTH; ++d) {
            uint32_t hi[RBP][4], lo[RBP][4];
            uint4 sv = make_uint4(0u, 0u, 0u, 0u);
            if constexpr (DELTA)
                sv = load_shared_16B(start_stage + ((warp * DEPTH + d) << 6));
#pragma unroll
            for (int rb = 0; rb < RBP; ++rb) {
                uint4 v = rb < RB ? load_shared_16B(src_stage + chunk_off[d] + rb * 8 * ROW_BYTES)
                                  : make_uint4(0u, 0u, 0u, 0u);
                if (DELTA && rb < RB)
                    v = delta_words<T>(v, sv);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    // nearest tf32 by integer arithmetic (the conversion instruction runs on
                    // the slow special-function pipe): add half a tf32 ulp, drop 13 bits
                    hi[rb][j] = (w[j] + 0x1000u) & 0xffffe000u;
                    lo[rb][j] = __float_as_uint(__uint_as_float(w[j]) - __uint_as_float(hi[rb][j]));
                }
            }
#pragma unroll
            for (int step = 0; step < 2; ++step) {
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
#pragma unroll
                    for (int nb = 0; nb < RB; ++nb) {
                        if (nb >= 2 * mb)
                            mma_step<T>(tile_h[mma_upper_index<R>(mb, nb)], hi[2 * mb][2 * step],
                                        hi[2 * mb + 1][2 * step], hi[2 * mb][2 * step + 1],
                                        hi[2 * mb + 1][2 * step + 1], hi[nb][2 * step], hi[nb][2 * step + 1]);
                        mma_step<T>(tile_c[mb * RB + nb], hi[2 * mb][2 * step], hi[2 * mb + 1][2 * step],
                                    hi[2 * mb][2 * step + 1], hi[2 * mb + 1][2 * step + 1], lo[nb][2 * step],
                                    lo[nb][2 * step + 1]);
                    }
                }
            }
        }
#pragma unroll
        for (int b = 0; b < UBLK; ++b)
#pragma unroll
            for (int r = 0; r < 4; ++r)
                acc[b][r] += tile_h[b][r];
#pragma unroll
        for (int b = 0; b < CBLK; ++b)
#pragma unroll
            for (int r = 0; r < 4; ++r)
                acc_c[b][r] += tile_c[b][r];
    }
}

template <typename T, int R, bool DELTA>
__device__ __forceinline__ void mma_clear(float (&acc)[MmaShape<T, R, DELTA>::UBLK][4],
                                          float (&acc_c)[MmaShape<T, R, DELTA>::CDIM][4])
{
    using S = MmaShape<T, R, DELTA>;
#pragma unroll
    for (int b = 0; b < S::UBLK; ++b)
#pragma unroll
        for (int r = 0; r < 4; ++r)
            acc[b][r] = 0.0f;
#pragma unroll
    for (int b = 0; b < S::CDIM; ++b)
#pragma unroll
        for (int r = 0; r < 4; ++r)
            acc_c[b][r] = 0.0f;
}

// Block reduction, first half: every warp parks its fragments in `slab_base` (SLAB_BYTES of shared
// memory that nobody else is using: stage memory whose tile has been consumed).  Begins with a
// barrier (every warp has finished reading the stage that becomes the slab).
template <typename T, int R, bool DELTA>
__device__ __forceinline__ void mma_park(float* slab_base, int warp, int lane,
                                         const float (&acc)[MmaShape<T, R, DELTA>::UBLK][4],
                                         const float (&acc_c)[MmaShape<T, R, DELTA>::CDIM][4])
{
    using S = MmaShape<T, R, DELTA>;
    constexpr int UBLK = S::UBLK, CBLK = S::CBLK, SLOTS = S::SLOTS;
    float* slab = slab_base + warp * SLOTS;
    __syncthreads();
#pragma unroll
    for (int b = 0; b < UBLK; ++b)
#pragma unroll
        for (int r = 0; r < 4; ++r)
            slab[(b * 4 + r) * 32 + lane] = acc[b][r];
#pragma unroll
    for (int b = 0; b < CBLK; ++b)
#pragma unroll
        for (int r = 0; r < 4; ++r)
            slab[((UBLK + b) * 4 + r) * 32 + lane] = acc_c[b][r];
}

// Second half: each slot is added over the warps in warp order and the packed upper triangle is
// written to dst[0 .. E).  The slab is free again once every thread has passed this function's
// last barrier, i.e. on return.
template <typename T, int R, bool DELTA>
__device__ __forceinline__ void mma_sum_store(const float* slab_base, float* __restrict__ dst)
{
    using S = MmaShape<T, R, DELTA>;
    constexpr int UBLK = S::UBLK, SLOTS = S::SLOTS, RB = S::RB;
    __shared__ float total[SLOTS];
    __syncthreads();
    for (int slot = threadIdx.x; slot < SLOTS; slot += kThreads) {
        const float* column = slab_base + slot;
        float sum = column[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w)
            sum = sum + column[w * SLOTS];
        total[slot] = sum;
    }
    __syncthreads();
    // entries (i <= j) of the packed upper triangle from the accumulator fragments
    for (int idx = threadIdx.x; idx < R * R; idx += kThreads) {
        const int i = idx / R, j = idx % R;
        if (i > j)
            continue;
        float v = total[mma_upper_index<R>(i / 16, j / 8) * 128 + mma_fragment_slot(i % 16, j % 8)];
        if (S::SPLIT) {
            v += total[(UBLK + (i / 16) * RB + j / 8) * 128 + mma_fragment_slot(i % 16, j % 8)];   // C_ij
            v += total[(UBLK + (j / 16) * RB + i / 8) * 128 + mma_fragment_slot(j % 16, i % 8)];   // C_ji
        }
        dst[gram_index(R, i, j)] = v;
    }
}

// The Gram matrix of one segment of the group whose first operand is ops.ptr[first], formed by the
// whole block (kThreads threads, mma_smem_bytes<T, R>() of dynamic shared memory) on the tensor cores
// and written to dst[0 .. E).
//
// The pipeline is the usual multi-stage one: wait for the oldest copy group, one __syncthreads
// per tile, refill the slot that was consumed in the previous iteration.
template <typename T, int R, bool VEC, bool DELTA = false>
__device__ __forceinline__ void gram_segment_mma(const OperandTable& ops, int first, int members, const Segment& seg,
                                                 float* __restrict__ dst, const void* start_ptr)
{
    using S = MmaShape<T, R, DELTA>;
    constexpr int STAGES = S::STAGES;
    extern __shared__ __align__(128) unsigned char stage_mem[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;

    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    const int64_t k0 = VEC ? begin / S::V * S::V : begin;
    const int ntiles = (int)((end - k0 + S::TILE_ELEMS - 1) / S::TILE_ELEMS);

    const uint32_t smem_base = static_cast<uint32_t>(__cvta_generic_to_shared(stage_mem));
    MmaCopier<T, R, VEC, DELTA> copier;
    copier.init(ops, first, members, start_ptr, smem_base);
    auto issue = [&](int tile, int stage) {
        if (tile < ntiles)
            copier.issue(begin, end, k0 + (int64_t)tile * S::TILE_ELEMS, stage);
        cp_async_commit();
    };

    float acc[S::UBLK][4], acc_c[S::CDIM][4];
    mma_clear<T, R, DELTA>(acc, acc_c);

#pragma unroll
    for (int st = 0; st < STAGES - 1; ++st)
        issue(st, st);

    int stage = 0;
    for (int tile = 0; tile < ntiles; ++tile) {
        cp_async_wait<STAGES - 2>();     // this thread's copies for `tile` have landed
        __syncthreads();                 // ... and everybody's; the previous tile's slot is free
        int refill = stage + STAGES - 1;
        if (refill >= STAGES)
            refill -= STAGES;
        issue(tile + STAGES - 1, refill);
        mma_multiply_tile<T, R, DELTA>(smem_base + stage * S::STAGE_BYTES, warp, g, t, acc, acc_c);
        if (++stage == STAGES)
            stage = 0;
    }
    cp_async_wait<0>();
    mma_park<T, R, DELTA>(reinterpret_cast<float*>(stage_mem), warp, lane, acc, acc_c);
    mma_sum_store<T, R, DELTA>(reinterpret_cast<const float*>(stage_mem), dst);
}

// grid = (segments, groups in this launch); block = kThreads; dynamic shared memory =
// mma_smem_bytes<T, R>().
template <typename T, int R, bool VEC, bool DELTA = false>
__global__ void __launch_bounds__(kThreads, mma_min_blocks<T, R>())
gram_partial_mma_kernel(const __grid_constant__ OperandTable ops, int operands,
                        const Segment* __restrict__ segments, float* __restrict__ partials,
                        int groups_total, int group_base, FinishArgs fin, const void* start_ptr)
{
    constexpr int E = gram_entries(R);
    const Segment seg = segments[blockIdx.x];
    const int first = blockIdx.y * R;
    const int members = min(R, operands - first);
    gram_segment_mma<T, R, VEC, DELTA>(ops, first, members, seg,
                                       partials + ((int64_t)blockIdx.x * groups_total + group_base + blockIdx.y) * E,
                                       start_ptr);
    finish_if_last<R>(fin, partials, seg.tensor, group_base + blockIdx.y, groups_total, members, (int)blockIdx.x);
}

// ---- pass 1 for groups of 64 fp16 / bf16 rows: tcgen05 ------------------------------------------
//
// At radix 64 the warp-level mma.sync path is bound by the tensor pipe.  The fifth-generation
// tensor core instruction takes both operands straight from shared memory and keeps the 64 x 64
// fp32 accumulator in tensor memory, so one thread issues a whole tile's multiplications and the
// other threads only move data.
//
// Tile = 64 rows x 1024 bytes (8 K-blocks of 64 elements), 64 KB, copied with coalesced cp.async
// (a warp moves 512 contiguous bytes of one row per instruction), laid out as eight
// [64 rows x 128 bytes] blocks in the 128-byte-swizzle K-major form the instruction's
// shared-memory descriptor expects: 16-byte chunk c of row r of a block sits at
// r * 128 + ((c ^ (r & 7)) * 16).  A and B are the SAME block (X X^T): M = N = 64, K = 16 per
// instruction, 32 instructions per tile.  With M = 64 the accumulator's rows 16 q .. 16 q + 15
// live in tensor-memory lanes 32 q .. 32 q + 15.
//
// Roles: all warps but the last copy (each warp whole half-rows), lane 0 of the last warp
// multiplies.  Per stage two mbarriers: `full` (the copying threads arrive when their pieces of
// the tile have landed and are fenced for the tensor core) and `empty` (the tensor core arrives
// when the multiplications that read the stage are done).  No block-wide barrier inside the loop.
//
// Every wait is bounded; if one runs out the thread records ADASUM_ERR_TIMEOUT in *status, stops
// waiting and keeps going (its block's numbers are then wrong, but every access stays in bounds),
// the block frees its tensor memory and returns.

constexpr int kTcKBlocks = 8;                 // K-blocks (64 elements, 128 bytes of a row) per tile
constexpr int kTcStages = 3;
constexpr int kTcAhead = kTcStages - 1;       // tiles in flight
constexpr int kTcThreads = 512;
constexpr int kTcProducerWarps = kTcThreads / 32 - 1;
constexpr int kTcProducers = kTcProducerWarps * 32;
constexpr int kTcHalfRows = 64 * kTcKBlocks / 4;                 // 512-byte pieces of rows per tile
constexpr int kTcRowsPerWarp = (kTcHalfRows + kTcProducerWarps - 1) / kTcProducerWarps;
constexpr int kTcTileBytes = kTcKBlocks * 8192;
constexpr int kTcPadBytes = 8 * 1024;         // slack after the last stage
constexpr size_t kTcSmemBytes = (size_t)kTcStages * kTcTileBytes + kTcPadBytes + 1024;   // + room to align to 1024
constexpr uint32_t kTcSpinLimit = 1u << 22;   // about a tenth of a second; a real wait is microseconds
constexpr uint32_t kTcSelftestSpinLimit = 1u << 14;   // the self-test's wait: long after every issued multiplication is done

__device__ __forceinline__ uint32_t mbarrier_try_wait_parity(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done)
                 : "r"(bar), "r"(parity)
                 : "memory");
    return done;
}

// Returns false if the barrier did not complete the phase within the spin limit.
__device__ __forceinline__ bool mbarrier_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = kTcSpinLimit)
{
    for (uint32_t spin = 0; spin < limit; ++spin)
        if (mbarrier_try_wait_parity(bar, parity))
            return true;
    return false;
}

__device__ __forceinline__ void mbarrier_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t tc_smem_descriptor(uint32_t smem_addr)
{
    const uint64_t start = (uint64_t)((smem_addr & 0x3ffffu) >> 4);          // bits 0..13
    const uint64_t leading = (uint64_t)1 << 16;                              // bits 16..29: unused with this swizzle
    const uint64_t stride = (uint64_t)(1024 >> 4) << 32;                     // bits 32..45: stride byte offset
    const uint64_t version = (uint64_t)1 << 46;                              // descriptor version of this architecture
    const uint64_t swizzle_128b = (uint64_t)2 << 61;                         // bits 61..63: layout type
    return start | leading | stride | version | swizzle_128b;
}

// grid = (segments, groups in this launch); block = kTcThreads; dynamic shared memory = kTcSmemBytes.
// Only for 16-byte aligned operands and launches in which every group has all 64 members.
template <typename T>
__global__ void __launch_bounds__(kTcThreads, 1)
gram_partial_tc64_kernel(const __grid_constant__ OperandTable ops, int operands,
                         const Segment* __restrict__ segments, float* __restrict__ partials,
                         int groups_total, int group_base, FinishArgs fin, int* __restrict__ status)
{
    static_assert(sizeof(T) == 2, "fp16 / bf16 only");
    constexpr int R = 64;
    constexpr int E = gram_entries(R);
    constexpr int V = 8;                                   // elements per 16-byte piece
    constexpr int TILE_ELEMS = 64 * kTcKBlocks;            // elements of one row in a tile
    extern __shared__ __align__(1024) unsigned char tc_smem_raw[];
    __shared__ __align__(8) unsigned long long full_bar[kTcStages], empty_bar[kTcStages];
    __shared__ uint32_t tmem_base_slot;

    const Segment seg = segments[blockIdx.x];
    const int first = blockIdx.y * R;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    const int64_t k0 = begin / V * V;
    const int ntiles = (int)((end - k0 + TILE_ELEMS - 1) / TILE_ELEMS);

    // stage memory, aligned to the 1024 bytes the swizzle pattern repeats with
    const uint32_t raw_base = static_cast<uint32_t>(__cvta_generic_to_shared(tc_smem_raw));
    const uint32_t smem_base = (raw_base + 1023u) & ~1023u;
    const uint32_t full0 = static_cast<uint32_t>(__cvta_generic_to_shared(&full_bar[0]));
    const uint32_t empty0 = static_cast<uint32_t>(__cvta_generic_to_shared(&empty_bar[0]));

    // ---- set-up: barriers, tensor memory (64 columns of fp32 accumulator)
    if (threadIdx.x == 0) {
#pragma unroll
        for (int st = 0; st < kTcStages; ++st) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full0 + 8 * st), "r"(kTcProducers));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(empty0 + 8 * st));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 64;" ::"r"(
            static_cast<uint32_t>(__cvta_generic_to_shared(&tmem_base_slot))));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = tmem_base_slot;

    bool timed_out = false;
    if (warp < kTcProducerWarps) {
        // ---- copying warps: warp w moves rows w, w + 7, ...; lane = 16-byte chunk of the 512-byte row
        const T* copy_src[kTcRowsPerWarp];
        uint32_t copy_off[kTcRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kTcRowsPerWarp; ++i) {
            // 512-byte piece h of the tile: row h / (pieces per row), chunks 32 (h % pieces per row) + lane
            const int h = warp + kTcProducerWarps * i;
            const int hh = h < kTcHalfRows ? h : 0;
            const int r = hh / (kTcKBlocks / 4), chunk = (hh % (kTcKBlocks / 4)) * 32 + lane;
            copy_src[i] = static_cast<const T*>(ops.ptr[first + r]) + chunk * V;
            copy_off[i] = (chunk >> 3) * 8192 + r * 128 + (((chunk & 7) ^ (r & 7)) << 4);
        }
        auto issue_copy = [&](int tile) {
            if (tile < ntiles) {
                const int stage = tile % kTcStages;
                if (tile >= kTcStages && !timed_out) {
                    // the multiplications of tile - S read this stage: wait for the tensor core
                    if (!mbarrier_wait_bounded(empty0 + 8 * stage, (uint32_t)((tile / kTcStages - 1) & 1)))
                        timed_out = true;
                }
                const uint32_t dst = smem_base + stage * kTcTileBytes;
                const int64_t tile_elem0 = k0 + (int64_t)tile * TILE_ELEMS;
                const bool interior = tile_elem0 >= begin && tile_elem0 + TILE_ELEMS <= end;
#pragma unroll
                for (int i = 0; i < kTcRowsPerWarp; ++i) {
                    const int h = warp + kTcProducerWarps * i;
                    if (h < kTcHalfRows) {
                        const int chunk = (h % (kTcKBlocks / 4)) * 32 + lane;
                        const int64_t e0 = tile_elem0 + (int64_t)chunk * V;
                        if (interior || (e0 >= begin && e0 + V <= end))
                            cp_async_16B_shared(dst + copy_off[i], copy_src[i] + tile_elem0);
                        else
                            store_shared_16B(dst + copy_off[i],
                                             load_masked_words<T>(copy_src[i] - chunk * V, e0, begin, end));
                    }
                }
            }
            cp_async_commit();
        };
#pragma unroll
        for (int tile = 0; tile < kTcAhead; ++tile)
            issue_copy(tile);
        for (int tile = 0; tile < ntiles; ++tile) {
            cp_async_wait<kTcAhead - 1>();                                 // this thread's pieces of `tile` have landed
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // ... and are visible to the tensor core
            mbarrier_arrive(full0 + 8 * (tile % kTcStages));
            issue_copy(tile + kTcAhead);
        }
        cp_async_wait<0>();
    } else if (lane == 0) {
        // ---- multiplying thread
        // instruction descriptor: fp32 accumulator, A and B of type T, both K-major, N = 64, M = 64
        constexpr uint32_t kFormat = __is_same(T, __half) ? 0u : 1u;     // 0 = fp16, 1 = bf16
        constexpr uint32_t kInstr =
            (1u << 4) | (kFormat << 7) | (kFormat << 10) | ((64u >> 3) << 17) | ((64u >> 4) << 24);
        for (int tile = 0; tile < ntiles; ++tile) {
            if (fin.selftest_timeout && tile == ntiles - 1)
                break;          // self-test: nothing arrives on this tile's `empty` barrier
            const int stage = tile % kTcStages;
            if (!timed_out && !mbarrier_wait_bounded(full0 + 8 * stage, (uint32_t)((tile / kTcStages) & 1)))
                timed_out = true;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tile_base = smem_base + stage * kTcTileBytes;
#pragma unroll
            for (int kb = 0; kb < kTcKBlocks; ++kb) {
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    // K-block kb, elements 16 ks .. 16 ks + 15 of it: 32 bytes further into the swizzled rows
                    const uint64_t desc = tc_smem_descriptor(tile_base + kb * 8192 + ks * 32);
                    const uint32_t accumulate = (tile > 0 || kb > 0 || ks > 0) ? 1u : 0u;
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                 ::"r"(tmem_acc), "l"(desc), "l"(desc), "r"(kInstr), "r"(accumulate)
                                 : "memory");
                }
            }
            // arrives on the barrier once everything issued so far has finished reading shared memory
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                             empty0 + 8 * stage)
                         : "memory");
        }
    }

    // ---- epilogue: wait for the last tile's multiplications, read the accumulator rows 0..63
    {
        const int last = ntiles - 1;
        if (!timed_out &&
            !mbarrier_wait_bounded(empty0 + 8 * (last % kTcStages), (uint32_t)((last / kTcStages) & 1),
                                   fin.selftest_timeout ? kTcSelftestSpinLimit : kTcSpinLimit))
            timed_out = true;
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (timed_out)
        atomicExch(status, (int)ADASUM_DEVICE_TIMEOUT);
    float* dst = partials + ((int64_t)blockIdx.x * groups_total + group_base + blockIdx.y) * E;
    if (warp < 4) {
        // With M = 64 the accumulator's rows 16 w .. 16 w + 15 live in tensor-memory lanes
        // 32 w .. 32 w + 15, which are the lanes warp w may read: lane l < 16 of warp w gets row
        // 16 w + l, 16 columns at a time.
        const int i = 16 * warp + lane;
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
            uint32_t r[16];
            const uint32_t taddr = tmem_acc + ((uint32_t)(32 * warp) << 16) + cb * 16;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                         : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                           "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                         : "r"(taddr)
                         : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (lane < 16) {
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const int j = cb * 16 + c;
                    if (j >= i)
                        dst[gram_index(R, i, j)] = __uint_as_float(r[c]);
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 64;" ::"r"(tmem_acc) : "memory");
    finish_if_last<R>(fin, partials, seg.tensor, group_base + blockIdx.y, groups_total, R, (int)blockIdx.x);
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

// The binary tree evaluated on a Gram matrix held in shared memory; called by every thread of a
// block of at least R threads.  Leaf weights start at 1; bottom-up over block widths 1, 2, 4, ...:
// the block [L, L+w) is paired with [L+w, L+2w) (a block without a right sibling is carried
// unchanged); with d = sum_{i in left, k in right} w_i w_k G_ik and the two blocks' squared norms
// the pair coefficients follow, every leaf weight of the left (right) block is multiplied by ca
// (cb), and the parent's squared norm is ca^2 |a|^2 + cb^2 |b|^2 + 2 ca cb d.
//
// opt.linear selects the other recursion of Section 3.4 instead: x = g_0, then x = Adasum(x, g_k)
// for k = 1, 2, ...; the same algebra with the left operand always the running result.
//
// Also written, when asked for: the sum of the leaves' squared norms (first level) and the
// orthogonality measure |result|^2 / sum_i |g_i|^2 of Section 3.6 (last level; NaN when every
// leaf is zero).
template <int R, typename W>
__device__ void tree_weights_from_gram(const double* gram, int members, W* __restrict__ dst,
                                       const TreeOptions& opt, int tensor, int group)
{
    __shared__ double weight[R], norm[R], row_dot[R], coef_a[R / 2 > 0 ? R / 2 : 1], coef_b[R / 2 > 0 ? R / 2 : 1];
    const int tid = threadIdx.x;
    if (tid < R) {
        // A leaf stored as s x its gradient starts with weight 1 / s instead of 1: every product
        // below then is the one of the gradients themselves, and the weight that comes out is the
        // one to apply to the stored values.
        double unit = 1.0;
        if (opt.leaf_scales != nullptr && opt.level_is_first && tid < members)
            unit = 1.0 / (double)opt.leaf_scales[((int64_t)group * R + tid) * opt.num_tensors + tensor];
        weight[tid] = unit;
        norm[tid] = tid < members ? gram[gram_index(R, tid, tid)] * unit * unit : 0.0;
    }
    __syncthreads();
    double leaf_sum = 0.0;
    if (tid == 0 && (opt.leaf_norm_sums != nullptr || opt.orthogonality != nullptr))
        for (int i = 0; i < members; ++i)
            leaf_sum += norm[i];
    __syncthreads();
    if (!opt.linear) {
        for (int w = 1; w < members; w *= 2) {
            // leaf i of a left block: weight_i * sum over the sibling block of weight_k G_ik
            if (tid < members) {
                const int left = tid / (2 * w) * (2 * w);
                const int mid = left + w;
                double acc = 0.0;
                if (tid < mid && mid < members) {
                    const int right_end = min(left + 2 * w, members);
                    for (int k = mid; k < right_end; ++k)
                        acc += weight[k] * gram[gram_index(R, tid, k)];
                    acc *= weight[tid];
                }
                row_dot[tid] = acc;
            }
            __syncthreads();
            // one thread per pair of sibling blocks
            const int pairs = (members + 2 * w - 1) / (2 * w);
            if (tid < pairs) {
                const int left = tid * 2 * w, mid = left + w;
                double ca = 1.0, cb = 1.0;
                if (mid < members) {
                    double dot = 0.0;
                    for (int i = left; i < mid; ++i)
                        dot += row_dot[i];
                    pair_coefficients(dot, norm[left], norm[mid], ca, cb);
                    norm[left] = ca * ca * norm[left] + cb * cb * norm[mid] + 2.0 * ca * cb * dot;
                }
                coef_a[tid] = ca;
                coef_b[tid] = cb;
            }
            __syncthreads();
            if (tid < members) {
                const int pair = tid / (2 * w);
                const int mid = pair * 2 * w + w;
                if (mid < members)
                    weight[tid] *= tid < mid ? coef_a[pair] : coef_b[pair];
            }
            __syncthreads();
        }
    } else if (opt.linear == 2) {
        // The binary tree taken top-down: the node over leaves [lo, hi) combines the results of
        // [lo, mid) and [mid, hi), mid = lo + (hi - lo) / 2.  Nodes are processed from the deepest
        // depth up; a thread finds the node of its leaf at a depth by walking down from the root.
        // A node's squared norm and coefficients are kept at index lo.
        __shared__ double node_ca[R], node_cb[R];
        int max_depth = 0;
        while ((1 << max_depth) < members)
            ++max_depth;
        for (int depth = max_depth - 1; depth >= 0; --depth) {
            int lo = 0, hi = members;
            bool active = tid < members;
            for (int t = 0; t < depth && active; ++t) {
                if (hi - lo < 2) {
                    active = false;          // this leaf's branch ended above `depth`
                } else {
                    const int m = lo + (hi - lo) / 2;
                    if (tid < m)
                        hi = m;
                    else
                        lo = m;
                }
            }
            active = active && hi - lo >= 2;
            const int mid = lo + (hi - lo) / 2;
            if (tid < R) {
                double acc = 0.0;
                if (active && tid < mid) {
                    for (int k = mid; k < hi; ++k)
                        acc += weight[k] * gram[gram_index(R, tid, k)];
                    acc *= weight[tid];
                }
                row_dot[tid] = acc;
            }
            __syncthreads();
            if (active && tid == lo) {
                double dot = 0.0;
                for (int i = lo; i < mid; ++i)
                    dot += row_dot[i];
                double ca, cb;
                pair_coefficients(dot, norm[lo], norm[mid], ca, cb);
                norm[lo] = ca * ca * norm[lo] + cb * cb * norm[mid] + 2.0 * ca * cb * dot;
                node_ca[lo] = ca;
                node_cb[lo] = cb;
            }
            __syncthreads();
            if (active)
                weight[tid] *= tid < mid ? node_ca[lo] : node_cb[lo];
            __syncthreads();
        }
    } else {
        for (int k = 1; k < members; ++k) {
            if (tid < k)
                row_dot[tid] = weight[tid] * weight[k] * gram[gram_index(R, tid, k)];
            __syncthreads();
            if (tid == 0) {
                double dot = 0.0;
                for (int i = 0; i < k; ++i)
                    dot += row_dot[i];
                double ca, cb;
                pair_coefficients(dot, norm[0], norm[k], ca, cb);
                norm[0] = ca * ca * norm[0] + cb * cb * norm[k] + 2.0 * ca * cb * dot;
                coef_a[0] = ca;
                coef_b[0] = cb;
            }
            __syncthreads();
            if (tid < k)
                weight[tid] *= coef_a[0];
            else if (tid == k)
                weight[tid] *= coef_b[0];
            __syncthreads();
        }
    }
    if (tid < R)
        dst[tid] = tid < members ? (W)weight[tid] : (W)0;
    if (tid == 0) {
        if (opt.leaf_norm_sums != nullptr && opt.level_is_first)
            opt.leaf_norm_sums[(int64_t)tensor * opt.groups_first + group] = leaf_sum;
        if (opt.orthogonality != nullptr && opt.level_is_last) {
            double denom = leaf_sum;
            if (!opt.level_is_first) {
                denom = 0.0;
                for (int gf = 0; gf < opt.groups_first; ++gf)
                    denom += opt.leaf_norm_sums[(int64_t)tensor * opt.groups_first + gf];
            }
            opt.orthogonality[tensor] = denom == 0.0 ? __int_as_float(0x7fc00000) : (float)(norm[0] / denom);
        }
    }
}

// Partial matrices of segments seg_begin .. seg_end added in fp64 by one block of kThreads threads
// into gram[0 .. E) (shared memory); ends with a block barrier.  Small groups: with Q = kThreads / E
// slices, slice q takes segments q, q + Q, ... in order and the slices are added in order.
// Partials were written by other blocks of the running kernel, hence the L2 loads.
template <int R>
__device__ void add_partials_in_block(const float* partials, int seg_begin, int seg_end, int group, int groups_total,
                                      double* gram)
{
    constexpr int E = gram_entries(R);
    const int64_t stride = (int64_t)groups_total * E;
    if constexpr (E <= kThreads) {
        constexpr int Q = kThreads / E;
        __shared__ double slice_sum[kThreads];
        const int q = threadIdx.x / E, kk = threadIdx.x - q * E;
        if (q < Q) {
            const float* src = partials + (int64_t)group * E + kk;
            double s = 0.0;
#pragma unroll 8
            for (int seg = seg_begin + q; seg < seg_end; seg += Q)
                s += (double)__ldcg(src + seg * stride);
            slice_sum[q * E + kk] = s;
        }
        __syncthreads();
        if (threadIdx.x < E) {
            double s = slice_sum[threadIdx.x];
            for (int qq = 1; qq < Q; ++qq)
                s += slice_sum[qq * E + threadIdx.x];
            gram[threadIdx.x] = s;
        }
    } else {
        // wide groups: every thread owns several entries and adds their partials in segment order
        // (blocks of more than kThreads threads: all of them)
        for (int k = threadIdx.x; k < E; k += (int)blockDim.x) {
            const float* src = partials + (int64_t)group * E + k;
            double s = 0.0;
#pragma unroll 8
            for (int seg = seg_begin; seg < seg_end; ++seg)
                s += (double)__ldcg(src + seg * stride);
            gram[k] = s;
        }
    }
    __syncthreads();
}

constexpr int kTreeThreadsMax = 1024;
// Entries of the packed Gram matrix handled by one block of gram_finish_kernel.
__host__ __device__ constexpr int tree_entries_per_block(int radix)
{
    return gram_entries(radix) < 256 ? gram_entries(radix) : 256;
}
__host__ __device__ constexpr int tree_entry_blocks(int radix)
{
    return (gram_entries(radix) + tree_entries_per_block(radix) - 1) / tree_entries_per_block(radix);
}

// grid = (tensors, groups, tree_entry_blocks(R)); block = 256 or 1024 threads (1024 when some
// tensor has many segments); dynamic shared memory = blockDim.x * 8 bytes.
// Adds the tensor's per-segment partial matrices in fp64: with Q = blockDim.x / entries slices,
// slice q takes segments q, q + Q, ... in order, then the slices are added in order (fixed order
// for a given block size: deterministic).  When the whole matrix fits one block (R <= 16) the
// same block goes on to run the tree and writes weights[(tensor * groups + group) * R + i];
// otherwise, or when sums_only is set (the sums are to be added across GPUs first), it stores
// its entries to gram64 and tree_weights_kernel finishes.
template <int R>
__global__ void __launch_bounds__(kTreeThreadsMax)
gram_finish_kernel(const float* __restrict__ partials, const int32_t* __restrict__ seg_first, int operands,
                   double* __restrict__ gram64, float* __restrict__ weights, TreeOptions opt, int sums_only)
{
    constexpr int E = gram_entries(R);
    constexpr int EPB = tree_entries_per_block(R);
    constexpr bool SINGLE = tree_entry_blocks(R) == 1;
    extern __shared__ __align__(16) unsigned char finish_smem[];
    double* slice_sum = reinterpret_cast<double*>(finish_smem);      // [Q][EPB]
    __shared__ double gram[SINGLE ? E : 1];

    const int Q = blockDim.x / EPB;
    const int tensor = blockIdx.x, group = blockIdx.y, groups = gridDim.y;
    const int s0 = seg_first[2 * tensor], s1 = seg_first[2 * tensor + 1];
    const int q = threadIdx.x / EPB, kk = threadIdx.x - q * EPB;
    const int k = blockIdx.z * EPB + kk;
    if (q < Q) {
        double s = 0.0;
        if (k < E) {
            const float* src = partials + (int64_t)group * E + k;
            const int64_t stride = (int64_t)groups * E;
#pragma unroll 4
            for (int seg = s0 + q; seg < s1; seg += Q)
                s += (double)__ldg(src + seg * stride);
        }
        slice_sum[q * EPB + kk] = s;
    }
    __syncthreads();
    if (q == 0 && k < E) {
        double s = slice_sum[kk];
        for (int qq = 1; qq < Q; ++qq)
            s += slice_sum[qq * EPB + kk];
        if (SINGLE && !sums_only)
            gram[kk] = s;
        else
            gram64[((int64_t)tensor * groups + group) * E + k] = s;
    }
    if (SINGLE && !sums_only) {      // sums_only is uniform over the grid
        __syncthreads();
        if (s0 == s1) {              // no segments: an empty tensor, or one that another kernel reduces
            opt.leaf_norm_sums = nullptr;
            opt.orthogonality = nullptr;
        }
        tree_weights_from_gram<R>(gram, min(R, operands - group * R),
                                  weights + ((int64_t)tensor * groups + group) * R, opt, tensor, group);
    }
}

// grid = (tensors, groups); block = kThreads.  The Gram matrix was finished into gram64 (by
// several blocks of gram_finish_kernel at radix >= 32, or to be summed across GPUs); load it and
// run the tree.
template <int R>
__global__ void __launch_bounds__(kThreads)
tree_weights_kernel(const double* __restrict__ gram64, int operands, float* __restrict__ weights, TreeOptions opt,
                    const int32_t* __restrict__ seg_first)
{
    constexpr int E = gram_entries(R);
    __shared__ double gram[E];
    const int tensor = blockIdx.x, group = blockIdx.y, groups = gridDim.y;
    // a tensor without segments (seg_first given): empty, or reduced by another kernel, which then
    // also reports its by-products
    if (seg_first != nullptr && seg_first[2 * tensor] == seg_first[2 * tensor + 1]) {
        opt.leaf_norm_sums = nullptr;
        opt.orthogonality = nullptr;
    }
    const double* src = gram64 + ((int64_t)tensor * groups + group) * E;
    for (int k = threadIdx.x; k < E; k += kThreads)
        gram[k] = src[k];
    __syncthreads();
    tree_weights_from_gram<R>(gram, min(R, operands - group * R), weights + ((int64_t)tensor * groups + group) * R,
                              opt, tensor, group);
}

// ---- pass 2: weighted sum ---------------------------------------------------------------------

// The weighted sum of one segment, dst[e] = sum_i w_i x_i[e], by the whole block.  wsrc[0 .. R)
// are the leaf weights (global or shared memory).  Rows are read eight at a time so that the
// loads of one batch are in flight together while the register count stays low enough for three
// blocks per SM.
//
// DELTA: the rows are (operand - ex.start), rounded to T.  ex.base (if any) is added to the sum
// and the result is stored in ex.out_dtype; dst may be the same buffer as ex.start / ex.base
// (every element is read by the thread that writes it, before it writes).
template <typename T, int R, bool VEC, bool DELTA = false, int UNROLL = 1>
__device__ __forceinline__ void weighted_sum_of_segment(const OperandTable& ops, int first, int members,
                                                        const Segment& seg, const float* wsrc,
                                                        void* dst, const PassExtras& ex)
{
    constexpr int V = Element<T>::kVec;
    constexpr int BATCH = R < 8 ? R : 8;
    // leaf weights: registers for small groups, shared memory for the wide ones
    constexpr bool W_IN_SMEM = R > 16;
    __shared__ float w_smem[W_IN_SMEM ? R : 1];
    float w_reg[W_IN_SMEM ? 1 : R];
    if constexpr (W_IN_SMEM) {
        if (threadIdx.x < R)
            w_smem[threadIdx.x] = threadIdx.x < members ? wsrc[threadIdx.x] : 0.0f;
        __syncthreads();
    } else {
#pragma unroll
        for (int i = 0; i < R; ++i)
            w_reg[i] = i < members ? wsrc[i] : 0.0f;
    }
    auto w = [&](int i) -> float {
        if constexpr (W_IN_SMEM)
            return w_smem[i];
        else
            return w_reg[i];
    };

    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    int64_t body_begin, body_end;
    split_segment<V, VEC>(begin, end, body_begin, body_end);

#pragma unroll(UNROLL)
    for (int64_t v = body_begin + (int64_t)threadIdx.x * V; v < body_end; v += (int64_t)kThreads * V) {
        float y[V];
#pragma unroll
        for (int j = 0; j < V; ++j)
            y[j] = 0.0f;
        uint4 sraw = make_uint4(0u, 0u, 0u, 0u);
        if constexpr (DELTA)
            sraw = load_plain_16B(static_cast<const T*>(ex.start) + v);
        // Two batches may be unrolled together; beyond that the loop stays rolled so that the
        // compiler cannot hoist every batch's loads and spill.
#pragma unroll(R / BATCH <= 2 ? 2 : 1)
        for (int b = 0; b < R; b += BATCH) {
            uint4 raw[BATCH];
#pragma unroll
            for (int i = 0; i < BATCH; ++i)
                if (b + i < members)
                    raw[i] = load_streaming_16B(static_cast<const T*>(ops.ptr[first + b + i]) + v);
#pragma unroll
            for (int i = 0; i < BATCH; ++i) {
                if (b + i < members) {
                    float x[V];
                    if constexpr (DELTA)
                        decode_vector<T>(delta_words<T>(raw[i], sraw), x);
                    else
                        decode_vector<T>(raw[i], x);
                    const float wi = w(b + i);
#pragma unroll
                    for (int j = 0; j < V; ++j)
                        y[j] = fmaf(wi, x[j], y[j]);
                }
            }
        }
        if (ex.base != nullptr)
            add_vector_as_float<V>(ex.base, ex.base_dtype, v, y);
        store_vector_from_float<V>(dst, ex.out_dtype, v, y);
    }
    for (int pass = 0; pass < 2; ++pass) {
        const int64_t lo = pass == 0 ? begin : body_end;
        const int64_t hi = pass == 0 ? body_begin : end;
        for (int64_t e = lo + threadIdx.x; e < hi; e += kThreads) {
            float y = 0.0f;
#pragma unroll
            for (int i = 0; i < R; ++i) {
                if (i < members) {
                    if constexpr (DELTA)
                        y = fmaf(w(i), delta_one(static_cast<const T*>(ops.ptr[first + i]),
                                                 static_cast<const T*>(ex.start), e), y);
                    else
                        y = fmaf(w(i), Element<T>::one(static_cast<const T*>(ops.ptr[first + i]) + e), y);
                }
            }
            if (ex.base != nullptr)
                y += load_as_float(ex.base, ex.base_dtype, e);
            store_from_float(dst, ex.out_dtype, e, y);
        }
    }
}

// grid = (segments, groups in this launch); block = kThreads.
// dst_base + (group_base + blockIdx.y) * dst_stride floats is the group's output buffer (fp32; a
// last level has one group and stride 0, and may store another type: ex.out_dtype).
template <typename T, int R, bool VEC, bool DELTA = false>
__global__ void __launch_bounds__(kThreads, 3)
weighted_sum_kernel(const __grid_constant__ OperandTable ops, int operands,
                    const Segment* __restrict__ segments, const float* __restrict__ weights,
                    int groups_total, int group_base, void* dst_base, int64_t dst_stride, PassExtras ex)
{
    // Segments are taken last to first: pass 1 walked them first to last, so the tail of the
    // operands is what the L2 still holds when this kernel starts.
    const Segment seg = segments[gridDim.x - 1 - blockIdx.x];
    const int first = blockIdx.y * R;
    const int members = min(R, operands - first);
    const int group = group_base + blockIdx.y;
    weighted_sum_of_segment<T, R, VEC, DELTA>(ops, first, members, seg,
                                              weights + ((int64_t)seg.tensor * groups_total + group) * R,
                                              static_cast<float*>(dst_base) + (int64_t)group * dst_stride, ex);
}

// ---- pass 2 of a level fused with pass 1 of the next ------------------------------------------
//
// Algorithm 1 applied level after level: the combine x' = ca a + cb b of one level writes exactly
// the vectors whose dot products [a'.b', a'.a', b'.b'] the next level needs.  This kernel forms the
// weighted sums of R2 adjacent groups of a level (R1 operands each), stores them as the level's
// outputs, and accumulates, from the same registers, the R2 x R2 Gram matrix of those outputs,
// which is the next level's pass 1: the intermediates are written once and read once instead of
// twice.  The next level's sums are finished here as well (last block per (tensor, next group)),
// so the next level only runs its pass 2.  R2 = 2 or 4: the Gram matrix on the fp32 pipes.
//
// grid = (segments, next-level groups in this launch); block = kThreads.
// weights[(tensor * groups_total + group) * R1 ...]: this level's leaf weights.
// dst_base + group * dst_stride floats: this level's output buffers (fp32).
// next_partials[(segment * next_groups_total + next group) * E2 + entry].
template <typename T, int R1, int R2, bool VEC>
__global__ void __launch_bounds__(kThreads, 2)
wsum_gram_kernel(const __grid_constant__ OperandTable ops, int operands,
                 const Segment* __restrict__ segments, const float* __restrict__ weights,
                 int groups_total, int group_base, float* __restrict__ dst_base, int64_t dst_stride,
                 float* __restrict__ next_partials, int next_groups_total, int next_group_base, FinishArgs next_fin)
{
    constexpr int V = Element<T>::kVec;
    constexpr int E2 = gram_entries(R2);
    constexpr int BATCH = R1 < 8 ? R1 : 8;
    __shared__ float w_smem[R2][R1];
    __shared__ float warp_sums[kWarps][E2];

    const Segment seg = segments[blockIdx.x];
    const int groups_here = (operands + R1 - 1) / R1;                 // this level's groups in this launch
    const int g_first = blockIdx.y * R2;                              // first of them that this block combines
    const int members_next = min(R2, groups_here - g_first);
    for (int k = threadIdx.x; k < R1 * R2; k += kThreads) {
        const int j = k / R1, i = k % R1;
        const bool live = j < members_next && (g_first + j) * R1 + i < operands;
        w_smem[j][i] = live ? weights[((int64_t)seg.tensor * groups_total + group_base + g_first + j) * R1 + i] : 0.0f;
    }
    __syncthreads();

    float acc[E2];
#pragma unroll
    for (int k = 0; k < E2; ++k)
        acc[k] = 0.0f;

    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    int64_t body_begin, body_end;
    split_segment<V, VEC>(begin, end, body_begin, body_end);

    for (int64_t v = body_begin + (int64_t)threadIdx.x * V; v < body_end; v += (int64_t)kThreads * V) {
        float y[R2][V];
#pragma unroll
        for (int j = 0; j < R2; ++j) {
#pragma unroll
            for (int c = 0; c < V; ++c)
                y[j][c] = 0.0f;
            if (j < members_next) {
                const int op0 = (g_first + j) * R1;
#pragma unroll(R1 / BATCH <= 2 ? 2 : 1)
                for (int bb = 0; bb < R1; bb += BATCH) {
                    uint4 raw[BATCH];
#pragma unroll
                    for (int i = 0; i < BATCH; ++i)
                        if (op0 + bb + i < operands)
                            raw[i] = load_streaming_16B(static_cast<const T*>(ops.ptr[op0 + bb + i]) + v);
#pragma unroll
                    for (int i = 0; i < BATCH; ++i) {
                        if (op0 + bb + i < operands) {
                            float x[V];
                            decode_vector<T>(raw[i], x);
                            const float wi = w_smem[j][bb + i];
#pragma unroll
                            for (int c = 0; c < V; ++c)
                                y[j][c] = fmaf(wi, x[c], y[j][c]);
                        }
                    }
                }
                float* out = dst_base + (int64_t)(group_base + g_first + j) * dst_stride + v;
#pragma unroll
                for (int c = 0; c < V; c += 4)
                    *reinterpret_cast<float4*>(out + c) = make_float4(y[j][c], y[j][c + 1], y[j][c + 2], y[j][c + 3]);
            }
        }
#pragma unroll
        for (int c = 0; c < V; ++c) {
            float col[R2];
#pragma unroll
            for (int j = 0; j < R2; ++j)
                col[j] = y[j][c];
            gram_accumulate<R2>(col, acc);
        }
    }
    // scalar head [begin, body_begin) and tail [body_end, end)
    for (int pass = 0; pass < 2; ++pass) {
        const int64_t lo = pass == 0 ? begin : body_end;
        const int64_t hi = pass == 0 ? body_begin : end;
        for (int64_t e = lo + threadIdx.x; e < hi; e += kThreads) {
            float col[R2];
#pragma unroll
            for (int j = 0; j < R2; ++j) {
                float yy = 0.0f;
                if (j < members_next) {
                    const int op0 = (g_first + j) * R1;
#pragma unroll
                    for (int i = 0; i < R1; ++i)
                        if (op0 + i < operands)
                            yy = fmaf(w_smem[j][i], Element<T>::one(static_cast<const T*>(ops.ptr[op0 + i]) + e), yy);
                    dst_base[(int64_t)(group_base + g_first + j) * dst_stride + e] = yy;
                }
                col[j] = yy;
            }
            gram_accumulate<R2>(col, acc);
        }
    }

    // block reduction: warp shuffles, then the warps' sums in warp order
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < E2; ++k) {
        float sum = acc[k];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1)
            sum += __shfl_xor_sync(0xffffffffu, sum, d);
        if (lane == 0)
            warp_sums[warp][k] = sum;
    }
    __syncthreads();
    float* dst = next_partials + ((int64_t)blockIdx.x * next_groups_total + next_group_base + blockIdx.y) * E2;
    for (int k = threadIdx.x; k < E2; k += kThreads) {
        float sum = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w)
            sum += warp_sums[w][k];
        dst[k] = sum;
    }
    finish_if_last<R2>(next_fin, next_partials, seg.tensor, next_group_base + blockIdx.y, next_groups_total, members_next,
                       (int)blockIdx.x);
}

// ---- both passes in one launch, for inputs that fit the L2 -------------------------------------
//
// One level, one group (n_workers <= 8), one cooperative launch whose blocks are all resident.
// HBM sees the operands once.  Work is dealt in two sizes:
//
//   - tensors of more than kWarpTensorElems elements are cut into segments, one per block.  A block
//     forms the Gram matrix of its segment, the grid synchronises, each block adds up its tensor's
//     partial matrices and derives the weights for itself (the same numbers in every block of a
//     tensor: fixed summation order), and writes the weighted sum of its segment.  When the segment
//     is short enough (a few 16-byte vectors per thread and row) the operands stay in registers
//     across the grid barrier and the second pass loads nothing; otherwise it reads them again,
//     out of the L2;
//   - tensors of at most kWarpTensorElems elements (beyond the short ones that the fp64 kernel
//     takes) are handled by one warp each, from the loads to the store, before the barrier: a fused
//     buffer with hundreds of small tensors (biases, normalisation parameters) then needs neither a
//     block nor a barrier per tensor.
//
// grid >= segments; block = kThreads; partials[segment * E + entry].

constexpr int kWarpTensorElems = 512;

// One tensor of at most kShortSlotElems elements: where it starts in the fused buffers, and where in
// the packed numbering of the short tensors' elements (used for the fp64 vectors that travel
// between the launches of adasum_short.cu).
struct ShortTensor {
    int64_t begin;
    int32_t len;
    int32_t tensor;
    int64_t packed;
};

// A small tensor that one warp reduces: `begin`, `len` in the fused buffers; `tensor` its index.
struct WarpTensor {
    int64_t begin;
    int32_t len;
    int32_t tensor;
};

// The binary tree (or the other two orders of Section 3.4) evaluated on a packed R x R Gram matrix
// by ONE thread, R <= 8: leaf weights w[0 .. members) and the squared norm of the result.  Same
// recursion as tree_weights_from_gram.
// With opt.leaf_scales (operand i holds scale x gradient) a leaf starts with weight 1 / scale, as in
// tree_weights_from_gram.  leaf_sum: the sum of the leaves' squared norms, in the gradients' units.
template <int R>
__device__ void tree_weights_serial(const double* gram, int members, const TreeOptions& opt, int tensor, double* w,
                                    double& root_norm, double& leaf_sum)
{
    const int order = opt.linear;
    double norm[R];
    leaf_sum = 0.0;
#pragma unroll
    for (int i = 0; i < R; ++i) {
        double unit = 1.0;
        if (opt.leaf_scales != nullptr && i < members)
            unit = 1.0 / (double)opt.leaf_scales[(int64_t)i * opt.num_tensors + tensor];
        w[i] = unit;
        norm[i] = i < members ? gram[gram_index(R, i, i)] * unit * unit : 0.0;
        leaf_sum += norm[i];
    }
    // a <- Adasum(a, b) for the nodes over leaves [lo, mid) and [mid, hi); norms kept at lo / mid
    auto combine = [&](int lo, int mid, int hi) {
        double dot = 0.0;
        for (int i = lo; i < mid; ++i) {
            double row = 0.0;
            for (int k = mid; k < hi; ++k)
                row += w[k] * gram[gram_index(R, i, k)];
            dot += w[i] * row;
        }
        double ca, cb;
        pair_coefficients(dot, norm[lo], norm[mid], ca, cb);
        for (int i = lo; i < mid; ++i)
            w[i] *= ca;
        for (int k = mid; k < hi; ++k)
            w[k] *= cb;
        norm[lo] = ca * ca * norm[lo] + cb * cb * norm[mid] + 2.0 * ca * cb * dot;
    };
    if (order == 1) {
        for (int k = 1; k < members; ++k)
            combine(0, k, k + 1);
    } else if (order == 2) {
        int max_depth = 0;
        while ((1 << max_depth) < members)
            ++max_depth;
        for (int depth = max_depth - 1; depth >= 0; --depth) {
            for (int j = 0; j < (1 << depth); ++j) {
                int lo = 0, hi = members;
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
                if (alive && hi - lo >= 2)
                    combine(lo, lo + (hi - lo) / 2, hi);
            }
        }
    } else {
        for (int width = 1; width < members; width *= 2)
            for (int left = 0; left + width < members; left += 2 * width)
                combine(left, left + width, min(left + 2 * width, members));
    }
    root_norm = norm[0];
}

// Block reduction of per-thread Gram accumulators: warp shuffles, then the warps' sums in warp
// order; entry k of the result goes to dst[k].  Ends without a barrier after the stores.
template <int E>
__device__ __forceinline__ void block_reduce_gram(const float (&acc)[E], float* __restrict__ dst)
{
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
    for (int k = threadIdx.x; k < E; k += kThreads) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w)
            s += warp_sums[w][k];
        dst[k] = s;
    }
}

// One small tensor, both passes, by one warp: 16-byte vectors over the aligned body (several
// independent vectors per lane in flight), scalars for the ragged ends.
template <typename T, int R, bool VEC, bool DELTA>
__device__ void reduce_warp_tensor(const OperandTable& ops, int members, const WarpTensor& wt, const TreeOptions& opt,
                                   void* out, const PassExtras& ex)
{
    constexpr int E = gram_entries(R);
    constexpr int V = Element<T>::kVec;
    constexpr int UNROLL = R <= 2 ? 4 : (R <= 4 ? 2 : 1);
    const int lane = threadIdx.x & 31;
    const T* src[R];
#pragma unroll
    for (int i = 0; i < R; ++i)
        src[i] = static_cast<const T*>(ops.ptr[i < members ? i : 0]);
    const T* start = static_cast<const T*>(ex.start);
    const int64_t begin = wt.begin, end = wt.begin + wt.len;
    int64_t body_begin, body_end;
    split_segment<V, VEC>(begin, end, body_begin, body_end);
    auto element = [&](int i, int64_t e) -> float {
        if constexpr (DELTA)
            return delta_one(src[i], start, e);
        else
            return Element<T>::one(src[i] + e);
    };
    auto vector = [&](int i, int64_t v, float (&x)[V]) {
        if constexpr (DELTA)
            decode_vector<T>(delta_words<T>(load_keep_16B(src[i] + v), load_plain_16B(start + v)), x);
        else
            Element<T>::vec(src[i] + v, x);
    };
    float acc[E];
#pragma unroll
    for (int k = 0; k < E; ++k)
        acc[k] = 0.0f;
#pragma unroll(UNROLL)
    for (int64_t v = body_begin + (int64_t)lane * V; v < body_end; v += 32 * V) {
        float x[R][V];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (i < members) {
                vector(i, v, x[i]);
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
    for (int pass = 0; pass < 2; ++pass) {
        const int64_t lo = pass == 0 ? begin : body_end, hi = pass == 0 ? body_begin : end;
        for (int64_t e = lo + lane; e < hi; e += 32) {
            float col[R];
#pragma unroll
            for (int i = 0; i < R; ++i)
                col[i] = i < members ? element(i, e) : 0.0f;
            gram_accumulate<R>(col, acc);
        }
    }
    // the lanes' sums (a few dozen products each) are added in fp64; every lane ends with the same bits
    double gram[E];
#pragma unroll
    for (int k = 0; k < E; ++k) {
        double s = (double)acc[k];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1)
            s += __shfl_xor_sync(0xffffffffu, s, d);
        gram[k] = s;
    }
    double w64[R], root = 0.0, leaf_sum = 0.0;
    tree_weights_serial<R>(gram, members, opt, wt.tensor, w64, root, leaf_sum);
    if (lane == 0 && opt.orthogonality != nullptr)
        opt.orthogonality[wt.tensor] = leaf_sum == 0.0 ? __int_as_float(0x7fc00000) : (float)(root / leaf_sum);
    float w[R];
#pragma unroll
    for (int i = 0; i < R; ++i)
        w[i] = i < members ? (float)w64[i] : 0.0f;
#pragma unroll(UNROLL)
    for (int64_t v = body_begin + (int64_t)lane * V; v < body_end; v += 32 * V) {
        float y[V];
#pragma unroll
        for (int j = 0; j < V; ++j)
            y[j] = 0.0f;
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (i < members) {
                float x[V];
                vector(i, v, x);
#pragma unroll
                for (int j = 0; j < V; ++j)
                    y[j] = fmaf(w[i], x[j], y[j]);
            }
        }
        if (ex.base != nullptr)
            add_vector_as_float<V>(ex.base, ex.base_dtype, v, y);
        store_vector_from_float<V>(out, ex.out_dtype, v, y);
    }
    for (int pass = 0; pass < 2; ++pass) {
        const int64_t lo = pass == 0 ? begin : body_end, hi = pass == 0 ? body_begin : end;
        for (int64_t e = lo + lane; e < hi; e += 32) {
            float y = 0.0f;
#pragma unroll
            for (int i = 0; i < R; ++i)
                if (i < members)
                    y = fmaf(w[i], element(i, e), y);
            if (ex.base != nullptr)
                y += load_as_float(ex.base, ex.base_dtype, e);
            store_from_float(out, ex.out_dtype, e, y);
        }
    }
}

// One tensor of at most kShortSlotElems elements by one warp, in fp64 from the loads to the store and
// with the operator applied literally (what adasum_short.cu does for the other paths): the leaves go
// to `slot` (this warp's R x kShortSlotElems doubles of shared memory), the tree runs in place.
template <typename T, int R, bool DELTA>
__device__ void reduce_short_tensor_warp(const OperandTable& ops, int members, const ShortTensor& st,
                                         const TreeOptions& opt, double* slot, void* out, const PassExtras& ex)
{
    const int lane = threadIdx.x & 31;
    const int len = st.len;
    double leaf_sum = 0.0;
    for (int i = 0; i < members; ++i) {
        const T* src = static_cast<const T*>(ops.ptr[i]);
        double sq = 0.0;
        for (int e = lane; e < len; e += 32) {
            double x;
            if constexpr (DELTA)
                x = (double)delta_one(src, static_cast<const T*>(ex.start), st.begin + e);
            else
                x = (double)Element<T>::one(src + st.begin + e);
            if (opt.leaf_scales != nullptr)        // the buffer holds scale x gradient
                x /= (double)opt.leaf_scales[(int64_t)i * opt.num_tensors + st.tensor];
            slot[i * kShortSlotElems + e] = x;
            sq += x * x;
        }
        leaf_sum += warp_sum(sq);
    }
    __syncwarp();
    warp_tree_in_place(slot, members, len, opt.linear);
    __syncwarp();
    if (opt.orthogonality != nullptr) {
        const double r0 = lane < len ? slot[lane] : 0.0, r1 = lane + 32 < len ? slot[lane + 32] : 0.0;
        const double norm = warp_sum(r0 * r0 + r1 * r1);
        if (lane == 0)
            opt.orthogonality[st.tensor] = leaf_sum == 0.0 ? __int_as_float(0x7fc00000) : (float)(norm / leaf_sum);
    }
    for (int e = lane; e < len; e += 32) {
        double y = slot[e];
        if (ex.base != nullptr)
            y += (double)load_as_float(ex.base, ex.base_dtype, st.begin + e);
        store_from_float(out, ex.out_dtype, st.begin + e, (float)y);
    }
    __syncwarp();
}

// The partial matrices of segments [seg_begin, seg_end) added in fp64 in a fixed order by the whole
// block, then the tree: leaf weights to weights_dst (shared memory), by-products as opt says.
// Thread (q, kk) adds the partials of segments q, q + Q, ... for entry kk; a warp then adds the Q
// slice sums of an entry (lane-strided, then a butterfly).
template <int R>
__device__ void finish_small(const float* partials, int seg_begin, int seg_end, int tensor, int members,
                             float* weights_dst, const TreeOptions& opt)
{
    constexpr int E = gram_entries(R);
    constexpr int Q = kThreads / E;
    static_assert(E <= kThreads, "one thread per entry at least");
    __shared__ double slice_sum[E * Q];
    __shared__ double gram[E];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q = threadIdx.x / E, kk = threadIdx.x - q * E;
    if (q < Q) {
        double s = 0.0;
#pragma unroll 4
        for (int seg = seg_begin + q; seg < seg_end; seg += Q)
            s += (double)__ldcg(partials + (int64_t)seg * E + kk);
        slice_sum[kk * Q + q] = s;
    }
    __syncthreads();
    for (int k = warp; k < E; k += kWarps) {
        double s = 0.0;
        for (int qq = lane; qq < Q; qq += 32)
            s += slice_sum[k * Q + qq];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1)
            s += __shfl_xor_sync(0xffffffffu, s, d);
        if (lane == 0)
            gram[k] = s;
    }
    __syncthreads();
    if constexpr (R <= 4) {
        if (threadIdx.x == 0) {
            double w64[R], root = 0.0, leaf_sum = 0.0;
            tree_weights_serial<R>(gram, members, opt, tensor, w64, root, leaf_sum);
            for (int i = 0; i < R; ++i)
                weights_dst[i] = i < members ? (float)w64[i] : 0.0f;
            if (opt.orthogonality != nullptr)
                opt.orthogonality[tensor] = leaf_sum == 0.0 ? __int_as_float(0x7fc00000) : (float)(root / leaf_sum);
        }
    } else {
        tree_weights_from_gram<R>(gram, members, weights_dst, opt, tensor, 0);
    }
    __syncthreads();
}

// 16-byte vectors per thread and row that stay in registers between the passes.
template <int R>
__host__ __device__ constexpr int small_keep_vectors() { return R <= 2 ? 4 : (R <= 4 ? 2 : 0); }

template <typename T, int R, bool VEC, bool DELTA = false>
__global__ void __launch_bounds__(kThreads, 2)
fused_small_kernel(const __grid_constant__ OperandTable ops, int operands,
                   const Segment* __restrict__ segments, int num_segments,
                   const WarpTensor* __restrict__ warp_tensors, int num_warp_tensors,
                   const ShortTensor* __restrict__ short_tensors, int num_short_tensors,
                   float* __restrict__ partials, FinishArgs fin, void* out, PassExtras ex, int* __restrict__ status)
{
    constexpr int E = gram_entries(R);
    constexpr int V = Element<T>::kVec;
    constexpr int K = small_keep_vectors<R>();
    constexpr int kSmallUnroll = R <= 2 ? 4 : (R <= 4 ? 2 : 1);      // vectors per thread in flight where nothing is kept
    __shared__ double short_slots[kWarps][R * kShortSlotElems];
    // This path uses no ticket counters, so the host does not clear them (one operation less in
    // front of a reduce that takes microseconds); the device status word, which lives beside
    // them and which adasum_device_status reads, is cleared here instead.
    if (blockIdx.x == 0 && threadIdx.x == 0)
        *status = 0;
    const int members = min(R, operands);
    const bool has_segment = (int)blockIdx.x < num_segments;
    const Segment seg = has_segment ? segments[blockIdx.x] : Segment{0, 0, 0};
    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    int64_t body_begin, body_end;
    split_segment<V, VEC>(begin, end, body_begin, body_end);
    const bool keep = K > 0 && VEC && has_segment && (body_end - body_begin) <= (int64_t)K * kThreads * V;

    // ---- pass 1 of this block's segment
    uint4 raw[R][K > 0 ? K : 1];
    if (keep) {
        const T* src[R];
#pragma unroll
        for (int i = 0; i < R; ++i)
            src[i] = static_cast<const T*>(ops.ptr[i < members ? i : 0]);
        // every load of the segment is issued before the first use
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const int64_t v = body_begin + ((int64_t)threadIdx.x + (int64_t)k * kThreads) * V;
            if (v < body_end) {
#pragma unroll
                for (int i = 0; i < R; ++i)
                    raw[i][k] = i < members ? load_keep_16B(src[i] + v) : make_uint4(0u, 0u, 0u, 0u);
            } else {
#pragma unroll
                for (int i = 0; i < R; ++i)
                    raw[i][k] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        if constexpr (DELTA) {
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const int64_t v = body_begin + ((int64_t)threadIdx.x + (int64_t)k * kThreads) * V;
                if (v < body_end) {
                    const uint4 sraw = load_plain_16B(static_cast<const T*>(ex.start) + v);
#pragma unroll
                    for (int i = 0; i < R; ++i)
                        if (i < members)
                            raw[i][k] = delta_words<T>(raw[i][k], sraw);
                }
            }
        }
        float acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e)
            acc[e] = 0.0f;
#pragma unroll
        for (int k = 0; k < K; ++k) {
            float x[R][V];
#pragma unroll
            for (int i = 0; i < R; ++i)
                decode_vector<T>(raw[i][k], x[i]);         // zero vectors beyond the segment add nothing
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
                for (int i = 0; i < R; ++i) {
                    if constexpr (DELTA)
                        col[i] = i < members ? delta_one(src[i], static_cast<const T*>(ex.start), e) : 0.0f;
                    else
                        col[i] = i < members ? Element<T>::one(src[i] + e) : 0.0f;
                }
                gram_accumulate<R>(col, acc);
            }
        }
        block_reduce_gram<E>(acc, partials + (int64_t)blockIdx.x * E);
    } else if (has_segment) {
        gram_of_segment<T, R, VEC, DELTA, kSmallUnroll>(ops, 0, members, seg, partials + (int64_t)blockIdx.x * E,
                                                        static_cast<const T*>(ex.start));
    }

    // ---- the small tensors, one warp each, while the segments' loads and stores drain
    {
        TreeOptions opt = fin.tree;
        const int warps_total = (int)gridDim.x * kWarps;
        // dealt from the last block backwards: the first blocks are the ones whose segments are longest
        const int first = ((int)gridDim.x - 1 - (int)blockIdx.x) * kWarps + (threadIdx.x >> 5);
        for (int s = first; s < num_warp_tensors; s += warps_total)
            reduce_warp_tensor<T, R, VEC, DELTA>(ops, members, warp_tensors[s], opt, out, ex);
        // ... and the tensors of at most 64 elements, in fp64
        for (int s = first; s < num_short_tensors; s += warps_total)
            reduce_short_tensor_warp<T, R, DELTA>(ops, members, short_tensors[s], opt, short_slots[threadIdx.x >> 5],
                                                  out, ex);
    }

    __threadfence();
    cooperative_groups::this_grid().sync();
    if (!has_segment)
        return;

    // ---- coefficients of this block's tensor, then pass 2 of its segment
    __shared__ float leaf_weights[R];
    const int s0 = fin.seg_first[2 * seg.tensor], s1 = fin.seg_first[2 * seg.tensor + 1];
    TreeOptions opt = fin.tree;
    if ((int)blockIdx.x != s0) {           // one block per tensor reports the by-products
        opt.leaf_norm_sums = nullptr;
        opt.orthogonality = nullptr;
    }
    finish_small<R>(partials, s0, s1, seg.tensor, members, leaf_weights, opt);
    if (keep) {
        float w[R];
#pragma unroll
        for (int i = 0; i < R; ++i)
            w[i] = leaf_weights[i];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const int64_t v = body_begin + ((int64_t)threadIdx.x + (int64_t)k * kThreads) * V;
            if (v < body_end) {
                float y[V];
#pragma unroll
                for (int j = 0; j < V; ++j)
                    y[j] = 0.0f;
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    float x[V];
                    decode_vector<T>(raw[i][k], x);
#pragma unroll
                    for (int j = 0; j < V; ++j)
                        y[j] = fmaf(w[i], x[j], y[j]);
                }
                if (ex.base != nullptr)
                    add_vector_as_float<V>(ex.base, ex.base_dtype, v, y);
                store_vector_from_float<V>(out, ex.out_dtype, v, y);
            }
        }
        for (int pass = 0; pass < 2; ++pass) {
            const int64_t lo = pass == 0 ? begin : body_end;
            const int64_t hi = pass == 0 ? body_begin : end;
            for (int64_t e = lo + threadIdx.x; e < hi; e += kThreads) {
                float y = 0.0f;
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    if (i < members) {
                        if constexpr (DELTA)
                            y = fmaf(w[i], delta_one(static_cast<const T*>(ops.ptr[i]), static_cast<const T*>(ex.start), e), y);
                        else
                            y = fmaf(w[i], Element<T>::one(static_cast<const T*>(ops.ptr[i]) + e), y);
                    }
                }
                if (ex.base != nullptr)
                    y += load_as_float(ex.base, ex.base_dtype, e);
                store_from_float(out, ex.out_dtype, e, y);
            }
        }
    } else {
        weighted_sum_of_segment<T, R, VEC, DELTA, kSmallUnroll>(ops, 0, members, seg, leaf_weights, out, ex);
    }
}

// n_workers = 1: the result is the input (with a start: start + (input - start), the difference
// rounded to T like everywhere else), stored in ex.out_dtype.
template <typename T>
__global__ void __launch_bounds__(kThreads)
convert_kernel(const T* src, void* dst, int64_t n, PassExtras ex)
{
    for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < n;
         e += (int64_t)gridDim.x * kThreads) {
        float y = ex.start != nullptr ? delta_one(src, static_cast<const T*>(ex.start), e) : Element<T>::one(src + e);
        if (ex.base != nullptr)
            y += load_as_float(ex.base, ex.base_dtype, e);
        store_from_float(dst, ex.out_dtype, e, y);
    }
}

}  // namespace adasum
