// Launchers of one level for operands of element type T: pass 1 (which of the Gram kernels), the
// coefficient step, pass 2, the kernels that fuse neighbouring steps.  Included by one translation
// unit per element type, which instantiates the entry points declared in adasum_internal.h.
#pragma once

#include "adasum_internal.h"

namespace adasum {

// ---- launches ----------------------------------------------------------------------------------

// Opt a kernel in to `bytes` of dynamic shared memory, once per device.
template <typename Kernel>
cudaError_t allow_dynamic_smem(Kernel kernel, size_t bytes, bool (&configured)[64])
{
    int device = 0;
    cudaError_t err = cudaGetDevice(&device);
    if (err != cudaSuccess)
        return err;
    if (device < 0 || device >= 64)
        return cudaErrorInvalidDevice;
    if (!configured[device]) {
        err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (err != cudaSuccess)
            return err;
        configured[device] = true;
    }
    return cudaSuccess;
}

template <typename T, int R, bool VEC, bool DELTA>
cudaError_t launch_gram_variant(GramKind kind, const OperandTable& ops, int operands, int groups_here,
                                const SegmentTable& tab, float* partials, int groups_total, int group_base,
                                const FinishArgs& fin, cudaStream_t stream, int* tc_status, const void* start)
{
    if constexpr (R == 64 && VEC && sizeof(T) == 2 && !DELTA) {
        // every group complete: the tcgen05 kernel (64 x 64 accumulator in tensor memory)
        if (kind == GRAM_MMA && tc_status != nullptr && operands == groups_here * 64) {
            auto kernel = gram_partial_tc64_kernel<T>;
            static bool configured[64] = {};
            cudaError_t err = allow_dynamic_smem(kernel, kTcSmemBytes, configured);
            if (err != cudaSuccess)
                return err;
            dim3 grid((unsigned)tab.num_segments, (unsigned)groups_here);
            kernel<<<grid, kTcThreads, kTcSmemBytes, stream>>>(ops, operands, tab.d_segments, partials, groups_total,
                                                               group_base, fin, tc_status);
            return cudaSuccess;
        }
    }
    if constexpr (R >= 8) {
        if (kind == GRAM_MMA) {
            if constexpr (R <= 32 || sizeof(T) == 2) {
                constexpr size_t smem = mma_smem_bytes<T, R, DELTA>();
                auto kernel = gram_partial_mma_kernel<T, R, VEC, DELTA>;
                static bool configured[64] = {};
                cudaError_t err = allow_dynamic_smem(kernel, smem, configured);
                if (err != cudaSuccess)
                    return err;
                dim3 grid((unsigned)tab.num_segments, (unsigned)groups_here);
                kernel<<<grid, kThreads, smem, stream>>>(ops, operands, tab.d_segments, partials, groups_total,
                                                         group_base, fin, start);
                return cudaSuccess;
            } else {
                return cudaErrorInvalidValue;
            }
        }
    }
    if constexpr (R <= 16) {
        if (kind == GRAM_SIMPLE) {
            dim3 grid((unsigned)tab.num_segments, (unsigned)groups_here);
            gram_partial_kernel<T, R, VEC, DELTA><<<grid, kThreads, 0, stream>>>(
                ops, operands, tab.d_segments, partials, groups_total, group_base, fin, start);
            return cudaSuccess;
        }
    }
    return cudaErrorInvalidValue;
}

// `start` != nullptr selects the kernels that read the operands as (operand - start); those exist
// for 16-byte aligned buffers only (the caller has checked).
template <typename T, int R, bool VEC>
cudaError_t launch_gram(GramKind kind, const OperandTable& ops, int operands, int groups_here,
                        const SegmentTable& tab, float* partials, int groups_total, int group_base,
                        const FinishArgs& fin, cudaStream_t stream, int* tc_status = nullptr,
                        const void* start = nullptr)
{
    if constexpr (VEC) {
        if (start != nullptr)
            return launch_gram_variant<T, R, true, true>(kind, ops, operands, groups_here, tab, partials, groups_total,
                                                         group_base, fin, stream, tc_status, start);
    }
    if (start != nullptr)
        return cudaErrorInvalidValue;
    return launch_gram_variant<T, R, VEC, false>(kind, ops, operands, groups_here, tab, partials, groups_total,
                                                 group_base, fin, stream, tc_status, nullptr);
}

template <typename T, int R, bool VEC>
void launch_wsum(const OperandTable& ops, int operands, int groups_here, const SegmentTable& tab,
                 const float* weights, int groups_total, int group_base, void* dst, int64_t dst_stride,
                 cudaStream_t stream, const PassExtras& ex = kNoExtras)
{
    dim3 grid((unsigned)tab.num_segments, (unsigned)groups_here);
    if constexpr (VEC) {
        if (ex.start != nullptr) {
            weighted_sum_kernel<T, R, true, true><<<grid, kThreads, 0, stream>>>(
                ops, operands, tab.d_segments, weights, groups_total, group_base, dst, dst_stride, ex);
            return;
        }
    }
    weighted_sum_kernel<T, R, VEC, false><<<grid, kThreads, 0, stream>>>(ops, operands, tab.d_segments, weights,
                                                                         groups_total, group_base, dst, dst_stride, ex);
}

template <int R>
cudaError_t launch_weights(const float* partials, const SegmentTable& tab, int32_t num_tensors, int operands,
                           int groups, double* gram64, float* weights, const TreeOptions& opt, cudaStream_t stream,
                           int* launches, bool sums_only = false)
{
    dim3 grid((unsigned)num_tensors, (unsigned)groups, (unsigned)tree_entry_blocks(R));
    // wide blocks only pay off when some tensor has many per-segment partials to add
    const int threads = tab.max_segments_per_tensor > 64 ? kTreeThreadsMax : 256;
    gram_finish_kernel<R><<<grid, threads, threads * sizeof(double), stream>>>(partials, tab.d_seg_first, operands,
                                                                                gram64, weights, opt, sums_only ? 1 : 0);
    *launches = 1;
    if (sums_only)
        return cudaSuccess;
    if constexpr (tree_entry_blocks(R) > 1) {
        dim3 grid2((unsigned)num_tensors, (unsigned)groups);
        tree_weights_kernel<R><<<grid2, kThreads, 0, stream>>>(gram64, operands, weights, opt, tab.d_seg_first);
        *launches = 2;
    }
    return cudaSuccess;
}

template <int R>
void launch_tree_from_sums(const double* gram64, int32_t num_tensors, int operands, int groups, float* weights,
                           const TreeOptions& opt, cudaStream_t stream)
{
    dim3 grid((unsigned)num_tensors, (unsigned)groups);
    tree_weights_kernel<R><<<grid, kThreads, 0, stream>>>(gram64, operands, weights, opt, nullptr);
}

template <typename T, int R, bool VEC>
cudaError_t launch_fused_small(const OperandTable& ops, int operands, const SegmentTable& tab, int resident_blocks,
                               float* partials, const FinishArgs& fin, void* out, const PassExtras& ex, int* status,
                               cudaStream_t stream)
{
    const void* kernel = (const void*)fused_small_kernel<T, R, VEC, false>;
    if constexpr (VEC) {
        if (ex.start != nullptr)
            kernel = (const void*)fused_small_kernel<T, R, true, true>;
    }
    if (!VEC && ex.start != nullptr)
        return cudaErrorInvalidValue;
    int operands_arg = operands;
    const Segment* segments = tab.d_segments;
    int num_segments = tab.num_segments;
    const WarpTensor* warp_tensors = tab.d_warp;
    int num_warp_tensors = (int)tab.h_warp.size();
    const ShortTensor* short_tensors = tab.d_short;
    int num_short_tensors = (int)tab.h_short.size();
    PassExtras ex_arg = ex;
    // one block per segment, and enough blocks for the small tensors' warps (never more than are resident)
    const int small = num_warp_tensors > num_short_tensors ? num_warp_tensors : num_short_tensors;
    int for_warps = (small + kWarps - 1) / kWarps;
    if (for_warps > resident_blocks)
        for_warps = resident_blocks;
    int grid = num_segments > for_warps ? num_segments : for_warps;
    if (grid < 1)
        grid = 1;
    void* args[] = {(void*)&ops,          (void*)&operands_arg,     (void*)&segments, (void*)&num_segments,
                    (void*)&warp_tensors, (void*)&num_warp_tensors, (void*)&short_tensors, (void*)&num_short_tensors,
                    (void*)&partials,     (void*)&fin,              (void*)&out,      (void*)&ex_arg,
                    (void*)&status};
    return cudaLaunchCooperativeKernel(kernel, dim3((unsigned)grid), dim3(kThreads), args, 0, stream);
}

template <typename T, bool VEC>
cudaError_t launch_fused_small_radix(int radix, const OperandTable& ops, int operands, const SegmentTable& tab,
                                     int resident_blocks, float* partials, const FinishArgs& fin, void* out,
                                     const PassExtras& ex, int* status, cudaStream_t stream)
{
    switch (radix) {
    case 2: return launch_fused_small<T, 2, VEC>(ops, operands, tab, resident_blocks, partials, fin, out, ex, status, stream);
    case 4: return launch_fused_small<T, 4, VEC>(ops, operands, tab, resident_blocks, partials, fin, out, ex, status, stream);
    case 8: return launch_fused_small<T, 8, VEC>(ops, operands, tab, resident_blocks, partials, fin, out, ex, status, stream);
    default: return cudaErrorInvalidValue;
    }
}

template <typename T, int R1, int R2>
adasum_status_t launch_wsum_gram(const LevelArgs& a)
{
    constexpr int kNextGroupsPerLaunch = kMaxOperandsPerLaunch / (R1 * R2);
    // (the next level's ticket counters per tensor end where its counters per run begin)
    const FinishArgs next_fin{a.fuse_tab->d_seg_first, a.counters, a.next_weights, a.next_tree, 0,
                              a.fuse_tab->d_group_first,
                              a.counters ? a.counters + (size_t)(a.num_tensors > 0 ? a.num_tensors : 1) * a.next_groups
                                         : nullptr,
                              a.run_sums};
    for (int ng0 = 0; ng0 < a.next_groups; ng0 += kNextGroupsPerLaunch) {
        const int next_here = a.next_groups - ng0 < kNextGroupsPerLaunch ? a.next_groups - ng0 : kNextGroupsPerLaunch;
        const int g0 = ng0 * R2, op0 = g0 * R1;
        const int ops_here = a.operands - op0 < kMaxOperandsPerLaunch ? a.operands - op0 : kMaxOperandsPerLaunch;
        OperandTable table;
        for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
            table.ptr[i] = a.operand_ptrs[op0 + (i < ops_here ? i : 0)];
        dim3 grid((unsigned)a.fuse_tab->num_segments, (unsigned)next_here);
        wsum_gram_kernel<T, R1, R2, true><<<grid, kThreads, 0, a.stream>>>(
            table, ops_here, a.fuse_tab->d_segments, a.weights, a.groups, g0, static_cast<float*>(a.dst), a.dst_stride,
            a.partials, a.next_groups, ng0, next_fin);
        profile_mark(a.stream, ADASUM_KERNEL_WSUM_GRAM, a.level, R1, false);
    }
    ADASUM_CUDA_CHECK(cudaGetLastError());
    return ADASUM_OK;
}

template <typename T, int R>
adasum_status_t run_level_typed(const LevelArgs& a)
{
    constexpr int kGroupsPerLaunch = kMaxOperandsPerLaunch / R;
    // the last block of every (tensor, group) in pass 1 also derives the weights
    const bool fused_finish = a.counters != nullptr && a.phase == PHASE_WHOLE;
    const FinishArgs fin{a.gram_tab->d_seg_first, fused_finish ? a.counters : nullptr, a.weights, a.tree,
                         a.selftest_timeout ? 1 : 0, a.gram_tab->d_group_first, a.run_counters, a.run_sums};
    // pass 1
    for (int g0 = 0; g0 < a.groups && a.phase != PHASE_APPLY && !a.skip_gram; g0 += kGroupsPerLaunch) {
        const int groups_here = a.groups - g0 < kGroupsPerLaunch ? a.groups - g0 : kGroupsPerLaunch;
        const int op0 = g0 * R;
        const int ops_here = a.operands - op0 < kMaxOperandsPerLaunch ? a.operands - op0 : kMaxOperandsPerLaunch;
        OperandTable table;
        for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
            table.ptr[i] = a.operand_ptrs[op0 + (i < ops_here ? i : 0)];
        if (a.vec)
            ADASUM_CUDA_CHECK((launch_gram<T, R, true>(a.kind, table, ops_here, groups_here, *a.gram_tab,
                                                       a.partials, a.groups, g0, fin, a.stream, a.tc_status,
                                                       a.extras.start)));
        else
            ADASUM_CUDA_CHECK((launch_gram<T, R, false>(a.kind, table, ops_here, groups_here, *a.gram_tab,
                                                        a.partials, a.groups, g0, fin, a.stream)));
        profile_mark(a.stream, ADASUM_KERNEL_GRAM_PARTIAL, a.level, R, false);
    }
    if (a.phase == PHASE_APPLY) {
        launch_tree_from_sums<R>(a.gram64, a.num_tensors, a.operands, a.groups, a.weights, a.tree, a.stream);
        profile_mark(a.stream, ADASUM_KERNEL_TREE_WEIGHTS, a.level, R, false);
    } else if (!fused_finish && !a.skip_gram) {
        int weight_launches = 0;
        ADASUM_CUDA_CHECK(launch_weights<R>(a.partials, *a.gram_tab, a.num_tensors, a.operands, a.groups,
                                            a.gram64, a.weights, a.tree, a.stream, &weight_launches,
                                            a.phase == PHASE_GRAM_SUMS));
        profile_mark(a.stream, ADASUM_KERNEL_TREE_WEIGHTS, a.level, R, false);
    }
    // pass 2, together with the next level's pass 1 where that is possible
    if constexpr (R <= 4) {
        if (a.fuse_next_radix == 2)
            return launch_wsum_gram<T, R, 2>(a);
        if (a.fuse_next_radix == 4)
            return launch_wsum_gram<T, R, 4>(a);
    }
    for (int g0 = 0; g0 < a.groups && a.phase != PHASE_GRAM_SUMS; g0 += kGroupsPerLaunch) {
        const int groups_here = a.groups - g0 < kGroupsPerLaunch ? a.groups - g0 : kGroupsPerLaunch;
        const int op0 = g0 * R;
        const int ops_here = a.operands - op0 < kMaxOperandsPerLaunch ? a.operands - op0 : kMaxOperandsPerLaunch;
        OperandTable table;
        for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
            table.ptr[i] = a.operand_ptrs[op0 + (i < ops_here ? i : 0)];
        if (a.vec)
            launch_wsum<T, R, true>(table, ops_here, groups_here, *a.wsum_tab, a.weights, a.groups, g0, a.dst,
                                    a.dst_stride, a.stream, a.extras);
        else
            launch_wsum<T, R, false>(table, ops_here, groups_here, *a.wsum_tab, a.weights, a.groups, g0, a.dst,
                                     a.dst_stride, a.stream, a.extras);
        profile_mark(a.stream, ADASUM_KERNEL_WEIGHTED_SUM, a.level, R, false);
    }
    ADASUM_CUDA_CHECK(cudaGetLastError());
    return ADASUM_OK;
}

template <typename T>
adasum_status_t run_level(int radix, const LevelArgs& a)
{
    switch (radix) {
    case 2: return run_level_typed<T, 2>(a);
    case 4: return run_level_typed<T, 4>(a);
    case 8: return run_level_typed<T, 8>(a);
    case 16: return run_level_typed<T, 16>(a);
    case 32: return run_level_typed<T, 32>(a);
    case 64:
        if constexpr (sizeof(T) == 2)
            return run_level_typed<T, 64>(a);
        else
            return fail(ADASUM_ERR_ARG, "radix 64 needs fp16 / bf16 operands");
    default: return fail(ADASUM_ERR_ARG, "unsupported radix %d", radix);
    }
}

template <typename T>
cudaError_t noalloc_launch(bool vec, const OperandTable& ops, const SegmentTable& tab, int32_t num_tensors,
                           float* partials, float* weights, float* out, cudaStream_t stream)
{
    const TreeOptions plain_tree{0, 1, 1, 1, nullptr, nullptr};
    const FinishArgs no_fusion{nullptr, nullptr, nullptr, plain_tree};
    cudaError_t err = vec ? launch_gram<T, 2, true>(GRAM_SIMPLE, ops, 2, 1, tab, partials, 1, 0, no_fusion, stream)
                          : launch_gram<T, 2, false>(GRAM_SIMPLE, ops, 2, 1, tab, partials, 1, 0, no_fusion, stream);
    if (err != cudaSuccess)
        return err;
    int weight_launches = 0;
    err = launch_weights<2>(partials, tab, num_tensors, 2, 1, nullptr, weights, plain_tree, stream, &weight_launches);
    if (err != cudaSuccess)
        return err;
    if (vec)
        launch_wsum<T, 2, true>(ops, 2, 1, tab, weights, 1, 0, out, 0, stream);
    else
        launch_wsum<T, 2, false>(ops, 2, 1, tab, weights, 1, 0, out, 0, stream);
    return cudaSuccess;
}

template <typename T>
cudaError_t launch_fused_small_any(bool vec, int radix, const OperandTable& ops, int operands,
                                   const SegmentTable& tab, int resident_blocks, float* partials,
                                   const FinishArgs& fin, void* out, const PassExtras& ex, int* status,
                                   cudaStream_t stream)
{
    return vec ? launch_fused_small_radix<T, true>(radix, ops, operands, tab, resident_blocks, partials, fin, out, ex,
                                                   status, stream)
               : launch_fused_small_radix<T, false>(radix, ops, operands, tab, resident_blocks, partials, fin, out, ex,
                                                    status, stream);
}

template <typename T>
cudaError_t launch_convert(const void* src, void* dst, int64_t n, const PassExtras& ex, cudaStream_t stream)
{
    const int64_t blocks = (n + kThreads - 1) / kThreads;
    const unsigned grid = (unsigned)(blocks < 148 * 16 ? blocks : 148 * 16);
    convert_kernel<T><<<grid, kThreads, 0, stream>>>(static_cast<const T*>(src), dst, n, ex);
    return cudaGetLastError();
}

#define ADASUM_INSTANTIATE_LEVELS(T)                                                                              \
    template adasum_status_t run_level<T>(int, const LevelArgs&);                                                 \
    template cudaError_t launch_fused_small_any<T>(bool, int, const OperandTable&, int, const SegmentTable&, int, \
                                                   float*, const FinishArgs&, void*, const PassExtras&, int*,     \
                                                   cudaStream_t);                                                 \
    template cudaError_t noalloc_launch<T>(bool, const OperandTable&, const SegmentTable&, int32_t, float*,       \
                                           float*, float*, cudaStream_t);                                         \
    template cudaError_t launch_convert<T>(const void*, void*, int64_t, const PassExtras&, cudaStream_t);

}  // namespace adasum
