// Host side of the C ABI declared in include/adasum.h: argument checks, the level plan, the cached
// segment tables and the kernel launches.  Nothing here synchronises the stream.
#include "adasum.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <memory>
#include <mutex>
#include <vector>

#include "adasum_kernels.cuh"
#include "adasum_f64.cuh"

namespace adasum {
namespace {

thread_local char g_error[512] = "";

adasum_status_t fail(adasum_status_t status, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof g_error, fmt, ap);
    va_end(ap);
    return status;
}

#define ADASUM_CUDA_CHECK(expr)                                                                  \
    do {                                                                                         \
        cudaError_t err__ = (expr);                                                              \
        if (err__ != cudaSuccess)                                                                \
            return fail(ADASUM_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(err__));            \
    } while (0)

// ---- optional per-launch timing ---------------------------------------------------------------
// When enabled, an event is recorded on the caller's stream before the first launch of a reduce
// and after every launch; launch i lasted from event i to event i + 1.  Meant for benchmarking
// from one thread.

struct ProfileMark {
    int32_t kernel, level, radix;
    bool starts_call;     // the event opens a reduce call: no launch ends here
};

struct Profiler {
    bool enabled = false;
    std::vector<cudaEvent_t> events;
    std::vector<ProfileMark> marks;
    size_t used = 0;
    bool overflow = false;
};

Profiler g_profiler;
std::mutex g_profiler_mutex;

void profile_mark(cudaStream_t stream, int kernel, int level, int radix, bool starts_call)
{
    if (!g_profiler.enabled)
        return;
    std::lock_guard<std::mutex> lock(g_profiler_mutex);
    if (!g_profiler.enabled)
        return;
    if (g_profiler.used >= g_profiler.events.size()) {
        g_profiler.overflow = true;
        return;
    }
    if (cudaEventRecord(g_profiler.events[g_profiler.used], stream) != cudaSuccess)
        return;
    g_profiler.marks[g_profiler.used] = ProfileMark{kernel, level, radix, starts_call};
    ++g_profiler.used;
}

constexpr size_t kAlign = 256;
size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

int dtype_bytes(adasum_dtype_t dtype) { return dtype == ADASUM_F64 ? 8 : (dtype == ADASUM_F32 ? 4 : 2); }

bool known_dtype(adasum_dtype_t dtype)
{
    return dtype == ADASUM_F32 || dtype == ADASUM_F16 || dtype == ADASUM_BF16 || dtype == ADASUM_F64;
}

int max_radix_for(adasum_dtype_t dtype) { return dtype == ADASUM_F32 ? 32 : 64; }

bool valid_radix(int r) { return r == 2 || r == 4 || r == 8 || r == 16 || r == 32 || r == 64; }

int pow2_ceil(int x)
{
    int p = 1;
    while (p < x)
        p *= 2;
    return p;
}

// Which Gram kernel serves a level.
enum GramKind {
    GRAM_SIMPLE,      // fp32 pipes, operands in registers (radix <= 4; radix 8 and 16 on request)
    GRAM_MMA          // tensor cores (radix >= 8)
};

GramKind gram_kind(int radix, bool simple_kernels)
{
    return (radix >= 32 || (radix >= 8 && !simple_kernels)) ? GRAM_MMA : GRAM_SIMPLE;
}

// Elements per segment.  One block accumulates a whole segment in fp32 (per thread: segment /
// 256 elements; on the tensor cores: per warp segment / 8), longer tensors are finished in fp64.
int gram_segment_length(GramKind kind, int64_t total)
{
    if (kind == GRAM_MMA)
        return total >= (int64_t(1) << 26) ? 32768 : (total >= (int64_t(1) << 23) ? 16384 : 8192);
    return total >= (int64_t(1) << 23) ? 8192 : 2048;
}
int min_gram_segment_length(int radix, int64_t total)
{
    const int a = gram_segment_length(gram_kind(radix, false), total);
    const int b = gram_segment_length(gram_kind(radix, true), total);
    return a < b ? a : b;
}
int wsum_segment_length(int64_t total)
{
    return total >= (int64_t(1) << 26) ? 8192 : (total >= (int64_t(1) << 23) ? 4096 : 2048);
}

struct Level {
    int radix;
    int operands;   // operands entering the level
    int groups;     // operands leaving it
};

struct LevelPlan {
    int num_levels = 0;
    Level level[ADASUM_MAX_LEVELS];
};

// TreeOptions::linear for this reduce: 0 bottom-up pairs, 1 sequential, 2 top-down halves (only
// when that is a different tree, i.e. the count is not a power of two).
int tree_order(int n_workers, uint32_t flags)
{
    if (flags & ADASUM_FLAG_LINEAR_ORDER)
        return 1;
    if ((flags & ADASUM_FLAG_TOP_DOWN_HALVES) && n_workers > 1 && (n_workers & (n_workers - 1)) != 0)
        return 2;
    return 0;
}

bool plan_levels(int n_workers, adasum_dtype_t dtype, uint32_t flags, LevelPlan* plan)
{
    const int first = (int)(flags & 0xffu), later_flag = (int)((flags >> 8) & 0xffu);
    if ((flags >> 22) != 0)
        return false;
    if ((flags & ADASUM_FLAG_LINEAR_ORDER) && (flags & ADASUM_FLAG_TOP_DOWN_HALVES))
        return false;
    if (first != 0 && (!valid_radix(first) || first > max_radix_for(dtype)))
        return false;
    if (later_flag != 0 && (!valid_radix(later_flag) || later_flag > max_radix_for(ADASUM_F32)))
        return false;
    if ((flags & ADASUM_FLAG_SIMPLE_KERNELS) && (first > 16 || later_flag > 16))
        return false;
    int later = later_flag != 0 ? later_flag : first;
    if (later > max_radix_for(ADASUM_F32))
        later = max_radix_for(ADASUM_F32);      // intermediates are fp32
    const int cap_auto = (flags & ADASUM_FLAG_SIMPLE_KERNELS) ? 16 : 64;
    if ((flags & ADASUM_FLAG_LINEAR_ORDER) || tree_order(n_workers, flags) == 2) {
        // the running result of the sequential recursion is a combination of ALL earlier leaves
        // (and the halves of a top-down split are not aligned groups of equal size):
        // one level whose Gram matrix covers every worker
        if (first != 0 || later_flag != 0)
            return false;
        const int radix = pow2_ceil(n_workers < 2 ? 2 : n_workers);
        if (radix > max_radix_for(dtype) || radix > cap_auto)
            return false;
        plan->num_levels = 0;
        if (n_workers > 1) {
            plan->num_levels = 1;
            plan->level[0] = Level{radix, n_workers, 1};
        }
        return true;
    }
    int m = n_workers;
    plan->num_levels = 0;
    while (m > 1) {
        if (plan->num_levels == ADASUM_MAX_LEVELS)
            return false;
        const bool first_level = plan->num_levels == 0;
        const int want = first_level ? first : later;
        int radix = want;
        if (radix == 0) {
            // Measured on B200: the tensor-core Gram pass keeps up with HBM at radix 16 for fp32
            // operands and at radix 32 for fp16 / bf16; beyond that mma.sync is bound by the tensor pipe.
            radix = (first_level && dtype != ADASUM_F32) ? 32 : 16;
            // fp16 / bf16 workers in complete groups of 64: the tcgen05 kernel, one level less
            if (first_level && dtype != ADASUM_F32 && m % 64 == 0 && !(flags & ADASUM_FLAG_NO_TCGEN05))
                radix = 64;
            radix = radix < cap_auto ? radix : cap_auto;
        }
        if (radix > pow2_ceil(m))
            radix = pow2_ceil(m);
        Level& lv = plan->level[plan->num_levels++];
        lv.radix = radix;
        lv.operands = m;
        lv.groups = (m + radix - 1) / radix;
        m = lv.groups;
    }
    return true;
}

int64_t segment_bound(int64_t total, int32_t num_tensors, int seg_len)
{
    return total / seg_len + 2 * (int64_t)num_tensors + 1;
}

struct Layout {
    size_t partials = 0, weights = 0, weights_alt = 0, gram64 = 0, counters = 0, leaf_sums = 0, buffer[2] = {0, 0};
    size_t partials_bytes = 0, weights_bytes = 0, gram64_bytes = 0, counters_bytes = 0, leaf_sums_bytes = 0,
           buffer_bytes[2] = {0, 0};
    int64_t padded_elems = 0;
    size_t total = 0;
};

Layout make_layout(const LevelPlan& plan, int64_t total_elems, int32_t num_tensors)
{
    Layout lay;
    lay.padded_elems = (total_elems + 63) / 64 * 64;
    for (int l = 0; l < plan.num_levels; ++l) {
        const Level& lv = plan.level[l];
        const size_t p = (size_t)segment_bound(total_elems, num_tensors,
                                               min_gram_segment_length(lv.radix, total_elems)) *
                         lv.groups * gram_entries(lv.radix) * sizeof(float);
        const size_t w = (size_t)(num_tensors > 0 ? num_tensors : 1) * lv.groups * lv.radix * sizeof(float);
        if (p > lay.partials_bytes)
            lay.partials_bytes = p;
        if (w > lay.weights_bytes)
            lay.weights_bytes = w;
        const size_t c = ((size_t)(num_tensors > 0 ? num_tensors : 1) * lv.groups + 1) * sizeof(int);
        if (c > lay.counters_bytes)       // + 1: the device status word sits after the ticket counters
            lay.counters_bytes = c;
        const size_t g64 = (size_t)(num_tensors > 0 ? num_tensors : 1) * lv.groups * gram_entries(lv.radix) *
                           sizeof(double);
        if (g64 > lay.gram64_bytes)
            lay.gram64_bytes = g64;
        if (l + 1 < plan.num_levels) {      // this level's output is an intermediate
            const size_t b = (size_t)lv.groups * lay.padded_elems * sizeof(float);
            if (b > lay.buffer_bytes[l & 1])
                lay.buffer_bytes[l & 1] = b;
        }
    }
    size_t off = 0;
    lay.partials = off;
    off += align_up(lay.partials_bytes);
    lay.weights = off;
    off += align_up(lay.weights_bytes);
    lay.weights_alt = off;          // odd levels: a fused kernel reads one level's weights while it writes the next's
    off += align_up(lay.weights_bytes);
    lay.gram64 = off;
    off += align_up(lay.gram64_bytes);
    lay.counters = off;
    off += align_up(lay.counters_bytes);
    if (plan.num_levels > 0)
        lay.leaf_sums_bytes = (size_t)(num_tensors > 0 ? num_tensors : 1) * plan.level[0].groups * sizeof(double);
    lay.leaf_sums = off;
    off += align_up(lay.leaf_sums_bytes);
    lay.buffer[0] = off;
    off += align_up(lay.buffer_bytes[0]);
    lay.buffer[1] = off;
    off += align_up(lay.buffer_bytes[1]);
    lay.total = off > 0 ? off : kAlign;
    return lay;
}

// ---- cached segment tables ---------------------------------------------------------------------

struct SegmentTable {
    int device = -1;
    int seg_len = 0;
    std::vector<int64_t> offsets;
    Segment* d_segments = nullptr;
    int32_t* d_seg_first = nullptr;
    int32_t num_segments = 0;
    int32_t max_segments_per_tensor = 0;
    std::vector<Segment> h_segments;
    std::vector<int32_t> h_seg_first;
};

std::mutex g_tables_mutex;
std::vector<std::unique_ptr<SegmentTable>> g_tables;
constexpr size_t kMaxCachedTables = 64;

// Segments are listed tensor by tensor, LARGEST tensor first (ties in index order): the blocks of
// pass 1 that run last then belong to small tensors, whose per-tensor finish (adding the partial
// matrices, tree weights) is short, instead of leaving one SM busy with a long tensor's finish
// while the rest of the GPU idles.  Each tensor's segments stay contiguous, in element order.
void build_segments(const int64_t* offsets, int32_t num_tensors, int seg_len, SegmentTable* tab)
{
    std::vector<int32_t> order((size_t)num_tensors);
    for (int32_t t = 0; t < num_tensors; ++t)
        order[t] = t;
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) {
        return offsets[x + 1] - offsets[x] > offsets[y + 1] - offsets[y];
    });
    tab->h_segments.clear();
    // h_seg_first[2 t], h_seg_first[2 t + 1]: first and one-past-last segment of tensor t
    tab->h_seg_first.assign(2 * (size_t)num_tensors + 2, 0);
    tab->max_segments_per_tensor = 0;
    for (int32_t t : order) {
        tab->h_seg_first[2 * (size_t)t] = (int32_t)tab->h_segments.size();
        int64_t b = offsets[t];
        const int64_t e = offsets[t + 1];
        while (b < e) {
            // cut on a 64-element grid of the fused buffer so that interior cuts keep 16-byte
            // alignment whatever the tensor's own start
            int64_t next = b / 64 * 64 + seg_len;
            if (next > e)
                next = e;
            tab->h_segments.push_back(Segment{b, (int32_t)(next - b), t});
            b = next;
        }
        tab->h_seg_first[2 * (size_t)t + 1] = (int32_t)tab->h_segments.size();
        const int32_t n = tab->h_seg_first[2 * (size_t)t + 1] - tab->h_seg_first[2 * (size_t)t];
        if (n > tab->max_segments_per_tensor)
            tab->max_segments_per_tensor = n;
    }
    tab->num_segments = (int32_t)tab->h_segments.size();
}

adasum_status_t get_segment_table(const int64_t* offsets, int32_t num_tensors, int seg_len,
                                  const SegmentTable** out)
{
    int device = 0;
    ADASUM_CUDA_CHECK(cudaGetDevice(&device));
    std::lock_guard<std::mutex> lock(g_tables_mutex);
    for (const auto& tab : g_tables) {
        if (tab->device == device && tab->seg_len == seg_len &&
            tab->offsets.size() == (size_t)num_tensors + 1 &&
            std::memcmp(tab->offsets.data(), offsets, sizeof(int64_t) * tab->offsets.size()) == 0) {
            *out = tab.get();
            return ADASUM_OK;
        }
    }
    if (g_tables.size() >= kMaxCachedTables) {
        // Drop the oldest table.  cudaFree waits for work already submitted to the device, so
        // kernels still reading the table finish first.
        SegmentTable* oldest = g_tables.front().get();
        int current = device;
        if (oldest->device != current)
            ADASUM_CUDA_CHECK(cudaSetDevice(oldest->device));
        cudaError_t e1 = cudaFree(oldest->d_segments), e2 = cudaFree(oldest->d_seg_first);
        if (oldest->device != current)
            ADASUM_CUDA_CHECK(cudaSetDevice(current));
        g_tables.erase(g_tables.begin());
        if (e1 != cudaSuccess || e2 != cudaSuccess)
            return fail(ADASUM_ERR_CUDA, "freeing an evicted segment table failed");
    }
    auto tab = std::make_unique<SegmentTable>();
    tab->device = device;
    tab->seg_len = seg_len;
    tab->offsets.assign(offsets, offsets + num_tensors + 1);
    build_segments(offsets, num_tensors, seg_len, tab.get());
    const size_t seg_bytes = sizeof(Segment) * (tab->h_segments.size() + 1);
    const size_t first_bytes = sizeof(int32_t) * tab->h_seg_first.size();
    ADASUM_CUDA_CHECK(cudaMalloc(&tab->d_segments, seg_bytes));
    cudaError_t err = cudaMalloc(&tab->d_seg_first, first_bytes);
    // Blocking copies: the table may be used from any stream afterwards.
    if (err == cudaSuccess && !tab->h_segments.empty())
        err = cudaMemcpy(tab->d_segments, tab->h_segments.data(),
                         sizeof(Segment) * tab->h_segments.size(), cudaMemcpyHostToDevice);
    if (err == cudaSuccess)
        err = cudaMemcpy(tab->d_seg_first, tab->h_seg_first.data(), first_bytes, cudaMemcpyHostToDevice);
    if (err != cudaSuccess) {
        cudaFree(tab->d_segments);
        cudaFree(tab->d_seg_first);
        return fail(ADASUM_ERR_CUDA, "segment table upload: %s", cudaGetErrorString(err));
    }
    *out = tab.get();
    g_tables.push_back(std::move(tab));
    return ADASUM_OK;
}

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

constexpr PassExtras kNoExtras{nullptr, nullptr, 0, 0};

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
        tree_weights_kernel<R><<<grid2, kThreads, 0, stream>>>(gram64, operands, weights, opt);
        *launches = 2;
    }
    return cudaSuccess;
}

template <int R>
void launch_tree_from_sums(const double* gram64, int32_t num_tensors, int operands, int groups, float* weights,
                           const TreeOptions& opt, cudaStream_t stream)
{
    dim3 grid((unsigned)num_tensors, (unsigned)groups);
    tree_weights_kernel<R><<<grid, kThreads, 0, stream>>>(gram64, operands, weights, opt);
}

// Which part of a level a call runs.
enum LevelPhase {
    PHASE_WHOLE = 0,        // pass 1, coefficients, pass 2
    PHASE_GRAM_SUMS = 1,    // pass 1, then this GPU's fp64 Gram sums to gram64 (to be added across GPUs)
    PHASE_APPLY = 2         // coefficients from gram64, then pass 2
};

// ---- single-launch path for inputs that fit the L2 ------------------------------------------------

constexpr int64_t kSmallInputBytes = int64_t(96) << 20;    // operands that the 126 MB L2 holds with room to spare
constexpr int kSmallBlocksPerSm = 2;                       // blocks per SM the grid is sized for (all variants keep >= 2 resident)
constexpr int kSmallSegmentGrain = 1024;

// Host-only rule (no device query): is this reduce served by fused_small_kernel, and with which
// segment length?  `blocks` is the number of blocks that can be resident at once.
bool small_input_plan(const LevelPlan& plan, int64_t total, int32_t num_tensors, int n_workers, int elem_bytes,
                      uint32_t flags, int blocks, int* seg_len)
{
    if (plan.num_levels != 1 || plan.level[0].radix > 8 || plan.level[0].groups != 1)
        return false;
    if (flags & (ADASUM_FLAG_SIMPLE_KERNELS | ADASUM_FLAG_SEPARATE_FINISH))
        return false;
    if (total <= 0 || (int64_t)n_workers * total * elem_bytes > kSmallInputBytes)
        return false;
    // every tensor ends with one ragged segment: budget for those first
    const int64_t room = (int64_t)blocks - 2 * (int64_t)num_tensors;
    if (room < 8)
        return false;
    int64_t len = (total + room - 1) / room;
    len = (len + kSmallSegmentGrain - 1) / kSmallSegmentGrain * kSmallSegmentGrain;
    if (len < 2048)
        len = 2048;
    if (len > (int64_t(1) << 20))
        return false;
    *seg_len = (int)len;
    return true;
}

template <typename T, int R, bool VEC>
cudaError_t launch_fused_small(const OperandTable& ops, int operands, const SegmentTable& tab, float* partials,
                               const FinishArgs& fin, void* out, const PassExtras& ex, int* status, cudaStream_t stream)
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
    PassExtras ex_arg = ex;
    void* args[] = {(void*)&ops, (void*)&operands_arg, (void*)&segments, (void*)&partials,
                    (void*)&fin, (void*)&out,          (void*)&ex_arg,   (void*)&status};
    return cudaLaunchCooperativeKernel(kernel, dim3((unsigned)tab.num_segments), dim3(kThreads), args, 0, stream);
}

template <typename T, bool VEC>
cudaError_t launch_fused_small_radix(int radix, const OperandTable& ops, int operands, const SegmentTable& tab,
                                     float* partials, const FinishArgs& fin, void* out, const PassExtras& ex,
                                     int* status, cudaStream_t stream)
{
    switch (radix) {
    case 2: return launch_fused_small<T, 2, VEC>(ops, operands, tab, partials, fin, out, ex, status, stream);
    case 4: return launch_fused_small<T, 4, VEC>(ops, operands, tab, partials, fin, out, ex, status, stream);
    case 8: return launch_fused_small<T, 8, VEC>(ops, operands, tab, partials, fin, out, ex, status, stream);
    default: return cudaErrorInvalidValue;
    }
}

// Blocks of fused_small_kernel that the current device keeps resident (0: no cooperative launch).
int resident_small_blocks()
{
    static int cached[64] = {};
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64)
        return 0;
    if (cached[device] == 0) {
        int sms = 0, coop = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device) != cudaSuccess || !coop || sms <= 0)
            cached[device] = -1;
        else
            cached[device] = sms * kSmallBlocksPerSm;
    }
    return cached[device] > 0 ? cached[device] : 0;
}

struct LevelArgs {
    const void* const* operand_ptrs;   // host array, `operands` entries
    int operands;
    int groups;
    GramKind kind;
    const SegmentTable* gram_tab;
    const SegmentTable* wsum_tab;
    int32_t num_tensors;
    float* partials;
    int* counters;      // ticket counters for finishing inside pass 1, or nullptr
    TreeOptions tree;
    LevelPhase phase;
    int* tc_status;     // status word for the tcgen05 kernel, or nullptr to keep to mma.sync
    double* gram64;
    float* weights;
    void* dst;
    int64_t dst_stride;
    PassExtras extras;   // start: this level's operands are (operand - start); base / out_dtype: last level
    bool vec;
    cudaStream_t stream;
    int level;
    // fusion of this level's pass 2 with the next level's pass 1 (wsum_gram_kernel)
    bool skip_gram;              // this level's Gram sums and weights were produced by the previous level's pass 2
    int fuse_next_radix;         // 0: plain pass 2; 2 or 4: also pass 1 of the next level, which has this radix
    const SegmentTable* fuse_tab;
    int next_groups;
    float* next_weights;
    TreeOptions next_tree;
};

// Measured on a B200: fusing pays while this level's groups are narrow (literal tree 0.60 -> 0.54 ms on
// the ResNet-50 list with 8 workers, 14.7 -> 13.0 ms on the BERT-Large list with 16); from radix 8 on
// the plain second pass, which keeps three blocks per SM busy, is faster than the saving.
bool fusable_radices(int radix, int next_radix) { return radix <= 4 && (next_radix == 2 || next_radix == 4); }

template <typename T, int R1, int R2>
adasum_status_t launch_wsum_gram(const LevelArgs& a)
{
    constexpr int kNextGroupsPerLaunch = kMaxOperandsPerLaunch / (R1 * R2);
    const FinishArgs next_fin{a.fuse_tab->d_seg_first, a.counters, a.next_weights, a.next_tree};
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
    const FinishArgs fin{a.gram_tab->d_seg_first, fused_finish ? a.counters : nullptr, a.weights, a.tree};
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

int launches_of(const LevelPlan& plan, int n_workers, uint32_t flags, int64_t total, int32_t num_tensors,
                int elem_bytes)
{
    if (n_workers == 1)
        return 1;
    int seg_len = 0;        // on a B200: 148 SMs
    if (small_input_plan(plan, total, num_tensors, n_workers, elem_bytes, flags, 148 * kSmallBlocksPerSm, &seg_len))
        return 1;
    int n = 0;
    bool gram_done = false;      // by the previous level's pass 2 (16-byte aligned buffers assumed)
    for (int l = 0; l < plan.num_levels; ++l) {
        const int radix = plan.level[l].radix;
        const int per_launch = kMaxOperandsPerLaunch / radix;
        const int batches = (plan.level[l].groups + per_launch - 1) / per_launch;
        if (!gram_done) {
            n += batches;
            if (flags & ADASUM_FLAG_SEPARATE_FINISH)        // otherwise done inside pass 1
                n += radix >= 32 ? 2 : 1;                   // gram_finish (+ tree_weights)
        }
        gram_done = l + 1 < plan.num_levels && fusable_radices(radix, plan.level[l + 1].radix) &&
                    !(flags & (ADASUM_FLAG_SEPARATE_FINISH | ADASUM_FLAG_NO_LEVEL_FUSION));
        if (gram_done) {
            const int next_per_launch = kMaxOperandsPerLaunch / (radix * plan.level[l + 1].radix);
            n += (plan.level[l + 1].groups + next_per_launch - 1) / next_per_launch;
        } else {
            n += batches;
        }
    }
    return n;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool ranges_overlap(const void* a, size_t a_bytes, const void* b, size_t b_bytes)
{
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + b_bytes && b0 < a0 + a_bytes;
}

adasum_status_t check_common(const int64_t* offsets, int32_t num_tensors, int32_t n_workers,
                             adasum_dtype_t dtype)
{
    if (!offsets)
        return fail(ADASUM_ERR_NULL, "tensor_offsets is NULL");
    if (!known_dtype(dtype))
        return fail(ADASUM_ERR_DTYPE, "unknown dtype %d", (int)dtype);
    if (n_workers < 1 || n_workers > ADASUM_MAX_WORKERS)
        return fail(ADASUM_ERR_ARG, "n_workers = %d outside 1..%d", n_workers, ADASUM_MAX_WORKERS);
    if (num_tensors < 0)
        return fail(ADASUM_ERR_ARG, "num_tensors = %d is negative", num_tensors);
    if (offsets[0] != 0)
        return fail(ADASUM_ERR_OFFSETS, "tensor_offsets[0] = %lld, expected 0", (long long)offsets[0]);
    for (int32_t t = 0; t < num_tensors; ++t)
        if (offsets[t + 1] < offsets[t])
            return fail(ADASUM_ERR_OFFSETS, "tensor_offsets decreases at tensor %d", t);
    return ADASUM_OK;
}

// `start` != nullptr: the delta form, out = start + Adasum_i(grads[i] - start).  `out` holds
// elements of out_dtype.
adasum_status_t reduce_impl(const void* const* grads, const int64_t* offsets, int32_t num_tensors,
                            int32_t n_workers, adasum_dtype_t dtype, void* out, float* orthogonality,
                            void* workspace, size_t workspace_bytes, uint32_t flags, cudaStream_t stream,
                            LevelPhase phase = PHASE_WHOLE, int only_level = -1, size_t* sums_offset = nullptr,
                            int64_t* sums_count = nullptr, const void* start = nullptr,
                            adasum_dtype_t out_dtype = ADASUM_F32)
{
    g_error[0] = '\0';
    if (dtype == ADASUM_F64)       // whole reduces of fp64 buffers go to reduce_f64_impl
        return fail(ADASUM_ERR_DTYPE, "the sharded calls take fp32, fp16 or bf16 gradients");
    if (!grads)
        return fail(ADASUM_ERR_NULL, "grads is NULL");
    if (orthogonality && n_workers < 2)
        return fail(ADASUM_ERR_ARG, "the orthogonality measure needs at least two workers");
    if (reinterpret_cast<uintptr_t>(orthogonality) & 3u)
        return fail(ADASUM_ERR_ARG, "orthogonality is not 4-byte aligned");
    adasum_status_t st = check_common(offsets, num_tensors, n_workers, dtype);
    if (st != ADASUM_OK)
        return st;
    LevelPlan plan;
    if (!plan_levels(n_workers, dtype, flags, &plan))
        return fail(ADASUM_ERR_ARG, "invalid flags 0x%x for %d workers of this dtype", flags, n_workers);
    const int64_t total = offsets[num_tensors];
    const bool sharded = phase != PHASE_WHOLE;
    if (sharded) {
        if (n_workers < 2)
            return fail(ADASUM_ERR_ARG, "the sharded calls need at least two workers");
        if (only_level < 0 || only_level >= plan.num_levels)
            return fail(ADASUM_ERR_ARG, "level %d outside 0..%d", only_level, plan.num_levels - 1);
        if (flags & ADASUM_FLAG_SEPARATE_FINISH)
            return fail(ADASUM_ERR_ARG, "ADASUM_FLAG_SEPARATE_FINISH has no meaning for the sharded calls");
    }
    if (total == 0 && !sharded)
        return ADASUM_OK;
    const bool need_out = phase != PHASE_GRAM_SUMS && total > 0;
    if (need_out && !out)
        return fail(ADASUM_ERR_NULL, "out is NULL");
    if (out_dtype != ADASUM_F32 && out_dtype != ADASUM_F16 && out_dtype != ADASUM_BF16)
        return fail(ADASUM_ERR_DTYPE, out_dtype == ADASUM_F64 ? "an fp64 output needs fp64 inputs" : "unknown output dtype %d",
                    (int)out_dtype);
    if (reinterpret_cast<uintptr_t>(out) & (uintptr_t)(dtype_bytes(out_dtype) - 1))
        return fail(ADASUM_ERR_ARG, "out is not aligned to its element size");
    const int eb = dtype_bytes(dtype);
    const size_t in_bytes = (size_t)total * eb, out_bytes = out ? (size_t)total * dtype_bytes(out_dtype) : 0;
    bool vec = out ? aligned16(out) : true;
    if (start != nullptr && total > 0) {
        if (!aligned16(start))
            return fail(ADASUM_ERR_ARG, "start is not 16-byte aligned");
        // the result may be written over start (the parameters are updated in place), nothing else
        const bool in_place = out == start && out_dtype == dtype;
        if (out && !in_place && ranges_overlap(start, in_bytes, out, out_bytes))
            return fail(ADASUM_ERR_ARG, "out overlaps start without being the same buffer of the same type");
        for (int w = 0; w < n_workers; ++w)
            if (grads[w] && ranges_overlap(start, in_bytes, grads[w], in_bytes))
                return fail(ADASUM_ERR_ARG, "start overlaps grads[%d]", w);
    }
    for (int w = 0; w < n_workers && total > 0; ++w) {
        if (!grads[w])
            return fail(ADASUM_ERR_NULL, "grads[%d] is NULL", w);
        if (reinterpret_cast<uintptr_t>(grads[w]) & (uintptr_t)(eb - 1))
            return fail(ADASUM_ERR_ARG, "grads[%d] is not aligned to its element size", w);
        if (out && ranges_overlap(grads[w], in_bytes, out, out_bytes))
            return fail(ADASUM_ERR_ARG, "out overlaps grads[%d]", w);
        vec = vec && aligned16(grads[w]);
    }
    if (start != nullptr && total > 0 && !vec)
        return fail(ADASUM_ERR_ARG, "the delta form needs every buffer 16-byte aligned");
    const Layout lay = make_layout(plan, total, num_tensors);
    if (n_workers > 1) {
        if (!workspace)
            return fail(ADASUM_ERR_WORKSPACE, "workspace is NULL");
        if (workspace_bytes < lay.total)
            return fail(ADASUM_ERR_WORKSPACE, "workspace has %zu bytes, need %zu", workspace_bytes, lay.total);
        if (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1))
            return fail(ADASUM_ERR_ARG, "workspace is not %zu-byte aligned", kAlign);
        if (out && total > 0 && ranges_overlap(workspace, lay.total, out, out_bytes))
            return fail(ADASUM_ERR_ARG, "workspace overlaps out");
        for (int w = 0; w < n_workers && total > 0; ++w)
            if (ranges_overlap(workspace, lay.total, grads[w], in_bytes))
                return fail(ADASUM_ERR_ARG, "workspace overlaps grads[%d]", w);
        if (start != nullptr && total > 0 && ranges_overlap(workspace, lay.total, start, in_bytes))
            return fail(ADASUM_ERR_ARG, "workspace overlaps start");
    }
    // what the last level adds and how it stores; the first level gets `start` as well
    const PassExtras last_extras{nullptr, start, (int)dtype, (int)out_dtype};

    profile_mark(stream, -1, 0, 0, true);
    if (n_workers == 1) {
        const int64_t blocks = (total + kThreads - 1) / kThreads;
        const unsigned grid = (unsigned)(blocks < 148 * 16 ? blocks : 148 * 16);
        PassExtras ex = last_extras;
        ex.start = start;
        if (dtype == ADASUM_F32)
            convert_kernel<float><<<grid, kThreads, 0, stream>>>((const float*)grads[0], out, total, ex);
        else if (dtype == ADASUM_F16)
            convert_kernel<__half><<<grid, kThreads, 0, stream>>>((const __half*)grads[0], out, total, ex);
        else
            convert_kernel<__nv_bfloat16><<<grid, kThreads, 0, stream>>>((const __nv_bfloat16*)grads[0], out, total, ex);
        ADASUM_CUDA_CHECK(cudaGetLastError());
        profile_mark(stream, ADASUM_KERNEL_CONVERT, 0, 1, false);
        return ADASUM_OK;
    }

    char* ws = static_cast<char*>(workspace);
    const bool separate_finish = (flags & ADASUM_FLAG_SEPARATE_FINISH) != 0 || sharded;
    // Inputs that fit the L2 are served by one cooperative launch that needs no ticket counters.
    int small_seg_len = 0;
    const int small_blocks = (sharded || total == 0 || num_tensors == 0) ? 0 : resident_small_blocks();
    const bool small_candidate =
        small_blocks > 0 && small_input_plan(plan, total, num_tensors, n_workers, eb, flags, small_blocks, &small_seg_len);
    // the workspace arrives with unknown contents
    auto clear_counters = [&]() { return cudaMemsetAsync(ws + lay.counters, 0, lay.counters_bytes, stream); };
    if (lay.counters_bytes > 0 && phase != PHASE_APPLY && !small_candidate)
        ADASUM_CUDA_CHECK(clear_counters());
    if (orthogonality && num_tensors > 0 && (!sharded || (phase == PHASE_APPLY && only_level == 0)))
        ADASUM_CUDA_CHECK(cudaMemsetAsync(orthogonality, 0xff, sizeof(float) * (size_t)num_tensors, stream));
    if (phase == PHASE_GRAM_SUMS) {
        const Level& lv = plan.level[only_level];
        const size_t count = (size_t)num_tensors * lv.groups * gram_entries(lv.radix);
        if (sums_offset)
            *sums_offset = lay.gram64;
        if (sums_count)
            *sums_count = (int64_t)count;
        if (total == 0 || num_tensors == 0) {           // this GPU holds no element: its sums are zero
            if (count > 0)
                ADASUM_CUDA_CHECK(cudaMemsetAsync(ws + lay.gram64, 0, count * sizeof(double), stream));
            return ADASUM_OK;
        }
    }
    if (total == 0 || num_tensors == 0)
        return ADASUM_OK;
    // per-launch timing: the first kernel's interval starts here, after the clearing of counters above
    profile_mark(stream, -1, 0, 0, true);
    std::vector<const void*> operand_ptrs(grads, grads + n_workers);

    // Inputs that fit the L2: one cooperative launch does both passes and HBM sees the operands once.
    if (small_candidate) {
        int* dev_status = reinterpret_cast<int*>(ws + lay.counters + lay.counters_bytes - sizeof(int));
        const SegmentTable* tab = nullptr;
        st = get_segment_table(offsets, num_tensors, small_seg_len, &tab);
        if (st != ADASUM_OK)
            return st;
        if (tab->num_segments <= small_blocks) {
            OperandTable table;
            for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
                table.ptr[i] = grads[i < n_workers ? i : 0];
            FinishArgs fin;
            fin.seg_first = tab->d_seg_first;
            fin.counters = nullptr;
            fin.weights = nullptr;
            fin.tree = TreeOptions{tree_order(n_workers, flags), 1, 1, 1,
                                   orthogonality ? reinterpret_cast<double*>(ws + lay.leaf_sums) : nullptr,
                                   orthogonality};
            float* partials = reinterpret_cast<float*>(ws + lay.partials);
            const int radix = plan.level[0].radix;
            PassExtras ex = last_extras;
            ex.start = start;
            cudaError_t err;
            if (dtype == ADASUM_F32)
                err = vec ? launch_fused_small_radix<float, true>(radix, table, n_workers, *tab, partials, fin, out, ex, dev_status, stream)
                          : launch_fused_small_radix<float, false>(radix, table, n_workers, *tab, partials, fin, out, ex, dev_status, stream);
            else if (dtype == ADASUM_F16)
                err = vec ? launch_fused_small_radix<__half, true>(radix, table, n_workers, *tab, partials, fin, out, ex, dev_status, stream)
                          : launch_fused_small_radix<__half, false>(radix, table, n_workers, *tab, partials, fin, out, ex, dev_status, stream);
            else
                err = vec ? launch_fused_small_radix<__nv_bfloat16, true>(radix, table, n_workers, *tab, partials, fin, out, ex, dev_status, stream)
                          : launch_fused_small_radix<__nv_bfloat16, false>(radix, table, n_workers, *tab, partials, fin, out, ex, dev_status, stream);
            if (err == cudaSuccess) {
                profile_mark(stream, ADASUM_KERNEL_FUSED_SMALL, 0, radix, false);
                return ADASUM_OK;
            }
            if (err != cudaErrorCooperativeLaunchTooLarge)
                return fail(ADASUM_ERR_CUDA, "cooperative launch: %s", cudaGetErrorString(err));
            (void)cudaGetLastError();       // too many blocks for this device after all: the two-pass path serves it
        }
        ADASUM_CUDA_CHECK(clear_counters());      // the two-pass path draws tickets
    }

    bool gram_done = false;      // the previous level's pass 2 has already produced this level's weights
    for (int l = 0; l < plan.num_levels; ++l) {
        const Level& lv = plan.level[l];
        if (only_level >= 0 && l != only_level) {       // other levels' operands: the intermediates
            if (l + 1 < plan.num_levels) {
                float* buf = reinterpret_cast<float*>(ws + lay.buffer[l & 1]);
                operand_ptrs.resize((size_t)lv.groups);
                for (int g = 0; g < lv.groups; ++g)
                    operand_ptrs[g] = buf + (int64_t)g * lay.padded_elems;
            }
            continue;
        }
        const bool simple_kernels = (flags & ADASUM_FLAG_SIMPLE_KERNELS) != 0;
        const GramKind kind = gram_kind(lv.radix, simple_kernels);
        const SegmentTable* gram_tab = nullptr;
        const SegmentTable* wsum_tab = nullptr;
        st = get_segment_table(offsets, num_tensors, gram_segment_length(kind, total), &gram_tab);
        if (st != ADASUM_OK)
            return st;
        st = get_segment_table(offsets, num_tensors, wsum_segment_length(total), &wsum_tab);
        if (st != ADASUM_OK)
            return st;
        const bool last = l + 1 == plan.num_levels;
        LevelArgs a;
        a.operand_ptrs = operand_ptrs.data();
        a.operands = lv.operands;
        a.groups = lv.groups;
        a.kind = kind;
        a.gram_tab = gram_tab;
        a.wsum_tab = wsum_tab;
        a.num_tensors = num_tensors;
        a.partials = reinterpret_cast<float*>(ws + lay.partials);
        a.weights = reinterpret_cast<float*>(ws + ((l & 1) ? lay.weights_alt : lay.weights));
        a.gram64 = reinterpret_cast<double*>(ws + lay.gram64);
        a.counters = separate_finish ? nullptr : reinterpret_cast<int*>(ws + lay.counters);
        a.phase = phase;
        // the status word is the last int of the (zeroed) counter region
        a.tc_status = (flags & ADASUM_FLAG_NO_TCGEN05)
                          ? nullptr
                          : reinterpret_cast<int*>(ws + lay.counters + lay.counters_bytes - sizeof(int));
        a.tree.linear = tree_order(n_workers, flags);
        a.tree.level_is_first = l == 0;
        a.tree.level_is_last = l + 1 == plan.num_levels;
        a.tree.groups_first = plan.level[0].groups;
        a.tree.leaf_norm_sums = orthogonality ? reinterpret_cast<double*>(ws + lay.leaf_sums) : nullptr;
        a.tree.orthogonality = orthogonality;
        a.dst = last ? out : static_cast<void*>(ws + lay.buffer[l & 1]);
        a.dst_stride = last ? 0 : lay.padded_elems;
        a.extras = last ? last_extras : kNoExtras;
        if (l == 0)
            a.extras.start = start;
        a.vec = vec;
        a.stream = stream;
        a.level = l;
        a.skip_gram = gram_done;
        a.fuse_next_radix = 0;
        a.fuse_tab = nullptr;
        a.next_groups = 0;
        a.next_weights = nullptr;
        a.next_tree = a.tree;
        gram_done = false;
        if (!last && !sharded && !separate_finish && vec && !(flags & ADASUM_FLAG_NO_LEVEL_FUSION) &&
            a.extras.start == nullptr && fusable_radices(lv.radix, plan.level[l + 1].radix)) {
            st = get_segment_table(offsets, num_tensors, gram_segment_length(GRAM_SIMPLE, total), &a.fuse_tab);
            if (st != ADASUM_OK)
                return st;
            a.fuse_next_radix = plan.level[l + 1].radix;
            a.next_groups = plan.level[l + 1].groups;
            a.next_weights = reinterpret_cast<float*>(ws + (((l + 1) & 1) ? lay.weights_alt : lay.weights));
            a.next_tree.level_is_first = 0;
            a.next_tree.level_is_last = l + 2 == plan.num_levels;
            gram_done = true;
        }
        if (l == 0) {
            if (dtype == ADASUM_F32)
                st = run_level<float>(lv.radix, a);
            else if (dtype == ADASUM_F16)
                st = run_level<__half>(lv.radix, a);
            else
                st = run_level<__nv_bfloat16>(lv.radix, a);
        } else {
            st = run_level<float>(lv.radix, a);
        }
        if (st != ADASUM_OK)
            return st;
        if (!last) {
            operand_ptrs.resize((size_t)lv.groups);
            for (int g = 0; g < lv.groups; ++g)
                operand_ptrs[g] = static_cast<float*>(a.dst) + (int64_t)g * lay.padded_elems;
        }
    }
    return ADASUM_OK;
}

// ---- fp64 gradients ------------------------------------------------------------------------------
//
// A family of its own (adasum_f64.cuh): levels of radix 2 or 4 on the fp64 pipes, doubles throughout.

// flags of an fp64 reduce: radix fields 0 (= 4), 2 or 4; the switches that select fp32 / 16-bit
// kernels are accepted and change nothing; the orders that need one Gram matrix over all workers
// are not offered.
bool plan_levels_f64(int n_workers, uint32_t flags, LevelPlan* plan)
{
    const int first = (int)(flags & 0xffu), later_flag = (int)((flags >> 8) & 0xffu);
    if ((flags >> 22) != 0)
        return false;
    if (flags & (ADASUM_FLAG_LINEAR_ORDER | ADASUM_FLAG_TOP_DOWN_HALVES | ADASUM_FLAG_SEPARATE_FINISH |
                 ADASUM_FLAG_SIMPLE_KERNELS))
        return false;
    if ((first != 0 && first != 2 && first != 4) || (later_flag != 0 && later_flag != 2 && later_flag != 4))
        return false;
    const int later = later_flag != 0 ? later_flag : first;
    int m = n_workers;
    plan->num_levels = 0;
    while (m > 1) {
        if (plan->num_levels == ADASUM_MAX_LEVELS)
            return false;
        int radix = plan->num_levels == 0 ? first : later;
        if (radix == 0)
            radix = 4;
        if (radix > pow2_ceil(m))
            radix = pow2_ceil(m);
        Level& lv = plan->level[plan->num_levels++];
        lv.radix = radix;
        lv.operands = m;
        lv.groups = (m + radix - 1) / radix;
        m = lv.groups;
    }
    return true;
}

int segment_length_f64(int64_t total) { return total >= (int64_t(1) << 22) ? 4096 : 1024; }

Layout make_layout_f64(const LevelPlan& plan, int64_t total_elems, int32_t num_tensors)
{
    Layout lay;
    lay.padded_elems = (total_elems + 63) / 64 * 64;
    const size_t tensors = (size_t)(num_tensors > 0 ? num_tensors : 1);
    for (int l = 0; l < plan.num_levels; ++l) {
        const Level& lv = plan.level[l];
        const size_t p = (size_t)segment_bound(total_elems, num_tensors, segment_length_f64(total_elems)) * lv.groups *
                         gram_entries(lv.radix) * sizeof(double);
        const size_t w = tensors * lv.groups * lv.radix * sizeof(double);
        const size_t c = (tensors * lv.groups + 1) * sizeof(int);
        lay.partials_bytes = p > lay.partials_bytes ? p : lay.partials_bytes;
        lay.weights_bytes = w > lay.weights_bytes ? w : lay.weights_bytes;
        lay.counters_bytes = c > lay.counters_bytes ? c : lay.counters_bytes;
        if (l + 1 < plan.num_levels) {
            const size_t b = (size_t)lv.groups * lay.padded_elems * sizeof(double);
            if (b > lay.buffer_bytes[l & 1])
                lay.buffer_bytes[l & 1] = b;
        }
    }
    if (plan.num_levels > 0)
        lay.leaf_sums_bytes = tensors * plan.level[0].groups * sizeof(double);
    size_t off = 0;
    lay.partials = off;
    off += align_up(lay.partials_bytes);
    lay.weights = off;
    off += align_up(lay.weights_bytes);
    lay.counters = off;
    off += align_up(lay.counters_bytes);
    lay.leaf_sums = off;
    off += align_up(lay.leaf_sums_bytes);
    lay.buffer[0] = off;
    off += align_up(lay.buffer_bytes[0]);
    lay.buffer[1] = off;
    off += align_up(lay.buffer_bytes[1]);
    lay.total = off > 0 ? off : kAlign;
    return lay;
}

struct LevelArgsF64 {
    const void* const* operand_ptrs;
    int operands, groups;
    const SegmentTable* tab;
    double* partials;
    FinishArgsF64 fin;
    void* dst;
    int64_t dst_stride;
    const double* start;     // first level of the delta form
    const double* base;      // last level of the delta form
    int out_f32;             // last level storing floats
    bool vec;
    cudaStream_t stream;
    int level;
};

template <int R>
adasum_status_t run_level_f64(const LevelArgsF64& a)
{
    constexpr int kGroupsPerLaunch = kMaxOperandsPerLaunch / R;
    for (int pass = 0; pass < 2; ++pass) {
        for (int g0 = 0; g0 < a.groups; g0 += kGroupsPerLaunch) {
            const int groups_here = a.groups - g0 < kGroupsPerLaunch ? a.groups - g0 : kGroupsPerLaunch;
            const int op0 = g0 * R;
            const int ops_here = a.operands - op0 < kMaxOperandsPerLaunch ? a.operands - op0 : kMaxOperandsPerLaunch;
            OperandTable table;
            for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
                table.ptr[i] = a.operand_ptrs[op0 + (i < ops_here ? i : 0)];
            dim3 grid((unsigned)a.tab->num_segments, (unsigned)groups_here);
            if (pass == 0) {
                if (a.vec)
                    gram_partial_f64_kernel<R, true><<<grid, kThreads, 0, a.stream>>>(
                        table, ops_here, a.tab->d_segments, a.partials, a.groups, g0, a.fin, a.start);
                else
                    gram_partial_f64_kernel<R, false><<<grid, kThreads, 0, a.stream>>>(
                        table, ops_here, a.tab->d_segments, a.partials, a.groups, g0, a.fin, a.start);
                profile_mark(a.stream, ADASUM_KERNEL_GRAM_PARTIAL, a.level, R, false);
            } else {
                if (a.vec)
                    weighted_sum_f64_kernel<R, true><<<grid, kThreads, 0, a.stream>>>(
                        table, ops_here, a.tab->d_segments, a.fin.weights, a.groups, g0, a.dst, a.dst_stride, a.start,
                        a.base, a.out_f32);
                else
                    weighted_sum_f64_kernel<R, false><<<grid, kThreads, 0, a.stream>>>(
                        table, ops_here, a.tab->d_segments, a.fin.weights, a.groups, g0, a.dst, a.dst_stride, a.start,
                        a.base, a.out_f32);
                profile_mark(a.stream, ADASUM_KERNEL_WEIGHTED_SUM, a.level, R, false);
            }
        }
    }
    ADASUM_CUDA_CHECK(cudaGetLastError());
    return ADASUM_OK;
}

// grads, start and (unless out_dtype is fp32) out hold doubles.
adasum_status_t reduce_f64_impl(const void* const* grads, const int64_t* offsets, int32_t num_tensors,
                                int32_t n_workers, void* out, adasum_dtype_t out_dtype, float* orthogonality,
                                void* workspace, size_t workspace_bytes, uint32_t flags, cudaStream_t stream,
                                const void* start)
{
    g_error[0] = '\0';
    if (!grads)
        return fail(ADASUM_ERR_NULL, "grads is NULL");
    if (orthogonality && n_workers < 2)
        return fail(ADASUM_ERR_ARG, "the orthogonality measure needs at least two workers");
    if (reinterpret_cast<uintptr_t>(orthogonality) & 3u)
        return fail(ADASUM_ERR_ARG, "orthogonality is not 4-byte aligned");
    adasum_status_t st = check_common(offsets, num_tensors, n_workers, ADASUM_F64);
    if (st != ADASUM_OK)
        return st;
    if (out_dtype != ADASUM_F64 && out_dtype != ADASUM_F32)
        return fail(ADASUM_ERR_DTYPE, "fp64 inputs are reduced to an fp64 or fp32 output");
    LevelPlan plan;
    if (!plan_levels_f64(n_workers, flags, &plan))
        return fail(ADASUM_ERR_ARG, "invalid flags 0x%x for %d fp64 workers (radix 2 or 4, binary tree only)", flags,
                    n_workers);
    const int64_t total = offsets[num_tensors];
    if (total == 0)
        return ADASUM_OK;
    if (!out)
        return fail(ADASUM_ERR_NULL, "out is NULL");
    const int out_f32 = out_dtype == ADASUM_F32;
    if (reinterpret_cast<uintptr_t>(out) & (uintptr_t)(out_f32 ? 3 : 7))
        return fail(ADASUM_ERR_ARG, "out is not aligned to its element size");
    const size_t in_bytes = (size_t)total * 8, out_bytes = (size_t)total * (out_f32 ? 4 : 8);
    bool vec = aligned16(out);
    if (start != nullptr) {
        if (reinterpret_cast<uintptr_t>(start) & 7u)
            return fail(ADASUM_ERR_ARG, "start is not 8-byte aligned");
        const bool in_place = out == start && !out_f32;
        if (!in_place && ranges_overlap(start, in_bytes, out, out_bytes))
            return fail(ADASUM_ERR_ARG, "out overlaps start without being the same buffer of the same type");
        vec = vec && aligned16(start);
    }
    for (int w = 0; w < n_workers; ++w) {
        if (!grads[w])
            return fail(ADASUM_ERR_NULL, "grads[%d] is NULL", w);
        if (reinterpret_cast<uintptr_t>(grads[w]) & 7u)
            return fail(ADASUM_ERR_ARG, "grads[%d] is not aligned to its element size", w);
        if (ranges_overlap(grads[w], in_bytes, out, out_bytes))
            return fail(ADASUM_ERR_ARG, "out overlaps grads[%d]", w);
        if (start != nullptr && ranges_overlap(start, in_bytes, grads[w], in_bytes))
            return fail(ADASUM_ERR_ARG, "start overlaps grads[%d]", w);
        vec = vec && aligned16(grads[w]);
    }
    const Layout lay = make_layout_f64(plan, total, num_tensors);
    if (n_workers > 1) {
        if (!workspace)
            return fail(ADASUM_ERR_WORKSPACE, "workspace is NULL");
        if (workspace_bytes < lay.total)
            return fail(ADASUM_ERR_WORKSPACE, "workspace has %zu bytes, need %zu", workspace_bytes, lay.total);
        if (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1))
            return fail(ADASUM_ERR_ARG, "workspace is not %zu-byte aligned", kAlign);
        if (ranges_overlap(workspace, lay.total, out, out_bytes))
            return fail(ADASUM_ERR_ARG, "workspace overlaps out");
        for (int w = 0; w < n_workers; ++w)
            if (ranges_overlap(workspace, lay.total, grads[w], in_bytes))
                return fail(ADASUM_ERR_ARG, "workspace overlaps grads[%d]", w);
        if (start != nullptr && ranges_overlap(workspace, lay.total, start, in_bytes))
            return fail(ADASUM_ERR_ARG, "workspace overlaps start");
    }
    profile_mark(stream, -1, 0, 0, true);
    if (n_workers == 1) {
        const int64_t blocks = (total + kThreads - 1) / kThreads;
        const unsigned grid = (unsigned)(blocks < 148 * 16 ? blocks : 148 * 16);
        convert_f64_kernel<<<grid, kThreads, 0, stream>>>(static_cast<const double*>(grads[0]), out, total,
                                                          static_cast<const double*>(start), out_f32);
        ADASUM_CUDA_CHECK(cudaGetLastError());
        profile_mark(stream, ADASUM_KERNEL_CONVERT, 0, 1, false);
        return ADASUM_OK;
    }
    char* ws = static_cast<char*>(workspace);
    ADASUM_CUDA_CHECK(cudaMemsetAsync(ws + lay.counters, 0, lay.counters_bytes, stream));
    if (orthogonality && num_tensors > 0)
        ADASUM_CUDA_CHECK(cudaMemsetAsync(orthogonality, 0xff, sizeof(float) * (size_t)num_tensors, stream));
    if (num_tensors == 0)
        return ADASUM_OK;
    const SegmentTable* tab = nullptr;
    st = get_segment_table(offsets, num_tensors, segment_length_f64(total), &tab);
    if (st != ADASUM_OK)
        return st;
    // per-launch timing: the first kernel's interval starts here, after the clearing of counters above
    profile_mark(stream, -1, 0, 0, true);
    std::vector<const void*> operand_ptrs(grads, grads + n_workers);
    for (int l = 0; l < plan.num_levels; ++l) {
        const Level& lv = plan.level[l];
        const bool last = l + 1 == plan.num_levels;
        LevelArgsF64 a;
        a.operand_ptrs = operand_ptrs.data();
        a.operands = lv.operands;
        a.groups = lv.groups;
        a.tab = tab;
        a.partials = reinterpret_cast<double*>(ws + lay.partials);
        a.fin.seg_first = tab->d_seg_first;
        a.fin.counters = reinterpret_cast<int*>(ws + lay.counters);
        a.fin.weights = reinterpret_cast<double*>(ws + lay.weights);
        a.fin.tree = TreeOptions{0, l == 0, last, plan.level[0].groups,
                                 orthogonality ? reinterpret_cast<double*>(ws + lay.leaf_sums) : nullptr, orthogonality};
        a.dst = last ? out : static_cast<void*>(ws + lay.buffer[l & 1]);
        a.dst_stride = last ? 0 : lay.padded_elems;
        a.start = l == 0 ? static_cast<const double*>(start) : nullptr;
        a.base = last ? static_cast<const double*>(start) : nullptr;
        a.out_f32 = last ? out_f32 : 0;
        a.vec = vec;
        a.stream = stream;
        a.level = l;
        st = lv.radix == 2 ? run_level_f64<2>(a) : run_level_f64<4>(a);
        if (st != ADASUM_OK)
            return st;
        if (!last) {
            operand_ptrs.resize((size_t)lv.groups);
            for (int g = 0; g < lv.groups; ++g)
                operand_ptrs[g] = static_cast<double*>(a.dst) + (int64_t)g * lay.padded_elems;
        }
    }
    return ADASUM_OK;
}

// ---- pair operator without any device allocation -------------------------------------------------
//
// Scratch for adasum_pair_noalloc: the segment table, the per-segment partial sums and the
// per-tensor coefficients live in one file-scope device array that every GPU loading this library
// holds until the process exits.  In host code `g_noalloc_scratch` is only a handle for
// cudaGetSymbolAddress; the kernels receive the device address obtained from it.

constexpr int64_t kNoallocMaxElems = ADASUM_NOALLOC_MAX_ELEMS;
constexpr int32_t kNoallocMaxTensors = ADASUM_NOALLOC_MAX_TENSORS;
constexpr int kNoallocSegLen = 8192;
constexpr int64_t kNoallocMaxSegments = kNoallocMaxElems / kNoallocSegLen + 2 * (int64_t)kNoallocMaxTensors + 1;
constexpr size_t kNoallocSegBytes = ((size_t)kNoallocMaxSegments * sizeof(Segment) + 255) / 256 * 256;
constexpr size_t kNoallocFirstBytes = ((size_t)(2 * kNoallocMaxTensors + 2) * sizeof(int32_t) + 255) / 256 * 256;
constexpr size_t kNoallocPartialBytes = ((size_t)kNoallocMaxSegments * gram_entries(2) * sizeof(float) + 255) / 256 * 256;
constexpr size_t kNoallocWeightBytes = ((size_t)kNoallocMaxTensors * 2 * sizeof(float) + 255) / 256 * 256;
constexpr size_t kNoallocScratchBytes = kNoallocSegBytes + kNoallocFirstBytes + kNoallocPartialBytes + kNoallocWeightBytes;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocScratchBytes];

constexpr int kNoallocMaxDevices = 64;
std::mutex g_noalloc_mutex;
unsigned char* g_noalloc_device_ptr[kNoallocMaxDevices] = {};

// Device address of the scratch array on the current device (looked up once per device).
adasum_status_t noalloc_scratch(unsigned char** ptr)
{
    int device = 0;
    ADASUM_CUDA_CHECK(cudaGetDevice(&device));
    if (device < 0 || device >= kNoallocMaxDevices)
        return fail(ADASUM_ERR_ARG, "device index %d is beyond the %d devices this entry point tracks", device,
                    kNoallocMaxDevices);
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_device_ptr[device]) {
        void* addr = nullptr;
        ADASUM_CUDA_CHECK(cudaGetSymbolAddress(&addr, g_noalloc_scratch));
        g_noalloc_device_ptr[device] = static_cast<unsigned char*>(addr);
    }
    *ptr = g_noalloc_device_ptr[device];
    return ADASUM_OK;
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

adasum_status_t pair_noalloc_impl(const void* a, const void* b, const int64_t* offsets, int32_t num_tensors,
                                  adasum_dtype_t dtype, float* out, cudaStream_t stream)
{
    g_error[0] = '\0';
    if (!a || !b)
        return fail(ADASUM_ERR_NULL, "an input pointer is NULL");
    adasum_status_t st = check_common(offsets, num_tensors, 2, dtype);
    if (st != ADASUM_OK)
        return st;
    if (dtype == ADASUM_F64)
        return fail(ADASUM_ERR_DTYPE, "adasum_pair_noalloc takes fp32, fp16 or bf16 inputs");
    const int64_t total = offsets[num_tensors];
    if (num_tensors > kNoallocMaxTensors)
        return fail(ADASUM_ERR_ARG, "num_tensors = %d exceeds the static scratch limit of %d tensors", num_tensors,
                    kNoallocMaxTensors);
    if (total > kNoallocMaxElems)
        return fail(ADASUM_ERR_ARG, "%lld elements exceed the static scratch limit of %lld elements",
                    (long long)total, (long long)kNoallocMaxElems);
    if (total == 0)
        return ADASUM_OK;
    if (!out)
        return fail(ADASUM_ERR_NULL, "out is NULL");
    if (reinterpret_cast<uintptr_t>(out) & 3u)
        return fail(ADASUM_ERR_ARG, "out is not 4-byte aligned");
    const int eb = dtype_bytes(dtype);
    const size_t in_bytes = (size_t)total * eb, out_bytes = (size_t)total * sizeof(float);
    const void* in[2] = {a, b};
    bool vec = aligned16(out);
    for (int w = 0; w < 2; ++w) {
        if (reinterpret_cast<uintptr_t>(in[w]) & (uintptr_t)(eb - 1))
            return fail(ADASUM_ERR_ARG, "input %d is not aligned to its element size", w);
        if (ranges_overlap(in[w], in_bytes, out, out_bytes))
            return fail(ADASUM_ERR_ARG, "out overlaps input %d", w);
        vec = vec && aligned16(in[w]);
    }

    unsigned char* scratch = nullptr;
    st = noalloc_scratch(&scratch);
    if (st != ADASUM_OK)
        return st;
    SegmentTable tab;                       // host-side only; its device pointers aim into the scratch
    build_segments(offsets, num_tensors, kNoallocSegLen, &tab);
    if ((int64_t)tab.num_segments > kNoallocMaxSegments)
        return fail(ADASUM_ERR_ARG, "segment table does not fit the static scratch");
    tab.d_segments = reinterpret_cast<Segment*>(scratch);
    tab.d_seg_first = reinterpret_cast<int32_t*>(scratch + kNoallocSegBytes);
    float* partials = reinterpret_cast<float*>(scratch + kNoallocSegBytes + kNoallocFirstBytes);
    float* weights = reinterpret_cast<float*>(scratch + kNoallocSegBytes + kNoallocFirstBytes + kNoallocPartialBytes);
    // The host vectors are pageable memory: cudaMemcpyAsync has read them completely when it
    // returns, and the copies are ordered before the kernels on `stream`.
    ADASUM_CUDA_CHECK(cudaMemcpyAsync(tab.d_segments, tab.h_segments.data(), sizeof(Segment) * tab.h_segments.size(),
                                      cudaMemcpyHostToDevice, stream));
    ADASUM_CUDA_CHECK(cudaMemcpyAsync(tab.d_seg_first, tab.h_seg_first.data(),
                                      sizeof(int32_t) * tab.h_seg_first.size(), cudaMemcpyHostToDevice, stream));
    OperandTable ops;
    for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
        ops.ptr[i] = in[i < 2 ? i : 0];
    if (dtype == ADASUM_F32)
        ADASUM_CUDA_CHECK(noalloc_launch<float>(vec, ops, tab, num_tensors, partials, weights, out, stream));
    else if (dtype == ADASUM_F16)
        ADASUM_CUDA_CHECK(noalloc_launch<__half>(vec, ops, tab, num_tensors, partials, weights, out, stream));
    else
        ADASUM_CUDA_CHECK(noalloc_launch<__nv_bfloat16>(vec, ops, tab, num_tensors, partials, weights, out, stream));
    ADASUM_CUDA_CHECK(cudaGetLastError());
    return ADASUM_OK;
}

}  // namespace
}  // namespace adasum

extern "C" {

size_t adasum_workspace_bytes(int64_t total_elems, int32_t num_tensors, int32_t n_workers,
                              adasum_dtype_t dtype, uint32_t flags)
{
    using namespace adasum;
    if (total_elems < 0 || num_tensors < 0 || n_workers < 1 || n_workers > ADASUM_MAX_WORKERS)
        return 0;
    if (!known_dtype(dtype))
        return 0;
    LevelPlan plan;
    if (dtype == ADASUM_F64)
        return plan_levels_f64(n_workers, flags, &plan) ? make_layout_f64(plan, total_elems, num_tensors).total : 0;
    if (!plan_levels(n_workers, dtype, flags, &plan))
        return 0;
    return make_layout(plan, total_elems, num_tensors).total;
}

adasum_status_t adasum_plan_info(int64_t total_elems, int32_t num_tensors, int32_t n_workers,
                                 adasum_dtype_t dtype, uint32_t flags, int32_t* radices,
                                 int32_t* num_levels, int32_t* num_launches)
{
    using namespace adasum;
    g_error[0] = '\0';
    if (total_elems < 0 || num_tensors < 0 || n_workers < 1 || n_workers > ADASUM_MAX_WORKERS)
        return fail(ADASUM_ERR_ARG, "invalid sizes");
    if (!known_dtype(dtype))
        return fail(ADASUM_ERR_DTYPE, "unknown dtype %d", (int)dtype);
    LevelPlan plan;
    if (dtype == ADASUM_F64 ? !plan_levels_f64(n_workers, flags, &plan) : !plan_levels(n_workers, dtype, flags, &plan))
        return fail(ADASUM_ERR_ARG, "invalid flags 0x%x", flags);
    if (radices)
        for (int l = 0; l < plan.num_levels; ++l)
            radices[l] = plan.level[l].radix;
    if (num_levels)
        *num_levels = plan.num_levels;
    if (num_launches) {
        // fp64: every level is two passes, nothing fused
        const uint32_t count_flags = dtype == ADASUM_F64 ? (flags | ADASUM_FLAG_NO_LEVEL_FUSION) : flags;
        *num_launches = total_elems == 0 ? 0
                                         : launches_of(plan, n_workers, count_flags, dtype == ADASUM_F64 ? -1 : total_elems,
                                                       num_tensors, dtype_bytes(dtype));
    }
    return ADASUM_OK;
}

adasum_status_t adasum_reduce(const void* const* grads, const int64_t* tensor_offsets,
                              int32_t num_tensors, int32_t n_workers, adasum_dtype_t dtype,
                              float* out, void* workspace, size_t workspace_bytes, uint32_t flags,
                              void* stream)
{
    if (dtype == ADASUM_F64)
        return adasum::reduce_f64_impl(grads, tensor_offsets, num_tensors, n_workers, out, ADASUM_F32, nullptr,
                                       workspace, workspace_bytes, flags, static_cast<cudaStream_t>(stream), nullptr);
    return adasum::reduce_impl(grads, tensor_offsets, num_tensors, n_workers, dtype, out, nullptr, workspace,
                               workspace_bytes, flags, static_cast<cudaStream_t>(stream));
}

adasum_status_t adasum_reduce_ex(const void* const* grads, const int64_t* tensor_offsets,
                                 int32_t num_tensors, int32_t n_workers, adasum_dtype_t dtype,
                                 float* out, float* orthogonality, void* workspace, size_t workspace_bytes,
                                 uint32_t flags, void* stream)
{
    if (dtype == ADASUM_F64)
        return adasum::reduce_f64_impl(grads, tensor_offsets, num_tensors, n_workers, out, ADASUM_F32, orthogonality,
                                       workspace, workspace_bytes, flags, static_cast<cudaStream_t>(stream), nullptr);
    return adasum::reduce_impl(grads, tensor_offsets, num_tensors, n_workers, dtype, out, orthogonality, workspace,
                               workspace_bytes, flags, static_cast<cudaStream_t>(stream));
}

adasum_status_t adasum_reduce_delta(const void* const* currents, const void* start,
                                    const int64_t* tensor_offsets, int32_t num_tensors, int32_t n_workers,
                                    adasum_dtype_t dtype, void* out, adasum_dtype_t out_dtype,
                                    float* orthogonality, void* workspace, size_t workspace_bytes, uint32_t flags,
                                    void* stream)
{
    if (dtype == ADASUM_F64)
        return adasum::reduce_f64_impl(currents, tensor_offsets, num_tensors, n_workers, out, out_dtype, orthogonality,
                                       workspace, workspace_bytes, flags, static_cast<cudaStream_t>(stream), start);
    return adasum::reduce_impl(currents, tensor_offsets, num_tensors, n_workers, dtype, out, orthogonality,
                               workspace, workspace_bytes, flags, static_cast<cudaStream_t>(stream),
                               adasum::PHASE_WHOLE, -1, nullptr, nullptr, start, out_dtype);
}

adasum_status_t adasum_sharded_gram(const void* const* grads, const int64_t* tensor_offsets,
                                    int32_t num_tensors, int32_t n_workers, adasum_dtype_t dtype,
                                    void* workspace, size_t workspace_bytes, uint32_t flags, int32_t level,
                                    size_t* sums_offset, int64_t* sums_count, void* stream)
{
    return adasum::reduce_impl(grads, tensor_offsets, num_tensors, n_workers, dtype, nullptr, nullptr, workspace,
                               workspace_bytes, flags, static_cast<cudaStream_t>(stream), adasum::PHASE_GRAM_SUMS,
                               level, sums_offset, sums_count);
}

adasum_status_t adasum_sharded_apply(const void* const* grads, const int64_t* tensor_offsets,
                                     int32_t num_tensors, int32_t n_workers, adasum_dtype_t dtype, float* out,
                                     float* orthogonality, void* workspace, size_t workspace_bytes, uint32_t flags,
                                     int32_t level, void* stream)
{
    return adasum::reduce_impl(grads, tensor_offsets, num_tensors, n_workers, dtype, out, orthogonality, workspace,
                               workspace_bytes, flags, static_cast<cudaStream_t>(stream), adasum::PHASE_APPLY, level);
}

adasum_status_t adasum_pair(const void* a, const void* b, const int64_t* tensor_offsets,
                            int32_t num_tensors, adasum_dtype_t dtype, float* out, void* workspace,
                            size_t workspace_bytes, uint32_t flags, void* stream)
{
    const void* grads[2] = {a, b};
    if (dtype == ADASUM_F64)
        return adasum::reduce_f64_impl(grads, tensor_offsets, num_tensors, 2, out, ADASUM_F32, nullptr, workspace,
                                       workspace_bytes, flags, static_cast<cudaStream_t>(stream), nullptr);
    return adasum::reduce_impl(grads, tensor_offsets, num_tensors, 2, dtype, out, nullptr, workspace,
                               workspace_bytes, flags, static_cast<cudaStream_t>(stream));
}

adasum_status_t adasum_pair_noalloc(const void* a, const void* b, const int64_t* tensor_offsets,
                                    int32_t num_tensors, adasum_dtype_t dtype, float* out, void* stream)
{
    return adasum::pair_noalloc_impl(a, b, tensor_offsets, num_tensors, dtype, out,
                                     static_cast<cudaStream_t>(stream));
}

adasum_status_t adasum_device_status(int64_t total_elems, int32_t num_tensors, int32_t n_workers,
                                     adasum_dtype_t dtype, uint32_t flags, const void* workspace, void* stream)
{
    using namespace adasum;
    g_error[0] = '\0';
    if (!workspace)
        return fail(ADASUM_ERR_NULL, "workspace is NULL");
    if (total_elems < 0 || num_tensors < 0 || n_workers < 1 || n_workers > ADASUM_MAX_WORKERS)
        return fail(ADASUM_ERR_ARG, "invalid sizes");
    if (!known_dtype(dtype))
        return fail(ADASUM_ERR_DTYPE, "unknown dtype %d", (int)dtype);
    if (dtype == ADASUM_F64)        // the fp64 kernels have no bounded waits
        return ADASUM_OK;
    LevelPlan plan;
    if (!plan_levels(n_workers, dtype, flags, &plan))
        return fail(ADASUM_ERR_ARG, "invalid flags 0x%x", flags);
    const Layout lay = make_layout(plan, total_elems, num_tensors);
    if (lay.counters_bytes < sizeof(int))
        return ADASUM_OK;
    int word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ADASUM_CUDA_CHECK(cudaMemcpyAsync(&word, static_cast<const char*>(workspace) + lay.counters + lay.counters_bytes -
                                                 sizeof(int),
                                      sizeof(int), cudaMemcpyDeviceToHost, s));
    ADASUM_CUDA_CHECK(cudaStreamSynchronize(s));
    if (word == ADASUM_DEVICE_TIMEOUT)
        return fail(ADASUM_ERR_TIMEOUT, "a bounded wait on the tensor core ran out");
    return ADASUM_OK;
}

const char* adasum_status_string(adasum_status_t status)
{
    switch (status) {
    case ADASUM_OK: return "ADASUM_OK";
    case ADASUM_ERR_NULL: return "ADASUM_ERR_NULL";
    case ADASUM_ERR_ARG: return "ADASUM_ERR_ARG";
    case ADASUM_ERR_OFFSETS: return "ADASUM_ERR_OFFSETS";
    case ADASUM_ERR_DTYPE: return "ADASUM_ERR_DTYPE";
    case ADASUM_ERR_WORKSPACE: return "ADASUM_ERR_WORKSPACE";
    case ADASUM_ERR_CUDA: return "ADASUM_ERR_CUDA";
    case ADASUM_ERR_TIMEOUT: return "ADASUM_ERR_TIMEOUT";
    }
    return "ADASUM_ERR_UNKNOWN";
}

const char* adasum_last_error(void) { return adasum::g_error; }

adasum_status_t adasum_profile_enable(int32_t max_launches)
{
    using namespace adasum;
    g_error[0] = '\0';
    if (max_launches < 1)
        return fail(ADASUM_ERR_ARG, "max_launches must be positive");
    std::lock_guard<std::mutex> lock(g_profiler_mutex);
    g_profiler.enabled = false;
    const size_t want = (size_t)max_launches * 3;    // room for the two call-opening events of every reduce too
    while (g_profiler.events.size() < want) {
        cudaEvent_t ev;
        cudaError_t err = cudaEventCreate(&ev);
        if (err != cudaSuccess)
            return fail(ADASUM_ERR_CUDA, "cudaEventCreate: %s", cudaGetErrorString(err));
        g_profiler.events.push_back(ev);
    }
    g_profiler.marks.resize(g_profiler.events.size());
    g_profiler.used = 0;
    g_profiler.overflow = false;
    g_profiler.enabled = true;
    return ADASUM_OK;
}

adasum_status_t adasum_profile_collect(adasum_launch_record_t* records, int32_t capacity, int32_t* count)
{
    using namespace adasum;
    g_error[0] = '\0';
    if (!count || (capacity > 0 && !records))
        return fail(ADASUM_ERR_NULL, "records / count is NULL");
    std::lock_guard<std::mutex> lock(g_profiler_mutex);
    g_profiler.enabled = false;
    int32_t n = 0;
    if (g_profiler.used > 0) {
        cudaError_t err = cudaEventSynchronize(g_profiler.events[g_profiler.used - 1]);
        if (err != cudaSuccess)
            return fail(ADASUM_ERR_CUDA, "cudaEventSynchronize: %s", cudaGetErrorString(err));
    }
    for (size_t i = 1; i < g_profiler.used; ++i) {
        const ProfileMark& m = g_profiler.marks[i];
        if (m.starts_call)
            continue;
        float ms = 0.0f;
        cudaError_t err = cudaEventElapsedTime(&ms, g_profiler.events[i - 1], g_profiler.events[i]);
        if (err != cudaSuccess)
            return fail(ADASUM_ERR_CUDA, "cudaEventElapsedTime: %s", cudaGetErrorString(err));
        if (n < capacity)
            records[n] = adasum_launch_record_t{m.kernel, m.level, m.radix, ms};
        ++n;
    }
    *count = n;
    const bool overflow = g_profiler.overflow;
    g_profiler.used = 0;
    g_profiler.overflow = false;
    if (overflow)
        return fail(ADASUM_ERR_ARG, "more launches than adasum_profile_enable() reserved; records are incomplete");
    return ADASUM_OK;
}

adasum_status_t adasum_shutdown(void)
{
    using namespace adasum;
    g_error[0] = '\0';
    {
        std::lock_guard<std::mutex> plock(g_profiler_mutex);
        g_profiler.enabled = false;
        for (cudaEvent_t ev : g_profiler.events)
            cudaEventDestroy(ev);
        g_profiler.events.clear();
        g_profiler.marks.clear();
        g_profiler.used = 0;
    }
    std::lock_guard<std::mutex> lock(g_tables_mutex);
    if (g_tables.empty())
        return ADASUM_OK;
    int current = 0;
    cudaError_t err = cudaGetDevice(&current);
    bool ok = err == cudaSuccess;
    for (auto& tab : g_tables) {
        if (ok && cudaSetDevice(tab->device) == cudaSuccess) {
            if (cudaFree(tab->d_segments) != cudaSuccess || cudaFree(tab->d_seg_first) != cudaSuccess)
                ok = false;
        } else {
            ok = false;
        }
    }
    g_tables.clear();
    if (err == cudaSuccess)
        cudaSetDevice(current);
    return ok ? ADASUM_OK : fail(ADASUM_ERR_CUDA, "adasum_shutdown: a CUDA call failed");
}

}  // extern "C"
