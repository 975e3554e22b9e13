// Interfaces between the translation units of the library (host side only; not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "adasum.h"

#include "adasum_kernels.cuh"

namespace adasum {

// ---- errors and per-launch timing (adasum_api.cu) ---------------------------------------------------

// Records the message for adasum_last_error() on the calling thread and returns `status`.
adasum_status_t fail(adasum_status_t status, const char* fmt, ...);

#define ADASUM_CUDA_CHECK(expr)                                                                  \
    do {                                                                                         \
        cudaError_t err__ = (expr);                                                              \
        if (err__ != cudaSuccess)                                                                \
            return ::adasum::fail(ADASUM_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(err__));  \
    } while (0)

// While per-launch timing is enabled: records an event on `stream` that closes the launch just made
// (or, with starts_call, opens a reduce call).
void profile_mark(cudaStream_t stream, int kernel, int level, int radix, bool starts_call);

// ---- tensors short enough to be reduced in fp64 from end to end (adasum_short.cu) -----------------

constexpr int kShortTensorElems = 64;            // tensors of at most this many elements take the fp64 path
constexpr int kShortChunkLeaves = 64;            // leaves a block reduces per round in shared memory

struct ShortArgs {
    const ShortTensor* table;     // device, one entry per short tensor (= per block)
    int order;                    // 0 bottom-up pairs with carry, 1 sequential, 2 top-down halves
    const void* start;            // delta form: every leaf is (operand - start), rounded to the operands' type
    // dynamic scaling: operand i of this launch is worker worker_base + i, whose buffer holds
    // leaf_scales[worker * num_tensors + tensor] times its gradient; nullptr: the gradients themselves
    const float* leaf_scales;
    int num_tensors, worker_base;
    // destination of this launch: either the final result ...
    void* out;                    // elements of out_dtype, indexed like the inputs; nullptr: not the final launch
    const void* base;             // added to the result (the delta form's start), or nullptr
    int base_dtype, out_dtype;    // 0 fp32, 1 fp16, 2 bf16
    float* orthogonality;         // [tensor], or nullptr
    // ... or the fp64 vector of this launch's sub-tree and the sum of its leaves' squared norms
    double* vec_out;              // [packed element]
    double* leaf_sum_out;         // [short tensor]
    // final launch over earlier launches' vectors: their leaf sums, `leaf_sum_launches` arrays
    // `leaf_sum_stride` doubles apart (nullptr: the leaves of this launch are the workers' gradients)
    const double* leaf_sum_in;    // set: the operands are such vectors, indexed by packed element
    int leaf_sum_launches;
    int64_t leaf_sum_stride;
};

// dtype: 0 fp32, 1 fp16, 2 bf16, 3 fp64 (the vectors of earlier launches).  `operands` <=
// kMaxOperandsPerLaunch leaves per tensor, taken from ops.ptr[0 .. operands).
cudaError_t launch_short_tensors(int dtype, const OperandTable& ops, int operands, int num_short,
                                 const ShortArgs& args, cudaStream_t stream);


// ---- what the level launchers (adasum_levels.cuh, one translation unit per element type) share
// ---- with the host logic (adasum_api.cu) ---------------------------------------------------------

// Which Gram kernel serves a level.
enum GramKind {
    GRAM_SIMPLE,      // fp32 pipes, operands in registers (radix <= 4; radix 8 and 16 on request)
    GRAM_MMA          // tensor cores (radix >= 8)
};

inline GramKind gram_kind(int radix, bool simple_kernels)
{
    return (radix >= 32 || (radix >= 8 && !simple_kernels)) ? GRAM_MMA : GRAM_SIMPLE;
}


struct SegmentTable {
    int device = -1;
    int seg_len = 0;
    std::vector<int64_t> offsets;
    Segment* d_segments = nullptr;
    int32_t* d_seg_first = nullptr;
    // d_seg_first + 2 * num_tensors + 2: per tensor of more than kSegmentsPerGroup segments the number
    // of its first run of that many segments (runs are numbered through those tensors; the two-step
    // finish keeps a counter and a sum per run); the same allocation
    int32_t* d_group_first = nullptr;
    int32_t num_runs = 0;
    bool owns_device_arrays = false;    // false: the arrays belong to somebody else (static scratch)
    int32_t num_segments = 0;
    int32_t max_segments_per_tensor = 0;
    std::vector<Segment> h_segments;
    std::vector<int32_t> h_seg_first;
    // Tensors of at most kShortTensorElems elements, when they are left to short_tensor_kernel:
    // they have no segments, and are listed here instead.
    bool skip_short = false;
    ShortTensor* d_short = nullptr;
    int64_t short_elems = 0;
    std::vector<ShortTensor> h_short;
    // Tensors of at most warp_limit elements (beyond the short ones), when the single-launch kernel
    // gives each of them to one warp: no segments either.
    int warp_limit = 0;
    // Tapered cutting (shorter segments at both ends of the table): what the table was asked for
    // (part of its identity in the cache) and what it was built with (0 if the buffer is too short).
    int taper_request = 0, taper_slots = 0;
    WarpTensor* d_warp = nullptr;
    std::vector<WarpTensor> h_warp;

    SegmentTable() = default;
    SegmentTable(const SegmentTable&) = delete;
    SegmentTable& operator=(const SegmentTable&) = delete;
    ~SegmentTable()
    {
        if (!owns_device_arrays || (!d_segments && !d_seg_first && !d_short && !d_warp))
            return;
        int current = 0;
        const bool have_current = cudaGetDevice(&current) == cudaSuccess;
        if (have_current && current != device)
            cudaSetDevice(device);
        cudaFree(d_segments);
        cudaFree(d_seg_first);
        cudaFree(d_short);
        cudaFree(d_warp);
        if (have_current && current != device)
            cudaSetDevice(current);
    }
};


// Which part of a level a call runs.
enum LevelPhase {
    PHASE_WHOLE = 0,        // pass 1, coefficients, pass 2
    PHASE_GRAM_SUMS = 1,    // pass 1, then this GPU's fp64 Gram sums to gram64 (to be added across GPUs)
    PHASE_APPLY = 2         // coefficients from gram64, then pass 2
};

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
    int* run_counters;  // zeroed, one per (run of segments, group): the two-step finish of long tensors
    double* run_sums;   // [run][group][entries of the Gram matrix]
    TreeOptions tree;
    LevelPhase phase;
    int* tc_status;     // status word for the tcgen05 kernel, or nullptr to keep to mma.sync
    bool selftest_timeout;   // ADASUM_FLAG_SELFTEST_TIMEOUT
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
inline bool fusable_radices(int radix, int next_radix) { return radix <= 4 && (next_radix == 2 || next_radix == 4); }

constexpr PassExtras kNoExtras{nullptr, nullptr, 0, 0};

// One level of a reduce whose operands have element type T (float, __half, __nv_bfloat16).
template <typename T>
adasum_status_t run_level(int radix, const LevelArgs& a);

// Both passes of a one-level reduce in one cooperative launch (fused_small_kernel), radix 2, 4 or 8.
template <typename T>
cudaError_t launch_fused_small_any(bool vec, int radix, const OperandTable& ops, int operands,
                                   const SegmentTable& tab, int resident_blocks, float* partials,
                                   const FinishArgs& fin, void* out, const PassExtras& ex, int* status,
                                   cudaStream_t stream);

// The three launches of adasum_pair_noalloc (pass 1, coefficients, pass 2), nothing fused.
template <typename T>
cudaError_t noalloc_launch(bool vec, const OperandTable& ops, const SegmentTable& tab, int32_t num_tensors,
                           float* partials, float* weights, float* out, cudaStream_t stream);

// n_workers = 1: convert (and, in the delta form, start + (input - start)).
template <typename T>
cudaError_t launch_convert(const void* src, void* dst, int64_t n, const PassExtras& ex, cudaStream_t stream);

}  // namespace adasum
