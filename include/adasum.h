/*
 * adasum.h — C ABI of the B200 (sm_100a) N-way Adasum combine.
 *
 * The operation (arXiv 2006.02924, Section 3 and Section 3.4; Algorithm 1 for the order):
 *
 *     Adasum(a, b) = (1 - a.b / (2 |a|^2)) a  +  (1 - a.b / (2 |b|^2)) b
 *
 * applied recursively over a binary tree whose first level pairs workers (2i, 2i+1), whose
 * second level pairs the results of blocks of two, and so on, independently for every tensor
 * (layer) of a fused gradient buffer (Section 3.6, Section 4.4.3).  |g|^2 is the squared L2
 * norm.  An operand whose squared norm is exactly zero contributes nothing and leaves the
 * other operand unchanged.  If the operand count at a level is odd, the last operand is
 * carried to the next level unchanged (the paper itself only treats powers of two).
 *
 * All N worker buffers live in the memory of ONE GPU.  Dot products and norms are accumulated
 * in fp32 inside blocks of at most a few thousand elements per thread block and in fp64 across
 * blocks (Section 4.4.1 asks for accumulation wider than the gradient type); all coefficient
 * arithmetic is fp64 on the device; intermediates between levels and the output are fp32.
 * Tensors of at most 64 elements are the exception: their result can be a small difference of
 * large terms (a one-element tensor whose workers disagree in sign), so adasum_reduce,
 * adasum_reduce_ex, adasum_reduce_scaled, adasum_reduce_delta and adasum_pair apply the operator to them literally, pair
 * by pair and level by level, in fp64 from the loads to the one rounding of the stored result (one
 * more small kernel when a buffer has such tensors, run beside the streaming passes on a stream of
 * the library's own that is forked from `stream` and joined to it again with events before the call
 * returns; the single-launch path does them inside its one kernel; the sharded calls, whose tensors
 * are spread over several GPUs, keep to the general path).
 *
 * Conventions for every entry point:
 *   - plain C, no exceptions; every call returns a status, and on any status other than
 *     ADASUM_OK nothing has been launched unless stated otherwise;
 *   - "device" pointers are CUDA device addresses on the current device, "host" pointers are
 *     ordinary host memory that is only read during the call;
 *   - the caller owns every buffer; inputs are never written; `out` and `workspace` must not
 *     overlap any input or each other;
 *   - calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = legacy
 *     default stream) and never synchronise it;
 *   - the library allocates nothing per call.  The first call with a tensor-offset table it
 *     has not seen on the current device builds a small segment table on the device
 *     (cudaMalloc plus a blocking copy); later calls with the same table reuse it.  The cache
 *     keeps the most recently used tables, up to 256 of them and 256 MB of device memory; a
 *     call that needs a new table beyond that drops the least recently used ones, and freeing
 *     them (cudaFree) waits for all work already submitted to the device.  A caller whose
 *     tensor grouping changes on every call therefore pays an allocation, a blocking copy and,
 *     once the cache is full, a device-wide wait per call; keep the set of offset tables small
 *     where that matters.  adasum_shutdown() frees them all.  A call that builds a table must
 *     not be made while the stream is being captured into a CUDA graph;
 *   - results are deterministic: the same inputs, sizes and flags give the same bits.
 */
#ifndef ADASUM_H_
#define ADASUM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Element type of the worker gradients.  adasum_reduce, adasum_reduce_ex and adasum_pair write
 * fp32 for every input type; adasum_reduce_delta takes the output type as an argument.
 *
 * ADASUM_F64 (the paper's implementation serves fp16, fp32 and fp64 tensors, Section 4.4): such
 * buffers are reduced in doubles throughout (fp64 products and sums, leaf weights, intermediates)
 * by kernels of their own, in levels of radix 2 or 4 (radix fields 0, 2 or 4; 0 = 4), as the
 * bottom-up binary tree only: ADASUM_FLAG_LINEAR_ORDER, ADASUM_FLAG_TOP_DOWN_HALVES,
 * ADASUM_FLAG_SEPARATE_FINISH and ADASUM_FLAG_SIMPLE_KERNELS are refused with ADASUM_ERR_ARG.
 * The output is fp64 or fp32 (adasum_reduce_delta with out_dtype ADASUM_F64 or ADASUM_F32; the
 * calls with a float* out store fp32).  The sharded calls and adasum_pair_noalloc refuse
 * ADASUM_F64 with ADASUM_ERR_DTYPE. */
typedef enum {
    ADASUM_F32 = 0,
    ADASUM_F16 = 1,   /* IEEE binary16 */
    ADASUM_BF16 = 2,
    ADASUM_F64 = 3
} adasum_dtype_t;

typedef enum {
    ADASUM_OK = 0,
    ADASUM_ERR_NULL = 1,        /* a required pointer is NULL */
    ADASUM_ERR_ARG = 2,         /* N < 1, num_tensors < 0, bad flags, misaligned out, overlap */
    ADASUM_ERR_OFFSETS = 3,     /* offsets[0] != 0 or decreasing offsets */
    ADASUM_ERR_DTYPE = 4,       /* unknown dtype */
    ADASUM_ERR_WORKSPACE = 5,   /* workspace NULL or smaller than adasum_workspace_bytes() */
    ADASUM_ERR_CUDA = 6,        /* a CUDA runtime call or a launch failed (see adasum_last_error) */
    ADASUM_ERR_TIMEOUT = 7      /* a bounded device-side wait ran out (the waits between the copying
                                   warps and the tensor core inside the tcgen05 Gram kernel, and
                                   the flag waits inside the single-launch kernels); reported by
                                   adasum_device_status, never by the call that launched */
} adasum_status_t;

/*
 * flags: how the tree is evaluated (the RESULT is the same binary tree in every case).
 *
 * A group of R = 2^j adjacent operands is a complete sub-tree of the binary tree, and every
 * node of that sub-tree is a linear combination of its R leaves.  One "level" of this library
 * therefore reads the operands once to form each group's R x R Gram matrix per tensor, derives
 * on the device the R leaf weights that the sub-tree's recursion produces, and reads the
 * operands a second time to write the group's weighted sum.  R = 2 is the literal
 * level-by-level tree (three scalars a.b, a.a, b.b per pair, as in Algorithm 1).
 *
 *   bits 0..7    radix of the first level: 0 = choose automatically, else 2, 4, 8, 16, 32 or,
 *                for fp16 / bf16 inputs only, 64
 *   bits 8..15   radix of the later levels (their operands are fp32): 0 = same rule as the
 *                first level, else 2 ... 32
 *   bit 16       ADASUM_FLAG_SIMPLE_KERNELS: form the Gram matrices on the fp32 pipes also at
 *                radix 8 and 16 instead of on the tensor cores (radices above 16 are then refused;
 *                same results up to rounding; for comparison and debugging)
 *   bit 17       ADASUM_FLAG_SEPARATE_FINISH: add up the per-segment Gram matrices and derive
 *                the leaf weights in a kernel of their own at every level, instead of inside
 *                the first pass; for comparison and debugging
 *   bit 18       ADASUM_FLAG_LINEAR_ORDER: a DIFFERENT result, the sequential recursion of
 *                Section 3.4, Adasum(g[0..n+1]) = Adasum(Adasum(g[0..n]), g[n+1]) (the order of
 *                the paper's ring implementation), instead of the binary tree.  The running
 *                result depends on all earlier workers, so the whole reduce is one level whose
 *                Gram matrix covers every worker: n_workers <= 32 for fp32 inputs, <= 64 for
 *                fp16 / bf16; the radix fields must be 0.  Otherwise ADASUM_ERR_ARG.
 *   bit 19       ADASUM_FLAG_NO_TCGEN05: form radix-64 Gram matrices with warp-level mma.sync
 *                instead of tcgen05 and tensor memory; for comparison and debugging
 *   bit 20       ADASUM_FLAG_TOP_DOWN_HALVES: the binary tree of Section 3.4 split from the top,
 *                Adasum(g[lo, hi)) = Adasum(Adasum(g[lo, mid)), Adasum(g[mid, hi))) with mid =
 *                lo + floor((hi - lo) / 2), instead of paired bottom-up with the odd operand
 *                carried.  The two are the same tree when n_workers is a power of two (the flag
 *                then changes nothing) and a DIFFERENT result otherwise; Algorithm 1 itself is
 *                stated for powers of two only.  For other counts the whole reduce is one level
 *                (same limits as ADASUM_FLAG_LINEAR_ORDER, radix fields 0); not together with
 *                ADASUM_FLAG_LINEAR_ORDER.  Otherwise ADASUM_ERR_ARG.
 *   bit 21       ADASUM_FLAG_NO_LEVEL_FUSION: always run the second pass of a level and the first
 *                pass of the next as separate kernels.  Without the flag, when a level has radix 2
 *                or 4 and so has the next (and the buffers are 16-byte aligned), one kernel writes a level's
 *                outputs and accumulates the next level's dot products from the same registers
 *                (Algorithm 1's "apply" of one level and its dot products of the next), so the
 *                intermediate vectors are read once less.  Same results up to rounding; for
 *                comparison and debugging.
 *   bit 22       ADASUM_FLAG_SELFTEST_TIMEOUT: a self-test of the device status path, not a way to
 *                reduce.  The radix-64 tensor-memory kernel leaves every segment's last tile
 *                unmultiplied, so nothing ever releases that tile's stage, and waits for the release
 *                with a limit of microseconds instead of the usual tenth of a second.  The wait runs
 *                out, the kernel records it, frees its tensor memory and returns; the output is
 *                wrong by construction and adasum_device_status reports ADASUM_ERR_TIMEOUT.  No other
 *                kernel looks at the flag.
 */
#define ADASUM_FLAG_SELFTEST_TIMEOUT (1u << 22)
#define ADASUM_FLAG_NO_LEVEL_FUSION (1u << 21)
#define ADASUM_FLAG_NO_TCGEN05 (1u << 19)
#define ADASUM_FLAG_TOP_DOWN_HALVES (1u << 20)
#define ADASUM_FLAG_SIMPLE_KERNELS (1u << 16)
#define ADASUM_FLAG_SEPARATE_FINISH (1u << 17)
#define ADASUM_FLAG_LINEAR_ORDER (1u << 18)
#define ADASUM_RADIX_AUTO 0u
#define ADASUM_FLAGS_RADIX(first, later) (((uint32_t)(first) & 0xffu) | (((uint32_t)(later) & 0xffu) << 8))

#define ADASUM_MAX_WORKERS 4096
#define ADASUM_MAX_LEVELS 12

/*
 * Bytes of device workspace that adasum_reduce / adasum_pair need for these sizes (an upper
 * bound that depends only on the arguments given here, not on the offset values).
 * Returns 0 on invalid arguments.  Host-only; touches no CUDA state.
 */
size_t adasum_workspace_bytes(int64_t total_elems, int32_t num_tensors, int32_t n_workers,
                              adasum_dtype_t dtype, uint32_t flags);

/*
 * How a reduce with these sizes will run: writes the radix of each level into radices[]
 * (room for ADASUM_MAX_LEVELS entries), the number of levels into *num_levels and the number
 * of kernel launches on a B200 into *num_launches (each may be NULL; a buffer that has tensors of
 * at most 64 elements takes one launch more, which this call cannot know).  Host-only.  A one-level
 * reduce of at most 8 workers whose operands total at most 96 MB is a single cooperative launch that
 * reads the operands from HBM once (the second pass finds them in the L2) unless flag bit 16 or 17
 * is set.
 */
adasum_status_t adasum_plan_info(int64_t total_elems, int32_t num_tensors, int32_t n_workers,
                                 adasum_dtype_t dtype, uint32_t flags, int32_t* radices,
                                 int32_t* num_levels, int32_t* num_launches);

/*
 * N-way Adasum combine (Section 3.4 tree of the Section 3 operator, per tensor).
 *
 *   grads           host array of n_workers device pointers; grads[w] is worker w's fused
 *                   gradient buffer of tensor_offsets[num_tensors] elements of `dtype`,
 *                   aligned to its element size (16-byte alignment of every buffer selects
 *                   the vectorised kernels; anything else falls back to scalar loads)
 *   tensor_offsets  host array of num_tensors + 1 element offsets into each buffer:
 *                   tensor_offsets[0] = 0, non-decreasing; empty tensors are allowed
 *   n_workers       1 .. ADASUM_MAX_WORKERS; n_workers = 1 converts grads[0] to fp32
 *   out             device, tensor_offsets[num_tensors] floats, 4-byte aligned
 *   workspace       device, at least adasum_workspace_bytes(...) bytes, 256-byte aligned;
 *                   contents on entry are ignored and on exit unspecified
 *   flags           see above; 0 is the recommended default
 *   stream          cudaStream_t
 *
 * A zero-element reduce (tensor_offsets[num_tensors] == 0) returns ADASUM_OK without a launch.
 */
adasum_status_t adasum_reduce(const void* const* grads, const int64_t* tensor_offsets,
                              int32_t num_tensors, int32_t n_workers, adasum_dtype_t dtype,
                              float* out, void* workspace, size_t workspace_bytes,
                              uint32_t flags, void* stream);

/*
 * adasum_reduce that also returns the per-tensor orthogonality measure of Section 3.6,
 *
 *     orthogonality[t] = |Adasum(g_1 .. g_N)|^2 / sum_i |g_i|^2      (tensor t),
 *
 * which is 1 for mutually orthogonal gradients and 1/N for identical ones.  It costs nothing
 * extra: both norms fall out of the Gram matrices the reduce forms anyway.
 *
 *   orthogonality   device, num_tensors floats, 4-byte aligned, or NULL (then this is
 *                   adasum_reduce).  NaN for a tensor that has no elements or whose gradients
 *                   are all zero.  Needs n_workers >= 2 (ADASUM_ERR_ARG otherwise).
 * Everything else as for adasum_reduce, including the workspace size.
 */
adasum_status_t adasum_reduce_ex(const void* const* grads, const int64_t* tensor_offsets,
                                 int32_t num_tensors, int32_t n_workers, adasum_dtype_t dtype,
                                 float* out, float* orthogonality, void* workspace,
                                 size_t workspace_bytes, uint32_t flags, void* stream);

/*
 * The reduce of gradients that are stored with a scale ("dynamic scaling", Section 4.4.1: in a
 * low-precision type every tensor is kept multiplied by a scale that holds its values inside the
 * type's range, and the scale is adjusted as training goes).  Worker w's buffer holds, for tensor t,
 *
 *     grads[w][e] = scales[w * num_tensors + t] * g_w[e]        (e in tensor t),
 *
 * and the call returns the combination of the gradients themselves, in fp32:
 *
 *     out = Adasum_w(g_w) = Adasum_w(grads[w] / scales[w][t])           per tensor.
 *
 * The operator is not linear, so workers with different scales cannot be combined as stored and
 * rescaled afterwards.  Nothing is rescaled in memory either: the dot products are formed of the
 * stored values as in adasum_reduce, and the fp64 coefficient step divides entry (i, k) of a
 * tensor's Gram matrix by scales[i][t] * scales[k][t] and the weight of worker i's stored values by
 * scales[i][t] (tensors of at most 64 elements: every loaded value is divided, in fp64).  Same
 * traffic, launches and plans as adasum_reduce_ex.
 *
 *   scales          device, n_workers * num_tensors floats (worker-major), 4-byte aligned; every
 *                   entry finite and > 0 (not checked: anything else gives Inf or NaN in that
 *                   tensor's output); read during the call's kernels, so it must stay unchanged
 *                   until they have run
 *   dtype           ADASUM_F32, ADASUM_F16 or ADASUM_BF16 (ADASUM_ERR_DTYPE for ADASUM_F64)
 *   n_workers       2 .. ADASUM_MAX_WORKERS (ADASUM_ERR_ARG for 1)
 *   orthogonality   as for adasum_reduce_ex (of the gradients themselves), or NULL
 *   everything else as for adasum_reduce_ex, including the workspace size and the flags.
 */
adasum_status_t adasum_reduce_scaled(const void* const* grads, const float* scales,
                                     const int64_t* tensor_offsets, int32_t num_tensors,
                                     int32_t n_workers, adasum_dtype_t dtype, float* out,
                                     float* orthogonality, void* workspace, size_t workspace_bytes,
                                     uint32_t flags, void* stream);

/*
 * The reduce wrapped around a local optimizer step (Section 4.1, the figure that applies the
 * operator after optimizer.step(); also "Low Precision Support" in Section 4.4.1 and the
 * delta-from-the-last-allreduce of Section 5.2).  Every worker has taken its own optimizer step
 * from the common parameters `start` and now holds currents[w]; the operator combines the
 * effective gradients currents[w] - start and the combination is added back:
 *
 *     out = start + Adasum_w(currents[w] - start)              per tensor.
 *
 * Nothing is materialised: the differences are formed while the operands stream through both
 * passes, `start` is added as the result is stored.  The cost over adasum_reduce is one more
 * operand read per pass ((n_workers + 1) / n_workers of the traffic).
 *
 *   currents        host array of n_workers device pointers, as `grads` of adasum_reduce
 *   start           device, total elements of `dtype`, 16-byte aligned; NULL: no start, the call
 *                   is adasum_reduce_ex with a choice of output type
 *   out             device, total elements of out_dtype.  May be `start` itself when out_dtype ==
 *                   dtype (the parameters are updated in place); may not overlap anything else
 *   out_dtype       ADASUM_F32, ADASUM_F16 or ADASUM_BF16 (round to nearest even on store); for
 *                   ADASUM_F64 inputs ADASUM_F64 or ADASUM_F32
 *   everything else as for adasum_reduce_ex, including the workspace size and the plan.
 *
 * Each difference currents[w][e] - start[e] is rounded once, to `dtype` (what `current - start`
 * gives in a framework); all later arithmetic is as in adasum_reduce.  With a start every buffer
 * must be 16-byte aligned (ADASUM_ERR_ARG otherwise).  The orthogonality measure, if asked for, is
 * that of the effective gradients.
 */
adasum_status_t adasum_reduce_delta(const void* const* currents, const void* start,
                                    const int64_t* tensor_offsets, int32_t num_tensors,
                                    int32_t n_workers, adasum_dtype_t dtype, void* out,
                                    adasum_dtype_t out_dtype, float* orthogonality, void* workspace,
                                    size_t workspace_bytes, uint32_t flags, void* stream);

/*
 * The same reduce with the ELEMENTS of every tensor spread over several GPUs (one process per GPU).
 *
 * Each GPU holds, for all n_workers workers, its own slice of every tensor: grads[w] is worker w's
 * fused buffer of this GPU's slices and tensor_offsets describes those local slices (the number of
 * tensors and their order are the same on every GPU; a tensor may be empty on some GPUs).  Dot
 * products and norms of a tensor are sums over all its elements, so one exchange per level is
 * needed, exactly the one of Algorithm 1 ("partial dot products", then an all-reduce of the
 * scalars, then "apply Adasum"): for level = 0 .. num_levels - 1 (adasum_plan_info)
 *
 *   1. adasum_sharded_gram(level)   streams this GPU's operands once and leaves this GPU's fp64
 *                                   Gram sums in the workspace, *sums_count doubles starting
 *                                   *sums_offset bytes into it (same count and layout on every GPU);
 *   2. the caller adds those doubles over all GPUs in place (e.g. ncclAllReduce, sum);
 *   3. adasum_sharded_apply(level)  derives the weights from the summed matrices and streams the
 *                                   operands a second time; after the last level `out` holds this
 *                                   GPU's slices of the result (and `orthogonality`, if not NULL,
 *                                   the per-tensor measure, identical on every GPU).
 *
 * Arguments as for adasum_reduce_ex; the workspace (adasum_workspace_bytes of the LOCAL sizes) must
 * be left untouched between the calls of one reduce, and all calls of one reduce must use the
 * same flags and be stream-ordered.  n_workers >= 2.  The library itself never communicates.
 * Errors as for adasum_reduce, plus ADASUM_ERR_ARG for a level outside the plan.
 */
adasum_status_t adasum_sharded_gram(const void* const* grads, const int64_t* tensor_offsets,
                                    int32_t num_tensors, int32_t n_workers, adasum_dtype_t dtype,
                                    void* workspace, size_t workspace_bytes, uint32_t flags,
                                    int32_t level, size_t* sums_offset, int64_t* sums_count,
                                    void* stream);
adasum_status_t adasum_sharded_apply(const void* const* grads, const int64_t* tensor_offsets,
                                     int32_t num_tensors, int32_t n_workers, adasum_dtype_t dtype,
                                     float* out, float* orthogonality, void* workspace,
                                     size_t workspace_bytes, uint32_t flags, int32_t level,
                                     void* stream);

/*
 * One application of the operator per tensor, out = Adasum(a, b) (Section 3; the "partial dot
 * products" and "apply Adasum" steps of Algorithm 1).  Same conventions as adasum_reduce with
 * n_workers = 2; `a` and `b` are device pointers.
 */
adasum_status_t adasum_pair(const void* a, const void* b, const int64_t* tensor_offsets,
                            int32_t num_tensors, adasum_dtype_t dtype, float* out,
                            void* workspace, size_t workspace_bytes, uint32_t flags,
                            void* stream);

/*
 * adasum_pair for callers that must not allocate device memory (the paper has no counterpart).
 *
 * Some hosts of this library cannot call cudaMalloc where they run the reduction: code inside a
 * framework's memory-pool callback, a process whose whole GPU budget was handed to another
 * allocator at start-up, a real-time loop that forbids driver allocations after initialisation.
 * adasum_pair needs a workspace from its caller and builds a cached segment table with cudaMalloc
 * on first use; this entry point needs neither.  Its scratch (segment table, per-segment partial
 * sums, per-tensor coefficients, the list of short tensors; about 0.6 MB) is a fixed array inside the library's device
 * image, so every GPU that loads the library carries it until the process exits.
 *
 *   a, b, tensor_offsets, num_tensors, dtype, out, stream   as for adasum_pair
 *
 * Limits: at most ADASUM_NOALLOC_MAX_ELEMS elements per input and ADASUM_NOALLOC_MAX_TENSORS
 * tensors; larger arguments return ADASUM_ERR_ARG with a message and launch nothing.  The result
 * equals adasum_pair's with default flags.
 *
 * The call performs no cudaMalloc / cudaFree and uses no allocating library routine; it enqueues
 * up to three small host-to-device copies (the segment table of this call, up to about 0.3 MB, staged
 * from ordinary host memory, so the call can briefly wait for the copy engine) and three or four
 * kernels on `stream`.  The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current); make that first call before any stream capture
 * begins.  Because the table is copied from host memory that lives only for the duration of the
 * call, a `stream` that is being captured is refused with ADASUM_ERR_ARG and nothing is recorded.
 *
 * All calls on a device share the one scratch array, which keeps the previous call's contents.
 * Every entry that a call reads is first rewritten by the same call, so nothing has to be
 * cleared; but two calls whose work overlaps on the GPU (different streams, no ordering between
 * them) race on it.  Serialise them with events or use adasum_pair with separate workspaces.
 */
#define ADASUM_NOALLOC_MAX_ELEMS 67108864    /* 2^26 elements per input */
#define ADASUM_NOALLOC_MAX_TENSORS 4096

adasum_status_t adasum_pair_noalloc(const void* a, const void* b, const int64_t* tensor_offsets,
                                    int32_t num_tensors, adasum_dtype_t dtype, float* out, void* stream);

/*
 * Device-side status of the last reduce that used this workspace (the paper has no counterpart).
 * The radix-64 tensor-memory kernel waits, with a limit, for the tensor core to release a
 * shared-memory stage; if such a wait ever runs out, the kernel records it and finishes (with
 * wrong numbers) instead of hanging.  This call copies that record back: it synchronises `stream`
 * and returns ADASUM_OK, ADASUM_ERR_TIMEOUT, or an argument / CUDA error.  Arguments as for the
 * reduce that is being asked about.
 */
adasum_status_t adasum_device_status(int64_t total_elems, int32_t num_tensors, int32_t n_workers,
                                     adasum_dtype_t dtype, uint32_t flags, const void* workspace,
                                     void* stream);

/* Static, human-readable name of a status code. */
const char* adasum_status_string(adasum_status_t status);

/* Detail of the most recent failure on the calling thread ("" if none); valid until the next
 * call into the library from the same thread. */
const char* adasum_last_error(void);

/*
 * Per-launch device timing, for benchmarks (the paper has no counterpart; it reports wall-clock
 * times only).  Between adasum_profile_enable() and adasum_profile_collect(), every reduce/pair
 * call records a CUDA event on its stream before its first kernel and after each kernel.
 * adasum_profile_collect() stops recording, waits for the last event and writes one record per
 * kernel launch in launch order (at most `capacity`; *count receives the number available).
 * `kernel` is one of the ADASUM_KERNEL_* values, `level` the tree level (0 = first), `radix`
 * the level's group size, `ms` the time from the previous event to the one after the launch.
 * Use from one thread, with all profiled calls on one stream.
 * Errors: ADASUM_ERR_ARG (max_launches < 1, or more launches happened than were reserved:
 * the records that were taken are still returned), ADASUM_ERR_NULL, ADASUM_ERR_CUDA.
 */
#define ADASUM_KERNEL_GRAM_PARTIAL 0
#define ADASUM_KERNEL_TREE_WEIGHTS 1
#define ADASUM_KERNEL_WEIGHTED_SUM 2
#define ADASUM_KERNEL_CONVERT 3
#define ADASUM_KERNEL_FUSED_SMALL 4   /* both passes in one cooperative launch (inputs that fit the L2) */
#define ADASUM_KERNEL_WSUM_GRAM 5     /* second pass of `level` and first pass of level + 1 in one kernel */
#define ADASUM_KERNEL_SHORT_TENSORS 6 /* the whole tree of the tensors of at most 64 elements, in fp64 */

typedef struct {
    int32_t kernel;
    int32_t level;
    int32_t radix;
    float ms;
} adasum_launch_record_t;

adasum_status_t adasum_profile_enable(int32_t max_launches);
adasum_status_t adasum_profile_collect(adasum_launch_record_t* records, int32_t capacity, int32_t* count);

/* Frees every cached segment table on every device and the profiling events.  Outstanding work that uses them must
 * have completed.  Returns ADASUM_OK or ADASUM_ERR_CUDA. */
adasum_status_t adasum_shutdown(void);

#ifdef __cplusplus
}
#endif

#endif /* ADASUM_H_ */
