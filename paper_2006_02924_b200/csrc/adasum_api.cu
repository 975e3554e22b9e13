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

#include "adasum_internal.h"
#include "adasum_kernels.cuh"
#include "adasum_f64.cuh"

namespace adasum {

thread_local char g_error[512] = "";

adasum_status_t fail(adasum_status_t status, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof g_error, fmt, ap);
    va_end(ap);
    return status;
}

namespace {

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

}  // namespace

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

namespace {

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

// Elements per segment.  One block accumulates a whole segment in fp32 (per thread: segment /
// 256 elements; on the tensor cores: per warp segment / 8), longer tensors are finished in fp64.
//
// Buffers below 8 M elements that one round of blocks can cover: the shortest power of two that
// still needs no second round (a one-tensor buffer of 256 K elements cut at 8192 would be 32 blocks
// on 148 SMs).  One round, not more: a pass-1 block costs 5 to 10 microseconds before its first
// tile is multiplied, so a second round of short blocks is slower than one round of long ones.
int filling_length(int64_t total, int slots, int shortest, int longest)
{
    int len = shortest;
    while (len < longest && (total + len - 1) / len > slots)
        len *= 2;
    return len;
}
// slots: blocks of the pass-1 kernel that the GPU holds at once (two per SM; one for the kernel
// that keeps its accumulator in tensor memory).
int gram_segment_length(GramKind kind, int64_t total, int slots = 296)
{
    if (kind == GRAM_MMA)
        return total >= (int64_t(1) << 26)   ? 32768
               : total >= (int64_t(1) << 23) ? 16384
                                             : filling_length(total, slots, 1024, 8192);
    return total >= (int64_t(1) << 23) ? 8192 : filling_length(total, slots, 512, 2048);
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
    if ((flags >> 23) != 0)
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

// Blocks that a pass-1 table's tapering is laid out for: two blocks on each of a B200's 148 SMs.
constexpr int kTaperSlots = 296;

// Upper bound of the segments of a table with this nominal segment length (tapered or not: the
// shorter segments at both ends of a tapered table add fewer than 4 per slot).
int64_t segment_bound(int64_t total, int32_t num_tensors, int seg_len)
{
    const bool may_taper = total >= 3 * (int64_t)kTaperSlots * seg_len;
    return total / seg_len + 2 * (int64_t)num_tensors + 1 + (may_taper ? 4 * kTaperSlots : 0);
}

// Upper bound of the runs of kSegmentsPerGroup segments in such a table.  Only tensors of more than
// kSegmentsPerGroup segments have runs, and such a tensor of n segments has at most n / 16 + 1 <=
// n / 8 of them.
int64_t run_bound(int64_t segments)
{
    return segments / (kSegmentsPerGroup / 2) + 1;
}

struct Layout {
    size_t partials = 0, weights = 0, weights_alt = 0, gram64 = 0, counters = 0, leaf_sums = 0, buffer[2] = {0, 0};
    size_t partials_bytes = 0, weights_bytes = 0, gram64_bytes = 0, counters_bytes = 0, leaf_sums_bytes = 0,
           buffer_bytes[2] = {0, 0};
    // short tensors of reduces with more workers than one launch carries: per launch an fp64 vector
    // over the short tensors' elements and the sum of its leaves' squared norms
    size_t short_vecs = 0, short_sums = 0, short_vecs_bytes = 0, short_sums_bytes = 0;
    size_t run_sums = 0, run_sums_bytes = 0;       // the two-step finish: one fp64 Gram matrix per run and group
    int64_t short_vec_stride = 0, short_sum_stride = 0;      // doubles between two launches' arrays
    int64_t padded_elems = 0;
    size_t total = 0;
};

Layout make_layout(const LevelPlan& plan, int64_t total_elems, int32_t num_tensors, int n_workers)
{
    Layout lay;
    lay.padded_elems = (total_elems + 63) / 64 * 64;
    if (n_workers > kMaxOperandsPerLaunch) {
        const int64_t launches = (n_workers + kMaxOperandsPerLaunch - 1) / kMaxOperandsPerLaunch;
        const int64_t bound = (int64_t)num_tensors * kShortTensorElems;
        lay.short_vec_stride = total_elems < bound ? total_elems : bound;
        lay.short_sum_stride = num_tensors;
        lay.short_vecs_bytes = (size_t)(launches * lay.short_vec_stride) * sizeof(double);
        lay.short_sums_bytes = (size_t)(launches * lay.short_sum_stride) * sizeof(double);
    }
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
        // ticket counters per (tensor, group), then per (run of segments, group); + 1: the device
        // status word sits after them
        const size_t runs = (size_t)run_bound(segment_bound(total_elems, num_tensors,
                                                            min_gram_segment_length(lv.radix, total_elems)));
        const size_t c = (((size_t)(num_tensors > 0 ? num_tensors : 1) + runs) * lv.groups + 1) * sizeof(int);
        if (c > lay.counters_bytes)
            lay.counters_bytes = c;
        const size_t rs = runs * lv.groups * gram_entries(lv.radix) * sizeof(double);
        if (rs > lay.run_sums_bytes)
            lay.run_sums_bytes = rs;
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
    lay.short_vecs = off;
    off += align_up(lay.short_vecs_bytes);
    lay.short_sums = off;
    off += align_up(lay.short_sums_bytes);
    lay.run_sums = off;
    off += align_up(lay.run_sums_bytes);
    lay.total = off > 0 ? off : kAlign;
    return lay;
}

// ---- cached segment tables ---------------------------------------------------------------------
//
// A table is shared between the cache and every call that is using it (TableRef), so dropping it
// from the cache never frees device memory that a call still intends to launch with: the device
// arrays go when the last reference does, and cudaFree then waits for the kernels that were
// enqueued with them.

using TableRef = std::shared_ptr<const SegmentTable>;

// Least recently used first.  The cache is bounded both by the number of tables and by the device
// bytes they hold.
std::mutex g_tables_mutex;
std::vector<std::shared_ptr<SegmentTable>> g_tables;
constexpr size_t kMaxCachedTables = 256;
constexpr size_t kMaxCachedTableBytes = size_t(256) << 20;

size_t table_device_bytes(const SegmentTable& tab)
{
    return sizeof(Segment) * (tab.h_segments.size() + 1) + sizeof(int32_t) * tab.h_seg_first.size() +
           sizeof(ShortTensor) * (tab.h_short.size() + 1) + sizeof(WarpTensor) * (tab.h_warp.size() + 1);
}

// Segments are listed tensor by tensor, LARGEST tensor first (ties in index order): the blocks of
// pass 1 that run last then belong to small tensors, whose per-tensor finish (adding the partial
// matrices, tree weights) is short, instead of leaving one SM busy with a long tensor's finish
// while the rest of the GPU idles.  Each tensor's segments stay contiguous, in element order.
//
// taper_slots > 0 (pass-1 tables of long buffers): the blocks of a launch are handed out in table
// order, `taper_slots` at a time.  Segments of one length would leave the machine half empty while
// the last round of blocks drains, and would keep the two blocks of an SM starting and ending
// together, pipelines empty at the same moments.  So the segments that the last one and a half
// rounds would cover are cut at half the length, those of the last half round at a quarter, and
// the first quarter round at half length, which staggers the blocks that share an SM.
void build_segments(const int64_t* offsets, int32_t num_tensors, int seg_len, bool skip_short, int warp_limit,
                    int taper_slots, SegmentTable* tab)
{
    tab->skip_short = skip_short;
    tab->warp_limit = warp_limit;
    tab->h_short.clear();
    tab->h_warp.clear();
    tab->short_elems = 0;
    const int64_t short_limit = skip_short ? kShortTensorElems : 0;
    for (int32_t t = 0; t < num_tensors && warp_limit > 0; ++t) {
        const int64_t len = offsets[t + 1] - offsets[t];
        if (len > short_limit && len <= warp_limit)
            tab->h_warp.push_back(WarpTensor{offsets[t], (int32_t)len, t});
    }
    if (skip_short) {
        for (int32_t t = 0; t < num_tensors; ++t) {
            const int64_t len = offsets[t + 1] - offsets[t];
            if (len > 0 && len <= kShortTensorElems) {
                tab->h_short.push_back(ShortTensor{offsets[t], (int32_t)len, t, tab->short_elems});
                tab->short_elems += len;
            }
        }
    }
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
    const auto in_segments = [&](int32_t t) {
        const int64_t len = offsets[t + 1] - offsets[t];
        return !((skip_short && len <= kShortTensorElems) || len <= warp_limit);
    };
    int64_t left = 0;           // elements that the segments from here to the end of the table cover
    for (int32_t t = 0; t < num_tensors; ++t)
        left += in_segments(t) ? offsets[t + 1] - offsets[t] : 0;
    const int64_t round = (int64_t)taper_slots * seg_len;
    if (left < 3 * round || seg_len < 4096)
        taper_slots = 0;        // too short a launch to have a middle, or blocks too short to matter
    tab->taper_slots = taper_slots;
    int64_t done = 0;
    for (int32_t t : order) {
        tab->h_seg_first[2 * (size_t)t] = (int32_t)tab->h_segments.size();
        int64_t b = offsets[t];
        const int64_t e = offsets[t + 1];
        if (!in_segments(t))
            b = e;
        while (b < e) {
            int64_t len = seg_len;
            if (taper_slots > 0) {
                if (left <= round / 2)
                    len = seg_len / 4;
                else if (left <= round + round / 2 || done < round / 4)
                    len = seg_len / 2;
            }
            // cut on a 64-element grid of the fused buffer so that interior cuts keep 16-byte
            // alignment whatever the tensor's own start
            int64_t next = b / 64 * 64 + len;
            if (next > e)
                next = e;
            tab->h_segments.push_back(Segment{b, (int32_t)(next - b), t});
            done += next - b;
            left -= next - b;
            b = next;
        }
        tab->h_seg_first[2 * (size_t)t + 1] = (int32_t)tab->h_segments.size();
        const int32_t n = tab->h_seg_first[2 * (size_t)t + 1] - tab->h_seg_first[2 * (size_t)t];
        if (n > tab->max_segments_per_tensor)
            tab->max_segments_per_tensor = n;
    }
    tab->num_segments = (int32_t)tab->h_segments.size();
    // runs of kSegmentsPerGroup segments, numbered through the tensors in their own order
    tab->h_seg_first.resize(3 * (size_t)num_tensors + 3, 0);
    int32_t runs = 0;
    for (int32_t t = 0; t < num_tensors; ++t) {
        tab->h_seg_first[2 * (size_t)num_tensors + 2 + t] = runs;
        const int32_t n = tab->h_seg_first[2 * (size_t)t + 1] - tab->h_seg_first[2 * (size_t)t];
        if (n > kSegmentsPerGroup)          // shorter tensors are finished in one step and need no runs
            runs += (n + kSegmentsPerGroup - 1) / kSegmentsPerGroup;
    }
    tab->h_seg_first[3 * (size_t)num_tensors + 2] = runs;
    tab->num_runs = runs;
}

// The table for (current device, offsets, seg_len), built and uploaded on first use.  The caller
// keeps the returned reference until it has enqueued its last launch that reads the table.
adasum_status_t get_segment_table(const int64_t* offsets, int32_t num_tensors, int seg_len, bool skip_short,
                                  TableRef* out, int warp_limit = 0, int taper_slots = 0)
{
    int device = 0;
    ADASUM_CUDA_CHECK(cudaGetDevice(&device));
    std::vector<std::shared_ptr<SegmentTable>> dropped;      // destroyed after the lock is released
    std::lock_guard<std::mutex> lock(g_tables_mutex);
    for (size_t i = 0; i < g_tables.size(); ++i) {
        const SegmentTable& tab = *g_tables[i];
        if (tab.device == device && tab.seg_len == seg_len && tab.skip_short == skip_short &&
            tab.warp_limit == warp_limit && tab.taper_request == taper_slots &&
            tab.offsets.size() == (size_t)num_tensors + 1 &&
            std::memcmp(tab.offsets.data(), offsets, sizeof(int64_t) * tab.offsets.size()) == 0) {
            // most recently used last
            std::rotate(g_tables.begin() + (ptrdiff_t)i, g_tables.begin() + (ptrdiff_t)i + 1, g_tables.end());
            *out = g_tables.back();
            return ADASUM_OK;
        }
    }
    auto tab = std::make_shared<SegmentTable>();
    tab->device = device;
    tab->seg_len = seg_len;
    tab->offsets.assign(offsets, offsets + num_tensors + 1);
    tab->taper_request = taper_slots;
    build_segments(offsets, num_tensors, seg_len, skip_short, warp_limit, taper_slots, tab.get());
    const size_t seg_bytes = sizeof(Segment) * (tab->h_segments.size() + 1);
    const size_t first_bytes = sizeof(int32_t) * tab->h_seg_first.size();
    const size_t short_bytes = sizeof(ShortTensor) * (tab->h_short.size() + 1) +
                               sizeof(WarpTensor) * (tab->h_warp.size() + 1);
    // Make room: least recently used tables leave the cache.  One that a call in flight still holds
    // lives on until that call lets go of it.
    size_t held = 0;
    for (const auto& t : g_tables)
        held += table_device_bytes(*t);
    while (!g_tables.empty() &&
           (g_tables.size() >= kMaxCachedTables ||
            held + seg_bytes + first_bytes + short_bytes > kMaxCachedTableBytes)) {
        held -= table_device_bytes(*g_tables.front());
        dropped.push_back(std::move(g_tables.front()));
        g_tables.erase(g_tables.begin());
    }
    tab->owns_device_arrays = true;
    cudaError_t err = cudaMalloc(&tab->d_segments, seg_bytes);
    if (err == cudaSuccess)
        err = cudaMalloc(&tab->d_seg_first, first_bytes);
    // Blocking copies: the table may be used from any stream afterwards.
    if (err == cudaSuccess && !tab->h_segments.empty())
        err = cudaMemcpy(tab->d_segments, tab->h_segments.data(),
                         sizeof(Segment) * tab->h_segments.size(), cudaMemcpyHostToDevice);
    if (err == cudaSuccess)
        err = cudaMemcpy(tab->d_seg_first, tab->h_seg_first.data(), first_bytes, cudaMemcpyHostToDevice);
    tab->d_group_first = tab->d_seg_first ? tab->d_seg_first + 2 * (size_t)num_tensors + 2 : nullptr;
    if (err == cudaSuccess && !tab->h_warp.empty()) {
        err = cudaMalloc(&tab->d_warp, sizeof(WarpTensor) * tab->h_warp.size());
        if (err == cudaSuccess)
            err = cudaMemcpy(tab->d_warp, tab->h_warp.data(), sizeof(WarpTensor) * tab->h_warp.size(),
                             cudaMemcpyHostToDevice);
    }
    if (err == cudaSuccess && !tab->h_short.empty()) {
        err = cudaMalloc(&tab->d_short, short_bytes);
        if (err == cudaSuccess)
            err = cudaMemcpy(tab->d_short, tab->h_short.data(), sizeof(ShortTensor) * tab->h_short.size(),
                             cudaMemcpyHostToDevice);
    }
    if (err != cudaSuccess)
        return fail(ADASUM_ERR_CUDA, "segment table upload: %s", cudaGetErrorString(err));
    g_tables.push_back(tab);
    *out = std::move(tab);
    return ADASUM_OK;
}

// ---- side streams ---------------------------------------------------------------------------------
//
// The kernel for the tensors of at most 64 elements is independent of the streaming passes (other
// elements of the output, its own part of the workspace), so it runs beside them: forked from the
// caller's stream with an event, on a stream of the library's own, joined with a second event
// before the call returns.  Both dependencies are ordinary stream operations (they are recorded
// like any other when the caller's stream is being captured).  A lane is borrowed for the duration
// of one call; lanes are created on demand and kept until adasum_shutdown().

struct SideLane {
    int device = -1;
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
};

std::mutex g_lanes_mutex;
std::vector<SideLane> g_lanes;

bool borrow_lane(SideLane* lane)
{
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess)
        return false;
    {
        std::lock_guard<std::mutex> lock(g_lanes_mutex);
        for (size_t i = 0; i < g_lanes.size(); ++i) {
            if (g_lanes[i].device == device) {
                *lane = g_lanes[i];
                g_lanes.erase(g_lanes.begin() + (ptrdiff_t)i);
                return true;
            }
        }
    }
    SideLane fresh;
    fresh.device = device;
    if (cudaStreamCreateWithFlags(&fresh.stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&fresh.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&fresh.join, cudaEventDisableTiming) != cudaSuccess) {
        if (fresh.stream)
            cudaStreamDestroy(fresh.stream);
        if (fresh.fork)
            cudaEventDestroy(fresh.fork);
        (void)cudaGetLastError();
        return false;
    }
    *lane = fresh;
    return true;
}

void return_lane(const SideLane& lane)
{
    std::lock_guard<std::mutex> lock(g_lanes_mutex);
    g_lanes.push_back(lane);
}

// Joins a forked lane into `stream` when the call ends, however it ends.
struct LaneJoin {
    SideLane lane;
    cudaStream_t stream = nullptr;
    bool forked = false;
    ~LaneJoin()
    {
        if (!forked)
            return;
        cudaEventRecord(lane.join, lane.stream);
        cudaStreamWaitEvent(stream, lane.join, 0);
        return_lane(lane);
    }
};

// ---- single-launch path for inputs that fit the L2 ------------------------------------------------

constexpr int64_t kSmallInputBytes = int64_t(96) << 20;    // operands that the 126 MB L2 holds with room to spare
constexpr int kSmallBlocksPerSm = 2;                       // blocks per SM the grid is sized for (all variants keep >= 2 resident)
constexpr int kSmallSegmentGrain = 1024;

// Segments that build_segments makes of the tensors of more than kWarpTensorElems elements at this
// segment length (cuts on the 64-element grid of the fused buffer).
int64_t count_long_segments(const int64_t* offsets, int32_t num_tensors, int64_t seg_len)
{
    int64_t n = 0;
    for (int32_t t = 0; t < num_tensors; ++t) {
        const int64_t b = offsets[t], e = offsets[t + 1];
        if (e - b <= kWarpTensorElems)
            continue;
        const int64_t first_cut = b / 64 * 64 + seg_len;
        n += first_cut >= e ? 1 : 1 + (e - first_cut + seg_len - 1) / seg_len;
    }
    return n;
}

// Host-only rule (no device query): is this reduce served by fused_small_kernel, and with which
// segment length?  `blocks` is the number of blocks that can be resident at once; only the tensors
// of more than kWarpTensorElems elements are cut into segments, one block each.  With the offsets
// the shortest segment length (a multiple of kSmallSegmentGrain) whose segments fit the blocks is
// found exactly; without them (offsets == nullptr, adasum_plan_info) every tensor is taken for a
// long one with two ragged ends.
bool small_input_plan(const LevelPlan& plan, int64_t total, int32_t num_tensors, const int64_t* offsets, int n_workers,
                      int elem_bytes, uint32_t flags, int blocks, int* seg_len)
{
    if (plan.num_levels != 1 || plan.level[0].radix > 8 || plan.level[0].groups != 1)
        return false;
    if (flags & (ADASUM_FLAG_SIMPLE_KERNELS | ADASUM_FLAG_SEPARATE_FINISH))
        return false;
    if (total <= 0 || (int64_t)n_workers * total * elem_bytes > kSmallInputBytes)
        return false;
    constexpr int64_t kLongest = int64_t(1) << 20;
    auto round_up = [](int64_t len) {
        len = (len + kSmallSegmentGrain - 1) / kSmallSegmentGrain * kSmallSegmentGrain;
        return len < 2048 ? int64_t(2048) : len;
    };
    if (offsets == nullptr) {
        const int64_t room = (int64_t)blocks - 2 * (int64_t)num_tensors;
        if (room < 8)
            return false;
        const int64_t len = round_up((total + room - 1) / room);
        if (len > kLongest)
            return false;
        *seg_len = (int)len;
        return true;
    }
    int64_t long_elems = 0;
    for (int32_t t = 0; t < num_tensors; ++t)
        if (offsets[t + 1] - offsets[t] > kWarpTensorElems)
            long_elems += offsets[t + 1] - offsets[t];
    int64_t len = round_up((long_elems + blocks - 1) / blocks);
    while (len <= kLongest && count_long_segments(offsets, num_tensors, len) > blocks)
        len += len < 16 * kSmallSegmentGrain ? kSmallSegmentGrain : len / 16 / kSmallSegmentGrain * kSmallSegmentGrain;
    if (len > kLongest)
        return false;
    *seg_len = (int)len;
    return true;
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

int launches_of(const LevelPlan& plan, int n_workers, uint32_t flags, int64_t total, int32_t num_tensors,
                int elem_bytes)
{
    if (n_workers == 1)
        return 1;
    int seg_len = 0;        // on a B200: 148 SMs
    if (small_input_plan(plan, total, num_tensors, nullptr, n_workers, elem_bytes, flags, 148 * kSmallBlocksPerSm, &seg_len))
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
                            adasum_dtype_t out_dtype = ADASUM_F32, const float* leaf_scales = nullptr)
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
    if (leaf_scales != nullptr) {
        if (n_workers < 2)
            return fail(ADASUM_ERR_ARG, "the scaled reduce needs at least two workers");
        if (reinterpret_cast<uintptr_t>(leaf_scales) & 3u)
            return fail(ADASUM_ERR_ARG, "scales is not 4-byte aligned");
    }
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
    const Layout lay = make_layout(plan, total, num_tensors, n_workers);
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
        PassExtras ex = last_extras;
        ex.start = start;
        if (dtype == ADASUM_F32)
            ADASUM_CUDA_CHECK(launch_convert<float>(grads[0], out, total, ex, stream));
        else if (dtype == ADASUM_F16)
            ADASUM_CUDA_CHECK(launch_convert<__half>(grads[0], out, total, ex, stream));
        else
            ADASUM_CUDA_CHECK(launch_convert<__nv_bfloat16>(grads[0], out, total, ex, stream));
        profile_mark(stream, ADASUM_KERNEL_CONVERT, 0, 1, false);
        return ADASUM_OK;
    }

    char* ws = static_cast<char*>(workspace);
    const bool separate_finish = (flags & ADASUM_FLAG_SEPARATE_FINISH) != 0 || sharded;
    // Inputs that fit the L2 are served by one cooperative launch that needs no ticket counters.
    int small_seg_len = 0;
    const int small_blocks = (sharded || total == 0 || num_tensors == 0) ? 0 : resident_small_blocks();
    const bool small_candidate = small_blocks > 0 && small_input_plan(plan, total, num_tensors, offsets, n_workers, eb,
                                                                      flags, small_blocks, &small_seg_len);
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

    // Tensors of at most kShortTensorElems elements are left out of the streaming kernels' segment
    // tables and reduced in fp64 by a kernel of their own, launched last.  Not in the sharded calls:
    // there a tensor's elements are spread over several GPUs and only its Gram sums travel.
    const bool skip_short = !sharded;
    TableRef short_ref;          // held for the whole call: every level's pass 2 uses this table too
    if (skip_short) {
        st = get_segment_table(offsets, num_tensors, wsum_segment_length(total), true, &short_ref);
        if (st != ADASUM_OK)
            return st;
    }
    bool short_done = false;
    auto run_short = [&](cudaStream_t stream) -> adasum_status_t {       // launches on the stream it is given
        const int num_short = short_ref ? (int)short_ref->h_short.size() : 0;
        if (num_short == 0 || short_done)
            return ADASUM_OK;
        short_done = true;
        ShortArgs sa{};
        sa.table = short_ref->d_short;
        sa.order = tree_order(n_workers, flags);
        sa.start = start;
        sa.leaf_scales = leaf_scales;
        sa.num_tensors = num_tensors;
        sa.worker_base = 0;
        sa.base_dtype = (int)dtype;
        sa.out_dtype = (int)out_dtype;
        OperandTable table;
        if (n_workers <= kMaxOperandsPerLaunch) {
            for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
                table.ptr[i] = grads[i < n_workers ? i : 0];
            sa.out = out;
            sa.base = start;
            sa.orthogonality = orthogonality;
            ADASUM_CUDA_CHECK(launch_short_tensors((int)dtype, table, n_workers, num_short, sa, stream));
            profile_mark(stream, ADASUM_KERNEL_SHORT_TENSORS, 0, 2, false);
            return ADASUM_OK;
        }
        // more workers than one launch carries: every launch reduces the complete sub-tree of its
        // kMaxOperandsPerLaunch workers to one fp64 vector, a last launch reduces those
        double* vecs = reinterpret_cast<double*>(ws + lay.short_vecs);
        double* sums = reinterpret_cast<double*>(ws + lay.short_sums);
        const int launches = (n_workers + kMaxOperandsPerLaunch - 1) / kMaxOperandsPerLaunch;
        for (int j = 0; j < launches; ++j) {
            const int w0 = j * kMaxOperandsPerLaunch;
            const int here = n_workers - w0 < kMaxOperandsPerLaunch ? n_workers - w0 : kMaxOperandsPerLaunch;
            for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
                table.ptr[i] = grads[w0 + (i < here ? i : 0)];
            ShortArgs part = sa;
            part.worker_base = w0;
            part.vec_out = vecs + (int64_t)j * lay.short_vec_stride;
            part.leaf_sum_out = sums + (int64_t)j * lay.short_sum_stride;
            ADASUM_CUDA_CHECK(launch_short_tensors((int)dtype, table, here, num_short, part, stream));
            profile_mark(stream, ADASUM_KERNEL_SHORT_TENSORS, 0, 2, false);
        }
        for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
            table.ptr[i] = vecs + (int64_t)(i < launches ? i : 0) * lay.short_vec_stride;
        sa.start = nullptr;
        sa.leaf_scales = nullptr;        // the vectors of the earlier launches are gradients already
        sa.out = out;
        sa.base = start;
        sa.orthogonality = orthogonality;
        sa.leaf_sum_in = sums;
        sa.leaf_sum_launches = launches;
        sa.leaf_sum_stride = lay.short_sum_stride;
        ADASUM_CUDA_CHECK(launch_short_tensors(3, table, launches, num_short, sa, stream));
        profile_mark(stream, ADASUM_KERNEL_SHORT_TENSORS, 1, 2, false);
        return ADASUM_OK;
    };
    if (short_ref && short_ref->num_segments == 0)        // every tensor is short
        return run_short(stream);
    // Beside the streaming passes, on a stream of the library's own (not while launches are being
    // timed one by one, and not where the single-launch kernel takes these tensors itself).
    LaneJoin lane_join;
    if (short_ref && !short_ref->h_short.empty() && !small_candidate && !g_profiler.enabled &&
        borrow_lane(&lane_join.lane)) {
        lane_join.stream = stream;
        if (cudaEventRecord(lane_join.lane.fork, stream) == cudaSuccess &&
            cudaStreamWaitEvent(lane_join.lane.stream, lane_join.lane.fork, 0) == cudaSuccess) {
            lane_join.forked = true;
            st = run_short(lane_join.lane.stream);
            if (st != ADASUM_OK)
                return st;
        } else {
            (void)cudaGetLastError();
            return_lane(lane_join.lane);
        }
    }

    // Inputs that fit the L2: one cooperative launch does both passes and HBM sees the operands once.
    if (small_candidate) {
        int* dev_status = reinterpret_cast<int*>(ws + lay.counters + lay.counters_bytes - sizeof(int));
        TableRef tab;
        st = get_segment_table(offsets, num_tensors, small_seg_len, skip_short, &tab, kWarpTensorElems);
        if (st != ADASUM_OK)
            return st;
        if (tab->num_segments <= small_blocks) {
            OperandTable table;
            for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
                table.ptr[i] = grads[i < n_workers ? i : 0];
            FinishArgs fin{};
            fin.seg_first = tab->d_seg_first;
            fin.counters = nullptr;
            fin.weights = nullptr;
            fin.selftest_timeout = 0;
            fin.tree = TreeOptions{tree_order(n_workers, flags), 1, 1, 1,
                                   orthogonality ? reinterpret_cast<double*>(ws + lay.leaf_sums) : nullptr,
                                   orthogonality, leaf_scales, num_tensors};
            float* partials = reinterpret_cast<float*>(ws + lay.partials);
            const int radix = plan.level[0].radix;
            PassExtras ex = last_extras;
            ex.start = start;
            cudaError_t err;
            if (dtype == ADASUM_F32)
                err = launch_fused_small_any<float>(vec, radix, table, n_workers, *tab, small_blocks, partials, fin, out, ex, dev_status, stream);
            else if (dtype == ADASUM_F16)
                err = launch_fused_small_any<__half>(vec, radix, table, n_workers, *tab, small_blocks, partials, fin, out, ex, dev_status, stream);
            else
                err = launch_fused_small_any<__nv_bfloat16>(vec, radix, table, n_workers, *tab, small_blocks, partials, fin, out, ex, dev_status, stream);
            if (err == cudaSuccess) {
                profile_mark(stream, ADASUM_KERNEL_FUSED_SMALL, 0, radix, false);
                return ADASUM_OK;          // the tensors of at most 64 elements included
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
        TableRef gram_tab, wsum_tab, fuse_tab;     // held until this level's launches are enqueued
        const bool tensor_memory_kernel = kind == GRAM_MMA && lv.radix == 64 && dtype != ADASUM_F32 && l == 0 &&
                                          !(flags & ADASUM_FLAG_NO_TCGEN05);
        st = get_segment_table(offsets, num_tensors, gram_segment_length(kind, total, tensor_memory_kernel ? 148 : 296),
                               skip_short, &gram_tab, 0, kTaperSlots);
        if (st != ADASUM_OK)
            return st;
        st = get_segment_table(offsets, num_tensors, wsum_segment_length(total), skip_short, &wsum_tab);
        if (st != ADASUM_OK)
            return st;
        const bool last = l + 1 == plan.num_levels;
        LevelArgs a;
        a.operand_ptrs = operand_ptrs.data();
        a.operands = lv.operands;
        a.groups = lv.groups;
        a.kind = kind;
        a.gram_tab = gram_tab.get();
        a.wsum_tab = wsum_tab.get();
        a.num_tensors = num_tensors;
        a.partials = reinterpret_cast<float*>(ws + lay.partials);
        a.weights = reinterpret_cast<float*>(ws + ((l & 1) ? lay.weights_alt : lay.weights));
        a.gram64 = reinterpret_cast<double*>(ws + lay.gram64);
        a.counters = separate_finish ? nullptr : reinterpret_cast<int*>(ws + lay.counters);
        a.run_counters = reinterpret_cast<int*>(ws + lay.counters) + (size_t)(num_tensors > 0 ? num_tensors : 1) * lv.groups;
        a.run_sums = reinterpret_cast<double*>(ws + lay.run_sums);
        a.phase = phase;
        // the status word is the last int of the (zeroed) counter region
        a.tc_status = (flags & ADASUM_FLAG_NO_TCGEN05)
                          ? nullptr
                          : reinterpret_cast<int*>(ws + lay.counters + lay.counters_bytes - sizeof(int));
        a.selftest_timeout = (flags & ADASUM_FLAG_SELFTEST_TIMEOUT) != 0;
        a.tree.linear = tree_order(n_workers, flags);
        a.tree.level_is_first = l == 0;
        a.tree.level_is_last = l + 1 == plan.num_levels;
        a.tree.groups_first = plan.level[0].groups;
        a.tree.leaf_norm_sums = orthogonality ? reinterpret_cast<double*>(ws + lay.leaf_sums) : nullptr;
        a.tree.orthogonality = orthogonality;
        a.tree.leaf_scales = leaf_scales;
        a.tree.num_tensors = num_tensors;
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
            st = get_segment_table(offsets, num_tensors, gram_segment_length(GRAM_SIMPLE, total), skip_short, &fuse_tab);
            if (st != ADASUM_OK)
                return st;
            a.fuse_tab = fuse_tab.get();
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
    return run_short(stream);       // unless they already run on the side stream
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
    if ((flags >> 23) != 0)
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
    TableRef tab;
    st = get_segment_table(offsets, num_tensors, segment_length_f64(total), false, &tab);
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
        a.tab = tab.get();
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
constexpr size_t kNoallocShortBytes = ((size_t)kNoallocMaxTensors * sizeof(ShortTensor) + 255) / 256 * 256;
constexpr size_t kNoallocScratchBytes =
    kNoallocSegBytes + kNoallocFirstBytes + kNoallocPartialBytes + kNoallocWeightBytes + kNoallocShortBytes;

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

    // This call's segment table is copied from host vectors that die when the call returns.  A
    // captured copy would read them at every replay, long after that, so a capturing stream is refused.
    cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
    ADASUM_CUDA_CHECK(cudaStreamIsCapturing(stream, &capture));
    if (capture != cudaStreamCaptureStatusNone)
        return fail(ADASUM_ERR_ARG, "adasum_pair_noalloc cannot be recorded into a CUDA graph: it uploads a "
                                    "per-call table from temporary host memory");
    unsigned char* scratch = nullptr;
    st = noalloc_scratch(&scratch);
    if (st != ADASUM_OK)
        return st;
    SegmentTable tab;                       // host-side only; its device pointers aim into the scratch
    build_segments(offsets, num_tensors, kNoallocSegLen, true, 0, 0, &tab);      // short tensors apart, as in adasum_pair
    if ((int64_t)tab.num_segments > kNoallocMaxSegments)
        return fail(ADASUM_ERR_ARG, "segment table does not fit the static scratch");
    tab.d_segments = reinterpret_cast<Segment*>(scratch);
    tab.d_seg_first = reinterpret_cast<int32_t*>(scratch + kNoallocSegBytes);
    float* partials = reinterpret_cast<float*>(scratch + kNoallocSegBytes + kNoallocFirstBytes);
    float* weights = reinterpret_cast<float*>(scratch + kNoallocSegBytes + kNoallocFirstBytes + kNoallocPartialBytes);
    ShortTensor* short_table = reinterpret_cast<ShortTensor*>(scratch + kNoallocSegBytes + kNoallocFirstBytes +
                                                              kNoallocPartialBytes + kNoallocWeightBytes);
    // The host vectors are pageable memory: cudaMemcpyAsync has read them completely when it
    // returns, and the copies are ordered before the kernels on `stream`.
    if (!tab.h_segments.empty())
        ADASUM_CUDA_CHECK(cudaMemcpyAsync(tab.d_segments, tab.h_segments.data(),
                                          sizeof(Segment) * tab.h_segments.size(), cudaMemcpyHostToDevice, stream));
    // (the segment ranges only: the run numbers that follow them are for the ticket finish, unused here)
    ADASUM_CUDA_CHECK(cudaMemcpyAsync(tab.d_seg_first, tab.h_seg_first.data(),
                                      sizeof(int32_t) * (2 * (size_t)num_tensors + 2), cudaMemcpyHostToDevice, stream));
    if (!tab.h_short.empty())
        ADASUM_CUDA_CHECK(cudaMemcpyAsync(short_table, tab.h_short.data(), sizeof(ShortTensor) * tab.h_short.size(),
                                          cudaMemcpyHostToDevice, stream));
    OperandTable ops;
    for (int i = 0; i < kMaxOperandsPerLaunch; ++i)
        ops.ptr[i] = in[i < 2 ? i : 0];
    if (tab.num_segments > 0) {
        if (dtype == ADASUM_F32)
            ADASUM_CUDA_CHECK(noalloc_launch<float>(vec, ops, tab, num_tensors, partials, weights, out, stream));
        else if (dtype == ADASUM_F16)
            ADASUM_CUDA_CHECK(noalloc_launch<__half>(vec, ops, tab, num_tensors, partials, weights, out, stream));
        else
            ADASUM_CUDA_CHECK(noalloc_launch<__nv_bfloat16>(vec, ops, tab, num_tensors, partials, weights, out, stream));
    }
    if (!tab.h_short.empty()) {         // tensors of at most kShortTensorElems elements: the fp64 kernel
        ShortArgs sa{};
        sa.table = short_table;
        sa.out = out;
        sa.base_dtype = (int)dtype;
        sa.out_dtype = (int)ADASUM_F32;
        ADASUM_CUDA_CHECK(launch_short_tensors((int)dtype, ops, 2, (int)tab.h_short.size(), sa, stream));
    }
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
    return make_layout(plan, total_elems, num_tensors, n_workers).total;
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

adasum_status_t adasum_reduce_scaled(const void* const* grads, const float* scales, const int64_t* tensor_offsets,
                                     int32_t num_tensors, int32_t n_workers, adasum_dtype_t dtype, float* out,
                                     float* orthogonality, void* workspace, size_t workspace_bytes, uint32_t flags,
                                     void* stream)
{
    if (!scales)
        return adasum::fail(ADASUM_ERR_NULL, "scales is NULL");
    if (dtype == ADASUM_F64)
        return adasum::fail(ADASUM_ERR_DTYPE, "the scaled reduce takes fp32, fp16 or bf16 gradients");
    return adasum::reduce_impl(grads, tensor_offsets, num_tensors, n_workers, dtype, out, orthogonality, workspace,
                               workspace_bytes, flags, static_cast<cudaStream_t>(stream), adasum::PHASE_WHOLE, -1,
                               nullptr, nullptr, nullptr, ADASUM_F32, scales);
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
    const Layout lay = make_layout(plan, total_elems, num_tensors, n_workers);
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
    {
        std::lock_guard<std::mutex> lock(g_lanes_mutex);
        for (const SideLane& lane : g_lanes) {
            int current = 0;
            const bool have = cudaGetDevice(&current) == cudaSuccess;
            if (have && current != lane.device)
                cudaSetDevice(lane.device);
            cudaStreamDestroy(lane.stream);
            cudaEventDestroy(lane.fork);
            cudaEventDestroy(lane.join);
            if (have && current != lane.device)
                cudaSetDevice(current);
        }
        g_lanes.clear();
    }
    std::vector<std::shared_ptr<SegmentTable>> dropped;
    {
        std::lock_guard<std::mutex> lock(g_tables_mutex);
        dropped.swap(g_tables);
    }
    if (dropped.empty())
        return ADASUM_OK;       // nothing to free: no CUDA call (the library may be loaded without a GPU)
    dropped.clear();            // frees the device arrays (cudaFree waits for the kernels that read them)
    const cudaError_t err = cudaGetLastError();
    return err == cudaSuccess ? ADASUM_OK : fail(ADASUM_ERR_CUDA, "adasum_shutdown: %s", cudaGetErrorString(err));
}

}  // extern "C"
