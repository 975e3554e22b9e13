// Pass 1 for complete groups of 64 fp16 / bf16 workers whose buffers are rows of ONE allocation
// (buffer w starts pitch * w bytes after buffer 0): tcgen05.mma fed by bulk tensor copies.
//
// Same arithmetic and tile shape as gram_partial_tc64_kernel (X X^T, M = N = 64, K = 16 per
// instruction, accumulator in tensor memory, eight 128-byte-swizzled K-blocks of 64 rows x 128 bytes
// per tile), but the 64 rows of a K-block arrive with one cp.async.bulk.tensor instruction from a
// two-dimensional tensor map {elements, workers} over this GPU's own buffers, box {64, 64}: the copy
// engine writes the swizzled layout itself and signals the stage's mbarrier with the byte count, so
// no warp spends its time issuing 16-byte copies and waiting for them.  One thread issues the
// copies, one issues the multiplications; the other warps only take part in the epilogue (warps
// 0-3 each read the 32 tensor-memory lanes of their own quarter) and in the finish.
//
// A segment may begin or end inside a K-block (tensor boundaries are arbitrary).  Such a K-block is
// filled by a helper warp with masked loads (zeros outside the segment) instead of a tensor copy;
// K-blocks that lie wholly outside the segment are not multiplied at all.  A stage's `full`
// barrier therefore expects two arrivals per tile: the copying thread's (with the byte count of the
// tensor copies it issued) and the helper's.
//
// Every wait is bounded, as in gram_partial_tc64_kernel.
#pragma once

#include <cuda.h>

#include "adasum_kernels.cuh"

namespace adasum {

constexpr int kTmaThreads = 256;      // the finish inside pass 1 is written for blocks of at least kThreads
constexpr int kTmaStages = 3;
constexpr size_t kTmaSmemBytes = (size_t)kTmaStages * kTcTileBytes + 1024;      // + room to align to 1024

__device__ __forceinline__ void mbarrier_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// One box of the tensor map to shared memory; completion is counted in bytes on `bar`.
__device__ __forceinline__ void tensor_copy_2d(uint32_t smem_dst, const CUtensorMap* map, int x, int y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
                 : "memory");
}

// grid = (segments, groups in this launch); block = kTmaThreads; dynamic shared memory = kTmaSmemBytes.
// `rows`: tensor map with dimension 0 = elements of a buffer, dimension 1 = the operands of this
// launch, box {64, 64}, 128-byte swizzle.  row0 / pitch_elems: the same buffers for the masked loads.
template <typename T>
__global__ void __launch_bounds__(kTmaThreads, 1)
gram_partial_tc64_tma_kernel(const __grid_constant__ CUtensorMap rows, const T* __restrict__ row0, int64_t pitch_elems,
                             const Segment* __restrict__ segments, float* __restrict__ partials, int groups_total,
                             int group_base, FinishArgs fin, int* __restrict__ status)
{
    static_assert(sizeof(T) == 2, "fp16 / bf16 only");
    constexpr int R = 64;
    constexpr int E = gram_entries(R);
    constexpr int V = 8;                                   // elements per 16-byte piece
    constexpr int KB_ELEMS = 64;                           // elements of a row in one K-block
    constexpr int TILE_ELEMS = KB_ELEMS * kTcKBlocks;
    extern __shared__ __align__(1024) unsigned char tma_smem_raw[];
    __shared__ __align__(8) unsigned long long full_bar[kTmaStages], empty_bar[kTmaStages];
    __shared__ uint32_t tmem_base_slot;

    const Segment seg = segments[blockIdx.x];
    const int first = blockIdx.y * R;                      // first operand of this block's group, in this launch
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    const int64_t begin = seg.begin, end = seg.begin + seg.len;
    const int64_t k0 = begin / V * V;
    const int ntiles = (int)((end - k0 + TILE_ELEMS - 1) / TILE_ELEMS);

    const uint32_t raw_base = static_cast<uint32_t>(__cvta_generic_to_shared(tma_smem_raw));
    const uint32_t smem_base = (raw_base + 1023u) & ~1023u;
    const uint32_t full0 = static_cast<uint32_t>(__cvta_generic_to_shared(&full_bar[0]));
    const uint32_t empty0 = static_cast<uint32_t>(__cvta_generic_to_shared(&empty_bar[0]));

    if (threadIdx.x == 0) {
#pragma unroll
        for (int st = 0; st < kTmaStages; ++st) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 2;" ::"r"(full0 + 8 * st));
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

    // K-block kb of tile t covers elements [e0, e0 + 64): 2 = wholly inside the segment (tensor copy),
    // 1 = partly inside (masked loads), 0 = outside (skipped)
    auto kblock_kind = [&](int tile, int kb) -> int {
        const int64_t e0 = k0 + (int64_t)tile * TILE_ELEMS + kb * KB_ELEMS;
        if (e0 >= end || e0 + KB_ELEMS <= begin)
            return 0;
        return (e0 >= begin && e0 + KB_ELEMS <= end) ? 2 : 1;
    };

    bool timed_out = false;
    if (warp == 0) {
        if (lane == 0) {
            // ---- copying thread
            for (int tile = 0; tile < ntiles; ++tile) {
                const int stage = tile % kTmaStages;
                if (tile >= kTmaStages && !timed_out &&
                    !mbarrier_wait_bounded(empty0 + 8 * stage, (uint32_t)((tile / kTmaStages - 1) & 1)))
                    timed_out = true;
                int whole = 0;
#pragma unroll
                for (int kb = 0; kb < kTcKBlocks; ++kb)
                    whole += kblock_kind(tile, kb) == 2;
                const uint32_t bar = full0 + 8 * stage;
                mbarrier_arrive_expect_tx(bar, (uint32_t)whole * 8192u);
                const uint32_t dst = smem_base + stage * kTcTileBytes;
                const int64_t tile_elem0 = k0 + (int64_t)tile * TILE_ELEMS;
#pragma unroll
                for (int kb = 0; kb < kTcKBlocks; ++kb)
                    if (kblock_kind(tile, kb) == 2)
                        tensor_copy_2d(dst + kb * 8192, &rows, (int)(tile_elem0 + kb * KB_ELEMS), first, bar);
            }
        }
    } else if (warp == 1) {
        // ---- helper warp: the K-blocks that a segment boundary cuts
        for (int tile = 0; tile < ntiles; ++tile) {
            const int stage = tile % kTmaStages;
            if (tile >= kTmaStages && !timed_out &&
                !mbarrier_wait_bounded(empty0 + 8 * stage, (uint32_t)((tile / kTmaStages - 1) & 1)))
                timed_out = true;
            const uint32_t dst = smem_base + stage * kTcTileBytes;
            bool wrote = false;
            for (int kb = 0; kb < kTcKBlocks; ++kb) {
                if (kblock_kind(tile, kb) != 1)
                    continue;
                const int64_t e0 = k0 + (int64_t)tile * TILE_ELEMS + kb * KB_ELEMS;
                for (int p = lane; p < R * 8; p += 32) {        // 64 rows x 8 pieces of 16 bytes
                    const int r = p >> 3, c = p & 7;
                    const T* row = row0 + (int64_t)(first + r) * pitch_elems;
                    store_shared_16B(dst + kb * 8192 + r * 128 + ((c ^ (r & 7)) << 4),
                                     load_masked_words<T>(row, e0 + c * V, begin, end));
                }
                wrote = true;
            }
            if (wrote)
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // visible to the tensor core
            __syncwarp();
            if (lane == 0)
                mbarrier_arrive(full0 + 8 * stage);
        }
    } else if (warp == 2 && lane == 0) {
        // ---- multiplying thread
        constexpr uint32_t kFormat = __is_same(T, __half) ? 0u : 1u;     // 0 = fp16, 1 = bf16
        constexpr uint32_t kInstr =
            (1u << 4) | (kFormat << 7) | (kFormat << 10) | ((64u >> 3) << 17) | ((64u >> 4) << 24);
        uint32_t accumulate = 0u;
        for (int tile = 0; tile < ntiles; ++tile) {
            const int stage = tile % kTmaStages;
            if (!timed_out && !mbarrier_wait_bounded(full0 + 8 * stage, (uint32_t)((tile / kTmaStages) & 1)))
                timed_out = true;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tile_base = smem_base + stage * kTcTileBytes;
#pragma unroll
            for (int kb = 0; kb < kTcKBlocks; ++kb) {
                if (kblock_kind(tile, kb) == 0)
                    continue;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t desc = tc_smem_descriptor(tile_base + kb * 8192 + ks * 32);
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                 ::"r"(tmem_acc), "l"(desc), "l"(desc), "r"(kInstr), "r"(accumulate)
                                 : "memory");
                    accumulate = 1u;
                }
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                             empty0 + 8 * stage)
                         : "memory");
        }
    }

    // ---- epilogue: wait for the last tile's multiplications, read the accumulator rows 0..63
    {
        const int last = ntiles - 1;
        if (!timed_out &&
            !mbarrier_wait_bounded(empty0 + 8 * (last % kTmaStages), (uint32_t)((last / kTmaStages) & 1)))
            timed_out = true;
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (timed_out)
        atomicExch(status, (int)ADASUM_DEVICE_TIMEOUT);
    float* dst = partials + ((int64_t)blockIdx.x * groups_total + group_base + blockIdx.y) * E;
    if (warp < 4) {
        // rows 16 w .. 16 w + 15 of the accumulator live in tensor-memory lanes 32 w .. 32 w + 15
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
    finish_if_last<R>(fin, partials, seg.tensor, group_base + blockIdx.y, groups_total, R);
}

}  // namespace adasum
