// Shared-memory layout and launch helper of the weight-streaming kernels.
#pragma once
#include "dot_core.cuh"

namespace fasttps {

constexpr int kStreamSmemMax = 227 * 1024 - 12 * 1024;   // dynamic shared memory opt-in (static arrays come on top)

// dynamic shared memory: [ring slots][full + empty barriers][abort word][partial tiles][norm scratch]
struct StreamSmemLayout {
    int nw, ipw, nslot, slot_bytes;
    size_t ring_off, bar_off, abort_off, part_off, red_off, total;
};

__host__ __device__ inline StreamSmemLayout stream_smem_layout(int n_in)
{
    StreamSmemLayout l;
    const WarpSplit s = warp_split(n_in);
    l.nw = s.nw; l.ipw = s.ipw;
    l.slot_bytes = kBlocksPerWarpPerSlot * (s.nw > 0 ? s.nw : 1) * kTileBytes;
    l.nslot = kRingBudget / l.slot_bytes;
    l.nslot = l.nslot >= 8 ? 8 : l.nslot >= 4 ? 4 : l.nslot >= 2 ? 2 : l.nslot;   // a power of two (ring indexing by mask and shift)
    l.ring_off = 0;
    l.bar_off = (size_t)l.nslot * l.slot_bytes;
    l.abort_off = l.bar_off + 2 * 8 * 8;
    l.part_off = l.abort_off + 16;
    l.red_off = l.part_off + sizeof(float) * 2 * (size_t)s.nw * 128;
    l.total = l.red_off + sizeof(float) * (size_t)s.nw * 8;
    return l;
}

template <class Args>
static int launch_stream_kernel(void (*kernel)(Args), int grid, int threads, size_t smem, cudaStream_t st, const Args *a)
{
    return launch_ex(kernel, dim3(grid), dim3(threads), smem, st, a);
}

template <class Args>
static cudaError_t allow_big_smem(void (*kernel)(Args))
{
    return cudaFuncSetAttribute(reinterpret_cast<const void *>(kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kStreamSmemMax);
}

}  // namespace fasttps
