// Shared-memory layout and launch helper of the weight-streaming kernels.
#pragma once
#include "async_copy.cuh"

namespace fasttps {

constexpr int kStreamSmemMax = 227 * 1024 - 20 * 1024;   // dynamic shared memory opt-in (static arrays come on top)

// dynamic shared memory: [ring slots][slot barriers][reduction scratch]
struct StreamSmemLayout {
    int nslot, slot_bytes, red_floats;
    size_t ring_off, bar_off, red_off, total;
};

__host__ __device__ inline StreamSmemLayout stream_smem_layout(int n_in, int R, int NB, int nwarps)
{
    StreamSmemLayout l;
    const int row_bytes = n_in * 2;
    l.nslot = ring_slots_for(row_bytes, R, kRingBudget);
    l.slot_bytes = R * row_bytes;
    l.red_floats = 2 * nwarps * R * NB > 32 * NB ? 2 * nwarps * R * NB : 32 * NB;
    l.ring_off = 0;
    l.bar_off = (size_t)l.nslot * l.slot_bytes;
    l.red_off = l.bar_off + 8 * 8;
    l.total = l.red_off + sizeof(float) * (size_t)l.red_floats;
    return l;
}

template <class Args>
static int launch_stream_kernel(void (*kernel)(Args), int grid, int threads, size_t smem, cudaStream_t st, const Args *a)
{
    void *params[] = {const_cast<Args *>(a)};
    FT_CUDA(cudaLaunchKernel(reinterpret_cast<const void *>(kernel), dim3(grid), dim3(threads), params, smem, st));
    return FASTTPS_OK;
}

template <class Args>
static cudaError_t allow_big_smem(void (*kernel)(Args))
{
    return cudaFuncSetAttribute(reinterpret_cast<const void *>(kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kStreamSmemMax);
}

}  // namespace fasttps
