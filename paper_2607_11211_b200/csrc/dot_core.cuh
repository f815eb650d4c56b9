// Weight-streaming dot-product core shared by the projection kernel and the
// gate_up half of the fused MLP kernel.
//
// Layout: W is [rows][n_in] bf16 with every row (one output feature) contiguous.
// A CTA of ceil(n_in / 8 / 32) warps owns a contiguous range of rows, which is one
// contiguous byte range of the matrix.  The range arrives through the shared-memory
// weight ring (bulk asynchronous copies, R rows per group, several groups in
// flight).  Thread t owns the 16-byte k-slice [8t, 8t+8) of EVERY row and keeps its
// slice of the activations in registers (FP32, NB batch rows).  The R*NB partial sums
// of a group are reduced with a halving butterfly (about one shuffle per value), meet
// in shared memory (one block barrier per group, double buffered) and are handed to
// the epilogue by the first R*NB threads.
#pragma once
#include "async_copy.cuh"

namespace fasttps {

template <int NB> struct RowsPerGroup { static constexpr int value = (NB <= 4) ? 8 : 4; };

constexpr int kRingBudget = 192 * 1024;     // shared memory given to the weight ring

// Loads this thread's activation slice: x[b][8t .. 8t+8) for NB batch rows, with an
// optional RMSNorm (gain g, eps) whose result is rounded to bf16 like a stored tensor.
// smem_red: at least 32 * NB floats.  All threads of the CTA must call.
template <int NB>
__device__ __forceinline__ void load_activations(float (&x)[NB][8], const __nv_bfloat16 *xg, int x_stride,
                                                 int batch, int n_in, const __nv_bfloat16 *g, float eps,
                                                 float *smem_red)
{
    const int t = threadIdx.x;
    const bool active = t * 8 < n_in;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        if (active && b < batch) {
            uint4 v = *reinterpret_cast<const uint4 *>(xg + (size_t)b * x_stride + t * 8);
            unpack8(v, x[b]);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) x[b][i] = 0.f;
        }
    }
    if (g == nullptr) return;
    const int lane = t & 31, warp = t >> 5, nwarps = (blockDim.x + 31) >> 5;
    float ss[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) s += x[b][i] * x[b][i];
        ss[b] = warp_sum(s);
    }
    if (lane == 0) {
#pragma unroll
        for (int b = 0; b < NB; ++b) smem_red[warp * NB + b] = ss[b];
    }
    __syncthreads();
    float gv[8];
    if (active) {
        uint4 v = *reinterpret_cast<const uint4 *>(g + t * 8);
        unpack8(v, gv);
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) gv[i] = 0.f;
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        float tot = 0.f;
        for (int w = 0; w < nwarps; ++w) tot += smem_red[w * NB + b];
        const float r = rsqrtf(tot / (float)n_in + eps);
#pragma unroll
        for (int i = 0; i < 8; ++i) x[b][i] = bf16_round(x[b][i] * r * gv[i]);
    }
    __syncthreads();   // smem_red may be reused by the caller
}

// Consumes ring groups [g0, g0 + ceil(nrows / R)) = rows [row0, row0 + nrows) of a matrix and
// calls epi(row, b, value) for every row and batch row b < NB, from threads 0 .. R*NB-1 (one
// (row, b) pair per thread and group).  smem_red: 2 * nwarps * R * NB floats.  All threads of
// the CTA must call.  Returns false if a bounded wait ran out (the CTA must then leave).
template <int NB, class Epi>
__device__ __forceinline__ bool dot_rows(WeightRing &ring, int g0, int n_in, int row0, int nrows,
                                         const float (&x)[NB][8], float *smem_red, Epi epi)
{
    constexpr int R = RowsPerGroup<NB>::value;
    constexpr int V = R * NB;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5, nwarps = (blockDim.x + 31) >> 5;
    const bool active = t * 8 < n_in;
    const int nvec = n_in >> 3;
    const int ngroups = (nrows + R - 1) / R;
    bool ok = true;
    for (int g = 0; g < ngroups; ++g) {
        const int buf = g & 1;
        const uint4 *slot = reinterpret_cast<const uint4 *>(ring.wait(g0 + g, ok));
        float p[V];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float wf[8];
            const uint4 w = active ? slot[r * nvec + t] : make_uint4(0, 0, 0, 0);
            unpack8(w, wf);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                float s = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) s = fmaf(wf[i], x[b][i], s);
                p[r * NB + b] = s;
            }
        }
        const float tot = warp_multi_reduce<V>(p, lane);
        constexpr int rep = 32 / V;                       // lanes sharing one value
        if ((lane & (rep - 1)) == 0) smem_red[(buf * nwarps + warp) * V + warp_multi_which<V>(lane)] = tot;
        if (!__syncthreads_and(ok ? 1 : 0)) return false; // every warp is done with the slot
        if (t == 0) ring.refill(g0 + g);
        if (t < V) {
            float s = 0.f;
            for (int w2 = 0; w2 < nwarps; ++w2) s += smem_red[(buf * nwarps + w2) * V + t];
            const int row = g * R + t / NB;
            if (row < nrows) epi(row0 + row, t % NB, s);
        }
    }
    return true;
}

}  // namespace fasttps
