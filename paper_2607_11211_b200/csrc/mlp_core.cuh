// Device-side phases of the fused SwiGLU MLP (Algorithm 4 / Eq. 1 / Eq. 31 of the paper), shared by the
// stand-alone MLP kernel and the persistent decode-step kernel.  A CTA owns `noct` consecutive j-octets
// (8 intermediate columns each):
//   gate_up phase  one 16-row tile per octet of the packed gate_up matrix (8 gate rows, then the 8
//                  matching up rows) times the activations on the tensor cores; the accumulator
//                  fragment of a lane holds a gate value and ITS up value (rows g and g + 8); the
//                  finished sums go through a = silu(gate) * up and stay in shared memory as a
//                  bf16 hi + lo pair (so the down projection sees ~16 mantissa bits of a),
//   down phase     the matching octets of the packed W_down (m16n8k8 fragments: 32 output columns x 8
//                  intermediate columns per 512-byte block) accumulate y^T[n, b] in registers, each
//                  warp owning a fixed set of output columns,
//   scatter        the partial y goes through shared memory into an FP32 accumulator in global memory
//                  with vector red.add.
#pragma once
#include "dot_core.cuh"

namespace fasttps {

constexpr int kMaxOctetsPerCta = 16;      // bounds the shared-memory intermediate

typedef __nv_bfloat16 ActTile[8][8];      // [batch row][j in octet]

template <int IPW>
__device__ __forceinline__ bool mlp_gate_up_phase(WeightRing &ring, int piece0, int noct, int nw,
                                                  const uint32_t (&bf)[IPW][4], float *smem_part, ActTile *s_hi,
                                                  ActTile *s_lo)
{
    return dot_tiles<IPW>(ring, piece0, noct, nw, bf, smem_part, [&](int tile, int cc, int b, float gate, float up) {
        const float act = gate / (1.f + __expf(-gate)) * up;
        const __nv_bfloat16 hi = __float2bfloat16_rn(act);
        s_hi[tile][b][cc] = hi;
        s_lo[tile][b][cc] = __float2bfloat16_rn(act - __bfloat162float(hi));
    });
}

// Consumes ring pieces [piece0, piece0 + noct * IPW / 4).  acc must be zero on entry.  `ok` is cleared on a
// failed wait (the caller turns it into a CTA-wide verdict at its next barrier).
template <int IPW>
__device__ __forceinline__ void mlp_down_phase(WeightRing &ring, int piece0, int noct, int nw, const ActTile *s_hi,
                                               const ActTile *s_lo, float (&acc)[IPW][2][4], bool &ok)
{
    constexpr int PPO = IPW / 4;                            // ring pieces per octet
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, g = lane >> 2, t4 = lane & 3;
#pragma unroll 1
    for (int o = 0; o < noct; ++o) {
        const uint32_t bh = *reinterpret_cast<const uint32_t *>(&s_hi[o][g][2 * t4]);
        const uint32_t bl = *reinterpret_cast<const uint32_t *>(&s_lo[o][g][2 * t4]);
#pragma unroll
        for (int q = 0; q < PPO; ++q) {
            const int piece = piece0 + o * PPO + q;
            const unsigned char *slot = ring.wait(piece, ok);
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                const uint4 r = *reinterpret_cast<const uint4 *>(slot + (size_t)(s * nw + w) * 512 + lane * 16);
                const int i = q * 4 + s;
                mma_bf16_k8(acc[i][0], r.x, r.y, bh);
                mma_bf16_k8(acc[i][0], r.x, r.y, bl);
                mma_bf16_k8(acc[i][1], r.z, r.w, bh);
                mma_bf16_k8(acc[i][1], r.z, r.w, bl);
            }
            ring.release(piece);
        }
    }
}

// One round of mlp_scatter_add: the staged chunks i0 .. i0 + nchunk - 1 go to global memory.  Out of line: the
// caller is unrolled over the chunks and would carry a copy of this loop for each of them.
static __device__ __noinline__ void mlp_scatter_drain(const float *stage, float *acc_g, int i0, int nchunk, int batch, int D,
                                                      int cw, int nct)
{
    const int t = threadIdx.x, per_row = cw >> 2;
    named_bar_sync(1, nct);
    for (int idx = t; idx < nchunk * batch * per_row; idx += nct) {
        const int cb = idx / per_row, j = idx - cb * per_row;      // cb = chunk * batch + b
        const int ch = cb / batch, b = cb - ch * batch;
        const float4 v = *reinterpret_cast<const float4 *>(stage + (size_t)cb * cw + 4 * j);
        red_add_v4(acc_g + (size_t)b * D + (size_t)cw * (i0 + ch) + 4 * j, v.x, v.y, v.z, v.w);
    }
}

// y^T fragments -> FP32 accumulator `acc_g` [batch][D] in global memory with vector red.add, staged
// through shared memory in IPW chunks of 32 * nw output columns (the columns the warps own for one
// value of i are one contiguous chunk), several chunks per round when the batch is small.  stage:
// 8 * 32 * nw floats that are idle (the partial-tile scratch of the gate_up phase).  Consumer threads
// only (named barrier 1).
template <int IPW>
__device__ __forceinline__ void mlp_scatter_add_block(const float (&acc)[IPW][2][4], float *stage, float *acc_g, int batch,
                                                int D, int nw)
{
    const int t = threadIdx.x, lane = t & 31, w = t >> 5, g = lane >> 2, t4 = lane & 3, nct = nw * 32;
    const int cw = 32 * nw;                                  // chunk width in columns
    // chunks staged per round: as many as the stage holds (all 8 at batch 1: one barrier instead of fifteen)
    const int R = batch <= 1 ? 8 : (batch <= 2 ? 4 : (batch <= 4 ? 2 : 1));
#pragma unroll
    for (int i = 0; i < IPW; ++i) {
        const int ir = i % R;                                // slot of chunk i inside the round
        if (ir == 0 && i > 0) named_bar_sync(1, nct);        // the previous round has been read
        float *st = stage + (size_t)ir * batch * cw;
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            const int n = 32 * w + 16 * m + g;
            const int b0 = 2 * t4;
            if (b0 < batch) { st[b0 * cw + n] = acc[i][m][0]; st[b0 * cw + n + 8] = acc[i][m][2]; }
            if (b0 + 1 < batch) { st[(b0 + 1) * cw + n] = acc[i][m][1]; st[(b0 + 1) * cw + n + 8] = acc[i][m][3]; }
        }
        if (ir == R - 1 || i == IPW - 1) mlp_scatter_drain(stage, acc_g, i - ir, ir + 1, batch, D, cw, nct);
    }
}


// One round of mlp_scatter_add_warp: the warp's staged rows go to global memory.  Out of line: the caller is
// unrolled over the chunks and would carry a copy of this loop for each of them.
static __device__ __noinline__ void mlp_scatter_drain_warp(const float *st, float *acc_g, int i0, int nrow, int batch, int D,
                                                           int nw)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    __syncwarp();
    for (int idx = lane; idx < nrow * 8; idx += 32) {
        const int row = idx >> 3, j = idx & 7;
        const int ch = row / batch, b = row - ch * batch;
        const float4 v = *reinterpret_cast<const float4 *>(st + row * 32 + (((j ^ row) & 7) << 2));
        red_add_v4(acc_g + (size_t)b * D + 32 * (nw * (i0 + ch) + w) + 4 * j, v.x, v.y, v.z, v.w);
    }
}

// The same scatter for larger batches, where the block-wide version would need two block-wide barriers per
// value of i.  For a given i a
// warp owns 32 contiguous output columns, 32 (nw i + w) .. + 32, so the transposition from fragment order to
// rows of 4 consecutive columns is private to the warp: it goes through the warp's own 1 KB of `stage`
// (8 * 32 * nw floats that are idle: the partial-tile scratch of the gate_up phase) with no block-wide barrier.
// The region holds R = 8 / batch' values of i at a time as rows [chunk][batch row][32 columns]; the eight
// 4-column groups of a row are XOR-swizzled with the row index, which makes both the fragment-order writes and
// the 16-byte row reads free of bank conflicts.
template <int IPW>
__device__ __forceinline__ void mlp_scatter_add_warp(const float (&acc)[IPW][2][4], float *stage, float *acc_g, int batch,
                                                int D, int nw)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, g = lane >> 2, t4 = lane & 3;
    const int R = batch <= 1 ? 8 : (batch <= 2 ? 4 : (batch <= 4 ? 2 : 1));
    float *st = stage + w * 256;
#pragma unroll
    for (int i = 0; i < IPW; ++i) {
        const int ir = i % R;                                // slot of chunk i inside the round
        if (ir == 0 && i > 0) __syncwarp();                  // the previous round has been read
#pragma unroll
        for (int m = 0; m < 2; ++m) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int b = 2 * t4 + (e & 1), n = 16 * m + g + 8 * (e >> 1);
                const int row = ir * batch + b;
                if (b < batch) st[row * 32 + ((((n >> 2) ^ row) & 7) << 2) + (n & 3)] = acc[i][m][e];
            }
        }
        if (ir == R - 1 || i == IPW - 1) mlp_scatter_drain_warp(st, acc_g, i - ir, (ir + 1) * batch, batch, D, nw);
    }
}

// WARP_PRIVATE: which of the two a caller wants (small batches: block-wide, one barrier in all; larger: per warp).
template <int IPW, bool WARP_PRIVATE>
__device__ __forceinline__ void mlp_scatter_add(const float (&acc)[IPW][2][4], float *stage, float *acc_g, int batch,
                                                int D, int nw)
{
    if (WARP_PRIVATE) mlp_scatter_add_warp<IPW>(acc, stage, acc_g, batch, D, nw);
    else mlp_scatter_add_block<IPW>(acc, stage, acc_g, batch, D, nw);
}

}  // namespace fasttps
