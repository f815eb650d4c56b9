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

// y^T fragments -> FP32 accumulator `acc_g` [batch][D] in global memory.  The packed W_down orders the 32
// output columns of a block so that the four rows a lane holds of its two MMA tiles (rows g and g + 8 of tile
// m = 0, then of tile m = 1) are the CONSECUTIVE columns 4 g .. 4 g + 3 of the block: every lane adds its
// accumulators with one 16-byte red.add per batch row it holds (2 t4 and 2 t4 + 1), straight from registers --
// no staging through shared memory, no barrier.  A warp-wide instruction covers 128 contiguous bytes of each of
// four batch rows.
template <int IPW>
__device__ __forceinline__ void mlp_scatter_add(const float (&acc)[IPW][2][4], float *acc_g, int batch, int D, int nw)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, g = lane >> 2, t4 = lane & 3;
    const int b0 = 2 * t4;
    float *col = acc_g + (size_t)b0 * D + 32 * w + 4 * g;    // one running address: the step per i is 32 nw columns
#pragma unroll
    for (int i = 0; i < IPW; ++i) {
        if (b0 < batch) red_add_v4(col, acc[i][0][0], acc[i][0][2], acc[i][1][0], acc[i][1][2]);
        if (b0 + 1 < batch) red_add_v4(col + D, acc[i][0][1], acc[i][0][3], acc[i][1][1], acc[i][1][3]);
        col += 32 * nw;
    }
}

}  // namespace fasttps
