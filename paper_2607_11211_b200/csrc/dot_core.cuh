// Tensor-core weight-streaming core shared by the projection kernel and the fused MLP kernel.
//
// Why tensor cores at batch 1: with FP32 FMAs every 16 bytes of bf16 weights cost 8 unpack
// instructions, 8 FMAs and a share of a cross-lane reduction; at the HBM rate of a B200 that is
// more warp-instructions than an SM with a handful of warps can issue (measured: issue-bound at
// ~5.3 TB/s).  One mma.sync.m16n8k16 consumes 512 bytes of weights with one instruction, takes
// bf16 directly, reduces over k inside the instruction and serves up to 8 batch rows for free.
//
// Packed layout ("tiled", written by the packing kernels): an [n_out][n_in] matrix is cut into
// tiles of 16 rows x 32 k, each tile stored row-major (1 KB), tiles ordered by (row tile, k block).
// A warp reads a tile with two conflict-free 16-byte shared loads per lane: lane (g = lane / 4,
// t4 = lane % 4) gets W[row g][8 t4 .. 8 t4 + 8) and W[row g + 8][same k].  Those 8 consecutive k
// of the two rows are exactly the A fragments of TWO m16n8k16 MMAs if the k index inside the MMA
// is permuted; the same permutation makes the B fragments of both MMAs one contiguous 16-byte
// piece x[batch row g][8 t4 .. 8 t4 + 8) of the bf16 activations.
//
// Work split inside a CTA: n_in / 32 k blocks per row tile are dealt round-robin to NW consumer
// warps, IPW blocks each (n_in = 32 * NW * IPW).  A warp keeps the B fragments of its IPW k
// blocks in registers for the whole kernel, accumulates a 16 x 8 partial tile over its blocks,
// and the NW partial tiles of a row tile meet in shared memory (one named barrier per 16 rows).
#pragma once
#include "async_copy.cuh"

namespace fasttps {

constexpr int kRingBudget = 192 * 1024;     // shared memory given to the weight ring
constexpr int kTileBytes = 1024;            // 16 rows x 32 k bf16
constexpr int kBlocksPerWarpPerSlot = 2;    // a slot holds 2 k blocks of every consumer warp

__device__ __forceinline__ void mma_bf16_k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16_k8(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0)
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(b0));
}

// How a reduction length n_in maps onto consumer warps: n_in = 32 * nw * ipw, ipw in {4, 8}.
struct WarpSplit { int nw, ipw; };
__host__ __device__ inline WarpSplit warp_split(int n_in)
{
    WarpSplit s = {0, 0};
    if (n_in >= 2048 && n_in % 256 == 0 && n_in / 256 <= 24) { s.nw = n_in / 256; s.ipw = 8; }
    else if (n_in % 128 == 0 && n_in / 128 <= 24) { s.nw = n_in / 128; s.ipw = 4; }
    return s;
}

// B fragments of this consumer thread: the bf16 activations x[g][32 (w + nw i) + 8 t4 .. + 8) for its
// IPW k blocks, batch row g = lane / 4 (zero for g >= batch), optionally RMS-normalised (gain gn, eps)
// with the result rounded to bf16 like a stored tensor.  Consumer threads only (named barrier 1).
// smem_red: nw * 8 floats.  If `add` is given (FP32 [batch][n_in], e.g. the MLP partial sums of the
// previous layer), the activation is bf16(x + add); if `store` is given, that activation (before the norm) is
// also written out, one share of its 16-byte chunks per CTA.  All loads bypass L1: inside a persistent kernel
// the activations were written by other SMs.
// The same for ONE batch row (batch 1): the 4 * IPW chunks of 8 elements a warp needs are spread over its lanes,
// one chunk per lane, instead of IPW chunks in each of the four lanes of row 0 -- an eighth of the loads,
// conversions and multiplies per thread -- and the finished chunks are handed out with shuffles.  The fragment
// words of the lanes of the unused batch columns (lane / 4 > 0) carry copies, which the products ignore.
template <int IPW>
__device__ __forceinline__ void load_b_frags_one_row(uint32_t (&bf)[IPW][4], const __nv_bfloat16 *x, int n_in, int nw,
                                                     const __nv_bfloat16 *gn, float eps, float *smem_red,
                                                     const float *add = nullptr, __nv_bfloat16 *store = nullptr,
                                                     int store_rem = 0, int store_mod = 1)
{
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    const int ci = lane >> 2 < IPW ? lane >> 2 : 0;            // this lane's chunk: k block ci of the warp, quarter lane % 4
    const bool mine = (lane >> 2) < IPW;
    const int k = 32 * (w + nw * ci) + 8 * (lane & 3);
    uint4 gq = make_uint4(0u, 0u, 0u, 0u);
    if (gn) gq = *reinterpret_cast<const uint4 *>(gn + k);
    uint4 v = ld_cg_u4(x + k);
    if (add) {
        const float4 a0 = ld_cg_f4(add + k), a1 = ld_cg_f4(add + k + 4);
        v.x = pack2(bf_lo(v.x) + a0.x, bf_hi(v.x) + a0.y);
        v.y = pack2(bf_lo(v.y) + a0.z, bf_hi(v.y) + a0.w);
        v.z = pack2(bf_lo(v.z) + a1.x, bf_hi(v.z) + a1.y);
        v.w = pack2(bf_lo(v.w) + a1.z, bf_hi(v.w) + a1.w);
    }
    if (store != nullptr && mine && (k >> 3) % store_mod == store_rem) *reinterpret_cast<uint4 *>(store + k) = v;
    uint32_t q[4] = {v.x, v.y, v.z, v.w};
    if (gn != nullptr) {
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float lo = bf_lo(q[j]), hi = bf_hi(q[j]);
            ss = fmaf(lo, lo, ss);
            ss = fmaf(hi, hi, ss);
        }
        if (!mine) ss = 0.f;
        ss = warp_sum(ss);
        if (lane == 0) smem_red[w] = ss;                        // row 0 of the [row][warp] layout
        named_bar_sync(1, nw * 32);
        float tot = 0.f;
        if ((nw & 3) == 0) {
            for (int w4 = 0; w4 < nw; w4 += 4) {
                const float4 p = *reinterpret_cast<const float4 *>(smem_red + w4);
                tot += (p.x + p.y) + (p.z + p.w);
            }
        } else {
            for (int w2 = 0; w2 < nw; ++w2) tot += smem_red[w2];
        }
        const float r = rsqrtf(tot / (float)n_in + eps);
        const uint32_t gg[4] = {gq.x, gq.y, gq.z, gq.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) q[j] = pack2(bf_lo(q[j]) * r * bf_lo(gg[j]), bf_hi(q[j]) * r * bf_hi(gg[j]));
        named_bar_sync(1, nw * 32);   // smem_red may be reused by the caller
    }
#pragma unroll
    for (int i = 0; i < IPW; ++i) {
        const int src = i * 4 + (lane & 3);
#pragma unroll
        for (int j = 0; j < 4; ++j) bf[i][j] = __shfl_sync(kFull, q[j], src);
    }
}

template <int IPW>
__device__ __forceinline__ void load_b_frags(uint32_t (&bf)[IPW][4], const __nv_bfloat16 *x, int x_stride, int batch,
                                             int n_in, int nw, const __nv_bfloat16 *gn, float eps, float *smem_red,
                                             const float *add = nullptr, __nv_bfloat16 *store = nullptr,
                                             int store_rem = 0, int store_mod = 1)
{
    const int t = threadIdx.x, lane = t & 31, w = t >> 5, g = lane >> 2, t4 = lane & 3;
    const bool live = g < batch;
    // Every load is issued unconditionally (rows beyond the batch read row 0 and are zeroed afterwards): with
    // no branch around them all loads of a thread go out back to back and cost ONE round trip to L2.
    const int gr = live ? g : 0;
#pragma unroll
    for (int i = 0; i < IPW; ++i) {
        const uint4 v = ld_cg_u4(x + (size_t)gr * x_stride + 32 * (w + nw * i) + 8 * t4);
        bf[i][0] = v.x; bf[i][1] = v.y; bf[i][2] = v.z; bf[i][3] = v.w;
    }
    if (add) {
#pragma unroll
        for (int h = 0; h < IPW; h += 4) {                  // four k blocks (32 registers) of addends in flight
            float4 a0[4], a1[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float *p = add + (size_t)gr * n_in + 32 * (w + nw * (h + u)) + 8 * t4;
                a0[u] = ld_cg_f4(p);
                a1[u] = ld_cg_f4(p + 4);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                uint32_t(&v)[4] = bf[h + u];
                v[0] = pack2(bf_lo(v[0]) + a0[u].x, bf_hi(v[0]) + a0[u].y);
                v[1] = pack2(bf_lo(v[1]) + a0[u].z, bf_hi(v[1]) + a0[u].w);
                v[2] = pack2(bf_lo(v[2]) + a1[u].x, bf_hi(v[2]) + a1[u].y);
                v[3] = pack2(bf_lo(v[3]) + a1[u].z, bf_hi(v[3]) + a1[u].w);
            }
        }
    }
    if (!live) {
#pragma unroll
        for (int i = 0; i < IPW; ++i) bf[i][0] = bf[i][1] = bf[i][2] = bf[i][3] = 0u;
    }
    if (store != nullptr && live) {
        // the activation before normalisation is kept as a tensor: of the grid's CTAs, which all hold it, the one
        // with number store_rem (of store_mod) writes every store_mod-th 16-byte chunk
#pragma unroll
        for (int i = 0; i < IPW; ++i) {
            const int k = 32 * (w + nw * i) + 8 * t4;
            if ((k >> 3) % store_mod == store_rem)
                *reinterpret_cast<uint4 *>(store + (size_t)g * x_stride + k) = make_uint4(bf[i][0], bf[i][1], bf[i][2], bf[i][3]);
        }
    }
    if (gn == nullptr) return;
    uint4 gv[IPW];                      // the gains are fetched before the reduction, not after its barrier
#pragma unroll
    for (int i = 0; i < IPW; ++i) gv[i] = *reinterpret_cast<const uint4 *>(gn + 32 * (w + nw * i) + 8 * t4);
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < IPW; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float lo = bf_lo(bf[i][j]), hi = bf_hi(bf[i][j]);
            ss = fmaf(lo, lo, ss);
            ss = fmaf(hi, hi, ss);
        }
    ss += __shfl_xor_sync(kFull, ss, 1);
    ss += __shfl_xor_sync(kFull, ss, 2);
    if (t4 == 0) smem_red[g * nw + w] = ss;             // [row][warp]: a row's partial sums are contiguous
    named_bar_sync(1, nw * 32);
    float tot = 0.f;
    if ((nw & 3) == 0) {
        for (int w4 = 0; w4 < nw; w4 += 4) {
            const float4 p = *reinterpret_cast<const float4 *>(smem_red + g * nw + w4);
            tot += (p.x + p.y) + (p.z + p.w);
        }
    } else {
        for (int w2 = 0; w2 < nw; ++w2) tot += smem_red[g * nw + w2];
    }
    const float r = rsqrtf(tot / (float)n_in + eps);
#pragma unroll
    for (int i = 0; i < IPW; ++i) {
        const uint32_t gg[4] = {gv[i].x, gv[i].y, gv[i].z, gv[i].w};
#pragma unroll
        for (int j = 0; j < 4; ++j)
            bf[i][j] = pack2(bf_lo(bf[i][j]) * r * bf_lo(gg[j]), bf_hi(bf[i][j]) * r * bf_hi(gg[j]));
    }
    named_bar_sync(1, nw * 32);   // smem_red may be reused by the caller
}

// Consumes ring pieces [g0, g0 + ntiles * IPW / 2) = `ntiles` row tiles of a tiled matrix and calls
// epi(tile, c, b, v_lo, v_hi) from consumer threads 0..63 with the finished sums of rows c and c + 8
// (c = 0..7) of the tile for batch row b = 0..7.  smem_part: 2 * nw * 128 floats.  Consumer threads
// only.  Returns false if a bounded wait ran out.
template <int IPW, class Epi>
__device__ __forceinline__ bool dot_tiles(WeightRing &ring, int g0, int ntiles, int nw, const uint32_t (&bf)[IPW][4],
                                          float *smem_part, Epi epi)
{
    constexpr int SPT = IPW / kBlocksPerWarpPerSlot;      // ring pieces per row tile
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    bool ok = true;
#pragma unroll 1
    for (int tile = 0; tile < ntiles; ++tile) {
        float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int q = 0; q < SPT; ++q) {
            const int piece = g0 + tile * SPT + q;
            const unsigned char *slot = ring.wait(piece, ok);
#pragma unroll
            for (int s = 0; s < kBlocksPerWarpPerSlot; ++s) {
                const unsigned char *blk = slot + (size_t)(s * nw + w) * kTileBytes + lane * 16;
                const uint4 lo = *reinterpret_cast<const uint4 *>(blk);          // row g,     k 8 t4 ..
                const uint4 hi = *reinterpret_cast<const uint4 *>(blk + 512);    // row g + 8, k 8 t4 ..
                const int i = q * kBlocksPerWarpPerSlot + s;
                mma_bf16_k16(c, lo.x, hi.x, lo.y, hi.y, bf[i][0], bf[i][1]);
                mma_bf16_k16(c, lo.z, hi.z, lo.w, hi.w, bf[i][2], bf[i][3]);
            }
            ring.release(piece);
        }
        // partial 16 x 8 tiles of the nw warps meet in shared memory (double buffered)
        float *part = smem_part + (size_t)(tile & 1) * nw * 128;
        *reinterpret_cast<float4 *>(part + (size_t)w * 128 + lane * 4) = make_float4(c[0], c[1], c[2], c[3]);
        if (!named_bar_and(1, nw * 32, ok)) return false;   // same verdict in every consumer thread
        for (int u = t; u < 64; u += nw * 32) {
            // fragment layout: lane (g, t4) holds rows g / g + 8, batch columns 2 t4 / 2 t4 + 1
            const int cc = u >> 3, b = u & 7;
            const int idx = (cc * 4 + (b >> 1)) * 4 + (b & 1);
            float v0 = 0.f, v1 = 0.f;
            for (int w2 = 0; w2 < nw; ++w2) {
                v0 += part[(size_t)w2 * 128 + idx];
                v1 += part[(size_t)w2 * 128 + idx + 2];
            }
            epi(tile, cc, b, v0, v1);
        }
    }
    return true;
}

}  // namespace fasttps
