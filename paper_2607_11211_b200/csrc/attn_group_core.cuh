// Decode attention for grouped-query models (Section 4.1 of the paper: G query heads read one K/V head;
// Algorithm 3 is otherwise unchanged): every cached K/V row is fetched ONCE for its whole group.
//
// With G query vectors per row the two products of Algorithm 3 are thin matrix products, so they run on the
// tensor cores (the FP32 dot products of attn_core.cuh already keep the ALUs as busy as HBM at G = 1; G times
// the arithmetic per byte would make the kernel compute-bound):
//   scores  S[head, key] = Q[head, :] . K[key, :]      mma m16n8k16, A = Q (8 heads in the rows; rows 8..15
//                                                       are padding), B = 8 keys of the tile
//   output  O[head, col] += P[head, key] V[key, col]    mma m16n8k16, A = P straight from two score fragments
// A tile of the ring holds 64 rows; consumer warps 0-3 own 16 rows each of the even pieces, warps 4-7 of the odd
// ones, and every warp keeps its own running (max, sum, output) for the G heads; the warps' states are merged
// per segment as in attn_core.cuh.
// Operand order is free inside a dot product, so the head_dim index is permuted such that one 16-byte load of a
// K row feeds two MMAs, and the output columns are permuted such that two V rows loaded as 32-bit words give
// the B operands of two MMAs after a byte permute (no transposing load, no swizzled tile).
// Precision.  The tensor cores take bf16 operands; K and V ARE bf16, but the rotated q and the softmax weights are
// FP32 values.  PRECISE (the default): both enter their product as a bf16 hi + lo pair (two MMAs each, about 16
// mantissa bits), so the result matches the FP32 path of attn_core.cuh to rounding and a layer built on it meets the
// same bars.  Without it (option "gqa_share" 2) they are rounded to bf16 once: faster, but the deviation of a layer
// output from the oracle was measured 4.5 times larger (rms 0.015 against 0.0034 on a Llama3-8B-shaped layer).
// FP8: the cache holds E4M3 codes (one byte per element, value = code * scale with one scale per tensor).  A tile of
// the ring then holds 128 rows (the same bytes as 64 bf16 rows); the codes are widened to fp16 in registers (exact:
// every E4M3 value, subnormals included, is a normal fp16 number), the MMAs take fp16 operands, q and the softmax
// weights go in as fp16 hi + lo pairs, and the two scales are applied to the scores and to the outputs once.
#pragma once
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include "attn_core.cuh"
#include "dot_core.cuh"

namespace fasttps {

constexpr int kMaxShareGroup = 16;       // query heads per K/V head this path serves (2 to 16)
constexpr int kHeadsPerWarp = 8;         // heads in the rows of one warp's MMAs
constexpr int kGroupWarps = 8;           // consumer warps: two sets of four, 16 rows of a tile each

template <int DH>
struct GroupScratch {
    alignas(16) float q[kMaxShareGroup][DH];            // rope(q) of the group, FP32
    alignas(16) __nv_bfloat16 knew[kMaxNB][DH];         // bf16(rope(k_new)): the rows that go into the cache (one per new token)
    alignas(16) __nv_bfloat16 vnew[kMaxNB][DH];
    float wm[kGroupWarps][kHeadsPerWarp], wl[kGroupWarps][kHeadsPerWarp];     // per warp and head slot: max (log2 domain), sum
    alignas(16) float wo[kGroupWarps][kHeadsPerWarp][DH];
    int last;
};


// The MMAs of this path use rows 0..7 of the 16-row tile only (rows 8..15 of A are zero): the lower half of the
// accumulator fragment is not kept (its inputs are constants, its outputs are dropped), which halves the
// registers the running outputs take.
template <bool F16 = false>
__device__ __forceinline__ void mma_top_k16(float (&c)[2], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    float d2, d3;
    if constexpr (F16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%5}, {%7,%8}, {%0,%1,%9,%9};"
                     : "+f"(c[0]), "+f"(c[1]), "=f"(d2), "=f"(d3)
                     : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1), "f"(0.f));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%5}, {%7,%8}, {%0,%1,%9,%9};"
                     : "+f"(c[0]), "+f"(c[1]), "=f"(d2), "=f"(d3)
                     : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1), "f"(0.f));
}

// the whole 16-row product (the output product: rows = 16 output columns, n = 8 members, k = 16 keys)
template <bool F16 = false>
__device__ __forceinline__ void mma_k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    if constexpr (F16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// two FP32 values as one register of two 16-bit floats (x in the low half), and what that rounding keeps of a value
template <bool F16>
__device__ __forceinline__ uint32_t pack2t(float x, float y)
{
    if constexpr (F16) {
        const __half2 h = __floats2half2_rn(x, y);
        return *reinterpret_cast<const uint32_t *>(&h);
    } else {
        return pack2(x, y);
    }
}
template <bool F16>
__device__ __forceinline__ float round16(float x)
{
    if constexpr (F16) return __half2float(__float2half_rn(x));
    else return bf16_round(x);
}
// two E4M3 codes (the low 16 bits of c) as two fp16 numbers
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t c)
{
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(c & 0xffffu), __NV_E4M3);
    return (uint32_t)h.x | ((uint32_t)h.y << 16);
}

// Consumer warps (kGroupWarps of them, threads 0 .. 255, synchronised by named barrier 1).  The segments of
// `src` are K/V heads (WalkSource with share = true).  Returns false in every thread if a bounded wait ran out.
template <int DH, bool PRECISE, bool FP8 = false>
__device__ __forceinline__ bool attn_consume_group(const AttnArgs &a, WeightRing &ring, int &piece, int cta, WalkSource src,
                                                   GroupScratch<DH> &sm)
{
    static_assert(PRECISE || !FP8, "the E4M3 path always takes q and the weights as hi + lo pairs");
    constexpr int HALF = DH / 2;
    constexpr int KB = DH / 32;                  // 32-wide blocks of head_dim in the score product
    constexpr int CB = DH / 32;                  // 32-column blocks of the output
    constexpr int EB = FP8 ? 1 : 2;              // bytes per cache element
    constexpr int TR = FP8 ? 2 * kAttnTileRows : kAttnTileRows;      // rows per tile of the ring
    constexpr int kRowBytes = DH * EB;
    constexpr int kPartStride = DH + 4;
    unsigned char *const kc8 = reinterpret_cast<unsigned char *>(a.k_cache), *const vc8 = reinterpret_cast<unsigned char *>(a.v_cache);
    unsigned char *const knew8 = reinterpret_cast<unsigned char *>(&sm.knew[0][0]), *const vnew8 = reinterpret_cast<unsigned char *>(&sm.vnew[0][0]);
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5, g = lane >> 2, t4 = lane & 3;
    const int nct = kGroupWarps * 32;
    const int Gh = a.n_q_heads / a.n_kv_heads, N = a.n_new;
    // The members of a group are the query heads of the K/V head, for every new token of the sequence: member
    // m = j * Gh + g2 is head g2 of the group for token j (N = 1: the decode step, members = query heads).
    const int G = Gh * N;
    // groups of up to 8: warps 0-3 take the even pieces, warps 4-7 the odd ones, all members each.  Larger groups
    // (up to 16): warps 0-3 take members 0-7 and warps 4-7 members 8-15, of every piece.
    const bool wide = G > kHeadsPerWarp;
    const int gh = g + (wide ? kHeadsPerWarp * (warp >> 2) : 0);      // the member of the group in this lane's MMA row
    const int my_tok = gh / Gh;                                       // its token: it sees the new rows 0 .. my_tok
    // scores in the log2 domain; with E4M3 codes the products are in units of the scales
    const float scale_log2 = (FP8 ? a.k_scale : 1.f) * (1.4426950408889634f / sqrtf((float)DH));
    const float out_scale = FP8 ? a.v_scale : 1.f;
    bool ok = true;

    Segment sg;
    while (src.next(sg)) {
        const int hk = sg.h, b = sg.b, L = sg.L;
        const bool has_new = sg.r1 > L;
        const int c1 = has_new ? L : sg.r1;
        const size_t slab = ((size_t)b * a.n_kv_heads + hk) * (size_t)a.max_seq * DH;

        // ---- joint RoPE of the G queries and k_new with one set of cos/sin (Algorithm 3, steps 6-8) ----
        for (int idx = t; idx < G * HALF; idx += nct) {
            const int m = idx / HALF, i = idx - m * HALF, j = m / Gh, g2 = m - j * Gh;
            const size_t row = (size_t)b * N + j;                          // token j of sequence b
            const float c = a.cos_tab[(size_t)(sg.pos + j) * HALF + i], sn = a.sin_tab[(size_t)(sg.pos + j) * HALF + i];
            const __nv_bfloat16 *qg = a.q + row * a.q_stride + (size_t)(hk * Gh + g2) * DH;
            const float x0 = __bfloat162float(ld_cg_bf16(qg + i)), x1 = __bfloat162float(ld_cg_bf16(qg + i + HALF));
            sm.q[m][i] = __fsub_rn(__fmul_rn(x0, c), __fmul_rn(x1, sn));
            sm.q[m][i + HALF] = __fadd_rn(__fmul_rn(x1, c), __fmul_rn(x0, sn));
            if (g2 == 0 && has_new) {
                const __nv_bfloat16 *kg = a.k_new + row * a.kv_stride + (size_t)hk * DH;
                const float k0 = __bfloat162float(ld_cg_bf16(kg + i)), k1 = __bfloat162float(ld_cg_bf16(kg + i + HALF));
                const float r0 = __fsub_rn(__fmul_rn(k0, c), __fmul_rn(k1, sn)), r1 = __fadd_rn(__fmul_rn(k1, c), __fmul_rn(k0, sn));
                const __nv_bfloat16 *vg = a.v_new + row * a.kv_stride + (size_t)hk * DH;
                if constexpr (FP8) {
                    // the codes that go into the cache: value / scale, nearest code (ties to even), saturating at 448
                    knew8[j * DH + i] = __nv_cvt_float_to_fp8(__fdiv_rn(r0, a.k_scale), __NV_SATFINITE, __NV_E4M3);
                    knew8[j * DH + i + HALF] = __nv_cvt_float_to_fp8(__fdiv_rn(r1, a.k_scale), __NV_SATFINITE, __NV_E4M3);
                    vnew8[j * DH + i] = __nv_cvt_float_to_fp8(__fdiv_rn(__bfloat162float(ld_cg_bf16(vg + i)), a.v_scale), __NV_SATFINITE, __NV_E4M3);
                    vnew8[j * DH + i + HALF] = __nv_cvt_float_to_fp8(__fdiv_rn(__bfloat162float(ld_cg_bf16(vg + i + HALF)), a.v_scale), __NV_SATFINITE, __NV_E4M3);
                } else {
                    sm.knew[j][i] = __float2bfloat16_rn(r0);
                    sm.knew[j][i + HALF] = __float2bfloat16_rn(r1);
                    sm.vnew[j][i] = ld_cg_bf16(vg + i);
                    sm.vnew[j][i + HALF] = ld_cg_bf16(vg + i + HALF);
                }
            }
        }
        named_bar_sync(1, nct);
        // ---- GKVC append (Eq. 2; Algorithm 3 steps 1 and 9): one write per row, no reload ----
        if (has_new) {
            // the N new rows are consecutive in the cache (rows L .. L + N - 1) and in shared memory
            for (int i = t; i < N * (kRowBytes / 16); i += nct) {
                reinterpret_cast<uint4 *>(kc8 + (slab + (size_t)L * DH) * EB)[i] = reinterpret_cast<const uint4 *>(knew8)[i];
                reinterpret_cast<uint4 *>(vc8 + (slab + (size_t)L * DH) * EB)[i] = reinterpret_cast<const uint4 *>(vnew8)[i];
            }
            asm volatile("fence.proxy.async;" ::: "memory");
        }

        // ---- A fragments of the score product: this lane's head of the group, 8 consecutive elements per block ----
        uint4 qhi[KB], qlo[PRECISE ? KB : 1];
#pragma unroll
        for (int kb = 0; kb < KB; ++kb) {
            float f[8];
            if (gh < G) {
                const float4 f0 = *reinterpret_cast<const float4 *>(&sm.q[gh][kb * 32 + 8 * t4]);
                const float4 f1 = *reinterpret_cast<const float4 *>(&sm.q[gh][kb * 32 + 8 * t4 + 4]);
                f[0] = f0.x; f[1] = f0.y; f[2] = f0.z; f[3] = f0.w; f[4] = f1.x; f[5] = f1.y; f[6] = f1.z; f[7] = f1.w;
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] = 0.f;
            }
            qhi[kb] = make_uint4(pack2t<FP8>(f[0], f[1]), pack2t<FP8>(f[2], f[3]), pack2t<FP8>(f[4], f[5]), pack2t<FP8>(f[6], f[7]));
            if constexpr (PRECISE) {
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] -= round16<FP8>(f[i]);          // what the rounding left out
                qlo[kb] = make_uint4(pack2t<FP8>(f[0], f[1]), pack2t<FP8>(f[2], f[3]), pack2t<FP8>(f[4], f[5]), pack2t<FP8>(f[6], f[7]));
            }
        }
        float m_run = -INFINITY, l_run = 0.f;      // of head g; the sum holds this lane's keys only until the end
        // output fragments, TRANSPOSED (rows of the product = output columns, n = members): acc[cb][m][i] belongs to
        // column 32 cb + 4 g + 2 m + (i >> 1) and member 2 t4 + (i & 1)
        float acc[CB][2][4];
#pragma unroll
        for (int cb = 0; cb < CB; ++cb)
#pragma unroll
            for (int m = 0; m < 2; ++m)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[cb][m][i] = 0.f;

        // One block of up to 16 keys: rows key0 .. key0 + 15 of the K tile `kt` / V tile `vt`, of which the rows below
        // `rows` exist.  Rows that do not exist are read from the last one that does (finite data) and get weight 0.
        // `causal`: the rows are the new tokens of the chunk: key i is visible to this lane's member only if i <= its token
        auto block = [&](const unsigned char *kt, const unsigned char *vt, int key0, int rows, bool causal = false) {
            // ---- scores (Algorithm 3 step 10): two sub-blocks of 8 keys; lane (g, t4) supplies keys key0 + g and
            //      key0 + 8 + g and receives keys key0 + 2 t4 (+1) and key0 + 8 + 2 t4 (+1) of its head.  Four
            //      independent accumulator chains (sub-block x half of the 32-wide block).
            const int kr0 = key0 + g < rows ? key0 + g : rows - 1, kr1 = key0 + 8 + g < rows ? key0 + 8 + g : rows - 1;
            // PRECISE: rows 8..15 of A carry the lo parts of the same members, so one product gives q_hi . k (elements 0, 1)
            // and q_lo . k (elements 2, 3)
            constexpr int SE = PRECISE ? 4 : 2;
            float sc[2][2][SE];
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int e = 0; e < SE; ++e) sc[u][c][e] = 0.f;
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                uint4 kv[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    if constexpr (FP8) {
                        const uint2 c8 = *reinterpret_cast<const uint2 *>(kt + (size_t)(u ? kr1 : kr0) * kRowBytes + kb * 32 + t4 * 8);
                        kv[u] = make_uint4(e4m3x2_to_f16x2(c8.x), e4m3x2_to_f16x2(c8.x >> 16), e4m3x2_to_f16x2(c8.y), e4m3x2_to_f16x2(c8.y >> 16));
                    } else {
                        kv[u] = *reinterpret_cast<const uint4 *>(kt + (size_t)(u ? kr1 : kr0) * kRowBytes + kb * 64 + t4 * 16);
                    }
                }
                // four accumulators: a product never follows the one it depends on by less than four instructions
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    if constexpr (PRECISE) {
                        mma_k16<FP8>(sc[u][0], qhi[kb].x, qlo[kb].x, qhi[kb].y, qlo[kb].y, kv[u].x, kv[u].y);
                        mma_k16<FP8>(sc[u][1], qhi[kb].z, qlo[kb].z, qhi[kb].w, qlo[kb].w, kv[u].z, kv[u].w);
                    } else {
                        mma_top_k16<FP8>(sc[u][0], qhi[kb].x, qhi[kb].y, kv[u].x, kv[u].y);
                        mma_top_k16<FP8>(sc[u][1], qhi[kb].z, qhi[kb].w, kv[u].z, kv[u].w);
                    }
                }
            }
            // ---- online softmax (step 11) ----
            int ka[4];
            bool see[4];
            float s[4];
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    ka[2 * u + e] = key0 + 8 * u + 2 * t4 + e;
                    float v = sc[u][0][e] + sc[u][1][e];
                    if constexpr (PRECISE) v += sc[u][0][2 + e] + sc[u][1][2 + e];
                    // a masked key gets weight 0 for this lane's member; the V row of the key still feeds the other members
                    see[2 * u + e] = ka[2 * u + e] < rows && !(causal && ka[2 * u + e] > my_tok);
                    s[2 * u + e] = see[2 * u + e] ? v * scale_log2 : -INFINITY;
                }
            float mt = fmaxf(fmaxf(s[0], s[1]), fmaxf(s[2], s[3]));
            mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 1));
            mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 2));
            const float m_new = fmaxf(m_run, mt);                  // finite: row key0 exists and is visible to every member
            const float corr = fast_exp2(m_run - m_new);           // 0 while m_run = -inf
            float pr[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) pr[e] = see[e] ? fast_exp2(s[e] - m_new) : 0.f;
            const uint32_t pa0 = pack2t<FP8>(pr[0], pr[1]), pa1 = pack2t<FP8>(pr[2], pr[3]);
            uint32_t pl0 = 0u, pl1 = 0u;
            if constexpr (PRECISE) {
                // the weights go in as hi + lo: the row sum is the sum of the weights themselves
                l_run = l_run * corr + ((pr[0] + pr[1]) + (pr[2] + pr[3]));
                pl0 = pack2t<FP8>(pr[0] - round16<FP8>(pr[0]), pr[1] - round16<FP8>(pr[1]));
                pl1 = pack2t<FP8>(pr[2] - round16<FP8>(pr[2]), pr[3] - round16<FP8>(pr[3]));
            } else {
                l_run = l_run * corr + ((bf16_round(pr[0]) + bf16_round(pr[1])) + (bf16_round(pr[2]) + bf16_round(pr[3])));
            }
            m_run = m_new;
            // ---- PV (step 12), transposed: O^T[column, member] += V^T[column, key] P^T[key, member].  The weights are
            //      the B operand exactly as the score fragments hold them (keys 2 t4 (+1) and 8 + 2 t4 (+1) of member g);
            //      V^T comes from four rows of V: four consecutive columns per lane and row, the same column of two
            //      keys paired by a byte permute.  All 16 rows of the product carry output columns. ----
            const unsigned char *vp[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) vp[e] = vt + (size_t)(ka[e] < rows ? ka[e] : rows - 1) * kRowBytes + g * 4 * EB;
            // the running maximum seldom moves after the first tiles: the rescaling is skipped when no lane needs it
            if (__any_sync(kFull, corr != 1.f)) {
                const float c0 = __shfl_sync(kFull, corr, 8 * t4), c1 = __shfl_sync(kFull, corr, 8 * t4 + 4);     // members 2 t4, 2 t4 + 1
#pragma unroll
                for (int cb = 0; cb < CB; ++cb)
#pragma unroll
                    for (int m = 0; m < 2; ++m) { acc[cb][m][0] *= c0; acc[cb][m][1] *= c1; acc[cb][m][2] *= c0; acc[cb][m][3] *= c1; }
            }
            // two column blocks at a time: loads first, then the products; the hi and lo product of an accumulator
            // are at least two (mostly four) instructions apart
#pragma unroll
            for (int cb0 = 0; cb0 < CB; cb0 += 2) {
                constexpr int kPair = 2;
                uint32_t av[kPair][2][4];          // [block][column pair m][a0..a3]
#pragma unroll
                for (int h = 0; h < kPair; ++h) {
                    if (cb0 + h < CB) {
                        const int cb = cb0 + h;
                        if constexpr (FP8) {
                            uint32_t x[4];             // codes of columns 32 cb + 4 g .. + 3 of the four rows
#pragma unroll
                            for (int e = 0; e < 4; ++e) x[e] = *reinterpret_cast<const uint32_t *>(vp[e] + cb * 32);
#pragma unroll
                            for (int m = 0; m < 2; ++m) {
                                av[h][m][0] = e4m3x2_to_f16x2(__byte_perm(x[0], x[1], m ? 0x0062 : 0x0040));
                                av[h][m][1] = e4m3x2_to_f16x2(__byte_perm(x[0], x[1], m ? 0x0073 : 0x0051));
                                av[h][m][2] = e4m3x2_to_f16x2(__byte_perm(x[2], x[3], m ? 0x0062 : 0x0040));
                                av[h][m][3] = e4m3x2_to_f16x2(__byte_perm(x[2], x[3], m ? 0x0073 : 0x0051));
                            }
                        } else {
                            uint2 x[4];                // columns 32 cb + 4 g .. + 3 of the four rows
#pragma unroll
                            for (int e = 0; e < 4; ++e) x[e] = *reinterpret_cast<const uint2 *>(vp[e] + cb * 64);
                            av[h][0][0] = __byte_perm(x[0].x, x[1].x, 0x5410); av[h][0][1] = __byte_perm(x[0].x, x[1].x, 0x7632);
                            av[h][0][2] = __byte_perm(x[2].x, x[3].x, 0x5410); av[h][0][3] = __byte_perm(x[2].x, x[3].x, 0x7632);
                            av[h][1][0] = __byte_perm(x[0].y, x[1].y, 0x5410); av[h][1][1] = __byte_perm(x[0].y, x[1].y, 0x7632);
                            av[h][1][2] = __byte_perm(x[2].y, x[3].y, 0x5410); av[h][1][3] = __byte_perm(x[2].y, x[3].y, 0x7632);
                        }
                    }
                }
#pragma unroll
                for (int h = 0; h < kPair; ++h)
                    if (cb0 + h < CB) {
#pragma unroll
                        for (int m = 0; m < 2; ++m)
                            mma_k16<FP8>(acc[cb0 + h][m], av[h][m][0], av[h][m][1], av[h][m][2], av[h][m][3], pa0, pa1);
                    }
                if constexpr (PRECISE) {
#pragma unroll
                    for (int h = 0; h < kPair; ++h)
                        if (cb0 + h < CB) {
#pragma unroll
                            for (int m = 0; m < 2; ++m)
                                mma_k16<FP8>(acc[cb0 + h][m], av[h][m][0], av[h][m][1], av[h][m][2], av[h][m][3], pl0, pl1);
                        }
                }
            }
        };

        // ---- stream the cached rows of the segment: warps 0-3 take the even pieces, warps 4-7 the odd ones, 16 rows
        //      of the tile each; every warp waits for and releases every piece (the ring protocol) ----
        for (int r = sg.r0; r < c1; r += TR, ++piece) {
            const unsigned char *slot = ring.wait(piece, ok);
            const int rows = (c1 - r) < TR ? (c1 - r) : TR;
            if constexpr (FP8) {
                // 128 rows per piece: every warp 16 of them (small groups), or 32 per warp of either set (large groups)
                if (ok && !wide && warp * 16 < rows) block(slot, slot + TR * kRowBytes, warp * 16, rows);
                if (ok && wide) {
                    if ((warp & 3) * 16 < rows) block(slot, slot + TR * kRowBytes, (warp & 3) * 16, rows);
                    if (64 + (warp & 3) * 16 < rows) block(slot, slot + TR * kRowBytes, 64 + (warp & 3) * 16, rows);
                }
            } else {
                if (ok && (wide || (piece & 1) == (warp >> 2)) && (warp & 3) * 16 < rows)
                    block(slot, slot + TR * kRowBytes, (warp & 3) * 16, rows);
            }
            ring.release(piece);
        }
        // ---- the new row, straight from shared memory (never re-read from the cache) ----
        if (has_new && (warp == 0 || (wide && warp == 4)))
            block(knew8, vnew8, 0, N, N > 1);

        // ---- the warps' states meet in shared memory ----
        l_run += __shfl_xor_sync(kFull, l_run, 1);
        l_run += __shfl_xor_sync(kFull, l_run, 2);
        // this lane's outputs: members 2 t4 (+1) in the warp's slots, two pairs of neighbouring columns per 32-column block
#pragma unroll
        for (int cb = 0; cb < CB; ++cb)
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                *reinterpret_cast<float2 *>(&sm.wo[warp][2 * t4][32 * cb + 4 * g + 2 * m]) = make_float2(acc[cb][m][0] * out_scale, acc[cb][m][2] * out_scale);
                *reinterpret_cast<float2 *>(&sm.wo[warp][2 * t4 + 1][32 * cb + 4 * g + 2 * m]) = make_float2(acc[cb][m][1] * out_scale, acc[cb][m][3] * out_scale);
            }
        if (gh < G && t4 == 0) { sm.wm[warp][g] = m_run; sm.wl[warp][g] = l_run; }
        if (!named_bar_and(1, nct, ok)) return false;
        const bool whole = sg.n_cta == 1;                // this CTA alone finishes the group right here
        for (int idx = t; idx < G * DH; idx += nct) {
            const int m = idx / DH, i = idx - m * DH, j = m / Gh, hq = hk * Gh + (m - j * Gh);
            const int ob = b * N + j;                        // output / partial row of member m: token j of sequence b
            // the warps that hold member m (all of them, or one set of four), in slot m mod 8
            const int sl = m & (kHeadsPerWarp - 1), w0 = wide ? 4 * (m >> 3) : 0, w1 = wide ? w0 + 4 : kGroupWarps;
            float M = -INFINITY;
            for (int w = w0; w < w1; ++w) M = fmaxf(M, sm.wm[w][sl]);
            float o = 0.f, l = 0.f;
            for (int w = w0; w < w1; ++w) {
                const float f = (sm.wm[w][sl] == -INFINITY) ? 0.f : fast_exp2(sm.wm[w][sl] - M);
                o += f * sm.wo[w][sl][i];
                l += f * sm.wl[w][sl];
            }
            if (whole) *attn_out_at(a, ob, hq * DH + i) = __float2bfloat16_rn(o / l);
            else {
                float *part = a.part + (((size_t)ob * a.n_q_heads + hq) * kMaxSplits + (cta - sg.first_cta)) * kPartStride;
                part[i] = o;
                if (i == 0) { part[DH] = M; part[DH + 1] = l; }
            }
        }
        if (!whole) {
            // ---- several CTAs share the K/V head: the partials are published, the last CTA merges the G heads ----
            __threadfence();
            named_bar_sync(1, nct);
            int *ticket = a.ticket + (size_t)b * N * a.n_q_heads + hk * Gh;
            if (t == 0) sm.last = (atomicAdd(ticket, 1) == sg.n_cta - 1);
            named_bar_sync(1, nct);
            if (sm.last) {
                __threadfence();
                // one warp per query head of the group, all heads at once: lane s holds (max, sum) of partial s and
                // the merge factor that goes with it; every lane finishes DH / 32 columns
                for (int hg = warp; hg < G; hg += kGroupWarps) {
                    const int mj = hg / Gh, mh = hk * Gh + (hg - mj * Gh), ob = b * N + mj;     // member hg: token mj, head mh
                    const float *hp = a.part + ((size_t)ob * a.n_q_heads + mh) * kMaxSplits * kPartStride;
                    const bool have = lane < sg.n_cta;
                    const float ms = have ? ld_cg_f32(hp + (size_t)lane * kPartStride + DH) : -INFINITY;
                    const float ls = have ? ld_cg_f32(hp + (size_t)lane * kPartStride + DH + 1) : 0.f;
                    float MM = ms;
#pragma unroll
                    for (int s = 16; s >= 1; s >>= 1) MM = fmaxf(MM, __shfl_xor_sync(kFull, MM, s));
                    const float f = (ms == -INFINITY) ? 0.f : fast_exp2(ms - MM);
                    const float ll = warp_sum(f * ls);
                    float oo[DH / 32];
#pragma unroll
                    for (int c = 0; c < DH / 32; ++c) oo[c] = 0.f;
                    for (int s0 = 0; s0 < sg.n_cta; s0 += 4) {
                        float v[4][DH / 32];
#pragma unroll
                        for (int u = 0; u < 4; ++u)
#pragma unroll
                            for (int c = 0; c < DH / 32; ++c)
                                v[u][c] = (s0 + u < sg.n_cta) ? ld_cg_f32(hp + (size_t)(s0 + u) * kPartStride + lane + 32 * c) : 0.f;
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const float fs = __shfl_sync(kFull, f, (s0 + u) & 31);
#pragma unroll
                            for (int c = 0; c < DH / 32; ++c) oo[c] = fmaf(fs, v[u][c], oo[c]);
                        }
                    }
#pragma unroll
                    for (int c = 0; c < DH / 32; ++c) *attn_out_at(a, ob, mh * DH + lane + 32 * c) = __float2bfloat16_rn(oo[c] / ll);
                }
                if (t == 0) *ticket = 0;
            }
        }
        named_bar_sync(1, nct);                              // the scratch is reused by the next segment
    }
    return true;
}

}  // namespace fasttps
