// Thin-GEMM path of the decode chain for batches of 9 to 32 rows (the batch-32 workload): every weight is read from
// HBM ONCE per product for all rows of the batch (Eq. 1 / Algorithm 4 and the projections of Figure 1 with N = 32).
//
// Why a path of its own: the kernels for up to 8 rows keep the activations of the whole reduction length as
// tensor-core B fragments in registers (32 registers for 8 rows); 32 rows would need 128, and 32 x 3072 bf16 of
// activations (192 KB) do not fit in shared memory beside the weight ring either.  Here the loop over k is the
// OUTER loop: a ring piece holds one k chunk of the activations of all rows (from the L2) next to the same k
// chunk of up to four 16-row weight tiles (from HBM), the sums of a CTA's tiles stay in registers across the whole
// reduction, and one weight fragment loaded from shared memory feeds the MMAs of all four 8-row batch tiles.
//
//   wide_linear_kernel   products over the tiled weight format (QKV, output projection, gate_up, logits): a CTA
//                        owns a contiguous range of 16-row tiles and works through it in passes of up to four
//                        tiles x the whole reduction; consumer warp w multiplies k block w of every chunk.  The
//                        epilogue stores bf16 / FP32 (+ residual, + running argmax) or applies siLu_Mul to the
//                        interlaced gate / up rows (Eq. 31) and writes the intermediate as a bf16 hi + lo pair.
//   wide_down_kernel     the down projection over the octet-block format: a CTA owns a contiguous range of units
//                        (128 output columns x 16 intermediate octets); partial sums leave with 16-byte
//                        reductions into an FP32 accumulator that the next kernel of the chain folds in.
//   prep_rows_kernel     between the products: x = residual + FP32 sums (rounded once to bf16, stored), RMSNorm
//                        (rounded to bf16 like a stored tensor), sums cleared; one CTA per batch row.
//
// The intermediate of the MLP (32 x K bf16 pairs, 1 MB for the Phi-3 shape) goes through global memory here: it is
// written and read back within microseconds and stays in the L2; HBM sees the weights once and nothing else.
#include "async_copy.cuh"
#include "dot_core.cuh"

namespace fasttps {

namespace {

constexpr int kWideWarps = 16;                                  // consumer warps: two per k block of a piece, two tiles each
constexpr int kWideThreads = (kWideWarps + 1) * 32;             // + the producer warp
constexpr int kWideTiles = 4;                                   // 16-row weight tiles per pass
constexpr int kWideTilesPerWarp = 2;
constexpr int kWideChunk = 8;                                   // k blocks (32 k each) per ring piece
constexpr int kWideXStride = kWideXRow * 2;                     // bytes between batch rows of an activation chunk: 512 + 64,
                                                                // so that the 16-byte loads of two neighbouring rows
                                                                // fall on different banks
constexpr int kWideXBytes = kWideMaxB * kWideXStride;           // 18 KB: one contiguous block of the chunked layout
static_assert(kWideChunk * 32 == kWideXChunk, "a ring piece holds one chunk of the activations");
constexpr int kWidePiece = kWideXBytes + kWideTiles * kWideChunk * kTileBytes;   // 50 KB
constexpr int kWideSlots = 4;
constexpr int kWideAccStride = 17;                              // floats between batch rows of the per-pass sums (16 + 1)

struct WideSmem {
    alignas(128) unsigned char slots[kWideSlots][kWidePiece];
    alignas(16) uint64_t bars[2 * kWideSlots];
    alignas(16) float sums[kWideTiles * kWideMaxB * kWideAccStride];     // [tile][batch row][row of the tile]
    float best_val[kWideMaxB];
    int best_idx[kWideMaxB];
    int abort;
    int last;
};

// Producer warp, all lanes: piece `g` = chunk c of the activations (one block of the chunked layout, all 32 rows)
// and k blocks [8 c, 8 c + kbs) of `nt` weight tiles starting at tile `t0`.  Lane 0 waits for the slot, announces
// the bytes and copies the activations; lane t copies weight tile t.
__device__ __forceinline__ bool wide_put(WeightRing &ring, int g, const WideArgs &a, int nkb, int t0, int nt, int c, int kbs)
{
    const int lane = threadIdx.x & 31;
    int okv = 1;
    const int s = ring.slot_of(g);
    unsigned char *slot = ring.slots + (size_t)s * ring.slot_bytes;
    if (lane == 0) {
        okv = ring.acquire(g) ? 1 : 0;
        if (okv) {
            mbar_expect_tx(&ring.full[s], (uint32_t)(kWideXBytes + nt * kbs * kTileBytes));
            bulk_g2s(slot, reinterpret_cast<const unsigned char *>(a.x) + (size_t)c * kWideXBytes, (uint32_t)kWideXBytes, &ring.full[s]);
        }
    }
    okv = __shfl_sync(kFull, okv, 0);
    if (!okv) return false;
    if (lane < nt)
        bulk_g2s_hint(slot + kWideXBytes + lane * (kWideChunk * kTileBytes),
                      reinterpret_cast<const unsigned char *>(a.w) + ((size_t)(t0 + lane) * nkb + (size_t)c * kWideChunk) * kTileBytes,
                      (uint32_t)(kbs * kTileBytes), &ring.full[s], ring.policy);
    return true;
}

__global__ void __launch_bounds__(kWideThreads, 1) wide_linear_kernel(WideArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    WideSmem &sm = *reinterpret_cast<WideSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int t = threadIdx.x, lane = t & 31, w = t >> 5, g = lane >> 2, t4 = lane & 3;
    constexpr int nct = kWideWarps * 32;

    const int n_tiles = (a.n_out + 15) >> 4, nkb = a.K >> 5, nchunk = (nkb + kWideChunk - 1) / kWideChunk;
    const int base = n_tiles / gridDim.x, rem = n_tiles % gridDim.x, cta = blockIdx.x;
    const int tile0 = cta * base + (cta < rem ? cta : rem), ntile = base + (cta < rem ? 1 : 0);

    WeightRing ring;
    ring.init(&sm.slots[0][0], sm.bars, &sm.abort, kWideSlots, kWidePiece, kWideWarps, nullptr, 0, nullptr, 0);
    if (t < kWideMaxB) { sm.best_val[t] = -INFINITY; sm.best_idx[t] = 0x7fffffff; }
    __syncthreads();

    if (w == kWideWarps) {
        // ---- producer warp.  The weights depend on nothing: the first pieces' worth is asked from HBM into the L2
        // at once; the activations were written by the previous kernel of the chain ----
        if (lane < (ntile < kWideTiles ? ntile : kWideTiles)) {
            const unsigned char *wp = reinterpret_cast<const unsigned char *>(a.w) + (size_t)(tile0 + lane) * nkb * kTileBytes;
            const int pre = nkb < 4 * kWideChunk ? nkb : 4 * kWideChunk;     // the k blocks of the first four pieces
            bulk_prefetch_l2(wp, (uint32_t)(pre * kTileBytes));
        }
        pdl_wait();
        ring.policy = l2_policy_evict_first();               // the weights are read once; the activations stay in the L2
        int piece = 0;
        for (int p0 = 0; p0 < ntile; p0 += kWideTiles) {
            const int nt = ntile - p0 < kWideTiles ? ntile - p0 : kWideTiles;
            for (int c = 0; c < nchunk; ++c, ++piece) {
                const int kbs = nkb - c * kWideChunk < kWideChunk ? nkb - c * kWideChunk : kWideChunk;
                if (!wide_put(ring, piece, a, nkb, tile0 + p0, nt, c, kbs)) {
                    if (lane == 0) ring.drain(piece);
                    return;
                }
            }
        }
        return;
    }

    // ---- consumer warps ----
    pdl_wait();
    pdl_launch_dependents();
    bool ok = true;
    int piece = 0;
    // running argmax of the batch row this thread finishes in the epilogue
    const int r = t & 15, eb = t >> 4;                       // epilogue: row r of a tile, batch row eb
    const int kb = w & (kWideChunk - 1), th = w >> 3;        // main loop: k block kb of every piece, tiles 2 th and 2 th + 1
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int p0 = 0; p0 < ntile; p0 += kWideTiles) {
        const int nt = ntile - p0 < kWideTiles ? ntile - p0 : kWideTiles;
        float acc[kWideTilesPerWarp][4][4];
#pragma unroll
        for (int i = 0; i < kWideTilesPerWarp; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;
        const unsigned char *slot = nullptr;
        for (int c = 0; c < nchunk; ++c, ++piece) {
            const int kbs = nkb - c * kWideChunk < kWideChunk ? nkb - c * kWideChunk : kWideChunk;
            slot = ring.wait(piece, ok);
            if (ok && kb < kbs && kWideTilesPerWarp * th < nt) {
                // B fragments of k block kb for the four batch tiles: rows 8 j + g, 8 consecutive k from 8 t4
                uint4 bq[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    bq[j] = *reinterpret_cast<const uint4 *>(slot + (8 * j + g) * kWideXStride + kb * 64 + t4 * 16);
#pragma unroll
                for (int i = 0; i < kWideTilesPerWarp; ++i) {
                    const int tile = kWideTilesPerWarp * th + i;
                    if (tile < nt) {
                        const unsigned char *blk = slot + kWideXBytes + (tile * kWideChunk + kb) * kTileBytes + lane * 16;
                        const uint4 lo = *reinterpret_cast<const uint4 *>(blk);          // row g,     k 8 t4 ..
                        const uint4 hi = *reinterpret_cast<const uint4 *>(blk + 512);    // row g + 8, k 8 t4 ..
                        // the two products into one accumulator are four instructions apart, not back to back
#pragma unroll
                        for (int j = 0; j < 4; ++j) mma_bf16_k16(acc[i][j], lo.x, hi.x, lo.y, hi.y, bq[j].x, bq[j].y);
#pragma unroll
                        for (int j = 0; j < 4; ++j) mma_bf16_k16(acc[i][j], lo.z, hi.z, lo.w, hi.w, bq[j].z, bq[j].w);
                    }
                }
            }
            if (c + 1 < nchunk) ring.release(piece);          // the slot of the pass's last piece is kept: see below
        }
        if (!named_bar_and(1, nct, ok)) {                     // every warp has read the last piece
            if (t == 0) atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT);
            return;
        }
        // ---- the sums of the eight k blocks of a tile pair meet: a merge tree over the eight warps (three levels, one
        //      block-wide barrier each), a warp's 32 sums travelling lane to lane through the slot of the pass's last
        //      piece, which is handed back to the producer afterwards.  (Shared-memory atomics straight into `sums`, eight
        //      warps on the same addresses, cost about 2 us per pass.)  A sender writes the region that only itself has
        //      read before, so one barrier per level is enough. ----
        {
            float *xb = reinterpret_cast<float *>(const_cast<unsigned char *>(slot)) + (size_t)th * 4 * 1024 + lane;
            for (int s = 4; s >= 1; s >>= 1) {
                if (kb >= s && kb < 2 * s) {
                    float *x = xb + (kb & 3) * 1024;
#pragma unroll
                    for (int i = 0; i < kWideTilesPerWarp; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j)
#pragma unroll
                            for (int e = 0; e < 4; ++e) x[((i * 4 + j) * 4 + e) * 32] = acc[i][j][e];
                }
                named_bar_sync(1, nct);
                if (kb < s) {
                    const float *x = xb + ((kb + s) & 3) * 1024;
#pragma unroll
                    for (int i = 0; i < kWideTilesPerWarp; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j)
#pragma unroll
                            for (int e = 0; e < 4; ++e) acc[i][j][e] += x[((i * 4 + j) * 4 + e) * 32];
                }
            }
            if (kb == 0) {
#pragma unroll
                for (int i = 0; i < kWideTilesPerWarp; ++i) {
                    const int tile = kWideTilesPerWarp * th + i;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // fragment: rows g / g + 8 of the tile, batch rows 8 j + 2 t4 / + 1
                        float *p = sm.sums + (size_t)(tile * kWideMaxB + 8 * j + 2 * t4) * kWideAccStride + g;
                        p[0] = acc[i][j][0];
                        p[kWideAccStride] = acc[i][j][1];
                        p[8] = acc[i][j][2];
                        p[kWideAccStride + 8] = acc[i][j][3];
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the slot goes back to the copy engine
            ring.release(piece - 1);
            named_bar_sync(1, nct);
        }
        // ---- epilogue: thread (r = t % 16, b = t / 16) finishes row r of every tile of the pass for batch row b ----
        {
            const int b = eb;
            for (int i = 0; i < nt; ++i) {
                float *p = sm.sums + (size_t)(i * kWideMaxB + b) * kWideAccStride;
                const int tile = tile0 + p0 + i;
                if (a.epi == kWideSilu) {
                    // rows c and c + 8 of a gate_up tile are a gate column and ITS up column (interlaced in blocks of 8)
                    if (r < 8) {
                        const float gate = p[r], up = p[r + 8];
                        if (b < a.batch) {
                            const float act = gate / (1.f + __expf(-gate)) * up;
                            const __nv_bfloat16 hi = __float2bfloat16_rn(act);
                            const size_t o = wide_a_index(b, tile * 8 + r);
                            a.a_hi[o] = hi;
                            a.a_lo[o] = __float2bfloat16_rn(act - __bfloat162float(hi));
                        }
                    }
                } else {
                    float v = p[r];
                    const int col = tile * 16 + (a.pair_rows ? ((r & 7) * 2 + (r >> 3)) : r);
                    if (b < a.batch && col < a.n_out) {
                        if (a.res) v += __bfloat162float(a.res[(size_t)b * a.res_stride + col]);
                        if (a.out_bf16) a.out_bf16[(size_t)b * a.out_stride + col] = __float2bfloat16_rn(v);
                        if (a.out_f32) a.out_f32[(size_t)b * a.out_stride + col] = v;
                        if (v > bv || (v == bv && col < bi)) { bv = v; bi = col; }
                    }
                }
            }
        }
        named_bar_sync(1, nct);                          // the sums have been read before the next pass writes them
    }
    if (a.next_ids == nullptr) return;

    // ---- greedy argmax: 16 threads per batch row -> CTA candidates -> the last CTA finishes (lowest index on ties) ----
#pragma unroll
    for (int s = 8; s >= 1; s >>= 1) {
        const float ov = __shfl_xor_sync(kFull, bv, s);
        const int oi = __shfl_xor_sync(kFull, bi, s);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (r == 0 && eb < a.batch) {
        a.amax_val[(size_t)eb * gridDim.x + cta] = bv;
        a.amax_idx[(size_t)eb * gridDim.x + cta] = bi;
    }
    __threadfence();
    named_bar_sync(1, nct);
    if (t == 0) sm.last = (atomicAdd(a.amax_ticket, 1) == (int)gridDim.x - 1);
    named_bar_sync(1, nct);
    if (!sm.last) return;
    __threadfence();
    for (int b = w; b < a.batch; b += kWideWarps) {      // one warp per batch row
        float v = -INFINITY; int ix = 0x7fffffff;
        for (int c = lane; c < (int)gridDim.x; c += 32) {
            const float cv = ld_cg_f32(a.amax_val + (size_t)b * gridDim.x + c);
            const int ci = ld_cg_s32(a.amax_idx + (size_t)b * gridDim.x + c);
            if (cv > v || (cv == v && ci < ix)) { v = cv; ix = ci; }
        }
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) {
            const float ov = __shfl_xor_sync(kFull, v, s);
            const int oi = __shfl_xor_sync(kFull, ix, s);
            if (ov > v || (ov == v && oi < ix)) { v = ov; ix = oi; }
        }
        if (lane == 0) {
            if (ix == 0x7fffffff) ix = 0;                // all-NaN row: fall back to index 0
            a.next_ids[b] = ix;
            if (a.adv_pos) a.adv_pos[b] += 1;
            if (a.adv_len) a.adv_len[b] += 1;
        }
    }
    if (t == 0) *a.amax_ticket = 0;
}

// ------------------------------------------------------------------------------------------- down projection

constexpr int kDownQuad = 4;                                    // intermediate octets per ring piece
constexpr int kDownBlocks = kWideWarps;                         // 32-column blocks per unit: one per consumer warp (512 columns)
constexpr int kDownChunkOct = kWideAChunk / 8;                  // octets per chunk of the chunked intermediate (16)
constexpr int kDownXStride = kWideARow * 2;                     // 272 bytes between batch rows: conflict-free 4-byte loads
constexpr int kDownXBytes = kWideMaxB * kDownXStride;           // one of hi / lo: one contiguous block of the chunked layout
constexpr int kDownRun = kDownBlocks * 512;                     // bytes of one octet's blocks of a column group: 8 KB
constexpr int kDownPiece = 2 * kDownXBytes + kDownQuad * kDownRun;   // 49 KB
constexpr int kDownSlots = 4;
static_assert(kDownChunkOct % kDownQuad == 0, "a piece lies inside one chunk of the intermediate");

__device__ __forceinline__ unsigned char *slot_of_piece(WeightRing &ring, int s) { return ring.slots + (size_t)s * ring.slot_bytes; }

struct DownSmem {
    alignas(128) unsigned char slots[kDownSlots][kDownPiece];
    alignas(16) uint64_t bars[2 * kDownSlots];
    int abort;
};

// A unit = four octets of the intermediate x sixteen 32-column blocks of the output (512 columns): in the packed
// W_down the sixteen blocks of an octet are 8 KB contiguous, so a ring piece is four weight copies plus the chunk of
// the intermediate (hi and lo) the octets belong to.  (Units of 16 octets x 4 blocks, sixteen 2 KB copies per piece,
// were bound by the rate at which one thread can issue bulk copies: 2.4 us per piece.)  Consumer warp w owns column
// block w of the unit; its sums stay in registers while the CTA's units stay in one column group.
__global__ void __launch_bounds__(kWideThreads, 1) wide_down_kernel(WideDownArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    DownSmem &sm = *reinterpret_cast<DownSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int t = threadIdx.x, lane = t & 31, w = t >> 5, g = lane >> 2, t4 = lane & 3;
    constexpr int nct = kWideWarps * 32;

    const int NT = a.D >> 5;                                   // 32-column blocks of an octet
    const int n_oct = a.K >> 3, noq = (n_oct + kDownQuad - 1) / kDownQuad, ncg = (NT + kDownBlocks - 1) / kDownBlocks;
    const int n_units = ncg * noq;                             // ordered by (column group, octet quad)
    const int base = n_units / gridDim.x, rem = n_units % gridDim.x, cta = blockIdx.x;
    const int u0 = cta * base + (cta < rem ? cta : rem), nu = base + (cta < rem ? 1 : 0);

    WeightRing ring;
    ring.init(&sm.slots[0][0], sm.bars, &sm.abort, kDownSlots, kDownPiece, kWideWarps, nullptr, 0, nullptr, 0);
    __syncthreads();

    if (w == kWideWarps) {
        pdl_wait();                                            // the intermediate was written by the previous kernel
        ring.policy = l2_policy_evict_first();
        for (int i = 0; i < nu; ++i) {
            const int u = u0 + i, cg = u / noq, oq = u - cg * noq;
            const int o0 = oq * kDownQuad, octs = n_oct - o0 < kDownQuad ? n_oct - o0 : kDownQuad;
            const int nbu = NT - cg * kDownBlocks < kDownBlocks ? NT - cg * kDownBlocks : kDownBlocks;
            const int chunk = o0 / kDownChunkOct;
            const int s = ring.slot_of(i);
            int okv = 1;
            if (lane == 0) {
                okv = ring.acquire(i) ? 1 : 0;
                if (okv) {
                    mbar_expect_tx(&ring.full[s], (uint32_t)(2 * kDownXBytes + octs * nbu * 512));
                    bulk_g2s(slot_of_piece(ring, s), reinterpret_cast<const unsigned char *>(a.a_hi) + (size_t)chunk * kDownXBytes, (uint32_t)kDownXBytes, &ring.full[s]);
                    bulk_g2s(slot_of_piece(ring, s) + kDownXBytes, reinterpret_cast<const unsigned char *>(a.a_lo) + (size_t)chunk * kDownXBytes, (uint32_t)kDownXBytes, &ring.full[s]);
                }
            }
            okv = __shfl_sync(kFull, okv, 0);
            if (!okv) { if (lane == 0) ring.drain(i); return; }
            unsigned char *slot = slot_of_piece(ring, s);
            if (lane < octs)
                bulk_g2s_hint(slot + 2 * kDownXBytes + lane * kDownRun,
                              reinterpret_cast<const unsigned char *>(a.w) + ((size_t)(o0 + lane) * NT + (size_t)cg * kDownBlocks) * 512,
                              (uint32_t)(nbu * 512), &ring.full[s], ring.policy);
        }
        return;
    }

    pdl_wait();
    pdl_launch_dependents();
    float acc[2][4][4];
    auto clear = [&]() {
#pragma unroll
        for (int m = 0; m < 2; ++m)
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[m][j][e] = 0.f;
    };
    // the four sums a lane holds of its two MMA tiles are four CONSECUTIVE columns (the order of the packed W_down):
    // one 16-byte reduction per batch row
    auto flush = [&](int cg) {
        if (cg * kDownBlocks + w >= NT) return;
        float *colp = a.acc + (size_t)((cg * kDownBlocks + w) * 32 + 4 * g);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int b0 = 8 * j + 2 * t4;
            if (b0 < a.batch) red_add_v4(colp + (size_t)b0 * a.D, acc[0][j][0], acc[0][j][2], acc[1][j][0], acc[1][j][2]);
            if (b0 + 1 < a.batch) red_add_v4(colp + (size_t)(b0 + 1) * a.D, acc[0][j][1], acc[0][j][3], acc[1][j][1], acc[1][j][3]);
        }
    };
    clear();
    bool ok = true;
    int cur_cg = nu > 0 ? u0 / noq : 0;
    for (int i = 0; i < nu; ++i) {
        const int u = u0 + i, cg = u / noq, oq = u - cg * noq;
        const int o0 = oq * kDownQuad, octs = n_oct - o0 < kDownQuad ? n_oct - o0 : kDownQuad;
        if (cg != cur_cg) { if (ok) flush(cur_cg); clear(); cur_cg = cg; }
        const unsigned char *slot = ring.wait(i, ok);
        if (ok && cg * kDownBlocks + w < NT) {
            const unsigned char *wb = slot + 2 * kDownXBytes + w * 512 + lane * 16;
            const int xo = (o0 % kDownChunkOct) * 16 + t4 * 4;        // the piece's first octet inside its chunk of the intermediate
            // two octets at a time as ONE k = 16 product (the A fragments of two octet blocks are the two k halves of an
            // m16n8k16 fragment); all hi products first, then the lo ones: the two products into an accumulator are
            // eight instructions apart
#pragma unroll
            for (int o = 0; o < kDownQuad; o += 2) {
                if (o + 1 < octs) {
                    const uint4 av = *reinterpret_cast<const uint4 *>(wb + o * kDownRun);
                    const uint4 aw = *reinterpret_cast<const uint4 *>(wb + (o + 1) * kDownRun);
                    uint32_t bh[4][2], bl[4][2];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const unsigned char *xp = slot + (8 * j + g) * kDownXStride + xo + o * 16;
                        bh[j][0] = *reinterpret_cast<const uint32_t *>(xp);
                        bh[j][1] = *reinterpret_cast<const uint32_t *>(xp + 16);
                        bl[j][0] = *reinterpret_cast<const uint32_t *>(xp + kDownXBytes);
                        bl[j][1] = *reinterpret_cast<const uint32_t *>(xp + kDownXBytes + 16);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        mma_bf16_k16(acc[0][j], av.x, av.y, aw.x, aw.y, bh[j][0], bh[j][1]);
                        mma_bf16_k16(acc[1][j], av.z, av.w, aw.z, aw.w, bh[j][0], bh[j][1]);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        mma_bf16_k16(acc[0][j], av.x, av.y, aw.x, aw.y, bl[j][0], bl[j][1]);
                        mma_bf16_k16(acc[1][j], av.z, av.w, aw.z, aw.w, bl[j][0], bl[j][1]);
                    }
                } else if (o < octs) {                            // an octet without a partner (a ragged last piece)
                    const uint4 av = *reinterpret_cast<const uint4 *>(wb + o * kDownRun);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const unsigned char *xp = slot + (8 * j + g) * kDownXStride + xo + o * 16;
                        const uint32_t bh = *reinterpret_cast<const uint32_t *>(xp);
                        const uint32_t bl = *reinterpret_cast<const uint32_t *>(xp + kDownXBytes);
                        mma_bf16_k8(acc[0][j], av.x, av.y, bh);
                        mma_bf16_k8(acc[1][j], av.z, av.w, bh);
                        mma_bf16_k8(acc[0][j], av.x, av.y, bl);
                        mma_bf16_k8(acc[1][j], av.z, av.w, bl);
                    }
                }
            }
        }
        ring.release(i);
    }
    if (!named_bar_and(1, nct, ok)) {
        if (t == 0) atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT);
        return;
    }
    if (nu > 0) flush(cur_cg);
}

// ------------------------------------------------------------------------------------------- between the products

__global__ void __launch_bounds__(256) prep_rows_kernel(PrepArgs a)
{
    __shared__ float s_part[8];
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x, t = threadIdx.x, lane = t & 31, w = t >> 5;
    const int nvec = a.D >> 3;
    const __nv_bfloat16 *xr = a.x ? a.x + (size_t)b * a.x_stride : nullptr;
    float *ar = a.acc ? a.acc + (size_t)b * a.D : nullptr;
    float ss = 0.f;
    // every thread keeps its (at most three) vectors of the row in registers between the two passes
    constexpr int kMaxVec = 3;                                  // D <= 6144: 768 vectors over 256 threads
    uint4 keep[kMaxVec];
#pragma unroll
    for (int i = 0; i < kMaxVec; ++i) {
        const int v = t + 256 * i;
        keep[i] = make_uint4(0u, 0u, 0u, 0u);
        if (v < nvec) {
            float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (xr) unpack8(*reinterpret_cast<const uint4 *>(xr + (size_t)v * 8), f);
            if (ar) {
                const float4 y0 = ld_cg_f4(ar + (size_t)v * 8), y1 = ld_cg_f4(ar + (size_t)v * 8 + 4);
                f[0] += y0.x; f[1] += y0.y; f[2] += y0.z; f[3] += y0.w;
                f[4] += y1.x; f[5] += y1.y; f[6] += y1.z; f[7] += y1.w;
                *reinterpret_cast<float4 *>(ar + (size_t)v * 8) = make_float4(0.f, 0.f, 0.f, 0.f);
                *reinterpret_cast<float4 *>(ar + (size_t)v * 8 + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            uint4 q;
            q.x = pack2(f[0], f[1]); q.y = pack2(f[2], f[3]); q.z = pack2(f[4], f[5]); q.w = pack2(f[6], f[7]);
            keep[i] = q;
            if (a.x_store) *reinterpret_cast<uint4 *>(a.x_store + (size_t)b * a.D + (size_t)v * 8) = q;
            const uint32_t qq[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float lo = bf_lo(qq[j]), hi = bf_hi(qq[j]);
                ss = fmaf(lo, lo, ss);
                ss = fmaf(hi, hi, ss);
            }
        }
    }
    if (a.n_out == nullptr) return;
    float r = 1.f;
    if (a.g) {
        ss = warp_sum(ss);
        if (lane == 0) s_part[w] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += s_part[i];
        r = rsqrtf(tot / (float)a.D + a.eps);
    }
#pragma unroll
    for (int i = 0; i < kMaxVec; ++i) {
        const int v = t + 256 * i;
        if (v < nvec) {
            uint4 q = keep[i];
            if (a.g) {
                const uint4 gq = *reinterpret_cast<const uint4 *>(a.g + (size_t)v * 8);
                q.x = pack2(bf_lo(q.x) * r * bf_lo(gq.x), bf_hi(q.x) * r * bf_hi(gq.x));
                q.y = pack2(bf_lo(q.y) * r * bf_lo(gq.y), bf_hi(q.y) * r * bf_hi(gq.y));
                q.z = pack2(bf_lo(q.z) * r * bf_lo(gq.z), bf_hi(q.z) * r * bf_hi(gq.z));
                q.w = pack2(bf_lo(q.w) * r * bf_lo(gq.w), bf_hi(q.w) * r * bf_hi(gq.w));
            }
            *reinterpret_cast<uint4 *>(a.n_out + wide_x_index(b, v * 8)) = q;
        }
    }
}

}  // namespace

int configure_wide_kernels()
{
    FT_CUDA(cudaFuncSetAttribute(wide_linear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(WideSmem) + 128));
    FT_CUDA(cudaFuncSetAttribute(wide_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DownSmem) + 128));
    return FASTTPS_OK;
}

int launch_wide_linear(Ctx *c, const WideArgs &a, int prof_class, cudaStream_t st)
{
    if (a.batch < 1 || a.batch > kWideMaxB || a.K < 32 || (a.K & 31) || a.n_out < 1) return FASTTPS_INVALID_ARG;
    const int n_tiles = (a.n_out + 15) / 16;
    int grid = c->n_sm < n_tiles ? c->n_sm : n_tiles;
    ProfScope prof(c, prof_class, st);
    const int rc = launch_ex(wide_linear_kernel, dim3(grid), dim3(kWideThreads), sizeof(WideSmem) + 128, st, &a);
    c->launches++;
    return rc;
}

int launch_wide_down(Ctx *c, const WideDownArgs &a, cudaStream_t st)
{
    if (a.batch < 1 || a.batch > kWideMaxB || (a.D & 31) || a.K < 8 || (a.K & 7)) return FASTTPS_INVALID_ARG;
    const int units = ((a.D / 32 + kDownBlocks - 1) / kDownBlocks) * ((a.K / 8 + kDownQuad - 1) / kDownQuad);
    int grid = c->n_sm < units ? c->n_sm : units;
    ProfScope prof(c, kProfMlp, st);
    const int rc = launch_ex(wide_down_kernel, dim3(grid), dim3(kWideThreads), sizeof(DownSmem) + 128, st, &a);
    c->launches++;
    return rc;
}

int launch_prep_rows(Ctx *c, const PrepArgs &a, int prof_class, cudaStream_t st)
{
    if (a.batch < 1 || a.D > 6144 || (a.D & 7)) return FASTTPS_INVALID_ARG;
    ProfScope prof(c, prof_class, st);
    const int rc = launch_ex(prep_rows_kernel, dim3(a.batch), dim3(256), 0, st, &a);
    c->launches++;
    return rc;
}

}  // namespace fasttps
