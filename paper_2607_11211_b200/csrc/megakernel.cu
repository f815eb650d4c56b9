// Persistent decode-step kernel: the whole token phase of the model -- embedding gather, then for
// every layer RMSNorm -> QKV -> attention (Algorithm 3) -> output projection -> RMSNorm -> fused MLP
// (Algorithm 4), then the final norm, the logits and the greedy argmax -- in ONE cooperative launch,
// for one or several consecutive tokens.
//
// Why: at batch 1 a layer is ~40 us of HBM streaming cut into four dependent products.  As separate
// kernels each of them pays a launch, a cold start of its copy pipeline and a drain (~5 us, more for
// attention), during which HBM idles.  Here one CTA per SM stays resident; a producer warp walks the
// CTA's share of EVERY weight matrix and K/V tile of the step in order and keeps the shared-memory
// ring (~190 KB per SM) full, never waiting for anything but free slots; the consumer warps meet at
// a grid-wide barrier after each product.  While they wait there, or run the latency-bound parts of
// attention, the bytes of the next product keep arriving, so HBM stays busy across all boundaries.
//
// Grid barrier: one arrival counter in global memory that only grows during a launch (the host zeroes it
// before the launch); every wait is bounded, and a CTA that gives up pushes the counter beyond every target so
// that nobody spins forever (the launch is cooperative, so all CTAs are resident).
//
// Two variants are compiled (template parameter DEFER, chosen by batch size at launch): where the softmax
// merge of a head shared by several CTAs happens, and how the MLP partial sums are staged.  Code that does not
// run is kept out of each variant: the kernel is sensitive to its instruction footprint and register pressure.
#include "step_core.cuh"

namespace fasttps {

namespace {

// DEFER: where the softmax merge of a head shared by several CTAs happens.  true (batch <= 2): every CTA only
// publishes its partials and the prologue of the output projection merges them on the fly -- no ticket chain in
// the short attention phase.  false: the CTA that finishes a head last merges it, hidden behind the long
// attention phase of a larger batch, where the merge loads of the prologue would serialise.  Two kernels
// rather than a run-time switch: code that does not run still costs instruction-cache reach and registers.
template <int IPW, int DH, bool DEFER>
__global__ void __launch_bounds__(kMegaThreadsMax, 1) decode_step_kernel(StepArgs a)
{
    extern __shared__ __align__(128) unsigned char dsm[];
    __shared__ __align__(16) ActTile s_hi[kMaxOctetsPerCta];
    __shared__ __align__(16) ActTile s_lo[kMaxOctetsPerCta];
    __shared__ float s_best_val[64];
    __shared__ int s_best_idx[64];
    __shared__ int s_go;
    __shared__ int s_tables_ready;                               // steps whose attention tables are built
    __shared__ LayerPtrs s_layers[kMaxStepLayers];               // the layer table: no global round trip per phase
    __shared__ SegmentList s_segs;                               // this CTA's attention share for the current step
    __shared__ unsigned char s_head_n[kMaxSegments];               // CTAs that share head (b, h) in the current step

    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    const int cta = blockIdx.x, ncta = gridDim.x;
    if (t == 0) s_tables_ready = 0;
    const MegaLayout lay = mega_layout<DH>(a.D);
    const int nw = lay.nw, nct = nw * 32;
    float *smem_part = reinterpret_cast<float *>(dsm + lay.part_off);
    float *smem_red = reinterpret_cast<float *>(dsm + lay.red_off);
    AttnScratch<DH> &scratch = *reinterpret_cast<AttnScratch<DH> *>(dsm + lay.scratch_off);

    const int D = a.D, B = a.batch;
    const int nq = a.n_q_heads * a.head_dim, nkv = a.n_kv_heads * a.head_dim, nqkv = nq + 2 * nkv;
    constexpr int SPT = IPW / kBlocksPerWarpPerSlot;      // ring pieces per 16-row tile
    constexpr int PPO = IPW / 4;                          // ring pieces per W_down octet
    const size_t tile_bytes = (size_t)D * 32;             // 16 rows x D (every reduction length here is D)
    const size_t oct_bytes = (size_t)D * 16;

    // this CTA's share of every product (the same for every layer)
    int q0, qn, o0, on, m0, mn, l0, ln;
    cta_range((nqkv + 15) >> 4, cta, ncta, q0, qn);
    cta_range((D + 15) >> 4, cta, ncta, o0, on);
    cta_range(a.K >> 3, cta, ncta, m0, mn);
    cta_range((a.V + 15) >> 4, cta, ncta, l0, ln);
    int ncta_attn = (kMaxSplits - 2) * a.n_q_heads;
    if (ncta_attn > ncta) ncta_attn = ncta;

    WeightRing ring;
    ring.init(dsm + lay.ring_off, reinterpret_cast<uint64_t *>(dsm + lay.bar_off),
              reinterpret_cast<int *>(dsm + lay.abort_off), lay.nslot, lay.slot_stride, nw, nullptr, 0, nullptr, 0);
    if (t < 64) { s_best_val[t] = -INFINITY; s_best_idx[t] = 0x7fffffff; }
    for (int i = t; i < a.n_layers * (int)(sizeof(LayerPtrs) / 8); i += blockDim.x)
        reinterpret_cast<unsigned long long *>(s_layers)[i] = reinterpret_cast<const unsigned long long *>(a.layers)[i];

    // Per-step attention tables (the lengths grow by one per step, so the split changes with the step, but
    // not with the layer): the segments of this CTA's share, and for every head the number of CTAs that
    // publish a partial for it.  Built by the consumer threads at the top of every step, after the barrier that
    // ends the step before; the producer waits for s_tables_ready before it fetches the step's first K/V tile.
    auto build_step_tables = [&](int step) {
        ShareWalk wk;
        wk.init(a.seq_lens, a.pos, step, B, a.n_q_heads, a.max_seq, cta, ncta_attn);
        if (t == 0) {
            int n = 0;
            Segment sg;
            while (wk.next(sg) && n < kMaxSegments) {
                PackedSegment p;
                p.r0 = sg.r0; p.r1 = sg.r1; p.bh = (unsigned short)(sg.b * a.n_q_heads + sg.h);
                p.first_cta = (unsigned char)sg.first_cta; p.n_cta = (unsigned char)sg.n_cta;
                s_segs.seg[n++] = p;
            }
            s_segs.n = n; s_segs.n_q_heads = a.n_q_heads;
            for (int bb = 0; bb < B; ++bb) { s_segs.len[bb] = wk.rows_of(bb) - 1; s_segs.pos[bb] = a.pos[bb] + step; }
        } else {
            long long head0 = 0;
            int b = 0, rows = wk.rows_of(0);
            for (int idx = t - 1; idx < B * a.n_q_heads; idx += nct - 1) {
                const int bb = idx / a.n_q_heads, hh = idx - bb * a.n_q_heads;
                while (b < bb) { head0 += (long long)a.n_q_heads * rows; ++b; rows = wk.rows_of(b); }
                const long long h0 = head0 + (long long)hh * rows;
                s_head_n[idx] = rows > 0 ? (unsigned char)(wk.owner_of(h0 + rows - 1) - wk.owner_of(h0) + 1) : 0;
            }
        }
    };
    __syncthreads();

    // =========================================================================== producer warp
    // One thread walks this CTA's share of every weight matrix and K/V tile of every step, in the order the
    // consumers need it, copies piece after piece into the shared-memory ring and blocks only on free slots.
    if (w >= nw) {
        if (w > nw || lane != 0) return;
        const uint32_t wp = (uint32_t)lay.wpiece;
        int piece = 0;
        auto weights = [&](const void *base, size_t first_byte, int npieces) -> bool {
            const unsigned char *p = static_cast<const unsigned char *>(base) + first_byte;
            for (int i = 0; i < npieces; ++i, ++piece)
                if (!ring.put(piece, p + (size_t)i * wp, wp)) return false;
            return true;
        };
        for (int step = 0; step < a.n_steps; ++step) {
            for (int l = 0; l < a.n_layers; ++l) {
                const LayerPtrs &lp = s_layers[l];
                if (!weights(lp.w_qkv, (size_t)q0 * tile_bytes, qn * SPT)) return;
                if (l == 0) {
                    // K/V tiles of this step include the rows appended by the step before it, and the share
                    // table is rebuilt per step: both are ready once the consumers have passed the barrier
                    // that ends that step and built the table (weights are never held back).  For all but
                    // toy models the flag is set long before the producer gets here.
                    const unsigned long long t0 = global_ns();
                    while (*reinterpret_cast<volatile int *>(&s_tables_ready) <= step) {
                        if (*ring.abort_flag || global_ns() - t0 > kGridWaitNanos) { *ring.abort_flag = 1; return; }
                        __nanosleep(64);
                    }
                    __threadfence_block();
                }
                const AttnArgs aa = attn_args_of(a, lp, step, ncta_attn);
                const bool kv_ok = attn_for_each_tile<DH>(aa, ListSource(&s_segs),
                                                          [&](const __nv_bfloat16 *k, const __nv_bfloat16 *v, uint32_t bytes) {
                    return ring.put2(piece++, k, v, bytes, kAttnTileRows * AttnTile<DH>::kRowBytes);
                });
                if (!kv_ok) return;
                if (!weights(lp.w_o, (size_t)o0 * tile_bytes, on * SPT)) return;
                if (!weights(lp.w_gu, (size_t)m0 * tile_bytes, mn * SPT)) return;
                if (!weights(lp.w_down, (size_t)m0 * oct_bytes, mn * PPO)) return;
            }
            if (!weights(a.w_lm, (size_t)l0 * tile_bytes, ln * SPT)) return;
        }
        return;
    }

    // =========================================================================== consumer warps
    GridBarrier gb;
    gb.count = a.bar; gb.status = a.status;
    gb.ncta = ncta; gb.s_go = &s_go;
    gb.target = (unsigned)ncta;
    if (cta == 0 && t == 0) {
        // sequences that cannot be served for all steps are reported once and contribute no rows
        for (int bb = 0; bb < B; ++bb) {
            const int L = a.seq_lens[bb], p = a.pos[bb];
            if (L < 0 || L + a.n_steps > a.max_seq) atomicOr(a.status, FASTTPS_DEV_CACHE_FULL);
            else if (p < 0 || p + a.n_steps > a.max_seq) atomicOr(a.status, FASTTPS_DEV_BAD_POSITION);
        }
    }

    // gathers the embedding rows of the current tokens into x0 (CTA 0 only)
    auto embed_rows = [&](const int32_t *ids) {
        for (int idx = t; idx < B * (D >> 3); idx += nct) {
            const int b = idx / (D >> 3), j = idx - b * (D >> 3);
            int id = ld_cg_s32(ids + b);
            if (id < 0 || id >= a.V) { if (j == 0) atomicOr(a.status, FASTTPS_DEV_BAD_TOKEN); id = 0; }
            reinterpret_cast<uint4 *>(a.x0 + (size_t)b * D)[j] = reinterpret_cast<const uint4 *>(a.embed + (size_t)id * D)[j];
        }
    };

    uint32_t bf[IPW][4];
    int piece = 0;
    bool ok = true;

    // optional timeline for profiling: the first and the last CTA stamp the global timer before and
    // after every grid barrier
    int n_stamp = 0;
    auto stamp = [&]() {
#ifdef FASTTPS_FINE_TRACE
        if (a.trace && t == 0 && cta == 0 && n_stamp < a.trace_len)
#else
        if (a.trace && t == 0 && (cta == 0 || cta == ncta - 1) && n_stamp < a.trace_len)
#endif
            a.trace[(size_t)(cta ? 1 : 0) * a.trace_len + n_stamp] = global_ns();
        ++n_stamp;
    };
#ifdef FASTTPS_FINE_TRACE
    // development build: CTA 0 also stamps, into the second half of the buffer, the end of every product's
    // prologue and of its tile loop (two stamps per product phase, none for attention)
    int n_fine = 0;
    auto fine = [&]() {
        if (a.trace && t == 0 && cta == 0 && n_fine < a.trace_len) a.trace[(size_t)a.trace_len + n_fine] = global_ns();
        ++n_fine;
    };
#define FT_FINE() fine()
#else
#define FT_FINE() ((void)0)
#endif
    auto sync_phase = [&]() -> bool {
        stamp();
        const bool go = grid_sync(gb, nct, /*ok=*/ok);
        stamp();
        return go;
    };

    if (cta == 0) embed_rows(a.token_ids);
    if (!sync_phase()) return;

    // One loop over all products of a step.  Every matrix product (QKV, output projection, gate_up, logits)
    // goes through the SAME copy of the B-fragment prologue and of the tile loop, selected by `kind`: the hot
    // code of the kernel stays small enough to live in the instruction cache from one product to the next.
    enum { kQkv = 0, kAttn = 1, kOproj = 2, kMlp = 3, kHead = 4 };
    const int L = a.n_layers;
    for (int step = 0; step < a.n_steps; ++step) {
        build_step_tables(step);
        named_bar_sync(1, nct);
        if (t == 0) {
            __threadfence_block();
            atomicExch(&s_tables_ready, step + 1);              // the producer may fetch this step's K/V rows now
        }
        for (int ph = 0; ph <= 4 * L; ++ph) {
            const int l = ph >> 2;
            const int kind = ph == 4 * L ? kHead : (ph & 3);
            const LayerPtrs &lp = s_layers[l < L ? l : L - 1];
            const int lprev = (kind == kHead ? L : l) - 1;                               // layer whose MLP sums feed x
            const float *y_prev = lprev >= 0 ? a.acc + (size_t)(lprev & 1) * B * D : nullptr;
            const __nv_bfloat16 *x_base = lprev >= 0 ? a.h : a.x0;                      // x = bf16(x_base + y_prev)

            // The gains of the norm two phases ahead are asked from L2 now (they come from HBM once per step):
            // one CTA, one thread per 128-byte line.
            if (cta == ncta - 1 && (kind == kAttn || kind == kMlp) && t * 64 < D) {
                const __nv_bfloat16 *gnext = kind == kAttn ? lp.g_mlp : (l + 1 < L ? s_layers[l + 1].g_attn : a.g_final);
                asm volatile("prefetch.global.L2 [%0];" ::"l"(gnext + t * 64));
            }
            if (kind == kAttn) {
                // ---- attention (Algorithm 3) ----
                const AttnArgs aa = attn_args_of(a, lp, step, ncta_attn);
                // every CTA publishes the partial (max, sum, output) of each of its segments; nobody merges
                // here: the output projection merges while it builds its B fragments
                ok = attn_consume<DH, DEFER>(aa, ring, piece, cta, ListSource(&s_segs), scratch, nw) && ok;
            } else {
                // ---- a matrix product: B fragments, then this CTA's row tiles ----
                const __nv_bfloat16 *src = x_base, *gain = nullptr;
                const float *add = y_prev;
                int tile0 = 0, ntile = 0;
                if (kind == kQkv) { gain = lp.g_attn; tile0 = q0; ntile = qn; }
                else if (kind == kOproj) { src = a.attn_out; add = nullptr; tile0 = o0; ntile = on; }
                else if (kind == kMlp) { src = a.h; add = nullptr; gain = lp.g_mlp; tile0 = m0; ntile = mn; }
                else { gain = a.g_final; tile0 = l0; ntile = ln; }
                // residual of the output projection for the first two tiles (all there are on a full grid),
                // fetched by the epilogue threads now instead of in the epilogue, where the tile loop would wait
                float res[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
                const bool res_pre = kind == kOproj && nct >= 64 && t < 64 && (t & 7) < B;
                if (res_pre) {
                    __nv_bfloat16 xb[2][2];
                    float ya[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        int row = (o0 + (q >> 1)) * 16 + (t >> 3) + 8 * (q & 1);
                        if (row >= D) row = D - 1;
                        xb[q >> 1][q & 1] = ld_cg_bf16(x_base + (size_t)(t & 7) * D + row);
                        if (y_prev) ya[q >> 1][q & 1] = ld_cg_f32(y_prev + (size_t)(t & 7) * D + row);
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float x = __bfloat162float(xb[q >> 1][q & 1]);
                        res[q >> 1][q & 1] = y_prev ? bf16_round(x + ya[q >> 1][q & 1]) : x;
                    }
                }
                if (DEFER && kind == kOproj) load_b_frags_attn<IPW, DH>(bf, a.attn_part, s_head_n, B, a.n_q_heads, nw);
                else load_b_frags<IPW>(bf, src, D, B, D, nw, gain, a.eps, smem_red, add);
                FT_FINE();
                if (kind == kHead) {
                    for (int u = t; u < 64; u += nct) { s_best_val[u] = -INFINITY; s_best_idx[u] = 0x7fffffff; }
                    named_bar_sync(1, nct);
                }
                ok = dot_tiles<IPW>(ring, piece, ntile, nw, bf, smem_part, [&](int tile, int cc, int b, float v0, float v1) {
                    if (kind == kMlp) {                      // siLu_Mul: rows cc / cc + 8 are a gate value and its up value
                        const float act = v0 / (1.f + __expf(-v0)) * v1;
                        const __nv_bfloat16 hi = __float2bfloat16_rn(act);
                        s_hi[tile][b][cc] = hi;
                        s_lo[tile][b][cc] = __float2bfloat16_rn(act - __bfloat162float(hi));
                        return;
                    }
                    if (b >= B) return;
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int row = (tile0 + tile) * 16 + cc + 8 * hh;
                        const float v = hh ? v1 : v0;
                        if (kind == kQkv) {
                            if (row < nqkv) a.qkv[(size_t)b * nqkv + row] = __float2bfloat16_rn(v);
                        } else if (kind == kOproj) {         // h = x_l + attn . W_o
                            if (row < D) {
                                float x;
                                if (res_pre && tile < 2) x = tile == 0 ? res[0][hh] : res[1][hh];
                                else {
                                    x = __bfloat162float(ld_cg_bf16(x_base + (size_t)b * D + row));
                                    if (y_prev) x = bf16_round(x + ld_cg_f32(y_prev + (size_t)b * D + row));
                                }
                                a.h[(size_t)b * D + row] = __float2bfloat16_rn(x + v);
                            }
                        } else if (row < a.V) {              // logits and the running argmax of this thread's rows
                            const int u = cc * 8 + b;
                            if (a.logits) a.logits[(size_t)b * a.V + row] = v;
                            if (v > s_best_val[u]) { s_best_val[u] = v; s_best_idx[u] = row; }
                        }
                    }
                }) && ok;
                piece += ntile * SPT;
                FT_FINE();

                if (kind == kMlp) {
                    // ---- down projection of this CTA's octets; the sums of all CTAs meet in acc[l & 1] ----
                    if (cta == 0 && y_prev) {
                        // layer l - 1's sums have been consumed by everyone (two barriers ago): zero them for layer l + 1
                        float *z = a.acc + (size_t)((l - 1) & 1) * B * D;
                        for (int idx = t; idx < B * (D >> 2); idx += nct) reinterpret_cast<float4 *>(z)[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                    named_bar_sync(1, nct);
                    float acc[IPW][2][4];
#pragma unroll
                    for (int i = 0; i < IPW; ++i)
#pragma unroll
                        for (int m = 0; m < 2; ++m)
#pragma unroll
                            for (int e = 0; e < 4; ++e) acc[i][m][e] = 0.f;
                    mlp_down_phase<IPW>(ring, piece, mn, nw, s_hi, s_lo, acc, ok);
                    piece += mn * PPO;
                    mlp_scatter_add<IPW, !DEFER>(acc, smem_part, a.acc + (size_t)(l & 1) * B * D, B, D, nw);
                } else if (kind == kHead) {
                    named_bar_sync(1, nct);
                    if (t < 8 && t < B) {
                        float bv = -INFINITY; int bi = 0x7fffffff;
                        for (int cc = 0; cc < 8; ++cc) {
                            const float v = s_best_val[cc * 8 + t]; const int i = s_best_idx[cc * 8 + t];
                            if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
                        }
                        a.amax_val[(size_t)t * ncta + cta] = bv;
                        a.amax_idx[(size_t)t * ncta + cta] = bi;
                    }
                }
            }
            if (!sync_phase()) return;
        }

        // ---- CTA 0 finishes the greedy argmax, advances the state and gathers the next embedding rows ----
        if (cta == 0) {
            // every thread fetches its share of the per-CTA candidates at once, then warps and the CTA reduce
            for (int b = 0; b < B; ++b) {
                float bv = -INFINITY; int bi = 0x7fffffff;
                for (int c = t; c < ncta; c += nct) {
                    const float v = ld_cg_f32(a.amax_val + (size_t)b * ncta + c);
                    const int i = ld_cg_s32(a.amax_idx + (size_t)b * ncta + c);
                    if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
                }
#pragma unroll
                for (int s = 16; s >= 1; s >>= 1) {
                    const float ov = __shfl_xor_sync(kFull, bv, s);
                    const int oi = __shfl_xor_sync(kFull, bi, s);
                    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
                }
                if (lane == 0) { s_best_val[w] = bv; s_best_idx[w] = bi; }
                named_bar_sync(1, nct);
                if (t == 0) {
                    for (int w2 = 0; w2 < nw; ++w2) {
                        const float v = s_best_val[w2]; const int i = s_best_idx[w2];
                        if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
                    }
                    if (bi == 0x7fffffff) bi = 0;      // all-NaN row: fall back to index 0
                    a.tok[b] = bi;
                    if (a.out_ids) a.out_ids[(size_t)step * B + b] = bi;
                    if (step == a.n_steps - 1) {
                        a.next_ids[b] = bi;
                        if (a.advance) { a.pos[b] += a.n_steps; a.seq_lens[b] += a.n_steps; }
                    }
                }
                named_bar_sync(1, nct);
            }
            // the last layer's MLP sums are consumed: back to zero (the other buffer was zeroed in the last MLP phase)
            float *z = a.acc + (size_t)((L - 1) & 1) * B * D;
            for (int idx = t; idx < B * (D >> 2); idx += nct) reinterpret_cast<float4 *>(z)[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (step + 1 < a.n_steps) {
                __threadfence();
                named_bar_sync(1, nct);
                embed_rows(a.tok);
            }
        }
        if (step + 1 < a.n_steps && !sync_phase()) return;
    }
}

}  // namespace

template <int IPW, int DH, bool DEFER>
static int launch_step_inst(Ctx *c, const StepArgs &a, cudaStream_t st)
{
    const MegaLayout lay = mega_layout<DH>(a.D);
    auto kernel = decode_step_kernel<IPW, DH, DEFER>;
    static bool configured[16] = {};
    if (!configured[c->cfg.device & 15]) {
        FT_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStreamSmemMax));
        int per_sm = 0;
        FT_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, (lay.nw + 1) * 32, lay.total));
        if (per_sm < 1) return FASTTPS_INVALID_ARG;
        configured[c->cfg.device & 15] = true;
    }
    if ((unsigned long long)(4 * a.n_layers + 3) * (unsigned long long)a.n_steps * (unsigned long long)c->n_sm >= kBarAbort)
        return FASTTPS_INVALID_ARG;                      // the arrival counter must stay below the abort mark
    // the barrier counter starts from zero every launch
    FT_CUDA(cudaMemsetAsync(c->grid_bar, 0, 64 * sizeof(unsigned), st));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(c->n_sm); cfg.blockDim = dim3((lay.nw + 1) * 32); cfg.dynamicSmemBytes = lay.total; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    void *params[] = {const_cast<StepArgs *>(&a)};
    ProfScope prof(c, kProfStep, st);
    FT_CUDA(cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(kernel), params));
    c->launches++;
    return FASTTPS_OK;
}

// True when the persistent kernel can serve this model shape and batch.
bool step_kernel_supported(const Ctx *c, int batch)
{
    const fasttps_config &f = c->cfg;
    const WarpSplit s = warp_split(f.hidden);
    if (batch < 1 || batch > kMaxNB) return false;
    if (f.n_q_heads * f.head_dim != f.hidden) return false;      // one reduction length for every product
    if (s.nw < 1 || s.nw > 12) return false;
    if (f.n_q_heads > kMaxStepHeads || f.n_layers > kMaxStepLayers) return false;
    if (batch * f.n_q_heads >= kMaxSegments || c->n_sm > 255) return false;   // segment table: capacity, 8-bit CTA index
    if (f.vocab < 1 || f.n_layers < 1) return false;
    return true;
}

int launch_step(Ctx *c, const StepArgs &a, cudaStream_t st)
{
    const int ipw = warp_split(a.D).ipw;
    const bool defer = a.batch <= 2;
#define FT_STEP(DHV)                                                                                     \
    case DHV:                                                                                            \
        if (defer) return ipw == 8 ? launch_step_inst<8, DHV, true>(c, a, st) : launch_step_inst<4, DHV, true>(c, a, st); \
        return ipw == 8 ? launch_step_inst<8, DHV, false>(c, a, st) : launch_step_inst<4, DHV, false>(c, a, st)
    switch (a.head_dim) {
        FT_STEP(32);
        FT_STEP(64);
        FT_STEP(96);
        FT_STEP(128);
    default: return FASTTPS_INVALID_ARG;
    }
#undef FT_STEP
}

}  // namespace fasttps
