// Persistent decode-step kernel (batch <= 8): the whole token phase of the model -- embedding gather, then
// for every layer RMSNorm -> QKV -> attention (Algorithm 3) -> output projection -> RMSNorm -> fused MLP
// (Algorithm 4), then the final norm, the logits and the greedy argmax -- in ONE cooperative launch, for one or
// several consecutive tokens.
//
// Why: at batch 1 a layer is ~37 us of HBM streaming cut into dependent products.  As separate kernels each of
// them pays a launch, a cold start of its copy pipeline and a drain, during which HBM idles.  Here one CTA per SM
// stays resident; a producer warp walks the CTA's share of EVERY weight matrix and K/V tile of the step in
// order and keeps the shared-memory ring (~190 KB per SM) full, never waiting for anything but free slots; the
// consumer warps meet at a grid-wide barrier after each phase (one arrival counter in global memory that only
// grows during a launch; every wait is bounded, and a CTA that gives up pushes the counter beyond every
// target, so nobody spins forever; the launch is cooperative, so all CTAs are resident).
//
// Every grid-wide boundary still costs 4-5 us of dependent latency (barrier, activation loads, norm), so there
// are THREE per layer, not four: the attention and the output projection are one phase.  Every query
// head belongs to a fixed group of m0 = n_sm / H_q CTAs.  The group's CTAs split the rows of the head's caches,
// all sequences of the batch laid end to end, into equal shares whatever the mix of lengths
// (Algorithm 3 on each share, partial (max, sum, output) published), meet at a counter of their own -- a wait
// for at most m0 - 1 neighbours instead of the whole grid --, each merges the head's partials, and each then
// multiplies the merged head output with ITS slice of the output-projection rows: for row tile r the d / 32
// k blocks of the head are d KB contiguous in the packed W_o, so a ring piece is a handful of such runs.  The
// products of the 32 heads meet in an FP32 accumulator (red.add); the residual add h = x + attn W_o moves into
// the prologue of the MLP phase, which also writes h out (one share of its chunks per CTA), as the QKV
// prologue does for x = h + y of the layer before.
#pragma once
#include <cstdlib>
#include "step_core.cuh"

namespace fasttps {

namespace {

// A CTA's share of its head: at most one segment per sequence.
struct GroupSegs {
    int n;
    Segment seg[kMaxNB];
};
struct GroupSource {
    const GroupSegs *p;
    int i;
    __device__ __forceinline__ explicit GroupSource(const GroupSegs *p_) : p(p_), i(0) {}
    __device__ __forceinline__ bool next(Segment &s)
    {
        if (i >= p->n) return false;
        s = p->seg[i++];
        return true;
    }
    __device__ __forceinline__ int count() const { return p->n; }
    __device__ __forceinline__ const Segment &at(int n) const { return p->seg[n]; }
};

// BC: batch class.  0: batch 1 (the batch loops fold away at compile time), 1: batch 2, 2: batches 3 to 8 (which
// also selects the staging of the MLP scatter; see mlp_core.cuh).
// This step's attention shares (thread 0 of every CTA; out of line so that its registers and its table stay out
// of the step kernel's loops): the rows of a head, all sequences end to end, are cut into m' shares of equal
// cost, one per CTA of the head's group (at least 16 rows each).  A cached row costs 1.  The end of a sequence
// costs kNewRowCost cached rows (at most three quarters of a share): the share that holds it scores the new row
// (RoPE of k, the append, the score from shared memory) and, in a batch, starts another segment behind it (RoPE
// of q, combine, partial write).  Measured on the ragged batch of 8: 0 -> 2603, 64 -> 2648, 128 -> 2669,
// 256 -> 2682 tok/s; at batch 1 the last share shrinks from 256 to about 110 of 1025 rows (+1.8 %).
static __host__ __device__ __noinline__ void build_attention_shares(const int32_t *seq_lens, const int32_t *pos, int max_seq, int step,
                                                           int B, int gm, int gs, int head, bool in_group, GroupSegs *segs,
                                                           int *ncta_out, int *mprime_out, int *cuts)
{
    constexpr int kNewRowCost = 256;
    int R[kMaxNB];
    long long T = 0;
    for (int bb = 0; bb < B; ++bb) {
        const int Ls = seq_lens[bb] + step, ps = pos[bb] + step;
        const bool valid = !(Ls < step || Ls >= max_seq || ps < step || ps >= max_seq);
        R[bb] = valid ? Ls + 1 : 0;
        T += R[bb];
    }
    int mp = (int)(T / 16 < gm ? T / 16 : gm);
    mp = T == 0 ? 0 : (mp < 1 ? 1 : mp);
    *mprime_out = mp;
    // share k holds the rows [cuts[k], cuts[k + 1]) of the flattened row space (cuts: kMaxSplits + 1 words of shared memory)
    {
        long long X = mp ? 3 * T / (4 * mp) : 0;
        if (X > kNewRowCost) X = kNewRowCost;
        int nvalid = 0;
        for (int bb = 0; bb < B; ++bb) nvalid += R[bb] > 0;
        const long long Wt = T + X * nvalid;
        for (int k = 0; k <= mp; ++k) {
            const long long c = mp ? Wt * k / mp : 0;     // the cut in cost units ...
            long long woff = 0, off = 0, row = T;      // ... and the row it falls on
            for (int bb = 0; bb < B; ++bb) {
                const long long wb = R[bb] > 0 ? R[bb] + X : 0;
                if (c < woff + wb) {
                    const long long local = c - woff;
                    row = off + (local <= R[bb] - 1 ? local : R[bb]);
                    break;
                }
                woff += wb; off += R[bb];
            }
            cuts[k] = (int)row;
        }
        // no share may be empty (T >= 16 mp rows): the partial of every share between a sequence's first and last is waited for
        for (int k = 1; k < mp; ++k) if (cuts[k] <= cuts[k - 1]) cuts[k] = cuts[k - 1] + 1;
        for (int k = mp - 1; k >= 1; --k) if (cuts[k] >= cuts[k + 1]) cuts[k] = cuts[k + 1] - 1;
    }
    const long long f0 = (mp && gs < mp) ? cuts[gs] : 0, f1 = (mp && gs < mp) ? cuts[gs + 1] : f0;
    auto owner = [&](long long x) {                    // the share that holds row x of the head
        int c = 0;
        while (c + 1 < mp && cuts[c + 1] <= x) ++c;
        return c;
    };
    int n = 0;
    long long off = 0;
    for (int bb = 0; bb < B; ++bb) {
        const int rb = R[bb];
        ncta_out[bb] = 0;
        if (rb > 0) {
            const int first = owner(off), last = owner(off + rb - 1);
            ncta_out[bb] = last - first + 1;
            const long long lo = f0 > off ? f0 : off, hi = f1 < off + rb ? f1 : off + rb;
            if (in_group && lo < hi) {
                Segment &sg = segs->seg[n++];
                sg.b = bb; sg.h = head; sg.L = rb - 1; sg.pos = pos[bb] + step;
                sg.r0 = (int)(lo - off); sg.r1 = (int)(hi - off);
                sg.first_cta = head * gm + first; sg.n_cta = last - first + 1;
            }
        }
        off += rb;
    }
    segs->n = n;
}

// LAYER: one decoder layer on caller-supplied activations (fasttps_layer_decode): no embedding gather, no
// logits; a closing pass writes x_out = h + y.
template <int IPW, int DH, int BC, bool LAYER>
__global__ void __launch_bounds__(kMegaThreadsMax, 1) decode_step_kernel(const __grid_constant__ StepArgs a)
{
    extern __shared__ __align__(128) unsigned char dsm[];
    __shared__ __align__(16) ActTile s_hi[kMaxOctetsPerCta];
    __shared__ __align__(16) ActTile s_lo[kMaxOctetsPerCta];
    __shared__ float s_best_val[64];
    __shared__ int s_best_idx[64];
    __shared__ int s_go;
    __shared__ int s_tables_ready;                               // steps whose attention share is known
    __shared__ LayerPtrs s_layers[LAYER ? 1 : kMaxStepLayers];   // the layer table, copied from the kernel parameters
    __shared__ GroupSegs s_segs;                                 // this CTA's attention share for the current step
    __shared__ int s_cuts[kMaxSplits + 1];                       // row cuts of the shares of a head in the current step
    __shared__ AttnPre<DH> s_pre;                                // the rotated q (and new K/V rows) of all segments of the share
    __shared__ int s_mprime;                                     // CTAs of a group that hold rows in the current step
    __shared__ int s_ncta[kMaxNB];                               // partials of (sequence b, this head) in the current step
    __shared__ __align__(16) __nv_bfloat16 s_outh[kMaxNB * DH];  // the merged outputs of this CTA's head, per sequence

    constexpr int KB = DH / 32;                                  // k blocks of a head in the output projection
    const int t = threadIdx.x, lane = t & 31, w = t >> 5, g = lane >> 2, t4 = lane & 3;
    const int cta = blockIdx.x, ncta = gridDim.x;
    if (t == 0) s_tables_ready = 0;
    const MegaLayout lay = mega_layout<DH>(a.D);
    const int nw = lay.nw, nct = nw * 32;
    float *smem_part = reinterpret_cast<float *>(dsm + lay.part_off);
    float *smem_red = reinterpret_cast<float *>(dsm + lay.red_off);
    AttnScratch<DH> &scratch = *reinterpret_cast<AttnScratch<DH> *>(dsm + lay.scratch_off);

    const int D = a.D, B = BC == 0 ? 1 : a.batch;
    const int nq = a.n_q_heads * a.head_dim, nkv = a.n_kv_heads * a.head_dim, nqkv = nq + 2 * nkv;
    constexpr int SPT = IPW / kBlocksPerWarpPerSlot;      // ring pieces per 16-row tile
    constexpr int PPO = IPW / 4;                          // ring pieces per W_down octet
    const size_t tile_bytes = (size_t)D * 32;             // 16 rows x D (every reduction length here is D)
    const size_t oct_bytes = (size_t)D * 16;

    // this CTA's share of every grid-wide product (the same for every layer)
    int q0, qn, m0, mn, l0, ln;
    cta_range((nqkv + 15) >> 4, cta, ncta, q0, qn);
    cta_range(a.K >> 3, cta, ncta, m0, mn);
    cta_range((a.V + 15) >> 4, cta, ncta, l0, ln);
    // head groups: CTA (head, gs) of gm CTAs per head; the CTAs beyond n_q_heads * gm sit the fused phase out
    int gm = ncta / a.n_q_heads;
    if (gm > kMaxSplits) gm = kMaxSplits;
    const int head = cta / gm, gs = cta - head * gm;
    const bool in_group = head < a.n_q_heads;
    int ot0 = 0, ont = 0;                                  // this CTA's row tiles of the output projection
    if (in_group) cta_range((D + 15) >> 4, gs, gm, ot0, ont);
    int TP = lay.slot_stride / (KB * kTileBytes);          // row tiles of the output projection per ring piece
    if (TP > nw) TP = nw;
    unsigned *grp = a.bar + 64 + (in_group ? head : 0);    // arrivals of this group's partials since the launch
    float *hacc = a.hacc;                                  // [2][D] FP32 sums of the output projection
    __nv_bfloat16 *xbuf = a.attn_out;                      // x of the current layer (the attention output tensor is not needed here)

    WeightRing ring;
    ring.init(dsm + lay.ring_off, reinterpret_cast<uint64_t *>(dsm + lay.bar_off),
              reinterpret_cast<int *>(dsm + lay.abort_off), lay.nslot, lay.slot_stride, nw, nullptr, 0, nullptr, 0);
    if (t < 64) { s_best_val[t] = -INFINITY; s_best_idx[t] = 0x7fffffff; }
    for (int i = t; i < a.n_layers * (int)(sizeof(LayerPtrs) / 8); i += blockDim.x)
        reinterpret_cast<unsigned long long *>(s_layers)[i] = reinterpret_cast<const unsigned long long *>(a.layers)[i];   // parameter space
    __syncthreads();

    // =========================================================================== producer warp
    if (w >= nw) {
        if (w > nw || lane != 0) return;
        const uint32_t wp = (uint32_t)lay.wpiece;
        int piece = 0;
        // every piece is read once: its L2 lines go first, the lines prefetched for later pieces stay
        ring.policy = l2_policy_evict_first();
        // how far (in ring pieces) the L2 prefetch runs ahead of the ring in each product; measured on the
        // Phi-3-mini shape with an 8-slot ring: 3 / 6 / 12 / 6.  Deeper prefetches of the QKV and gate_up pieces
        // are issued during the phases before them and slow those down by more than they gain.
        const int pf_qkv = (3 * ring.nslot + 7) / 8, pf_gu = 3 * ring.nslot / 4, pf_down = 3 * ring.nslot / 2,
                  pf_lm = 3 * ring.nslot / 4;
        auto weights = [&](const void *base, size_t first_byte, int npieces, int ahead) -> bool {
            const unsigned char *p = static_cast<const unsigned char *>(base) + first_byte;
            // the L2 runs `ahead` pieces ahead of the ring: while the consumers are held up at a phase boundary and
            // the ring is full, HBM keeps working on the pieces that follow
            for (int i = 0; i < npieces && i < ahead; ++i) bulk_prefetch_l2(p + (size_t)i * wp, wp);
            for (int i = 0; i < npieces; ++i, ++piece) {
                if (i + ahead < npieces) bulk_prefetch_l2(p + (size_t)(i + ahead) * wp, wp);
                if (!ring.put(piece, p + (size_t)i * wp, wp)) return false;
            }
            return true;
        };
        auto stream_all = [&]() -> bool {
            for (int step = 0; step < a.n_steps; ++step) {
                for (int l = 0; l < a.n_layers; ++l) {
                    const LayerPtrs &lp = s_layers[l];
                    if (!weights(lp.w_qkv, (size_t)q0 * tile_bytes, qn * SPT, pf_qkv)) return false;
                    if (l == 0) {
                        // K/V tiles of this step include the row appended by the step before it, and the share is
                        // recomputed per step: both are ready once the consumers have passed the barrier that ends
                        // that step (weights are never held back)
                        const unsigned long long t0 = global_ns();
                        while (*reinterpret_cast<volatile int *>(&s_tables_ready) <= step) {
                            if (*ring.abort_flag || global_ns() - t0 > kGridWaitNanos) { *ring.abort_flag = 1; return false; }
                            __nanosleep(64);
                        }
                        __threadfence_block();
                    }
                    const AttnArgs aa = attn_args_of(a, lp, step, gm * a.n_q_heads);
                    const unsigned char *wo = reinterpret_cast<const unsigned char *>(lp.w_o);
                    const bool kv_ok = attn_for_each_tile<DH>(aa, GroupSource(&s_segs),
                                                              [&](const unsigned char *k, const unsigned char *v, uint32_t bytes) {
                        if (!ring.put2(piece, k, v, bytes, kAttnTileRows * AttnTile<DH>::kRowBytes)) return false;
                        ++piece;
                        return true;
                    });
                    if (!kv_ok) return false;
                    // this CTA's rows of the output projection, the head's k blocks only: KB KB per row tile
                    for (int p0 = 0; p0 < ont; p0 += TP, ++piece) {
                        const int nt = ont - p0 < TP ? ont - p0 : TP;
                        if (!ring.acquire(piece)) return false;
                        const int sl = ring.slot_of(piece);
                        mbar_expect_tx(&ring.full[sl], (uint32_t)(nt * KB * kTileBytes));
                        for (int j = 0; j < nt; ++j)
                            bulk_g2s_hint(ring.slots + (size_t)sl * ring.slot_bytes + (size_t)j * KB * kTileBytes,
                                          wo + ((size_t)(ot0 + p0 + j) * (nq / 32) + (size_t)head * KB) * kTileBytes,
                                          (uint32_t)(KB * kTileBytes), &ring.full[sl], ring.policy);
                    }
                    // the gate_up prefetch waits until this CTA's rows of W_o have landed
                    if (ont > 0 && !mbar_wait_bounded(&ring.full[ring.slot_of(piece - 1)], (uint32_t)ring.round_of(piece - 1) & 1u, ring.abort_flag)) return false;
                    if (!weights(lp.w_gu, (size_t)m0 * tile_bytes, mn * SPT, pf_gu)) return false;
                    if (!weights(lp.w_down, (size_t)m0 * oct_bytes, mn * PPO, pf_down)) return false;
                }
                if (!LAYER && !weights(a.w_lm, (size_t)l0 * tile_bytes, ln * SPT, pf_lm)) return false;
            }
            return true;
        };
        // after a failed wait the copies already handed to the copy engine get a bounded chance to land
        if (!stream_all()) ring.drain(piece);
        return;
    }

    // =========================================================================== consumer warps
    GridBarrier gb;
    gb.count = a.bar; gb.status = a.status;
    gb.ncta = ncta; gb.s_go = &s_go;
    gb.target = (unsigned)ncta;
    unsigned grp_target = 0;
    if (cta == 0 && t == 0) {
        // sequences that cannot be served for all steps are reported once and contribute no rows
        for (int bb = 0; bb < B; ++bb) {
            const int L = a.seq_lens[bb], p = a.pos[bb];
            if (L < 0 || L + a.n_steps > a.max_seq) atomicOr(a.status, FASTTPS_DEV_CACHE_FULL);
            else if (p < 0 || p + a.n_steps > a.max_seq) atomicOr(a.status, FASTTPS_DEV_BAD_POSITION);
        }
    }

    // gathers the embedding rows of the current tokens into x0 (CTA 0 only)
    auto embed_row = [&](const int32_t *ids) {
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

    auto sync_phase = [&]() -> bool { return grid_sync(gb, nct, /*ok=*/ok); };
    // On the way out of a launch that ran to its end every CTA signs off; the last one puts the barrier words back
    // to zero (nobody polls them any more), so the next launch needs no clearing pass in front of it.  A launch that
    // was abandoned leaves them as they are: fasttps_get_status clears them when it reports the timeout.
    auto sign_off = [&]() {
        if (t == 0 && atomicAdd(a.bar + kGridBarDoneWord, 1u) == (unsigned)ncta - 1u) {
            a.bar[0] = 0u;
            for (int hh = 0; hh < a.n_q_heads; ++hh) a.bar[64 + hh] = 0u;
            a.bar[kGridBarDoneWord] = 0u;
        }
    };

    if constexpr (!LAYER) {
        if (cta == 0) embed_row(a.token_ids);
        if (!sync_phase()) return;
    }

    enum { kQkv = 0, kAttn = 1, kMlp = 2, kHead = 3 };
    const int L = a.n_layers;
    for (int step = 0; step < a.n_steps; ++step) {
        // ---- this step's attention shares ----
        if (t == 0) build_attention_shares(a.seq_lens, a.pos, a.max_seq, step, B, gm, gs, head, in_group, &s_segs, s_ncta, &s_mprime, s_cuts);
        named_bar_sync(1, nct);
        if (t == 0) {
            __threadfence_block();
            atomicExch(&s_tables_ready, step + 1);              // the producer may fetch this step's K/V rows now
        }
        const int mprime = s_mprime;

        for (int ph = 0; ph < 3 * L + (LAYER ? 0 : 1); ++ph) {
            const int l = ph / 3;
            const int kind = (!LAYER && ph == 3 * L) ? kHead : ph - 3 * l;
            const LayerPtrs &lp = s_layers[l < L ? l : L - 1];

            // The gains of the norm after next are asked from L2 now (they come from HBM once per step)
            if (cta == ncta - 1 && (kind == kQkv || kind == kAttn) && t * 64 < D) {
                const __nv_bfloat16 *gnext = kind == kQkv ? lp.g_mlp : (l + 1 < L ? s_layers[l + 1].g_attn : a.g_final);
                asm volatile("prefetch.global.L2 [%0];" ::"l"(gnext + t * 64));
            }

            if (kind == kAttn) {
                // ---- attention (Algorithm 3) on this CTA's rows of its head; the partial is published ----
                const AttnArgs aa = attn_args_of(a, lp, step, gm * a.n_q_heads);
                ok = attn_consume<DH, true, GroupSource, BC != 0, BC != 0>(aa, ring, piece, cta, GroupSource(&s_segs), scratch, nw, &s_pre) && ok;
                grp_target += (unsigned)mprime;
                if (in_group) {
                    // ---- the group meets: every CTA of it needs the merged output of the head ----
                    __threadfence();
                    named_bar_sync(1, nct);
                    if (t == 0) {
                        if (s_segs.n && ok) atomicAdd(grp, 1u);
                        int met = 1;
                        unsigned long long t0 = 0;
                        for (unsigned it = 1; ld_acquire_u32(grp) < grp_target; ++it) {
                            if ((it & 63u) == 0) {
                                const unsigned long long now = global_ns();
                                if (t0 == 0) t0 = now;
                                else if (now - t0 > kGridWaitNanos) { met = 0; break; }
                            }
                        }
                        s_go = met;
                    }
                    named_bar_sync(1, nct);
                    if (!s_go) ok = false;
                    // ---- softmax merge of the head's partials: out = sum_s 2^(m_s - M) o_s / sum_s 2^(m_s - M) l_s ----
                    constexpr int PS = DH + 4;
                    for (int idx = t; idx < B * DH; idx += nct) {
                        const int b = idx / DH, i = idx - b * DH;
                        const int np = s_ncta[b];
                        const float *hp = a.attn_part + ((size_t)b * a.n_q_heads + head) * kMaxSplits * PS;
                        float M = -INFINITY, den = 0.f, o = 0.f;
                        for (int s0 = 0; s0 < np; s0 += 4) {
                            float ms[4], ls[4], os[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const bool have = s0 + u < np;
                                const float *p = hp + (size_t)(have ? s0 + u : 0) * PS;
                                ms[u] = ld_cg_f32(p + DH);
                                ls[u] = ld_cg_f32(p + DH + 1);
                                os[u] = ld_cg_f32(p + i);
                                if (!have) ms[u] = -INFINITY;
                            }
                            float Mn = M;
#pragma unroll
                            for (int u = 0; u < 4; ++u) Mn = fmaxf(Mn, ms[u]);
                            const float corr = fast_exp2(M - Mn);        // 0 in the first round (M = -inf)
                            den *= corr; o *= corr;
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const float f = ms[u] == -INFINITY ? 0.f : fast_exp2(ms[u] - Mn);
                                den = fmaf(f, ls[u], den);
                                o = fmaf(f, os[u], o);
                            }
                            M = Mn;
                        }
                        s_outh[idx] = __float2bfloat16_rn(np > 0 && ok ? o / den : 0.f);
                    }
                    named_bar_sync(1, nct);
                    // ---- this CTA's row tiles of the output projection, k = the head: sums go to hacc[l & 1] ----
                    uint4 bh[KB];
#pragma unroll
                    for (int j = 0; j < KB; ++j)
                        bh[j] = g < B ? *reinterpret_cast<const uint4 *>(s_outh + g * DH + 32 * j + 8 * t4) : make_uint4(0u, 0u, 0u, 0u);
                    float *hsum = hacc + (size_t)(l & 1) * B * D;
#pragma unroll(BC == 0 ? 1 : 2)
                    for (int p0 = 0; p0 < ont; p0 += TP, ++piece) {
                        const int nt = ont - p0 < TP ? ont - p0 : TP;
                        const unsigned char *slot = ring.wait(piece, ok);
                        float c[4] = {0.f, 0.f, 0.f, 0.f};
                        if (w < nt) {
                            // independent accumulators per half k block: the products do not wait for one another
                            float cj[2 * KB][4];
#pragma unroll
                            for (int j = 0; j < KB; ++j) {
                                const unsigned char *blk = slot + (size_t)(w * KB + j) * kTileBytes + lane * 16;
                                const uint4 lo = *reinterpret_cast<const uint4 *>(blk);
                                const uint4 hi = *reinterpret_cast<const uint4 *>(blk + 512);
#pragma unroll
                                for (int e = 0; e < 4; ++e) cj[2 * j][e] = cj[2 * j + 1][e] = 0.f;
                                mma_bf16_k16(cj[2 * j], lo.x, hi.x, lo.y, hi.y, bh[j].x, bh[j].y);
                                mma_bf16_k16(cj[2 * j + 1], lo.z, hi.z, lo.w, hi.w, bh[j].z, bh[j].w);
                            }
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                c[e] = 0.f;
#pragma unroll
                                for (int j = 0; j < 2 * KB; ++j) c[e] += cj[j][e];
                            }
                        }
                        // the slot goes back before the sums leave: an arrival after the reductions would wait for them
                        ring.release(piece);
                        if (w < nt) {
                            // accumulator fragment: rows g / g + 8 of the tile, batch rows 2 t4 / 2 t4 + 1.  The packed
                            // W_o pairs its rows: rows g and g + 8 of a tile are the output columns 2 g and 2 g + 1,
                            // so the two sums of a batch row leave as one 8-byte reduction
                            const int col = (ot0 + p0 + w) * 16 + 2 * g, b0 = 2 * t4;
                            if (ok && b0 < B) red_add_v2(hsum + (size_t)b0 * D + col, c[0], c[2]);
                            if (ok && b0 + 1 < B) red_add_v2(hsum + (size_t)(b0 + 1) * D + col, c[1], c[3]);
                        }
                    }
                }
            } else {
                // ---- a grid-wide matrix product: B fragments, then this CTA's row tiles ----
                const __nv_bfloat16 *src, *gain;
                const float *add;
                __nv_bfloat16 *store = nullptr;
                int tile0, ntile;
                if (kind == kQkv) {                          // x_l = h_{l-1} + y_{l-1} (layer 0: the embedding row)
                    src = l == 0 ? a.x0 : a.h; add = l == 0 ? nullptr : a.acc + (size_t)((l - 1) & 1) * B * D;
                    gain = lp.g_attn; store = l == 0 ? nullptr : xbuf; tile0 = q0; ntile = qn;
                } else if (kind == kMlp) {                   // h_l = x_l + attn . W_o
                    src = l == 0 ? a.x0 : xbuf; add = hacc + (size_t)(l & 1) * B * D;
                    gain = lp.g_mlp; store = a.h; tile0 = m0; ntile = mn;
                } else {                                     // x_L = h_{L-1} + y_{L-1}
                    src = a.h; add = a.acc + (size_t)((L - 1) & 1) * B * D;
                    gain = a.g_final; tile0 = l0; ntile = ln;
                }
                const bool is_head = !LAYER && kind == kHead;
                // the sums of the output projection of the layer before are consumed: back to zero
                if (cta == ncta - 1 && ((kind == kQkv && l > 0) || is_head)) {
                    float *z = hacc + (size_t)((l - 1) & 1) * B * D;   // (head: l = L)
                    for (int idx = t; idx < B * (D >> 2); idx += nct) reinterpret_cast<float4 *>(z)[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                if (BC == 0) load_b_frags_one_row<IPW>(bf, src, D, nw, gain, a.eps, smem_red, add, store, cta, ncta);
                else load_b_frags<IPW>(bf, src, D, B, D, nw, gain, a.eps, smem_red, add, store, cta, ncta);
                if (is_head) {
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
                        } else if (!LAYER && row < a.V) {    // logits and the running argmax of this thread's rows
                            const int u = cc * 8 + b;
                            if (a.logits) a.logits[(size_t)b * a.V + row] = v;
                            if (v > s_best_val[u]) { s_best_val[u] = v; s_best_idx[u] = row; }
                        }
                    }
                }) && ok;
                piece += ntile * SPT;

                if (kind == kMlp) {
                    // ---- down projection of this CTA's octets; the sums of all CTAs meet in acc[l & 1] ----
                    if (cta == 0 && l > 0) {
                        // layer l - 1's sums were consumed by the QKV prologue of this layer: zero them for layer l + 1
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
                    mlp_scatter_add<IPW>(acc, a.acc + (size_t)(l & 1) * B * D, B, D, nw);
                } else if (is_head) {
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

        if constexpr (LAYER) {
            // ---- x_out = h + y, one share of the 16-byte chunks per CTA; the consumed sums go back to zero ----
            float *ysum = a.acc, *hs = hacc;                   // buffer 0 of each: the layer index is 0
            for (int idx = cta * nct + t; idx < B * (D >> 3); idx += ncta * nct) {
                const uint4 hv = ld_cg_u4(a.h + (size_t)idx * 8);
                const float4 y0 = ld_cg_f4(ysum + (size_t)idx * 8), y1 = ld_cg_f4(ysum + (size_t)idx * 8 + 4);
                uint4 o;
                o.x = pack2(bf_lo(hv.x) + y0.x, bf_hi(hv.x) + y0.y);
                o.y = pack2(bf_lo(hv.y) + y0.z, bf_hi(hv.y) + y0.w);
                o.z = pack2(bf_lo(hv.z) + y1.x, bf_hi(hv.z) + y1.y);
                o.w = pack2(bf_lo(hv.w) + y1.z, bf_hi(hv.w) + y1.w);
                *reinterpret_cast<uint4 *>(a.x_out + (size_t)idx * 8) = o;
                const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
                *reinterpret_cast<float4 *>(ysum + (size_t)idx * 8) = z;
                *reinterpret_cast<float4 *>(ysum + (size_t)idx * 8 + 4) = z;
                *reinterpret_cast<float4 *>(hs + (size_t)idx * 8) = z;
                *reinterpret_cast<float4 *>(hs + (size_t)idx * 8 + 4) = z;
            }
            sign_off();
            return;
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
                embed_row(a.tok);
            }
        }
        if (step + 1 < a.n_steps && !sync_phase()) return;
    }
    sign_off();
}

}  // namespace

template <int IPW, int DH, int BC, bool LAYER>
static int launch_step_inst(Ctx *c, const StepArgs &a, cudaStream_t st)
{
    const MegaLayout lay = mega_layout<DH>(a.D);
    auto kernel = decode_step_kernel<IPW, DH, BC, LAYER>;
    // the dynamic shared memory this instantiation has been allowed so far, per device (its static arrays
    // come on top: the opt-in is for what the model shape needs, not for the maximum)
    static size_t configured[16] = {};
    if (configured[c->cfg.device & 15] < lay.total) {
        FT_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lay.total));
        int per_sm = 0;
        FT_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, (lay.nw + 1) * 32, lay.total));
        if (per_sm < 1) return FASTTPS_INVALID_ARG;
        configured[c->cfg.device & 15] = lay.total;
    }
    if ((unsigned long long)(3 * a.n_layers + 3) * (unsigned long long)a.n_steps * (unsigned long long)c->n_sm >= kBarAbort)
        return FASTTPS_INVALID_ARG;                      // the arrival counter must stay below the abort mark
    // the barrier counter and the group counters are zero here: the workspace starts out cleared, every launch that
    // runs to its end clears them on its way out, and fasttps_get_status clears them after an abandoned one
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(c->n_sm); cfg.blockDim = dim3((lay.nw + 1) * 32); cfg.dynamicSmemBytes = lay.total; cfg.stream = st;
    // (launching it as a programmatic dependent of its predecessor as well, so that the producer warps stream the
    // first weights while the predecessor's last CTAs finish, was measured on the one-layer workloads: no change)
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


}  // namespace fasttps
