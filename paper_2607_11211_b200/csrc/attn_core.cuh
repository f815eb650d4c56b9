// Device-side core of the fused decode attention (Algorithm 3 of the paper, "GKVC & TPSFLAT"):
// joint RoPE of the new q and k, in-place append of the k/v rows at the address of Eq. 2, QK^T,
// softmax and PV over the cache.  Used by the stand-alone attention kernel and by the persistent
// decode-step kernel.
//
// Work split.  The paper keeps one head's whole stream in one NPU core.  Here all rows that
// have to be read -- for every sequence b and query head h the L_b cached rows plus the new
// row -- form one flattened row space that is cut into equal contiguous shares, one per CTA.
// A share is a few "segments" (b, h, row range); every CTA streams the same number of bytes
// whatever the batch size or the mix of lengths.  A head that spans several CTAs is finished by
// whichever of them arrives last (an arrival ticket, no waiting) from the partial
// (max, sum, output) triples.
//
// Data movement.  The rows of one head are contiguous in the [B, H, max_seq, d] cache, so a
// tile of 64 rows of K (or V) is ONE contiguous block.  The producer thread fetches tile after
// tile with bulk asynchronous copies into the shared-memory ring (K tile, then V tile, in one
// slot), ahead of the consumer warps and across segment boundaries.  The new row never makes a
// round trip through global memory: it is scored from shared memory and written to the cache
// exactly once.
//
// Grouped-query attention (Section 4.1: several query heads read one K/V head): here a segment is one
// query head, and a group's rows are streamed once per query head.  attn_group_core.cuh holds the
// variant that streams a K/V head once for its whole group.
#pragma once
#include "async_copy.cuh"

namespace fasttps {

constexpr int kAttnTileRows = 64;        // rows per ring piece (K tile + V tile)
constexpr int kAttnMaxWorkers = 8;       // warps that score rows: one 8-row group each per tile
constexpr int kLanesPerRow = 4;

// One contiguous piece of a CTA's share: rows [r0, r1) of head h of sequence b, where row index
// L (= the sequence's cached length) stands for the new row.
struct Segment {
    int b, h, L, pos, r0, r1;
    int first_cta, n_cta;        // CTAs that share this head, and the first of them
};

// Walks the segments of CTA `cta` of `ncta`.  Consumers and the producer run the same walk.
// `add` is added to every length and position (the step index inside a multi-step launch).
struct ShareWalk {
    const int32_t *seq_lens, *pos;
    int B, H, max_seq, ncta, add;
    int N = 1;                   // new tokens per sequence: row bb of the walk is token bb % N of sequence bb / N
    int need = 1;                // new rows per sequence that must fit into its cache (N, or the chunk length when the
                                 // walk runs over sequences and the chunk's tokens share the pass)
    long long T, f, f_end;       // total rows, cursor, end of this CTA's share
    int b, h;
    long long head0;             // flattened index of row 0 of head (b, h)
    int rows_b;                  // rows per head of sequence b (L_b + 1, or 0 if the sequence is skipped)

    // rows of one head of walk row bb: the cached rows plus ONE for the new rows (with N new tokens per sequence
    // the last "row" of token j stands for the new rows 0 .. j, which never come from the cache)
    __host__ __device__ __forceinline__ int rows_of(int bb) const
    {
        const int L = seq_lens[bb / N] + add, p = pos[bb / N] + add;
        return (L < add || L + need > max_seq || p < add || p + need > max_seq) ? 0 : L + 1;
    }
    __host__ __device__ __forceinline__ long long share_begin(int c) const { return (T * c) / ncta; }
    // the CTA whose share holds flattened row x
    __host__ __device__ __forceinline__ int owner_of(long long x) const
    {
        int c = (int)((x * ncta) / T);
        while (c + 1 < ncta && share_begin(c + 1) <= x) ++c;
        while (c > 0 && share_begin(c) > x) --c;
        return c;
    }
    __host__ __device__ __forceinline__ void init(const int32_t *sl, const int32_t *ps, int add_, int B_, int H_, int max_seq_,
                                         int cta, int ncta_)
    {
        seq_lens = sl; pos = ps; add = add_; B = B_; H = H_; max_seq = max_seq_;
        T = 0;
        int live = 0, rows0 = 0, rmax = 0;
        bool uniform = true;
        for (int bb = 0; bb < B; ++bb) {
            const int r = rows_of(bb);
            T += (long long)H * r;
            rmax = r > rmax ? r : rmax;
            if (r > 0) {
                if (live == 0) rows0 = r;
                else if (r != rows0) uniform = false;
                ++live;
            }
        }
        // only as many CTAs take part as can get at least 16 rows each: every share is then
        // non-empty, so the CTAs that share a head are exactly first_cta .. first_cta + n_cta - 1
        const long long want = T / 16;
        ncta = want < 1 ? 1 : (want < ncta_ ? (int)want : ncta_);
        // a head has kMaxSplits partial records: a share is at least 1 / (kMaxSplits - 3) of the longest head (less
        // up to a sixteenth for the rounding of the cuts, shares being at least 16 rows), so that no head spans
        // more than kMaxSplits shares (whole shares plus a cut one at either end)
        if (rmax > 0) {
            const long long cap = (long long)(kMaxSplits - 3) * T / rmax;
            if (ncta > cap) ncta = cap < 1 ? 1 : (int)cap;
        }
        // equal lengths and no more heads than CTAs: a whole number of CTAs per head, so that every share
        // is ONE segment and every head has the same, small number of partials
        if (uniform && live > 0 && live * H <= ncta) ncta = live * H * (ncta / (live * H));
        const bool in = T > 0 && cta < ncta;
        f = in ? share_begin(cta) : 0;
        f_end = in ? share_begin(cta + 1) : 0;
        // locate the head that holds f
        b = 0; head0 = 0; rows_b = B > 0 ? rows_of(0) : 0;
        while (b < B && head0 + (long long)H * rows_b <= f) {
            head0 += (long long)H * rows_b;
            ++b;
            rows_b = b < B ? rows_of(b) : 0;
        }
        h = 0;
        if (b < B && rows_b > 0) {
            h = (int)((f - head0) / rows_b);
            head0 += (long long)h * rows_b;
        }
    }
    __host__ __device__ __forceinline__ bool next(Segment &s)
    {
        while (f < f_end) {
            if (rows_b == 0 || h >= H) {          // step to the next sequence
                ++b; h = 0;
                if (b >= B) return false;
                rows_b = rows_of(b);
                continue;
            }
            const long long head1 = head0 + rows_b;
            const long long e = head1 < f_end ? head1 : f_end;
            s.b = b; s.h = h; s.L = rows_b - 1; s.pos = pos[b / N] + add + b % N;
            s.r0 = (int)(f - head0); s.r1 = (int)(e - head0);
            s.first_cta = owner_of(head0);
            s.n_cta = owner_of(head1 - 1) - s.first_cta + 1;
            f = e;
            if (e == head1) { head0 = head1; ++h; }
            return true;
        }
        return false;
    }
};

// where element `col` of the attention output of sequence (token row) b goes
__device__ __forceinline__ __nv_bfloat16 *attn_out_at(const AttnArgs &a, int b, int col)
{
    return a.out + (a.out_chunked ? wide_x_index(b, col) : (size_t)b * a.out_stride + col);
}

template <int DH>
struct AttnScratch {
    alignas(16) float q[DH];                 // rope(q), FP32
    alignas(16) __nv_bfloat16 knew[DH];      // bf16(rope(k_new)): the row that goes into the cache
    alignas(16) __nv_bfloat16 vnew[DH];
    float wm[kAttnMaxWorkers], wl[kAttnMaxWorkers];   // per-warp softmax state (log2 domain max, sum)
    float mf[kMaxSplits];                    // merge factors of the partials of a shared head
    alignas(16) float wo[kAttnMaxWorkers][DH];
    int last;
};

// PRE (attn_consume): rope(q), bf16(rope(k_new)) and v_new of ALL segments of a share, prepared in one pass
template <int DH>
struct AttnPre {
    alignas(16) float q[kMaxNB][DH];
    alignas(16) __nv_bfloat16 knew[kMaxNB][DH];
    alignas(16) __nv_bfloat16 vnew[kMaxNB][DH];
};

// MULTI (attn_consume): the rotated K rows and the V rows of the new tokens 0 .. j of the sequence a segment belongs to
template <int DH>
struct AttnMulti {
    alignas(16) __nv_bfloat16 knew[kMaxNB][DH];
    alignas(16) __nv_bfloat16 vnew[kMaxNB][DH];
};

template <int DH> struct AttnTile {
    static constexpr int kRowBytes = DH * 2;
    static constexpr int kPieceBytes = 2 * kAttnTileRows * kRowBytes;     // K tile then V tile
};

// Segment sources: `bool next(Segment &)`.
struct WalkSource {
    ShareWalk walk;
    // share: the flattened row space runs over the K/V heads (segment.h is then a K/V head) of the SEQUENCES: the new
    // tokens of a sequence and the query heads of a K/V head all share one pass
    __device__ __forceinline__ WalkSource(const AttnArgs &a, int cta, int ncta, bool share = false)
    {
        walk.N = share ? 1 : a.n_new;
        walk.need = a.n_new;
        walk.init(a.seq_lens, a.pos, a.len_add, share ? a.batch / a.n_new : a.batch, share ? a.n_kv_heads : a.n_q_heads,
                  a.max_seq, cta, ncta);
    }
    __device__ __forceinline__ bool next(Segment &s) { return walk.next(s); }
};
// Calls f(k_tile, v_tile, bytes_each) for every K/V tile of this CTA's share, in walk order; stops and
// returns false as soon as f does.  EB: bytes per cache element (2: bf16, 1: E4M3 codes); TR: rows per tile.
template <int DH, bool SHARE = false, int EB = 2, int TR = kAttnTileRows, class Src, class F>
__device__ __forceinline__ bool attn_for_each_tile(const AttnArgs &a, Src src, F f)
{
    const int G = SHARE ? 1 : a.n_q_heads / a.n_kv_heads;
    const unsigned char *kc = reinterpret_cast<const unsigned char *>(a.k_cache), *vc = reinterpret_cast<const unsigned char *>(a.v_cache);
    Segment sg;
    while (src.next(sg)) {
        const int c1 = sg.r1 < sg.L ? sg.r1 : sg.L;              // cached rows of the segment: [r0, c1)
        const size_t slab = ((size_t)(SHARE ? sg.b : sg.b / a.n_new) * a.n_kv_heads + sg.h / G) * (size_t)a.max_seq * DH;
        for (int r = sg.r0; r < c1; r += TR) {
            const int rows = (c1 - r) < TR ? (c1 - r) : TR;
            if (!f(kc + (slab + (size_t)r * DH) * EB, vc + (slab + (size_t)r * DH) * EB, (uint32_t)rows * DH * EB))
                return false;
        }
    }
    return true;
}

// Producer thread: issues the K/V tiles of this CTA's share, in walk order, as ring pieces starting at `piece`.
template <int DH, bool SHARE = false, int EB = 2, int TR = kAttnTileRows>
__device__ __forceinline__ bool attn_produce(const AttnArgs &a, WeightRing &ring, int &piece, int cta, int ncta)
{
    const bool done = attn_for_each_tile<DH, SHARE, EB, TR>(a, WalkSource(a, cta, ncta, SHARE), [&](const unsigned char *k, const unsigned char *v, uint32_t bytes) {
        if (!ring.put2(piece, k, v, bytes, TR * DH * EB)) return false;
        ++piece;
        return true;
    });
    if (!done) ring.drain(piece);      // the copies in flight get a bounded chance to land before the CTA leaves
    return done;
}

// Consumer warps (nwc of them, threads 0 .. 32 nwc - 1, synchronised by named barrier 1): the attention
// of this CTA's share.  The first min(nwc, 8) warps score rows; the others only keep the ring protocol.
// Returns false (in every consumer thread alike) if a bounded wait ran out.
// DEFER: the partial of every segment is published (even when the CTA owns the whole head) and nobody
// merges here; the caller merges the partials of a head itself (the persistent step kernel does, per group).
// MULTI: several new tokens per sequence (a.n_new <= 8): the segment of token j scores the cached rows and then the
// new rows 0 .. j of its sequence from shared memory (causal inside the chunk), and appends row j.
template <int DH, bool DEFER, class Src, bool LATE_FENCE = false, bool PRE = false, bool MULTI = false>
__device__ __forceinline__ bool attn_consume(const AttnArgs &a, WeightRing &ring, int &piece, int cta, Src src,
                                             AttnScratch<DH> &sm, int nwc, AttnPre<DH> *pre = nullptr,
                                             AttnMulti<DH> *mt = nullptr)
{
    static_assert(!(MULTI && PRE), "the multi-token path prepares its rows per segment");
    constexpr int EPL = DH / kLanesPerRow;      // elements per lane of a row
    constexpr int VPL = EPL / 8;                // 16-byte vectors per lane
    constexpr int HALF = DH / 2;
    constexpr int kRowBytes = AttnTile<DH>::kRowBytes;
    constexpr int kPartStride = DH + 4;         // partial = o[DH], max, sum, pad (16-byte aligned records)
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int nct = nwc * 32;
    const int nwork = nwc < kAttnMaxWorkers ? nwc : kAttnMaxWorkers;
    const bool worker = warp < nwork;
    const int G = a.n_q_heads / a.n_kv_heads;
    const int sub = lane & (kLanesPerRow - 1);       // which quarter of the row
    const int rgrp = lane >> 2;                      // row within an 8-row group
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
    bool ok = true;
    bool appended = false;

    // element i (and i + HALF) of the rotated q of segment s, and of its new K/V row when the segment holds it
    auto rope_one = [&](const Segment &s, int i, float *qv, __nv_bfloat16 *knew, __nv_bfloat16 *vnew) {
        const int hq = s.h, hk = hq / G, b = s.b;
        const float c = a.cos_tab[(size_t)s.pos * HALF + i], sn = a.sin_tab[(size_t)s.pos * HALF + i];
        const __nv_bfloat16 *qg = a.q + (size_t)b * a.q_stride + (size_t)hq * DH;
        const float x0 = __bfloat162float(ld_cg_bf16(qg + i)), x1 = __bfloat162float(ld_cg_bf16(qg + i + HALF));
        qv[i] = __fsub_rn(__fmul_rn(x0, c), __fmul_rn(x1, sn));
        qv[i + HALF] = __fadd_rn(__fmul_rn(x1, c), __fmul_rn(x0, sn));
        if (s.r1 > s.L) {
            const __nv_bfloat16 *kg = a.k_new + (size_t)b * a.kv_stride + (size_t)hk * DH;
            const float k0 = __bfloat162float(ld_cg_bf16(kg + i)), k1 = __bfloat162float(ld_cg_bf16(kg + i + HALF));
            knew[i] = __float2bfloat16_rn(__fsub_rn(__fmul_rn(k0, c), __fmul_rn(k1, sn)));
            knew[i + HALF] = __float2bfloat16_rn(__fadd_rn(__fmul_rn(k1, c), __fmul_rn(k0, sn)));
            const __nv_bfloat16 *vg = a.v_new + (size_t)b * a.kv_stride + (size_t)hk * DH;
            vnew[i] = ld_cg_bf16(vg + i);
            vnew[i + HALF] = ld_cg_bf16(vg + i + HALF);
        }
    };
    if constexpr (PRE) {
        // every (segment, element) pair of the share has a thread of its own: the loads of all segments go out
        // together and cost one round trip to the L2, not one per segment
        const int nseg = src.count();
        for (int idx = t; idx < nseg * HALF; idx += nct) {
            const int n = idx / HALF;
            rope_one(src.at(n), idx - n * HALF, pre->q[n], pre->knew[n], pre->vnew[n]);
        }
        named_bar_sync(1, nct);
    }

    Segment sg;
    int segi = 0;
    for (; src.next(sg); ++segi) {
        const int hq = sg.h, hk = hq / G, b = sg.b, L = sg.L;
        const bool has_new = sg.r1 > L;
        const int c1 = has_new ? L : sg.r1;
        const int tok = MULTI ? b % a.n_new : 0;                  // this token's index among its sequence's new tokens
        const size_t slab = ((size_t)(MULTI ? b / a.n_new : b) * a.n_kv_heads + hk) * (size_t)a.max_seq * DH;

        // ---- joint RoPE of q and k_new with one set of cos/sin (Algorithm 3, steps 6-8) ----
        float *qv = PRE ? pre->q[segi] : sm.q;
        __nv_bfloat16 *knew = PRE ? pre->knew[segi] : sm.knew, *vnew = PRE ? pre->vnew[segi] : sm.vnew;
        if constexpr (MULTI) {
            // q of this token at its own position; K / V rows of the new tokens 0 .. tok at theirs
            const int n_rows = has_new ? tok + 1 : 0;
            for (int idx = t; idx < (1 + n_rows) * HALF; idx += nct) {
                const int which = idx / HALF, i = idx - which * HALF;
                if (which == 0) {
                    const float c = a.cos_tab[(size_t)sg.pos * HALF + i], sn = a.sin_tab[(size_t)sg.pos * HALF + i];
                    const __nv_bfloat16 *qg = a.q + (size_t)b * a.q_stride + (size_t)hq * DH;
                    const float x0 = __bfloat162float(ld_cg_bf16(qg + i)), x1 = __bfloat162float(ld_cg_bf16(qg + i + HALF));
                    qv[i] = __fsub_rn(__fmul_rn(x0, c), __fmul_rn(x1, sn));
                    qv[i + HALF] = __fadd_rn(__fmul_rn(x1, c), __fmul_rn(x0, sn));
                } else {
                    const int r = which - 1, row = b - tok + r, p = sg.pos - tok + r;     // token r of the same sequence
                    const float c = a.cos_tab[(size_t)p * HALF + i], sn = a.sin_tab[(size_t)p * HALF + i];
                    const __nv_bfloat16 *kg = a.k_new + (size_t)row * a.kv_stride + (size_t)hk * DH;
                    const float k0 = __bfloat162float(ld_cg_bf16(kg + i)), k1 = __bfloat162float(ld_cg_bf16(kg + i + HALF));
                    mt->knew[r][i] = __float2bfloat16_rn(__fsub_rn(__fmul_rn(k0, c), __fmul_rn(k1, sn)));
                    mt->knew[r][i + HALF] = __float2bfloat16_rn(__fadd_rn(__fmul_rn(k1, c), __fmul_rn(k0, sn)));
                    const __nv_bfloat16 *vg = a.v_new + (size_t)row * a.kv_stride + (size_t)hk * DH;
                    mt->vnew[r][i] = ld_cg_bf16(vg + i);
                    mt->vnew[r][i + HALF] = ld_cg_bf16(vg + i + HALF);
                }
            }
            named_bar_sync(1, nct);
            knew = mt->knew[tok]; vnew = mt->vnew[tok];          // the row this token appends
        } else if (!PRE) {
            for (int i = t; i < HALF; i += nct) rope_one(sg, i, qv, knew, vnew);
            named_bar_sync(1, nct);
        }
        // ---- GKVC append (Eq. 2; Algorithm 3 steps 1 and 9): one write per row, no reload ----
        if (has_new && (hq % G) == 0) {
            const size_t arow = (size_t)(L + tok) * DH;           // token j of the chunk goes into row L + j
            for (int i = t; i < DH / 8; i += nct) {
                reinterpret_cast<uint4 *>(a.k_cache + slab + arow)[i] = reinterpret_cast<const uint4 *>(knew)[i];
                reinterpret_cast<uint4 *>(a.v_cache + slab + arow)[i] = reinterpret_cast<const uint4 *>(vnew)[i];
            }
            // bulk copies of a later step of the same launch must see these rows: the stores are ordered before the
            // asynchronous proxy, here or (LATE_FENCE) after the last segment
            if (LATE_FENCE) appended = true;
            else asm volatile("fence.proxy.async;" ::: "memory");
        }

        float qr[EPL];
#pragma unroll
        for (int i = 0; i < EPL; ++i) qr[i] = qv[sub * EPL + i];
        float m_run = -INFINITY, l_run = 0.f;
        float acc[EPL];
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] = 0.f;

        auto dot_row = [&](const unsigned char *rowp) -> float {
            float s = 0.f;
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                float f[8];
                unpack8(*reinterpret_cast<const uint4 *>(rowp + (sub * VPL + v) * 16), f);
#pragma unroll
                for (int i = 0; i < 8; ++i) s = fmaf(f[i], qr[v * 8 + i], s);
            }
            s += __shfl_xor_sync(kFull, s, 1);
            s += __shfl_xor_sync(kFull, s, 2);
            return s * scale_log2;
        };
        // online-softmax step with one (possibly invalid) row per lane group
        auto update = [&](float sc, bool valid, const unsigned char *vrow) {
            float mt = valid ? sc : -INFINITY;
            mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 4));
            mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 8));
            mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 16));
            const float m_new = fmaxf(m_run, mt);
            if (m_new == -INFINITY) return;              // nothing valid yet (warp-uniform)
            // the maximum is the same in every lane of the warp and seldom moves after the first tiles
            if (m_new != m_run) {
                const float corr = fast_exp2(m_run - m_new); // 0 when m_run = -inf
                l_run *= corr;
#pragma unroll
                for (int i = 0; i < EPL; ++i) acc[i] *= corr;
                m_run = m_new;
            }
            if (valid) {
                const float pj = fast_exp2(sc - m_new);
                if (sub == 0) l_run += pj;
#pragma unroll
                for (int v = 0; v < VPL; ++v) {
                    float f[8];
                    unpack8(*reinterpret_cast<const uint4 *>(vrow + (sub * VPL + v) * 16), f);
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[v * 8 + i] = fmaf(pj, f[i], acc[v * 8 + i]);
                }
            }
        };

        // ---- stream the cached rows of the segment (Algorithm 3 steps 10-12) ----
        for (int r = sg.r0; r < c1; r += kAttnTileRows, ++piece) {
            // every consumer warp waits for the piece before it releases it, workers or not: a warp that
            // ran ahead would arrive on a slot's "empty" barrier in the wrong phase
            const unsigned char *slot = ring.wait(piece, ok);
            if (worker) {
                const int rows = (c1 - r) < kAttnTileRows ? (c1 - r) : kAttnTileRows;
                for (int rg = warp; rg < kAttnTileRows / 8; rg += nwork) {
                    const int row = rg * 8 + rgrp;
                    const bool valid = ok && row < rows;
                    const unsigned char *krow = slot + row * kRowBytes;
                    const float sc = dot_row(krow);                // all lanes: shuffles inside
                    update(sc, valid, krow + kAttnTileRows * kRowBytes);
                }
            }
            ring.release(piece);
        }

        // ---- the new row, straight from shared memory (never re-read from the cache) ----
        if (has_new && warp == 0) {
            if constexpr (MULTI) {
                // one new row per lane group: rows 0 .. tok of the chunk are visible to this token, the later ones are not
                const int r = rgrp <= tok ? rgrp : 0;
                const float sc = dot_row(reinterpret_cast<const unsigned char *>(mt->knew[r]));
                update(sc, rgrp <= tok, reinterpret_cast<const unsigned char *>(mt->vnew[r]));
            } else {
                const float sc = dot_row(reinterpret_cast<const unsigned char *>(knew));
                update(sc, rgrp == 0, reinterpret_cast<const unsigned char *>(vnew));
            }
        }

        // ---- combine the row groups of a warp, then the warps of the CTA ----
        if (worker) {
            // The eight row groups of a warp hold partial sums of the same EPL elements.  They are added by halving:
            // in each of three rounds a lane keeps one half of what it holds and gets the partner's sums of that
            // half, so the element count per lane goes EPL -> EPL/2 -> EPL/4 -> EPL/8 (7 EPL / 8 shuffles instead of
            // 3 EPL) and every lane ends with EPL / 8 finished elements.
            static_assert(EPL % 8 == 0, "head_dim must be a multiple of 32");
#pragma unroll
            for (int s = 4; s <= 16; s <<= 1) l_run += __shfl_xor_sync(kFull, l_run, s);
            l_run = __shfl_sync(kFull, l_run, 0);          // the sum was kept by the sub == 0 lanes
            int first = 0;                                  // index (within the lane's EPL) of the elements it still holds
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                const int half = EPL >> (r + 1);
                const bool upper = (lane >> (4 - r)) & 1;   // rounds pair lanes 16, 8, 4 apart
#pragma unroll
                for (int i = 0; i < half; ++i) {
                    const float send = upper ? acc[i] : acc[i + half];
                    const float keep = upper ? acc[i + half] : acc[i];
                    acc[i] = keep + __shfl_xor_sync(kFull, send, 16 >> r);
                }
                first += upper ? half : 0;
            }
#pragma unroll
            for (int i = 0; i < EPL / 8; ++i) sm.wo[warp][sub * EPL + first + i] = acc[i];
            if (lane == 0) { sm.wm[warp] = m_run; sm.wl[warp] = l_run; }
        }
        if (!named_bar_and(1, nct, ok)) return false;
        float M = -INFINITY;
        for (int w = 0; w < nwork; ++w) M = fmaxf(M, sm.wm[w]);
        float *hp = a.part + ((size_t)b * a.n_q_heads + hq) * kMaxSplits * kPartStride;
        float *part = hp + (size_t)(cta - sg.first_cta) * kPartStride;
        const bool whole = !DEFER && sg.n_cta == 1;      // this CTA alone finishes the head right here
        for (int i = t; i < DH; i += nct) {
            float o = 0.f, l = 0.f;
            for (int w = 0; w < nwork; ++w) {
                const float f = (sm.wm[w] == -INFINITY) ? 0.f : fast_exp2(sm.wm[w] - M);
                o += f * sm.wo[w][i];
                l += f * sm.wl[w];
            }
            if (whole) *attn_out_at(a, b, hq * DH + i) = __float2bfloat16_rn(o / l);
            else {
                part[i] = o;
                if (i == 0) { part[DH] = M; part[DH + 1] = l; }
            }
        }
        if (!DEFER && sg.n_cta > 1) {
            // ---- several CTAs share the head: the partial is published, the last one merges ----
            __threadfence();
            named_bar_sync(1, nct);
            int *ticket = a.ticket + (size_t)b * a.n_q_heads + hq;
            if (t == 0) sm.last = (atomicAdd(ticket, 1) == sg.n_cta - 1);
            named_bar_sync(1, nct);
            if (sm.last) {
                __threadfence();
                // all loads of the merge are issued side by side: one lane per partial for (max, sum) ...
                if (warp == 0) {
                    const bool have = lane < sg.n_cta;
                    const float ms = have ? ld_cg_f32(hp + (size_t)lane * kPartStride + DH) : -INFINITY;
                    const float ls = have ? ld_cg_f32(hp + (size_t)lane * kPartStride + DH + 1) : 0.f;
                    float MM = ms;
#pragma unroll
                    for (int s = 16; s >= 1; s >>= 1) MM = fmaxf(MM, __shfl_xor_sync(kFull, MM, s));
                    const float f = (ms == -INFINITY) ? 0.f : fast_exp2(ms - MM);
                    sm.mf[lane] = f;
                    const float ll = warp_sum(f * ls);
                    if (lane == 0) sm.wl[0] = ll;
                }
                named_bar_sync(1, nct);
                // ... and one thread per output element, eight partials in flight at a time
                for (int i = t; i < DH; i += nct) {
                    float oo = 0.f;
                    for (int s0 = 0; s0 < sg.n_cta; s0 += 8) {
                        float v[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            v[u] = (s0 + u < sg.n_cta) ? ld_cg_f32(hp + (size_t)(s0 + u) * kPartStride + i) : 0.f;
#pragma unroll
                        for (int u = 0; u < 8; ++u) oo = fmaf(sm.mf[(s0 + u) & (kMaxSplits - 1)], v[u], oo);
                    }
                    *attn_out_at(a, b, hq * DH + i) = __float2bfloat16_rn(oo / sm.wl[0]);
                }
                if (t == 0) *ticket = 0;
            }
        }
        named_bar_sync(1, nct);                          // the scratch is reused by the next segment
    }
    // LATE_FENCE: off the path of the rows that were still to be scored (worth it when a share holds several segments)
    if (LATE_FENCE && appended) asm volatile("fence.proxy.async;" ::: "memory");
    return true;
}

}  // namespace fasttps
