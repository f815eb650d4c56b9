// Fused decode attention (Algorithm 3 of the paper, "GKVC & TPSFLAT"): joint RoPE of the
// new q and k, in-place append of the k/v rows at the address of Eq. 2, QK^T, softmax and
// PV over the cache in one kernel.
//
// Work split.  The paper keeps one head's whole stream in one NPU core.  Here all rows that
// have to be read -- for every sequence b and query head h the L_b cached rows plus the new
// row -- form one flattened row space that is cut into equal contiguous shares, one per CTA
// (one CTA per SM).  A share is a few "segments" (b, h, row range); every CTA streams the same
// number of bytes whatever the batch size or the mix of lengths.  A head that spans several
// CTAs is finished by whichever of them arrives last (an arrival ticket, no waiting) from the
// partial (max, sum, output) triples.
//
// Data movement.  The rows of one head are contiguous in the [B, H, max_seq, d] cache, so a
// tile of 64 rows of K (or V) is ONE contiguous block.  A producer warp fetches tile after tile
// with bulk asynchronous copies (cp.async.bulk, the 1-D TMA path) into a ring of shared-memory
// slots guarded by full/empty mbarriers, up to 8 tiles (K and V) ahead of the consumer warps and
// across segment boundaries.  The new row never makes a round trip through global memory: it is
// scored from shared memory and written to the cache exactly once.
#include "async_copy.cuh"

namespace fasttps {

namespace {

constexpr int kAttnTileRows = 64;                       // rows per ring slot (K tile + V tile)
constexpr int kAttnWarps = 8;                           // consumer warps: one 8-row group each per tile
constexpr int kAttnThreads = (kAttnWarps + 1) * 32;     // + the producer warp
constexpr int kLanesPerRow = 4;

// One contiguous piece of a CTA's share: rows [r0, r1) of head h of sequence b, where row index
// L (= the sequence's cached length) stands for the new row.
struct Segment {
    int b, h, L, pos, r0, r1;
    int first_cta, n_cta;        // CTAs that share this head, and the first of them
};

// Walks the segments of CTA `cta` of `ncta`.  Consumers and the producer run the same walk.
struct ShareWalk {
    const int32_t *seq_lens, *pos;
    int B, H, max_seq, ncta;
    long long T, f, f_end;       // total rows, cursor, end of this CTA's share
    int b, h;
    long long head0;             // flattened index of row 0 of head (b, h)
    int rows_b;                  // rows per head of sequence b (L_b + 1, or 0 if the sequence is skipped)

    __device__ __forceinline__ int rows_of(int bb) const
    {
        const int L = seq_lens[bb], p = pos[bb];
        return (L < 0 || L >= max_seq || p < 0 || p >= max_seq) ? 0 : L + 1;
    }
    __device__ __forceinline__ long long share_begin(int c) const { return (T * c) / ncta; }
    // the CTA whose share holds flattened row x
    __device__ __forceinline__ int owner_of(long long x) const
    {
        int c = (int)((x * ncta) / T);
        while (c + 1 < ncta && share_begin(c + 1) <= x) ++c;
        while (c > 0 && share_begin(c) > x) --c;
        return c;
    }
    __device__ __forceinline__ void init(const int32_t *sl, const int32_t *ps, int B_, int H_, int max_seq_, int cta, int ncta_)
    {
        seq_lens = sl; pos = ps; B = B_; H = H_; max_seq = max_seq_;
        T = 0;
        for (int bb = 0; bb < B; ++bb) T += (long long)H * rows_of(bb);
        // only as many CTAs take part as can get at least 16 rows each: every share is then
        // non-empty, so the CTAs that share a head are exactly first_cta .. first_cta + n_cta - 1
        const long long want = T / 16;
        ncta = want < 1 ? 1 : (want < ncta_ ? (int)want : ncta_);
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
    __device__ __forceinline__ bool next(Segment &s)
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
            s.b = b; s.h = h; s.L = rows_b - 1; s.pos = pos[b];
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

template <int DH>
struct AttnSmem {
    static constexpr int kRowBytes = DH * 2;
    static constexpr int kSlotBytes = 2 * kAttnTileRows * kRowBytes;       // K tile then V tile
    static constexpr int kSlots = (192 * 1024 / kSlotBytes) < 8 ? (192 * 1024 / kSlotBytes) : 8;
    alignas(128) unsigned char slots[kSlots][kSlotBytes];
    alignas(16) uint64_t bars[2 * kSlots];
    alignas(16) float q[DH];                 // rope(q), FP32
    alignas(16) __nv_bfloat16 knew[DH];      // bf16(rope(k_new)): the row that goes into the cache
    alignas(16) __nv_bfloat16 vnew[DH];
    float wm[kAttnWarps], wl[kAttnWarps];    // per-warp softmax state (log2 domain max, sum)
    float mf[kMaxSplits];                    // merge factors of the partials of a shared head
    alignas(16) float wo[kAttnWarps][DH];
    int last;
    int abort;
};

template <int DH>
__global__ void __launch_bounds__(kAttnThreads, 1) attn_decode_kernel(AttnArgs a)
{
    constexpr int EPL = DH / kLanesPerRow;      // elements per lane of a row
    constexpr int VPL = EPL / 8;                // 16-byte vectors per lane
    constexpr int HALF = DH / 2;
    constexpr int NCT = kAttnWarps * 32;        // consumer threads
    using Smem = AttnSmem<DH>;
    constexpr int kAttnSlots = Smem::kSlots;
    extern __shared__ unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int G = a.n_q_heads / a.n_kv_heads;

    uint64_t *full = sm.bars, *empty = sm.bars + kAttnSlots;
    if (t == 0) {
        for (int s = 0; s < kAttnSlots; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kAttnWarps); }
        sm.abort = 0;
        mbar_fence_init();
    }
    __syncthreads();

    // The share of this CTA depends on seq_lens, which the previous kernel in the stream may have
    // written (a model step advances them at its very end): nothing is read before it has finished.
    pdl_wait();
    pdl_launch_dependents();

    ShareWalk walk;
    walk.init(a.seq_lens, a.pos, a.batch, a.n_q_heads, a.max_seq, blockIdx.x, gridDim.x);
    Segment sg;

    // ------------------------------------------------------------------ producer warp
    if (warp == kAttnWarps) {
        if (lane != 0) return;
        int piece = 0;
        while (walk.next(sg)) {
            const int c1 = sg.r1 < sg.L ? sg.r1 : sg.L;              // cached rows of the segment: [r0, c1)
            const size_t slab = ((size_t)sg.b * a.n_kv_heads + sg.h / G) * (size_t)a.max_seq * DH;
            for (int r = sg.r0; r < c1; r += kAttnTileRows, ++piece) {
                const int s = piece % kAttnSlots;
                if (piece >= kAttnSlots &&
                    !mbar_wait_bounded(&empty[s], (uint32_t)(piece / kAttnSlots - 1) & 1u, &sm.abort)) {
                    sm.abort = 1;
                    return;
                }
                const int rows = (c1 - r) < kAttnTileRows ? (c1 - r) : kAttnTileRows;
                const uint32_t bytes = (uint32_t)rows * Smem::kRowBytes;
                mbar_expect_tx(&full[s], 2 * bytes);
                bulk_g2s(sm.slots[s], a.k_cache + slab + (size_t)r * DH, bytes, &full[s]);
                bulk_g2s(sm.slots[s] + kAttnTileRows * Smem::kRowBytes, a.v_cache + slab + (size_t)r * DH, bytes, &full[s]);
            }
        }
        return;
    }

    // ------------------------------------------------------------------ consumer warps
    if (blockIdx.x == 0 && t == 0) {
        // sequences that cannot be served are reported once and contribute no rows
        for (int bb = 0; bb < a.batch; ++bb) {
            const int L = a.seq_lens[bb], p = a.pos[bb];
            if (L < 0 || L >= a.max_seq) atomicOr(a.status, FASTTPS_DEV_CACHE_FULL);
            else if (p < 0 || p >= a.max_seq) atomicOr(a.status, FASTTPS_DEV_BAD_POSITION);
        }
    }
    const int sub = lane & (kLanesPerRow - 1);       // which quarter of the row
    const int rgrp = lane >> 2;                      // row within the warp's 8-row group
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
    int piece = 0;
    bool ok = true;

    while (walk.next(sg)) {
        const int hq = sg.h, hk = hq / G, b = sg.b, L = sg.L;
        const bool has_new = sg.r1 > L;
        const int c1 = has_new ? L : sg.r1;
        const size_t slab = ((size_t)b * a.n_kv_heads + hk) * (size_t)a.max_seq * DH;

        // ---- joint RoPE of q and k_new with one set of cos/sin (Algorithm 3, steps 6-8) ----
        if (t < HALF) {
            const float c = a.cos_tab[(size_t)sg.pos * HALF + t], s = a.sin_tab[(size_t)sg.pos * HALF + t];
            const __nv_bfloat16 *qg = a.q + (size_t)b * a.q_stride + (size_t)hq * DH;
            const float x0 = __bfloat162float(qg[t]), x1 = __bfloat162float(qg[t + HALF]);
            sm.q[t] = __fsub_rn(__fmul_rn(x0, c), __fmul_rn(x1, s));
            sm.q[t + HALF] = __fadd_rn(__fmul_rn(x1, c), __fmul_rn(x0, s));
            if (has_new) {
                const __nv_bfloat16 *kg = a.k_new + (size_t)b * a.kv_stride + (size_t)hk * DH;
                const float k0 = __bfloat162float(kg[t]), k1 = __bfloat162float(kg[t + HALF]);
                sm.knew[t] = __float2bfloat16_rn(__fsub_rn(__fmul_rn(k0, c), __fmul_rn(k1, s)));
                sm.knew[t + HALF] = __float2bfloat16_rn(__fadd_rn(__fmul_rn(k1, c), __fmul_rn(k0, s)));
            }
        } else if (has_new && t >= 64 && t < 64 + DH / 8) {
            const uint4 *vg = reinterpret_cast<const uint4 *>(a.v_new + (size_t)b * a.kv_stride + (size_t)hk * DH);
            reinterpret_cast<uint4 *>(sm.vnew)[t - 64] = vg[t - 64];
        }
        named_bar_sync(1, NCT);
        // ---- GKVC append (Eq. 2; Algorithm 3 steps 1 and 9): one write per row, no reload ----
        if (has_new && (hq % G) == 0 && t < DH / 8) {
            reinterpret_cast<uint4 *>(a.k_cache + slab + (size_t)L * DH)[t] = reinterpret_cast<const uint4 *>(sm.knew)[t];
            reinterpret_cast<uint4 *>(a.v_cache + slab + (size_t)L * DH)[t] = reinterpret_cast<const uint4 *>(sm.vnew)[t];
        }

        float qr[EPL];
#pragma unroll
        for (int i = 0; i < EPL; ++i) qr[i] = sm.q[sub * EPL + i];
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
            const float corr = fast_exp2(m_run - m_new); // 0 when m_run = -inf
            l_run *= corr;
#pragma unroll
            for (int i = 0; i < EPL; ++i) acc[i] *= corr;
            m_run = m_new;
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
            const int s = piece % kAttnSlots;
            bool mine = ok;
            if (mine) mine = mbar_wait_bounded(&full[s], (uint32_t)(piece / kAttnSlots) & 1u, &sm.abort);
            mine = __all_sync(kFull, mine);
            if (!mine && ok) sm.abort = 1;
            ok = mine;
            const int rows = (c1 - r) < kAttnTileRows ? (c1 - r) : kAttnTileRows;
            const int row = warp * 8 + rgrp;
            const bool valid = ok && row < rows;
            const unsigned char *krow = sm.slots[s] + row * Smem::kRowBytes;
            const float sc = dot_row(krow);                    // all lanes: shuffles inside
            update(sc, valid, krow + kAttnTileRows * Smem::kRowBytes);
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }

        // ---- the new row, straight from shared memory (never re-read from the cache) ----
        if (has_new && warp == 0) {
            const float sc = dot_row(reinterpret_cast<const unsigned char *>(sm.knew));
            update(sc, rgrp == 0, reinterpret_cast<const unsigned char *>(sm.vnew));
        }

        // ---- combine the row groups of a warp, then the warps of the CTA ----
#pragma unroll
        for (int s = 4; s <= 16; s <<= 1) {
            l_run += __shfl_xor_sync(kFull, l_run, s);
#pragma unroll
            for (int i = 0; i < EPL; ++i) acc[i] += __shfl_xor_sync(kFull, acc[i], s);
        }
        l_run = __shfl_sync(kFull, l_run, 0);          // the sum was kept by the sub == 0 lanes
        if (lane < kLanesPerRow) {
#pragma unroll
            for (int i = 0; i < EPL; ++i) sm.wo[warp][sub * EPL + i] = acc[i];
            if (lane == 0) { sm.wm[warp] = m_run; sm.wl[warp] = l_run; }
        }
        if (!named_bar_and(1, NCT, ok)) {
            if (t == 0) atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT);
            return;
        }
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, sm.wm[w]);
        float o = 0.f, l = 0.f;
        if (t < DH) {
#pragma unroll
            for (int w = 0; w < kAttnWarps; ++w) {
                const float f = (sm.wm[w] == -INFINITY) ? 0.f : fast_exp2(sm.wm[w] - M);
                o += f * sm.wo[w][t];
                l += f * sm.wl[w];
            }
        }
        __nv_bfloat16 *outp = a.out + (size_t)b * a.out_stride + (size_t)hq * DH;
        if (sg.n_cta == 1) {
            if (t < DH) outp[t] = __float2bfloat16_rn(o / l);
        } else {
            // ---- several CTAs share the head: publish the partial, the last one merges ----
            float *hp = a.part + ((size_t)b * a.n_q_heads + hq) * kMaxSplits * (DH + 2);
            float *part = hp + (size_t)(blockIdx.x - sg.first_cta) * (DH + 2);
            if (t < DH) part[2 + t] = o;
            if (t == 0) { part[0] = M; part[1] = l; }
            __threadfence();
            named_bar_sync(1, NCT);
            int *ticket = a.ticket + (size_t)b * a.n_q_heads + hq;
            if (t == 0) sm.last = (atomicAdd(ticket, 1) == sg.n_cta - 1);
            named_bar_sync(1, NCT);
            if (sm.last) {
                __threadfence();
                // all loads of the merge are issued side by side: one lane per partial for (max, sum) ...
                if (warp == 0) {
                    const bool have = lane < sg.n_cta;
                    const float ms = have ? ld_cg_f32(hp + (size_t)lane * (DH + 2)) : -INFINITY;
                    const float ls = have ? ld_cg_f32(hp + (size_t)lane * (DH + 2) + 1) : 0.f;
                    float MM = ms;
#pragma unroll
                    for (int s = 16; s >= 1; s >>= 1) MM = fmaxf(MM, __shfl_xor_sync(kFull, MM, s));
                    const float f = (ms == -INFINITY) ? 0.f : fast_exp2(ms - MM);
                    sm.mf[lane] = f;
                    const float ll = warp_sum(f * ls);
                    if (lane == 0) sm.wl[0] = ll;
                }
                named_bar_sync(2, NCT);
                // ... and one thread per output element, eight partials in flight at a time
                if (t < DH) {
                    float oo = 0.f;
                    for (int s0 = 0; s0 < sg.n_cta; s0 += 8) {
                        float v[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            v[u] = (s0 + u < sg.n_cta) ? ld_cg_f32(hp + (size_t)(s0 + u) * (DH + 2) + 2 + t) : 0.f;
#pragma unroll
                        for (int u = 0; u < 8; ++u) oo = fmaf(sm.mf[(s0 + u) & (kMaxSplits - 1)], v[u], oo);
                    }
                    outp[t] = __float2bfloat16_rn(oo / sm.wl[0]);
                }
                if (t == 0) *ticket = 0;
            }
        }
        named_bar_sync(1, NCT);                          // shared scratch is reused by the next segment
    }
}

}  // namespace

// Number of CTAs the attention kernel uses for this batch (one per SM, fewer for tiny problems so that
// no head is shared by more than kMaxSplits CTAs).
int attn_splits_for(const Ctx *c, int batch)
{
    int n = c->n_sm;
    (void)batch;
    const int cap = (kMaxSplits - 2) * c->cfg.n_q_heads;
    if (n > cap) n = cap;
    return n < 1 ? 1 : n;
}

template <int DH>
static int launch_attn_dh(Ctx *c, const AttnArgs &a, cudaStream_t st)
{
    const size_t smem = sizeof(AttnSmem<DH>) + 128;
    dim3 grid(a.n_splits);
    ProfScope prof(c, kProfAttn, st);
    const int rc = launch_ex(attn_decode_kernel<DH>, grid, dim3(kAttnThreads), smem, st, &a);
    c->launches++;
    return rc;
}

int configure_attn_kernels()
{
    FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttnSmem<32>) + 128));
    FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttnSmem<64>) + 128));
    FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<96>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttnSmem<96>) + 128));
    FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttnSmem<128>) + 128));
    return FASTTPS_OK;
}

int launch_attn(Ctx *c, const AttnArgs &a, cudaStream_t st)
{
    switch (a.head_dim) {
    case 32: return launch_attn_dh<32>(c, a, st);
    case 64: return launch_attn_dh<64>(c, a, st);
    case 96: return launch_attn_dh<96>(c, a, st);
    case 128: return launch_attn_dh<128>(c, a, st);
    default: return FASTTPS_INVALID_ARG;
    }
}

}  // namespace fasttps
