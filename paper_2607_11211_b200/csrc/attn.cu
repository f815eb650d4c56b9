// Fused decode attention (Algorithm 3 of the paper, "GKVC & TPSFLAT"): joint RoPE of the
// new q and k, in-place append of the k/v rows at the address of Eq. 2, QK^T, softmax and
// PV over the cache in one kernel.  The paper keeps one head's whole stream in one NPU core;
// on a B200 the stream of a (sequence, head) pair is cut into n_splits row ranges
// (split-KV), each range is one CTA, and the partial (max, sum, output) triples are merged
// by whichever CTA of the head finishes last (an arrival ticket, no waiting).
//
// Data movement: the rows of one head are contiguous in the [B, H, max_seq, d] cache, so a
// tile of T rows of K (or V) is ONE contiguous block that a single thread fetches with a
// bulk asynchronous copy (cp.async.bulk, the 1-D TMA path) into a ring of shared-memory
// stages guarded by mbarriers.  The new row never makes a round trip through global
// memory: it is scored from registers/shared memory and written to the cache once.
#include "async_copy.cuh"

namespace fasttps {

namespace {

constexpr int kAttnThreads = 128;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kTileRows = 64;          // rows per stage (K tile + V tile)
constexpr int kStages = 3;
constexpr int kLanesPerRow = 4;
constexpr int kRowsPerPass = 32 / kLanesPerRow;                  // 8 rows per warp pass
constexpr int kPasses = kTileRows / (kAttnWarps * kRowsPerPass); // passes per warp per tile
template <int DH>
struct AttnSmem {
    static constexpr int kRowBytes = DH * 2;
    static constexpr int kTileBytes = kTileRows * kRowBytes;
    alignas(128) unsigned char k[kStages][kTileBytes];
    alignas(128) unsigned char v[kStages][kTileBytes];
    alignas(16) uint64_t full[kStages];
    alignas(16) float q[DH];                 // rope(q), FP32
    alignas(16) __nv_bfloat16 knew[DH];      // bf16(rope(k_new)): the row that goes into the cache
    alignas(16) __nv_bfloat16 vnew[DH];
    float wm[kAttnWarps], wl[kAttnWarps];    // per-warp softmax state (log2 domain max, sum)
    alignas(16) float wo[kAttnWarps][DH];
    int last;
    int abort;
};

// Row range of split s for a sequence with L cached rows: [s*rps, min(L, (s+1)*rps)).
__device__ __forceinline__ int rows_per_split(int L, int n_splits)
{
    int rps = (L + n_splits - 1) / n_splits;
    rps = (rps + 15) & ~15;
    return rps < 16 ? 16 : rps;
}

template <int DH>
__global__ void __launch_bounds__(kAttnThreads) attn_decode_kernel(AttnArgs a)
{
    constexpr int EPL = DH / kLanesPerRow;      // elements per lane of a row
    constexpr int VPL = EPL / 8;                // 16-byte vectors per lane
    constexpr int HALF = DH / 2;
    using Smem = AttnSmem<DH>;
    extern __shared__ unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int split = blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
    const int G = a.n_q_heads / a.n_kv_heads;
    const int hk = hq / G;

    const int L = a.seq_lens[b];
    const int p = a.pos[b];
    if (L < 0 || L >= a.max_seq) { if (t == 0) atomicOr(a.status, FASTTPS_DEV_CACHE_FULL); return; }
    if (p < 0 || p >= a.max_seq) { if (t == 0) atomicOr(a.status, FASTTPS_DEV_BAD_POSITION); return; }

    const int rps = rows_per_split(L, a.n_splits);
    int n_act = (L + rps - 1) / rps;             // splits that own cached rows
    if (n_act < 1) n_act = 1;
    if (split >= n_act) return;
    const int r0 = split * rps;
    const int r1 = (r0 + rps < L) ? r0 + rps : L;
    const int nrows = r1 > r0 ? r1 - r0 : 0;
    const bool owns_new = (split == n_act - 1);  // this CTA scores (and, for the group's first head, stores) the new row
    const int ntiles = (nrows + kTileRows - 1) / kTileRows;

    const size_t slab = ((size_t)b * a.n_kv_heads + hk) * (size_t)a.max_seq * DH;
    const unsigned char *kbase = reinterpret_cast<const unsigned char *>(a.k_cache + slab + (size_t)r0 * DH);
    const unsigned char *vbase = reinterpret_cast<const unsigned char *>(a.v_cache + slab + (size_t)r0 * DH);

    if (t == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&sm.full[s], 1);
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto issue_tile = [&](int tile) {
        const int stage = tile % kStages;
        const int rows = (nrows - tile * kTileRows) < kTileRows ? (nrows - tile * kTileRows) : kTileRows;
        const uint32_t bytes = (uint32_t)rows * Smem::kRowBytes;
        mbar_expect_tx(&sm.full[stage], 2 * bytes);
        bulk_g2s(sm.k[stage], kbase + (size_t)tile * Smem::kTileBytes, bytes, &sm.full[stage]);
        bulk_g2s(sm.v[stage], vbase + (size_t)tile * Smem::kTileBytes, bytes, &sm.full[stage]);
    };
    if (t == 0) {
        for (int tile = 0; tile < ntiles && tile < kStages; ++tile) issue_tile(tile);
    }

    // ---- joint RoPE of q and k_new with one set of cos/sin (Algorithm 3, steps 6-8) ----
    if (t < HALF) {
        const float c = a.cos_tab[(size_t)p * HALF + t], s = a.sin_tab[(size_t)p * HALF + t];
        const __nv_bfloat16 *qg = a.q + (size_t)b * a.q_stride + (size_t)hq * DH;
        const float x0 = __bfloat162float(qg[t]), x1 = __bfloat162float(qg[t + HALF]);
        sm.q[t] = __fsub_rn(__fmul_rn(x0, c), __fmul_rn(x1, s));
        sm.q[t + HALF] = __fadd_rn(__fmul_rn(x1, c), __fmul_rn(x0, s));
        if (owns_new) {
            const __nv_bfloat16 *kg = a.k_new + (size_t)b * a.kv_stride + (size_t)hk * DH;
            const float k0 = __bfloat162float(kg[t]), k1 = __bfloat162float(kg[t + HALF]);
            sm.knew[t] = __float2bfloat16_rn(__fsub_rn(__fmul_rn(k0, c), __fmul_rn(k1, s)));
            sm.knew[t + HALF] = __float2bfloat16_rn(__fadd_rn(__fmul_rn(k1, c), __fmul_rn(k0, s)));
        }
    } else if (owns_new && t >= 64 && t < 64 + DH / 8) {
        const uint4 *vg = reinterpret_cast<const uint4 *>(a.v_new + (size_t)b * a.kv_stride + (size_t)hk * DH);
        reinterpret_cast<uint4 *>(sm.vnew)[t - 64] = vg[t - 64];
    }
    __syncthreads();
    // ---- GKVC append (Eq. 2; Algorithm 3 steps 1 and 9): one write per row, no reload ----
    if (owns_new && (hq % G) == 0 && t < DH / 8) {
        uint4 *kdst = reinterpret_cast<uint4 *>(a.k_cache + slab + (size_t)L * DH);
        uint4 *vdst = reinterpret_cast<uint4 *>(a.v_cache + slab + (size_t)L * DH);
        kdst[t] = reinterpret_cast<const uint4 *>(sm.knew)[t];
        vdst[t] = reinterpret_cast<const uint4 *>(sm.vnew)[t];
    }

    // this lane's slice of q
    const int sub = lane & (kLanesPerRow - 1);       // which quarter of the row
    const int rgrp = lane >> 2;                      // row within a pass
    float qr[EPL];
#pragma unroll
    for (int i = 0; i < EPL; ++i) qr[i] = sm.q[sub * EPL + i];
    const float scale_log2 = rsqrtf((float)DH) * 1.4426950408889634f;

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
    auto axpy_row = [&](const unsigned char *rowp, float pj) {
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            float f[8];
            unpack8(*reinterpret_cast<const uint4 *>(rowp + (sub * VPL + v) * 16), f);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[v * 8 + i] = fmaf(pj, f[i], acc[v * 8 + i]);
        }
    };
    // online-softmax update with up to kPasses scores per lane
    auto update = [&](const float (&sc)[kPasses], const bool (&valid)[kPasses],
                      const unsigned char *const (&vrow)[kPasses]) {
        float mt = -INFINITY;
#pragma unroll
        for (int ps = 0; ps < kPasses; ++ps) mt = fmaxf(mt, valid[ps] ? sc[ps] : -INFINITY);
        mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 4));
        mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 8));
        mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, 16));
        const float m_new = fmaxf(m_run, mt);
        if (m_new == -INFINITY) return;              // nothing valid yet (warp-uniform)
        const float corr = fast_exp2(m_run - m_new);     // 0 when m_run = -inf
        l_run *= corr;
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] *= corr;
        m_run = m_new;
#pragma unroll
        for (int ps = 0; ps < kPasses; ++ps) {
            if (valid[ps]) {
                const float pj = fast_exp2(sc[ps] - m_new);
                if (sub == 0) l_run += pj;
                axpy_row(vrow[ps], pj);
            }
        }
    };

    // ---- stream the cached rows (Algorithm 3 steps 10-12) ----
    int tile = 0;
    for (; tile < ntiles; ++tile) {
        const int stage = tile % kStages;
        const uint32_t parity = (uint32_t)(tile / kStages) & 1u;
        bool ok = mbar_wait_bounded(&sm.full[stage], parity);
        if (!ok) sm.abort = 1;
        ok = __all_sync(kFull, ok);
        if (ok) {
            const int rows = (nrows - tile * kTileRows) < kTileRows ? (nrows - tile * kTileRows) : kTileRows;
            float sc[kPasses];
            bool valid[kPasses];
            const unsigned char *vrow[kPasses];
#pragma unroll
            for (int ps = 0; ps < kPasses; ++ps) {
                const int r = (ps * kAttnWarps + warp) * kRowsPerPass + rgrp;
                valid[ps] = r < rows;
                vrow[ps] = sm.v[stage] + r * Smem::kRowBytes;
                const float s = dot_row(sm.k[stage] + r * Smem::kRowBytes);   // all lanes: shuffles inside
                sc[ps] = valid[ps] ? s : -INFINITY;
            }
            update(sc, valid, vrow);
        }
        __syncthreads();                              // every warp is done with this stage
        if (sm.abort) break;
        if (t == 0 && tile + kStages < ntiles) issue_tile(tile + kStages);
    }
    if (sm.abort) {
        // a copy never landed: report, give outstanding copies one more bounded chance, leave
        if (t == 0) {
            atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT);
            for (int u = tile; u < ntiles && u < tile + kStages; ++u)
                (void)mbar_wait_bounded(&sm.full[u % kStages], (uint32_t)(u / kStages) & 1u);
        }
        return;
    }

    // ---- the new row, straight from shared memory (never re-read from the cache) ----
    if (owns_new && warp == 0) {
        float sc[kPasses];
        bool valid[kPasses];
        const unsigned char *vrow[kPasses];
#pragma unroll
        for (int ps = 0; ps < kPasses; ++ps) { sc[ps] = -INFINITY; valid[ps] = false; vrow[ps] = nullptr; }
        valid[0] = (rgrp == 0);
        vrow[0] = reinterpret_cast<const unsigned char *>(sm.vnew);
        const float s = dot_row(reinterpret_cast<const unsigned char *>(sm.knew));   // all lanes: shuffles inside
        sc[0] = valid[0] ? s : -INFINITY;
        update(sc, valid, vrow);
    }

    // ---- combine the row groups of a warp, then the warps of the CTA ----
#pragma unroll
    for (int s = 4; s <= 16; s <<= 1) {
        l_run += __shfl_xor_sync(kFull, l_run, s);
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] += __shfl_xor_sync(kFull, acc[i], s);
    }
    // (all lanes of a warp share m_run; l_run was accumulated by sub == 0 lanes only)
    l_run = __shfl_sync(kFull, l_run, 0);
    if (lane < kLanesPerRow) {
#pragma unroll
        for (int i = 0; i < EPL; ++i) sm.wo[warp][sub * EPL + i] = acc[i];
        if (lane == 0) { sm.wm[warp] = m_run; sm.wl[warp] = l_run; }
    }
    __syncthreads();

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
    if (n_act == 1) {
        if (t < DH) outp[t] = __float2bfloat16_rn(o / l);
        return;
    }

    // ---- split-KV: publish the partial, the last CTA of this head merges ----
    float *part = a.part + (((size_t)b * a.n_q_heads + hq) * kMaxSplits + split) * (DH + 2);
    if (t < DH) part[2 + t] = o;
    if (t == 0) { part[0] = M; part[1] = l; }
    __threadfence();
    __syncthreads();
    int *ticket = a.ticket + (size_t)b * a.n_q_heads + hq;
    if (t == 0) sm.last = (atomicAdd(ticket, 1) == n_act - 1);
    __syncthreads();
    if (!sm.last) return;
    __threadfence();
    const float *hp = a.part + ((size_t)b * a.n_q_heads + hq) * kMaxSplits * (DH + 2);
    float MM = -INFINITY;
    for (int s = 0; s < n_act; ++s) MM = fmaxf(MM, ld_cg_f32(hp + (size_t)s * (DH + 2)));
    if (t < DH) {
        float oo = 0.f, ll = 0.f;
        for (int s = 0; s < n_act; ++s) {
            const float ms = ld_cg_f32(hp + (size_t)s * (DH + 2));
            const float f = (ms == -INFINITY) ? 0.f : fast_exp2(ms - MM);
            oo += f * ld_cg_f32(hp + (size_t)s * (DH + 2) + 2 + t);
            ll += f * ld_cg_f32(hp + (size_t)s * (DH + 2) + 1);
        }
        outp[t] = __float2bfloat16_rn(oo / ll);
    }
    if (t == 0) *ticket = 0;
}

}  // namespace

int attn_splits_for(const Ctx *c, int batch)
{
    const int heads = batch * c->cfg.n_q_heads;
    const int target = c->n_sm * 18;                       // several waves of 3 CTAs per SM
    int s = (target + heads - 1) / heads;
    const int by_len = (c->cfg.max_seq + kTileRows - 1) / kTileRows;
    if (s > by_len) s = by_len;
    if (s > kMaxSplits) s = kMaxSplits;
    return s < 1 ? 1 : s;
}

template <int DH>
static int launch_attn_dh(Ctx *c, const AttnArgs &a, cudaStream_t st)
{
    const size_t smem = sizeof(AttnSmem<DH>) + 128;
    static bool configured[16] = {};
    if (!configured[c->cfg.device & 15]) {
        FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured[c->cfg.device & 15] = true;
    }
    dim3 grid(a.n_splits, a.n_q_heads, a.batch);
    ProfScope prof(c, kProfAttn, st);
    attn_decode_kernel<DH><<<grid, kAttnThreads, smem, st>>>(a);
    c->launches++;
    FT_CUDA(cudaGetLastError());
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
