// Stand-alone fused decode attention kernel (Algorithm 3 of the paper, "GKVC & TPSFLAT"):
// one CTA per SM, 8 consumer warps + 1 producer warp around the shared-memory ring.
// The algorithm lives in attn_core.cuh.
#include <type_traits>
#include "attn_group_core.cuh"

namespace fasttps {

namespace {

constexpr int kAttnWarps = 8;                           // consumer warps
constexpr int kAttnThreads = (kAttnWarps + 1) * 32;     // + the producer warp
static_assert(kAttnWarps == kGroupWarps, "the grouped-query path divides the tiles among exactly kGroupWarps consumer warps");

// Grouped-query attention with 2 to 16 query heads per K/V head streams every cached row once for the whole
// group, with the two products on the tensor cores; other ratios stream it once per query head.
// The members of a group are its query heads times the new tokens of the sequence (n_new > 1: a chunk).
inline bool attn_shares_groups(int n_q_heads, int n_kv_heads, int n_new = 1)
{
    const int G = (n_kv_heads > 0 ? n_q_heads / n_kv_heads : 1) * n_new;
    return G > 1 && G <= kMaxShareGroup;
}

template <int DH>
struct AttnSmem {
    // a power of two (the ring finds slot and round of a piece by mask and shift): 8 pieces of up to 24 KB,
    // 4 of the 32 KB pieces of head_dim 128
    static constexpr int kFit = 192 * 1024 / AttnTile<DH>::kPieceBytes;
    static constexpr int kSlots = kFit >= 8 ? 8 : kFit >= 4 ? 4 : 2;
    static_assert((kSlots & (kSlots - 1)) == 0 && kSlots <= kFit, "ring slot count must be a power of two that fits");
    alignas(128) unsigned char slots[kSlots][AttnTile<DH>::kPieceBytes];
    alignas(16) uint64_t bars[2 * kSlots];
    AttnScratch<DH> scratch;
    AttnMulti<DH> multi;             // rows of the new tokens of a chunk (several new tokens per sequence)
    int abort;
};
template <int DH>
struct AttnSmemShare {
    // the per-warp outputs of a whole group take DH KB: the ring gives up slots for them at head_dim 96
    static constexpr int kFit = (int)(226 * 1024 - sizeof(GroupScratch<DH>)) / AttnTile<DH>::kPieceBytes;
    static constexpr int kSlots = kFit >= 8 ? 8 : kFit >= 4 ? 4 : 2;
    alignas(128) unsigned char slots[kSlots][AttnTile<DH>::kPieceBytes];
    alignas(16) uint64_t bars[2 * kSlots];
    GroupScratch<DH> scratch;
    int abort;
};

// SHARE: one pass per K/V head for its group of query heads (tensor cores; PRECISE: q and the softmax weights as bf16
// hi + lo pairs).  MULTI: several new tokens per sequence.  FP8: the cache holds E4M3 codes (SHARE and PRECISE).
template <int DH, bool SHARE, bool MULTI = false, bool PRECISE = false, bool FP8 = false>
__global__ void __launch_bounds__(kAttnThreads, 1) attn_decode_kernel(AttnArgs a)
{
    static_assert(!FP8 || (SHARE && PRECISE), "the E4M3 cache is served by the one-pass-per-K/V-head kernel");
    static_assert(!(SHARE && MULTI), "the multi-token path is the one-pass-per-query-head kernel");
    using Smem = typename std::conditional<SHARE, AttnSmemShare<DH>, AttnSmem<DH>>::type;
    extern __shared__ unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int t = threadIdx.x, warp = t >> 5;

    WeightRing ring;
    ring.init(&sm.slots[0][0], sm.bars, &sm.abort, Smem::kSlots, AttnTile<DH>::kPieceBytes, kAttnWarps, nullptr, 0, nullptr, 0);
    __syncthreads();

    // The share of this CTA depends on seq_lens, which the previous kernel in the stream may have
    // written (a model step advances them at its very end): nothing is read before it has finished.
    pdl_wait();
    pdl_launch_dependents();

    int piece = 0;
    if (warp == kAttnWarps) {
        if ((t & 31) == 0) (void)attn_produce<DH, SHARE, FP8 ? 1 : 2, FP8 ? 2 * kAttnTileRows : kAttnTileRows>(a, ring, piece, blockIdx.x, gridDim.x);
        return;
    }
    if (blockIdx.x == 0 && t == 0) {
        // sequences that cannot be served are reported once and contribute no rows
        for (int bb = 0; bb < a.batch / a.n_new; ++bb) {
            const int L = a.seq_lens[bb], p = a.pos[bb];
            if (L < 0 || L + a.n_new > a.max_seq) atomicOr(a.status, FASTTPS_DEV_CACHE_FULL);
            else if (p < 0 || p + a.n_new > a.max_seq) atomicOr(a.status, FASTTPS_DEV_BAD_POSITION);
        }
    }
    bool done;
    if constexpr (SHARE)
        done = attn_consume_group<DH, PRECISE, FP8>(a, ring, piece, blockIdx.x, WalkSource(a, blockIdx.x, gridDim.x, true), sm.scratch);
    else if constexpr (MULTI)
        done = attn_consume<DH, false, WalkSource, false, false, true>(a, ring, piece, blockIdx.x, WalkSource(a, blockIdx.x, gridDim.x),
                                                                       sm.scratch, kAttnWarps, nullptr, &sm.multi);
    else
        done = attn_consume<DH, false>(a, ring, piece, blockIdx.x, WalkSource(a, blockIdx.x, gridDim.x), sm.scratch, kAttnWarps);
    if (!done && t == 0) atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT);
}

}  // namespace

// Number of CTAs the attention kernel is launched with: one per SM.  How many of them take part is decided on
// the device from the lengths (the share walk): every share holds at least 16 rows, and no head is cut into
// more shares than it has partial records.
int attn_splits_for(const Ctx *c, int batch)
{
    (void)batch;
    return c->n_sm < 1 ? 1 : c->n_sm;
}

template <int DH>
static int launch_attn_dh(Ctx *c, const AttnArgs &a, cudaStream_t st, bool fp8)
{
    dim3 grid(a.n_splits);
    ProfScope prof(c, kProfAttn, st);
    const bool share = attn_shares_groups(a.n_q_heads, a.n_kv_heads, a.n_new);
    const int rc = fp8 ? launch_ex(attn_decode_kernel<DH, true, false, true, true>, grid, dim3(kAttnThreads), sizeof(AttnSmemShare<DH>) + 128, st, &a)
                   : (c->opt_gqa_share == 1 && share)
                       ? launch_ex(attn_decode_kernel<DH, true, false, true>, grid, dim3(kAttnThreads), sizeof(AttnSmemShare<DH>) + 128, st, &a)
                   : (c->opt_gqa_share && share)
                       ? launch_ex(attn_decode_kernel<DH, true>, grid, dim3(kAttnThreads), sizeof(AttnSmemShare<DH>) + 128, st, &a)
                   : a.n_new > 1
                       ? launch_ex(attn_decode_kernel<DH, false, true>, grid, dim3(kAttnThreads), sizeof(AttnSmem<DH>) + 128, st, &a)
                       : launch_ex(attn_decode_kernel<DH, false>, grid, dim3(kAttnThreads), sizeof(AttnSmem<DH>) + 128, st, &a);
    c->launches++;
    return rc;
}

template <int DH>
static int configure_attn_dh()
{
    FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<DH, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttnSmem<DH>) + 128));
    FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<DH, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttnSmemShare<DH>) + 128));
    FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<DH, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttnSmemShare<DH>) + 128));
    FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<DH, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttnSmem<DH>) + 128));
    FT_CUDA(cudaFuncSetAttribute(attn_decode_kernel<DH, true, false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttnSmemShare<DH>) + 128));
    return FASTTPS_OK;
}

int configure_attn_kernels()
{
    int rc;
    if ((rc = configure_attn_dh<32>()) != FASTTPS_OK) return rc;
    if ((rc = configure_attn_dh<64>()) != FASTTPS_OK) return rc;
    if ((rc = configure_attn_dh<96>()) != FASTTPS_OK) return rc;
    return configure_attn_dh<128>();
}

// fp8: the caches hold E4M3 codes (a.k_scale / a.v_scale set); the group (query heads x new tokens) is 1 to 16 members
int launch_attn(Ctx *c, const AttnArgs &a, cudaStream_t st, bool fp8)
{
    if (fp8) {
        const int G = (a.n_kv_heads > 0 ? a.n_q_heads / a.n_kv_heads : 0) * a.n_new;
        if (G < 1 || G > kMaxShareGroup) return FASTTPS_INVALID_ARG;
    }
    switch (a.head_dim) {
    case 32: return launch_attn_dh<32>(c, a, st, fp8);
    case 64: return launch_attn_dh<64>(c, a, st, fp8);
    case 96: return launch_attn_dh<96>(c, a, st, fp8);
    case 128: return launch_attn_dh<128>(c, a, st, fp8);
    default: return FASTTPS_INVALID_ARG;
    }
}

}  // namespace fasttps

// Diagnostic entry point: the share walk of the stand-alone attention kernel, run on the host by the same code the
// kernel runs on the device, for every CTA in turn; the segments go to the caller.
extern "C" int fasttps_attention_walk(const int32_t *seq_lens, const int32_t *pos, int batch, int heads, int max_seq, int n_cta,
                                      int32_t *seg_out, int max_segs)
{
    using namespace fasttps;
    if (!seq_lens || !pos || !seg_out || batch < 1 || heads < 1 || max_seq < 1 || n_cta < 1 || max_segs < 0)
        return FASTTPS_INVALID_ARG;
    int n = 0;
    for (int cta = 0; cta < n_cta; ++cta) {
        ShareWalk w;
        w.init(seq_lens, pos, 0, batch, heads, max_seq, cta, n_cta);
        Segment sg;
        while (w.next(sg)) {
            if (n < max_segs) {
                int32_t *o = seg_out + (size_t)n * 7;
                o[0] = cta; o[1] = sg.b; o[2] = sg.h; o[3] = sg.r0; o[4] = sg.r1; o[5] = sg.first_cta; o[6] = sg.n_cta;
            }
            ++n;
        }
    }
    return n;
}
