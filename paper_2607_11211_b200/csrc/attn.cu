// Stand-alone fused decode attention kernel (Algorithm 3 of the paper, "GKVC & TPSFLAT"):
// one CTA per SM, 8 consumer warps + 1 producer warp around the shared-memory ring.
// The algorithm lives in attn_core.cuh.
#include "attn_core.cuh"

namespace fasttps {

namespace {

constexpr int kAttnWarps = 8;                           // consumer warps
constexpr int kAttnThreads = (kAttnWarps + 1) * 32;     // + the producer warp

template <int DH>
struct AttnSmem {
    static constexpr int kSlots = (192 * 1024 / AttnTile<DH>::kPieceBytes) < 8 ? (192 * 1024 / AttnTile<DH>::kPieceBytes) : 8;
    alignas(128) unsigned char slots[kSlots][AttnTile<DH>::kPieceBytes];
    alignas(16) uint64_t bars[2 * kSlots];
    AttnScratch<DH> scratch;
    int abort;
};

template <int DH>
__global__ void __launch_bounds__(kAttnThreads, 1) attn_decode_kernel(AttnArgs a)
{
    using Smem = AttnSmem<DH>;
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
        if ((t & 31) == 0) (void)attn_produce<DH>(a, ring, piece, blockIdx.x, gridDim.x);
        return;
    }
    if (blockIdx.x == 0 && t == 0) {
        // sequences that cannot be served are reported once and contribute no rows
        for (int bb = 0; bb < a.batch; ++bb) {
            const int L = a.seq_lens[bb], p = a.pos[bb];
            if (L < 0 || L >= a.max_seq) atomicOr(a.status, FASTTPS_DEV_CACHE_FULL);
            else if (p < 0 || p >= a.max_seq) atomicOr(a.status, FASTTPS_DEV_BAD_POSITION);
        }
    }
    if (!attn_consume<DH, false>(a, ring, piece, blockIdx.x, WalkSource(a, blockIdx.x, gridDim.x), sm.scratch, kAttnWarps) && t == 0)
        atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT);
}

}  // namespace

// Number of CTAs the attention kernel uses (one per SM, fewer for tiny head counts so that
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
