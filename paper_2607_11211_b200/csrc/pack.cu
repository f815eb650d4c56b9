// One-time weight re-layout (the offline interlacing of Section 3.2, item 1 of the paper,
// taken further: the packed form is the order in which the tensor-core fragments are read)
// and the embedding-row gather that starts a full-stack decode step.
//
// Packed layouts
//   QKV, O, GATE_UP, LM_HEAD ("tiled"): the [n_out][n_in] matrix (n_out padded to a multiple
//     of 16 with zero rows) cut into tiles of 16 rows x 32 k, each tile row-major (1 KB),
//     tiles ordered by (row tile, k block).  For GATE_UP packed row r of row tile J is gate
//     column 8J + r for r < 8 and up column 8J + r - 8 otherwise (interlaced in blocks of 8).
//     For O packed row r of row tile J is output column 16J + 2r for r < 8 and 16J + 2(r - 8) + 1
//     otherwise: the two rows a thread of the tensor-core product holds are neighbouring columns.
//   DOWN ("octet blocks"): for intermediate octet o and output block nb (32 columns) one
//     512-byte block; lane (g, t4) of a warp owns 16 bytes of it: the pairs
//     (W[8o + 2 t4][n], W[8o + 2 t4 + 1][n]) for n = 32 nb + 4 g + {0, 1, 2, 3}, i.e. the A
//     fragments of two m16n8k8 MMAs whose rows g, g + 8 (first MMA) and g, g + 8 (second) are
//     four consecutive output columns: the products leave the registers as 16-byte vectors.
//     Blocks ordered by (o, nb).
#include "common.cuh"

namespace fasttps {

namespace {

struct PackDesc {
    int kind;          // fasttps_weight_kind
    int n_in, n_out;   // reduction length, logical output count
    int interlaceK;    // K for GATE_UP, else 0
    int src_is_out_in; // 1 when the logical matrix is [n_out][n_in] (LM_HEAD)
};

__device__ __forceinline__ int logical_col(int r, int interlaceK, int kind)
{
    // W_o: rows g and g + 8 of a tile are the output columns 2 g and 2 g + 1 (a thread's two sums are neighbours)
    if (kind == FASTTPS_W_O) return (r & ~15) + ((r & 8) ? 2 * (r & 7) + 1 : 2 * (r & 7));
    if (interlaceK == 0) return r;
    const int o = r >> 4, half = (r >> 3) & 1, c = r & 7;
    return half * interlaceK + o * 8 + c;
}

// one thread per packed 16-byte vector (8 consecutive k of one packed row)
__global__ void pack_tiled_kernel(const __nv_bfloat16 *logical, __nv_bfloat16 *packed, PackDesc d, size_t nvec, int inverse)
{
    const size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= nvec) return;
    const int KB = d.n_in >> 5;
    const size_t tile = v >> 6;
    const int within = (int)(v & 63), r = within >> 2, kc = within & 3;
    const int rt = (int)(tile / KB), kb = (int)(tile % KB);
    const int row = 16 * rt + r, k0 = 32 * kb + 8 * kc;
    __nv_bfloat16 *pv = packed + v * 8;
    if (row >= d.n_out) {
        if (!inverse)
            for (int e = 0; e < 8; ++e) pv[e] = __float2bfloat16_rn(0.f);
        return;
    }
    const int col = logical_col(row, d.interlaceK, d.kind);
    for (int e = 0; e < 8; ++e) {
        const size_t li = d.src_is_out_in ? (size_t)col * d.n_in + (k0 + e) : (size_t)(k0 + e) * d.n_out + col;
        if (inverse) const_cast<__nv_bfloat16 *>(logical)[li] = pv[e];
        else pv[e] = logical[li];
    }
}

// one thread per packed 16-byte vector of the DOWN layout; logical is [K][D]
__global__ void pack_down_kernel(const __nv_bfloat16 *logical, __nv_bfloat16 *packed, int K, int D, size_t nvec, int inverse)
{
    const size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= nvec) return;
    const int NT = D >> 5;
    const size_t blk = v >> 5;
    const int lane = (int)(v & 31), g = lane >> 2, t4 = lane & 3;
    const int o = (int)(blk / NT), nb = (int)(blk % NT);
    __nv_bfloat16 *pv = packed + v * 8;
    for (int e = 0; e < 8; ++e) {
        const int j = 8 * o + 2 * t4 + (e & 1), n = 32 * nb + 4 * g + (e >> 1);
        const size_t li = (size_t)j * D + n;
        if (inverse) const_cast<__nv_bfloat16 *>(logical)[li] = pv[e];
        else pv[e] = logical[li];
    }
}

struct EmbedArgs {
    const __nv_bfloat16 *embed;
    const int32_t *ids;
    __nv_bfloat16 *x;
    int D, vocab;
    uint32_t *status;
};

__global__ void embed_gather_kernel(EmbedArgs a)
{
    pdl_wait();                    // the token ids come from the previous step's argmax
    pdl_launch_dependents();
    const int b = blockIdx.x;
    int id = a.ids[b];
    if (id < 0 || id >= a.vocab) {
        if (threadIdx.x == 0) atomicOr(a.status, FASTTPS_DEV_BAD_TOKEN);
        id = 0;
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(a.embed + (size_t)id * a.D);
    uint4 *dst = reinterpret_cast<uint4 *>(a.x + (size_t)b * a.D);
    for (int i = threadIdx.x; i < a.D / 8; i += blockDim.x) dst[i] = src[i];
}

}  // namespace

int launch_embed(Ctx *c, const __nv_bfloat16 *embed, const int32_t *ids, __nv_bfloat16 *x, int batch, cudaStream_t st)
{
    ProfScope prof(c, kProfEmbed, st);
    EmbedArgs a = {embed, ids, x, c->cfg.hidden, c->cfg.vocab, c->status};
    const int rc = launch_ex(embed_gather_kernel, dim3(batch), dim3(128), 0, st, &a);
    c->launches++;
    return rc;
}

size_t packed_elems(const fasttps_config &f, int kind)
{
    const size_t nq = (size_t)f.n_q_heads * f.head_dim, nkv = (size_t)f.n_kv_heads * f.head_dim;
    auto pad16 = [](size_t n) { return (n + 15) / 16 * 16; };
    switch (kind) {
    case FASTTPS_W_QKV: return pad16(nq + 2 * nkv) * f.hidden;
    case FASTTPS_W_O: return pad16(f.hidden) * nq;
    case FASTTPS_W_GATE_UP: return pad16(2 * (size_t)f.inter) * f.hidden;
    case FASTTPS_W_DOWN: return (size_t)f.inter * f.hidden;
    case FASTTPS_W_LM_HEAD: return pad16(f.vocab) * f.hidden;
    default: return 0;
    }
}

int launch_pack(Ctx *c, int kind, const void *src, void *dst, bool inverse, cudaStream_t st)
{
    // forward: src = logical, dst = packed; inverse: src = packed, dst = logical
    const fasttps_config &f = c->cfg;
    const __nv_bfloat16 *logical = static_cast<const __nv_bfloat16 *>(inverse ? dst : src);
    __nv_bfloat16 *packed = static_cast<__nv_bfloat16 *>(inverse ? const_cast<void *>(src) : dst);
    const size_t nvec = packed_elems(f, kind) / 8;
    if (nvec == 0) return FASTTPS_INVALID_ARG;
    const unsigned grid = (unsigned)((nvec + 255) / 256);
    if (kind == FASTTPS_W_DOWN) {
        pack_down_kernel<<<grid, 256, 0, st>>>(logical, packed, f.inter, f.hidden, nvec, inverse ? 1 : 0);
    } else {
        PackDesc d;
        d.kind = kind; d.interlaceK = 0; d.src_is_out_in = 0;
        const int nq = f.n_q_heads * f.head_dim, nkv = f.n_kv_heads * f.head_dim;
        switch (kind) {
        case FASTTPS_W_QKV: d.n_in = f.hidden; d.n_out = nq + 2 * nkv; break;
        case FASTTPS_W_O: d.n_in = nq; d.n_out = f.hidden; break;
        case FASTTPS_W_GATE_UP: d.n_in = f.hidden; d.n_out = 2 * f.inter; d.interlaceK = f.inter; break;
        case FASTTPS_W_LM_HEAD: d.n_in = f.hidden; d.n_out = f.vocab; d.src_is_out_in = 1; break;
        default: return FASTTPS_INVALID_ARG;
        }
        pack_tiled_kernel<<<grid, 256, 0, st>>>(logical, packed, d, nvec, inverse ? 1 : 0);
    }
    FT_CUDA(cudaGetLastError());
    return FASTTPS_OK;
}

}  // namespace fasttps
