// One-time weight re-layout (the offline interlacing of Section 3.2, item 1 of the paper)
// and the embedding-row gather that starts a full-stack decode step.
#include "common.cuh"

namespace fasttps {

namespace {

// dst[r][c] = src[c][r_src(r)]  for a logical [n_in][n_out] source and a packed
// [n_out][n_in] destination; r_src maps a packed row to its logical column.
// gate_up: packed row r -> octet o = r / 16, half = (r / 8) & 1, c = r & 7 -> logical column half*K + 8*o + c.
__device__ __forceinline__ int logical_col(int r, int interlaceK)
{
    if (interlaceK == 0) return r;
    const int o = r >> 4, half = (r >> 3) & 1, c = r & 7;
    return half * interlaceK + o * 8 + c;
}

__global__ void transpose_pack_kernel(const __nv_bfloat16 *src, __nv_bfloat16 *dst, int n_in, int n_out,
                                      int interlaceK, int inverse)
{
    __shared__ __nv_bfloat16 tile[32][33];
    const int in0 = blockIdx.x * 32, out0 = blockIdx.y * 32;
    const int tx = threadIdx.x, ty = threadIdx.y;     // 32 x 8
    if (!inverse) {
        // read logical [in][out] coalesced along out (packed-row order), write packed [out][in] along in
        for (int i = ty; i < 32; i += 8) {
            const int in = in0 + i, r = out0 + tx;
            if (in < n_in && r < n_out) tile[i][tx] = src[(size_t)in * n_out + logical_col(r, interlaceK)];
        }
        __syncthreads();
        for (int i = ty; i < 32; i += 8) {
            const int r = out0 + i, in = in0 + tx;
            if (in < n_in && r < n_out) dst[(size_t)r * n_in + in] = tile[tx][i];
        }
    } else {
        for (int i = ty; i < 32; i += 8) {
            const int r = out0 + i, in = in0 + tx;
            if (in < n_in && r < n_out) tile[tx][i] = src[(size_t)r * n_in + in];
        }
        __syncthreads();
        for (int i = ty; i < 32; i += 8) {
            const int in = in0 + i, r = out0 + tx;
            if (in < n_in && r < n_out) dst[(size_t)in * n_out + logical_col(r, interlaceK)] = tile[i][tx];
        }
    }
}

__global__ void embed_gather_kernel(const __nv_bfloat16 *embed, const int32_t *ids, __nv_bfloat16 *x,
                                    int D, int vocab, uint32_t *status)
{
    const int b = blockIdx.x;
    int id = ids[b];
    if (id < 0 || id >= vocab) {
        if (threadIdx.x == 0) atomicOr(status, FASTTPS_DEV_BAD_TOKEN);
        id = 0;
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(embed + (size_t)id * D);
    uint4 *dst = reinterpret_cast<uint4 *>(x + (size_t)b * D);
    for (int i = threadIdx.x; i < D / 8; i += blockDim.x) dst[i] = src[i];
}

}  // namespace

int launch_embed(Ctx *c, const __nv_bfloat16 *embed, const int32_t *ids, __nv_bfloat16 *x, int batch, cudaStream_t st)
{
    ProfScope prof(c, kProfEmbed, st);
    embed_gather_kernel<<<batch, 128, 0, st>>>(embed, ids, x, c->cfg.hidden, c->cfg.vocab, c->status);
    c->launches++;
    FT_CUDA(cudaGetLastError());
    return FASTTPS_OK;
}

int launch_pack(Ctx *c, int kind, const void *src, void *dst, bool inverse, cudaStream_t st)
{
    const fasttps_config &f = c->cfg;
    int n_in = 0, n_out = 0, interlaceK = 0;
    switch (kind) {
    case FASTTPS_W_QKV: n_in = f.hidden; n_out = (f.n_q_heads + 2 * f.n_kv_heads) * f.head_dim; break;
    case FASTTPS_W_O: n_in = f.n_q_heads * f.head_dim; n_out = f.hidden; break;
    case FASTTPS_W_GATE_UP: n_in = f.hidden; n_out = 2 * f.inter; interlaceK = f.inter; break;
    case FASTTPS_W_DOWN:
        FT_CUDA(cudaMemcpyAsync(dst, src, (size_t)f.inter * f.hidden * 2, cudaMemcpyDeviceToDevice, st));
        return FASTTPS_OK;
    case FASTTPS_W_LM_HEAD:
        FT_CUDA(cudaMemcpyAsync(dst, src, (size_t)f.vocab * f.hidden * 2, cudaMemcpyDeviceToDevice, st));
        return FASTTPS_OK;
    default: return FASTTPS_INVALID_ARG;
    }
    dim3 grid((n_in + 31) / 32, (n_out + 31) / 32), block(32, 8);
    transpose_pack_kernel<<<grid, block, 0, st>>>(static_cast<const __nv_bfloat16 *>(src),
                                                  static_cast<__nv_bfloat16 *>(dst), n_in, n_out, interlaceK,
                                                  inverse ? 1 : 0);
    FT_CUDA(cudaGetLastError());
    return FASTTPS_OK;
}

}  // namespace fasttps
