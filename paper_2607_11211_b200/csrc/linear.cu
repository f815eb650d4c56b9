// Projection kernel of the decode chain: out = [rmsnorm](x) . W^T (+ residual), with an
// optional fused greedy argmax (lm_head).  Used for the QKV projection, the
// attention output projection and the logits (Figure 1 of the paper; these
// products are weight-bound thin GEMMs at decode time).
//
// One CTA per SM owns a contiguous range of 16-row tiles of the tiled weight matrix (a single
// contiguous byte range).  A producer warp streams it through the shared-memory ring; the
// consumer warps multiply it with the activations on the tensor cores (dot_core.cuh).
#include "stream_launch.cuh"

namespace fasttps {

template <int IPW, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) linear_kernel(LinearArgs a)
{
    extern __shared__ __align__(128) unsigned char dsm[];
    __shared__ float s_best_val[64];
    __shared__ int s_best_idx[64];
    __shared__ int s_last;

    const int t = threadIdx.x;
    const StreamSmemLayout lay = stream_smem_layout(a.n_in);
    const int nw = lay.nw;
    float *smem_part = reinterpret_cast<float *>(dsm + lay.part_off);
    float *smem_red = reinterpret_cast<float *>(dsm + lay.red_off);

    // contiguous, balanced range of row tiles of this CTA
    const int n_tiles = (a.n_out + 15) >> 4;
    const int base = n_tiles / gridDim.x, rem = n_tiles % gridDim.x;
    const int cta = blockIdx.x;
    const int tile0 = cta * base + (cta < rem ? cta : rem);
    const int ntile = base + (cta < rem ? 1 : 0);
    const size_t tile_bytes = (size_t)a.n_in * 32;            // 16 rows x n_in bf16

    WeightRing ring;
    ring.init(dsm + lay.ring_off, reinterpret_cast<uint64_t *>(dsm + lay.bar_off),
              reinterpret_cast<int *>(dsm + lay.abort_off), lay.nslot, lay.slot_bytes, nw,
              reinterpret_cast<const unsigned char *>(a.w) + (size_t)tile0 * tile_bytes, (long long)ntile * tile_bytes,
              nullptr, 0);
    if (t < 64) { s_best_val[t] = -INFINITY; s_best_idx[t] = 0x7fffffff; }
    __syncthreads();

    if (t >= nw * 32) {
        // producer warp: the weights do not depend on the activations, so streaming starts at once
        if (t == nw * 32) ring.produce();
        return;
    }

    // everything below reads what the previous kernel wrote, or writes what it may still read
    pdl_wait();
    pdl_launch_dependents();

    uint32_t bf[IPW][4];
    load_b_frags<IPW>(bf, a.x, a.x_stride, a.batch, a.n_in, nw, a.g, a.eps, smem_red);

    const bool ok = dot_tiles<IPW>(ring, 0, ntile, nw, bf, smem_part, [&](int tile, int cc, int b, float v0, float v1) {
        if (b >= a.batch) return;
        const int u = cc * 8 + b;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int row = (tile0 + tile) * 16 + (a.pair_rows ? 2 * cc + h : cc + 8 * h);
            if (row >= a.n_out) continue;
            float v = h ? v1 : v0;
            if (a.res) v += __bfloat162float(a.res[(size_t)b * a.res_stride + row]);
            if (a.out_bf16) a.out_bf16[(size_t)b * a.out_stride + row] = __float2bfloat16_rn(v);
            if (a.out_f32) a.out_f32[(size_t)b * a.out_stride + row] = v;
            if (v > s_best_val[u]) { s_best_val[u] = v; s_best_idx[u] = row; }   // rows ascend: first max kept
        }
    });
    if (!ok) {
        if (t == 0) atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT);
        return;
    }
    if (a.next_ids == nullptr) return;

    // greedy argmax: CTA best per batch row -> global partials -> last CTA finishes
    named_bar_sync(1, nw * 32);
    if (t < 8 && t < a.batch) {
        float bv = -INFINITY; int bi = 0x7fffffff;
        for (int cc = 0; cc < 8; ++cc) {
            const float v = s_best_val[cc * 8 + t]; const int i = s_best_idx[cc * 8 + t];
            if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
        }
        a.amax_val[(size_t)t * gridDim.x + cta] = bv;
        a.amax_idx[(size_t)t * gridDim.x + cta] = bi;
    }
    __threadfence();
    named_bar_sync(1, nw * 32);
    if (t == 0) s_last = (atomicAdd(a.amax_ticket, 1) == (int)gridDim.x - 1);
    named_bar_sync(1, nw * 32);
    if (!s_last) return;
    __threadfence();
    // every thread fetches its share of the per-CTA candidates at once, then warps and the CTA reduce
    const int lane = t & 31, w = t >> 5;
    for (int b = 0; b < a.batch; ++b) {
        float bv = -INFINITY; int bi = 0x7fffffff;
        for (int c = t; c < (int)gridDim.x; c += nw * 32) {
            const float v = ld_cg_f32(a.amax_val + (size_t)b * gridDim.x + c);
            const int i = ld_cg_s32(a.amax_idx + (size_t)b * gridDim.x + c);
            if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
        }
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) {
            const float ov = __shfl_xor_sync(kFull, bv, s);
            const int oi = __shfl_xor_sync(kFull, bi, s);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { s_best_val[w] = bv; s_best_idx[w] = bi; }
        named_bar_sync(1, nw * 32);
        if (t == 0) {
            for (int w2 = 0; w2 < nw; ++w2) {
                const float v = s_best_val[w2]; const int i = s_best_idx[w2];
                if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
            }
            if (bi == 0x7fffffff) bi = 0;      // all-NaN row: fall back to index 0
            a.next_ids[b] = bi;
            if (a.adv_pos) a.adv_pos[b] += 1;
            if (a.adv_len) a.adv_len[b] += 1;
        }
        named_bar_sync(1, nw * 32);
    }
    if (t == 0) *a.amax_ticket = 0;
}

int configure_linear_kernels()
{
    FT_CUDA(allow_big_smem(linear_kernel<4, 416>));
    FT_CUDA(allow_big_smem(linear_kernel<4, 800>));
    FT_CUDA(allow_big_smem(linear_kernel<8, 416>));
    FT_CUDA(allow_big_smem(linear_kernel<8, 544>));
    FT_CUDA(allow_big_smem(linear_kernel<8, 800>));
    return FASTTPS_OK;
}

static int launch_linear_tile(Ctx *c, const LinearArgs &a, cudaStream_t st)
{
    const StreamSmemLayout lay = stream_smem_layout(a.n_in);
    if (lay.nw < 1 || lay.nslot < 2) return FASTTPS_INVALID_ARG;
    const int threads = (lay.nw + 1) * 32;                  // consumer warps + the producer warp
    const int n_tiles = (a.n_out + 15) / 16;
    int grid = c->n_sm;
    if (grid > n_tiles) grid = n_tiles;
    ProfScope prof(c, a.prof_class, st);
    // the register budget follows the block size: one instantiation per size class
    int rc;
    if (lay.ipw == 8)
        // 17 warps (hidden 4096: 16 consumer warps) get a register budget of their own: under the 800-thread bound a
        // thread has 72 registers and the tile loops spill
        rc = threads <= 416   ? launch_stream_kernel(linear_kernel<8, 416>, grid, threads, lay.total, st, &a)
             : threads <= 544 ? launch_stream_kernel(linear_kernel<8, 544>, grid, threads, lay.total, st, &a)
                              : launch_stream_kernel(linear_kernel<8, 800>, grid, threads, lay.total, st, &a);
    else
        rc = threads <= 416 ? launch_stream_kernel(linear_kernel<4, 416>, grid, threads, lay.total, st, &a)
                            : launch_stream_kernel(linear_kernel<4, 800>, grid, threads, lay.total, st, &a);
    c->launches++;
    return rc;
}

// Batches above kMaxNB are served in tiles of kMaxNB rows (the weights are re-read per tile).
int launch_linear(Ctx *c, const LinearArgs &a0, cudaStream_t st)
{
    for (int b0 = 0; b0 < a0.batch; b0 += kMaxNB) {
        LinearArgs a = a0;
        a.batch = a0.batch - b0 < kMaxNB ? a0.batch - b0 : kMaxNB;
        a.x = a0.x + (size_t)b0 * a0.x_stride;
        if (a.res) a.res = a0.res + (size_t)b0 * a0.res_stride;
        if (a.out_bf16) a.out_bf16 = a0.out_bf16 + (size_t)b0 * a0.out_stride;
        if (a.out_f32) a.out_f32 = a0.out_f32 + (size_t)b0 * a0.out_stride;
        if (a.next_ids) a.next_ids = a0.next_ids + b0;
        if (a.adv_pos) a.adv_pos = a0.adv_pos + b0;
        if (a.adv_len) a.adv_len = a0.adv_len + b0;
        const int rc = launch_linear_tile(c, a, st);
        if (rc != FASTTPS_OK) return rc;
    }
    return FASTTPS_OK;
}

}  // namespace fasttps
