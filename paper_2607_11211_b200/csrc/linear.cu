// Projection kernel of the decode chain: out = [rmsnorm](x) . W^T (+ residual), with an
// optional fused greedy argmax (lm_head).  Used for the QKV projection, the
// attention output projection and the logits (Figure 1 of the paper; these
// products are weight-bound GEMVs at decode time).
#include "dot_core.cuh"
#include "stream_launch.cuh"

namespace fasttps {

template <int NB, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) linear_kernel(LinearArgs a)
{
    constexpr int R = RowsPerGroup<NB>::value;
    extern __shared__ __align__(128) unsigned char dsm[];
    __shared__ float s_best_val[R * NB];
    __shared__ int s_best_idx[R * NB];
    __shared__ int s_last;

    const int t = threadIdx.x;
    const StreamSmemLayout lay = stream_smem_layout(a.n_in, R, NB, (blockDim.x + 31) >> 5);
    float *smem = reinterpret_cast<float *>(dsm + lay.red_off);

    // contiguous, balanced row range of this CTA
    const int base = a.n_out / gridDim.x, rem = a.n_out % gridDim.x;
    const int cta = blockIdx.x;
    const int row0 = cta * base + (cta < rem ? cta : rem);
    const int nrows = base + (cta < rem ? 1 : 0);

    // the weights do not depend on the activations: start streaming them first
    WeightRing ring;
    ring.init(dsm + lay.ring_off, reinterpret_cast<uint64_t *>(dsm + lay.bar_off), lay.nslot, a.n_in * 2, R,
              a.w + (size_t)row0 * a.n_in, nrows, nullptr, 0);
    __syncthreads();
    if (t == 0) ring.start();

    float x[NB][8];
    load_activations<NB>(x, a.x, a.x_stride, a.batch, a.n_in, a.g, a.eps, smem);

    float best_val = -INFINITY;
    int best_idx = 0x7fffffff;
    const bool ok = dot_rows<NB>(ring, 0, a.n_in, row0, nrows, x, smem, [&](int row, int b, float v) {
        if (b >= a.batch) return;
        if (a.res) v += __bfloat162float(a.res[(size_t)b * a.res_stride + row]);
        if (a.out_bf16) a.out_bf16[(size_t)b * a.out_stride + row] = __float2bfloat16_rn(v);
        if (a.out_f32) a.out_f32[(size_t)b * a.out_stride + row] = v;
        if (v > best_val) { best_val = v; best_idx = row; }       // rows ascend per thread: first max kept
    });
    if (!ok) {
        if (t == 0) { atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT); ring.drain(0); }
        return;
    }

    if (a.next_ids == nullptr) return;

    // greedy argmax: CTA best per batch row -> global partials -> last CTA finishes
    if (t < R * NB) { s_best_val[t] = best_val; s_best_idx[t] = best_idx; }
    __syncthreads();
    if (t < NB && t < a.batch) {
        float bv = -INFINITY; int bi = 0x7fffffff;
        for (int r = 0; r < R; ++r) {
            float v = s_best_val[r * NB + t]; int i = s_best_idx[r * NB + t];
            if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
        }
        a.amax_val[(size_t)t * gridDim.x + cta] = bv;
        a.amax_idx[(size_t)t * gridDim.x + cta] = bi;
    }
    __threadfence();
    __syncthreads();
    if (t == 0) s_last = (atomicAdd(a.amax_ticket, 1) == (int)gridDim.x - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (t < NB && t < a.batch) {
        float bv = -INFINITY; int bi = 0x7fffffff;
        for (int c = 0; c < (int)gridDim.x; ++c) {
            float v = ld_cg_f32(a.amax_val + (size_t)t * gridDim.x + c);
            int i = ld_cg_s32(a.amax_idx + (size_t)t * gridDim.x + c);
            if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
        }
        if (bi == 0x7fffffff) bi = 0;          // all-NaN row: fall back to index 0
        a.next_ids[t] = bi;
        if (a.adv_pos) a.adv_pos[t] += 1;
        if (a.adv_len) a.adv_len[t] += 1;
    }
    if (t == 0) *a.amax_ticket = 0;
}

int linear_grid(const Ctx *c, int n_out)
{
    int g = c->n_sm;
    if (g > n_out) g = n_out;
    return g < 1 ? 1 : g;
}

template <int NB>
static cudaError_t configure_linear_nb()
{
    cudaError_t e = allow_big_smem(linear_kernel<NB, 128>);
    if (e == cudaSuccess) e = allow_big_smem(linear_kernel<NB, 256>);
    if (e == cudaSuccess) e = allow_big_smem(linear_kernel<NB, 384>);
    if (e == cudaSuccess) e = allow_big_smem(linear_kernel<NB, 512>);
    if (e == cudaSuccess) e = allow_big_smem(linear_kernel<NB, 768>);
    return e;
}

int configure_linear_kernels()
{
    FT_CUDA(configure_linear_nb<1>());
    FT_CUDA(configure_linear_nb<2>());
    FT_CUDA(configure_linear_nb<4>());
    FT_CUDA(configure_linear_nb<8>());
    return FASTTPS_OK;
}

template <int NB>
static int launch_linear_nb(Ctx *c, const LinearArgs &a, cudaStream_t st)
{
    constexpr int R = RowsPerGroup<NB>::value;
    const int threads = ((a.n_in / 8) + 31) / 32 * 32;
    const StreamSmemLayout lay = stream_smem_layout(a.n_in, R, NB, threads / 32);
    if (lay.nslot < 2) return FASTTPS_INVALID_ARG;
    const int grid = linear_grid(c, a.n_out);
    ProfScope prof(c, a.prof_class, st);
    int rc;
    // the register budget follows the block size: one instantiation per size class
    if (threads <= 128) rc = launch_stream_kernel(linear_kernel<NB, 128>, grid, threads, lay.total, st, &a);
    else if (threads <= 256) rc = launch_stream_kernel(linear_kernel<NB, 256>, grid, threads, lay.total, st, &a);
    else if (threads <= 384) rc = launch_stream_kernel(linear_kernel<NB, 384>, grid, threads, lay.total, st, &a);
    else if (threads <= 512) rc = launch_stream_kernel(linear_kernel<NB, 512>, grid, threads, lay.total, st, &a);
    else rc = launch_stream_kernel(linear_kernel<NB, 768>, grid, threads, lay.total, st, &a);
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
        int rc;
        if (a.batch == 1) rc = launch_linear_nb<1>(c, a, st);
        else if (a.batch == 2) rc = launch_linear_nb<2>(c, a, st);
        else if (a.batch <= 4) rc = launch_linear_nb<4>(c, a, st);
        else rc = launch_linear_nb<8>(c, a, st);
        if (rc != FASTTPS_OK) return rc;
    }
    return FASTTPS_OK;
}

}  // namespace fasttps
