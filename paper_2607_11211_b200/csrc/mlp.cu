// Fully fused SwiGLU MLP for decode (Algorithm 4 / Eq. 1 / Eq. 31 of the paper).
//
// The paper fuses gate and up into one interlaced Matmul with a siLu_Mul epilogue and
// sends the intermediate through L3 to a separate down projection.  Here the intermediate
// never leaves the SM: a CTA owns a contiguous range of j-octets (8 intermediate columns
// each).  For its range it
//   1. streams the 16 interlaced rows per octet of the packed gate_up matrix (8 gate rows,
//      then the 8 matching up rows; each row = the D weights of one output, contiguous) and
//      reduces them to FP32 gate/up values (dot_rows),
//   2. applies a = silu(gate) * up in shared memory,
//   3. streams the matching rows j of W_down [K, D] (each thread owns 8 output columns) and
//      accumulates y[:, 8t..8t+8) += a_j * W_down[j, 8t..8t+8) in registers,
//   4. adds its partial y into an FP32 accumulator in global memory (vector red.add); the
//      CTA that arrives last adds the residual, rounds to bf16 and re-zeroes the accumulator.
// Both weight slices of a CTA are contiguous byte ranges and go through ONE shared-memory
// ring of bulk asynchronous copies, so the W_down rows are already in flight while the
// gate_up reduction and the SiLU step are still running.
#include "dot_core.cuh"
#include "stream_launch.cuh"

namespace fasttps {

namespace {

constexpr int kMaxOctetsPerCta = 16;      // bounds the shared-memory intermediate

template <int NB, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) mlp_decode_kernel(MlpArgs a)
{
    constexpr int R = RowsPerGroup<NB>::value;               // rows per ring group, both phases
    extern __shared__ __align__(128) unsigned char dsm[];
    __shared__ float s_gu[kMaxOctetsPerCta * 16][NB];       // gate/up values of this CTA's rows
    __shared__ float s_act[kMaxOctetsPerCta * 8][NB];       // silu(gate) * up
    __shared__ int s_last;

    const int t = threadIdx.x;
    const StreamSmemLayout lay = stream_smem_layout(a.D, R, NB, (blockDim.x + 31) >> 5);
    float *smem = reinterpret_cast<float *>(dsm + lay.red_off);

    const int n_oct = a.K >> 3;
    const int base = n_oct / gridDim.x, rem = n_oct % gridDim.x;
    const int cta = blockIdx.x;
    const int oct0 = cta * base + (cta < rem ? cta : rem);
    const int noct = base + (cta < rem ? 1 : 0);
    const bool active = t * 8 < a.D;
    const int row0 = oct0 * 16, nrows_gu = noct * 16, nj = noct * 8;

    // both weight slices of this CTA, back to back through one ring
    WeightRing ring;
    ring.init(dsm + lay.ring_off, reinterpret_cast<uint64_t *>(dsm + lay.bar_off), lay.nslot, a.D * 2, R,
              a.w_gu + (size_t)row0 * a.D, nrows_gu, a.w_down + (size_t)oct0 * 8 * a.D, nj);
    __syncthreads();
    if (t == 0) ring.start();

    // ---- Algorithm 4 step 1 (optional): RMSNorm of the block input ----
    float x[NB][8];
    load_activations<NB>(x, a.x, a.D, a.batch, a.D, a.g, a.eps, smem);

    // ---- steps 2-10: interlaced gate_up product for rows [16*oct0, 16*(oct0+noct)) ----
    bool ok = dot_rows<NB>(ring, 0, a.D, 0, nrows_gu, x, smem, [&](int row, int b, float v) { s_gu[row][b] = v; });
    if (!ok) {
        if (t == 0) { atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT); ring.drain(0); }
        return;
    }
    __syncthreads();

    // ---- step 11: siLu_Mul (first half of an interlaced block is gate, second half up) ----
    for (int i = t; i < nj * NB; i += blockDim.x) {
        const int j = i / NB, b = i % NB;
        const int o = j >> 3, c = j & 7;
        const float g = s_gu[o * 16 + c][b], u = s_gu[o * 16 + 8 + c][b];
        s_act[j][b] = g / (1.f + __expf(-g)) * u;
    }
    __syncthreads();

    // ---- steps 13-15: down projection of this CTA's slice of the intermediate ----
    float acc[NB][8];
#pragma unroll
    for (int b = 0; b < NB; ++b)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[b][i] = 0.f;
    const int nvec = a.D >> 3;
    const int g_down0 = ring.groups0;
    const int ngroups_down = nj / R;                         // nj is a multiple of 8, hence of R
    for (int g = 0; g < ngroups_down; ++g) {
        const uint4 *slot = reinterpret_cast<const uint4 *>(ring.wait(g_down0 + g, ok));
        if (active) {
#pragma unroll
            for (int u = 0; u < R; ++u) {
                float wf[8];
                unpack8(slot[u * nvec + t], wf);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const float av = s_act[g * R + u][b];
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[b][i] = fmaf(av, wf[i], acc[b][i]);
                }
            }
        }
        if (!__syncthreads_and(ok ? 1 : 0)) {
            if (t == 0) { atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT); ring.drain(g_down0 + g); }
            return;
        }
        if (t == 0) ring.refill(g_down0 + g);
    }

    // ---- partial sums of all CTAs meet in the FP32 accumulator ----
    if (active) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (b < a.batch) {
                float *dst = a.acc + (size_t)b * a.D + t * 8;
                red_add_v4(dst, acc[b][0], acc[b][1], acc[b][2], acc[b][3]);
                red_add_v4(dst + 4, acc[b][4], acc[b][5], acc[b][6], acc[b][7]);
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (t == 0) s_last = (atomicAdd(a.ticket, 1) == (int)gridDim.x - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // last CTA: y (+ residual) -> bf16, accumulator back to zero for the next call
    if (active) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (b < a.batch) {
                float *src = a.acc + (size_t)b * a.D + t * 8;
                float4 y0, y1;
                asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(y0.x), "=f"(y0.y), "=f"(y0.z), "=f"(y0.w) : "l"(src));
                asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(y1.x), "=f"(y1.y), "=f"(y1.z), "=f"(y1.w) : "l"(src + 4));
                float r[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                if (a.res) unpack8(*reinterpret_cast<const uint4 *>(a.res + (size_t)b * a.D + t * 8), r);
                uint4 o;
                o.x = pack2(y0.x + r[0], y0.y + r[1]);
                o.y = pack2(y0.z + r[2], y0.w + r[3]);
                o.z = pack2(y1.x + r[4], y1.y + r[5]);
                o.w = pack2(y1.z + r[6], y1.w + r[7]);
                *reinterpret_cast<uint4 *>(a.out + (size_t)b * a.D + t * 8) = o;
                *reinterpret_cast<float4 *>(src) = make_float4(0.f, 0.f, 0.f, 0.f);
                *reinterpret_cast<float4 *>(src + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    }
    if (t == 0) *a.ticket = 0;
}

template <int NB>
cudaError_t configure_mlp_nb()
{
    cudaError_t e = allow_big_smem(mlp_decode_kernel<NB, 128>);
    if (e == cudaSuccess) e = allow_big_smem(mlp_decode_kernel<NB, 256>);
    if (e == cudaSuccess) e = allow_big_smem(mlp_decode_kernel<NB, 384>);
    if (e == cudaSuccess) e = allow_big_smem(mlp_decode_kernel<NB, 512>);
    if (e == cudaSuccess) e = allow_big_smem(mlp_decode_kernel<NB, 768>);
    return e;
}

template <int NB>
int launch_mlp_nb(Ctx *c, const MlpArgs &a, cudaStream_t st)
{
    constexpr int R = RowsPerGroup<NB>::value;
    const int threads = ((a.D / 8) + 31) / 32 * 32;
    const StreamSmemLayout lay = stream_smem_layout(a.D, R, NB, threads / 32);
    if (lay.nslot < 2) return FASTTPS_INVALID_ARG;
    const int n_oct = a.K / 8;
    int grid = c->n_sm;
    if (grid > n_oct) grid = n_oct;
    while ((n_oct + grid - 1) / grid > kMaxOctetsPerCta) grid *= 2;   // tiny GPUs / huge K only
    ProfScope prof(c, kProfMlp, st);
    int rc;
    if (threads <= 128) rc = launch_stream_kernel(mlp_decode_kernel<NB, 128>, grid, threads, lay.total, st, &a);
    else if (threads <= 256) rc = launch_stream_kernel(mlp_decode_kernel<NB, 256>, grid, threads, lay.total, st, &a);
    else if (threads <= 384) rc = launch_stream_kernel(mlp_decode_kernel<NB, 384>, grid, threads, lay.total, st, &a);
    else if (threads <= 512) rc = launch_stream_kernel(mlp_decode_kernel<NB, 512>, grid, threads, lay.total, st, &a);
    else rc = launch_stream_kernel(mlp_decode_kernel<NB, 768>, grid, threads, lay.total, st, &a);
    c->launches++;
    return rc;
}

}  // namespace

int configure_mlp_kernels()
{
    FT_CUDA(configure_mlp_nb<1>());
    FT_CUDA(configure_mlp_nb<2>());
    FT_CUDA(configure_mlp_nb<4>());
    FT_CUDA(configure_mlp_nb<8>());
    return FASTTPS_OK;
}

// Batches above kMaxNB are served in tiles of kMaxNB rows (the weights are re-read per tile).
int launch_mlp(Ctx *c, const MlpArgs &a0, cudaStream_t st)
{
    for (int b0 = 0; b0 < a0.batch; b0 += kMaxNB) {
        MlpArgs a = a0;
        a.batch = a0.batch - b0 < kMaxNB ? a0.batch - b0 : kMaxNB;
        a.x = a0.x + (size_t)b0 * a0.D;
        if (a.res) a.res = a0.res + (size_t)b0 * a0.D;
        a.out = a0.out + (size_t)b0 * a0.D;
        a.acc = a0.acc + (size_t)b0 * a0.D;
        int rc;
        if (a.batch == 1) rc = launch_mlp_nb<1>(c, a, st);
        else if (a.batch == 2) rc = launch_mlp_nb<2>(c, a, st);
        else if (a.batch <= 4) rc = launch_mlp_nb<4>(c, a, st);
        else rc = launch_mlp_nb<8>(c, a, st);
        if (rc != FASTTPS_OK) return rc;
    }
    return FASTTPS_OK;
}

}  // namespace fasttps
