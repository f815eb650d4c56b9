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
// Both weight streams are strictly sequential per CTA.
#include "dot_core.cuh"

namespace fasttps {

namespace {

constexpr int kMaxOctetsPerCta = 16;      // bounds the shared-memory intermediate

template <int NB> struct DownUnroll { static constexpr int value = (NB <= 2) ? 8 : 4; };

template <int NB, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) mlp_decode_kernel(MlpArgs a)
{
    constexpr int U = DownUnroll<NB>::value;
    extern __shared__ float smem[];                         // reduction scratch of dot_rows
    __shared__ float s_gu[kMaxOctetsPerCta * 16][NB];       // gate/up values of this CTA's rows
    __shared__ float s_act[kMaxOctetsPerCta * 8][NB];       // silu(gate) * up
    __shared__ int s_last;

    const int t = threadIdx.x;
    const int n_oct = a.K >> 3;
    const int base = n_oct / gridDim.x, rem = n_oct % gridDim.x;
    const int cta = blockIdx.x;
    const int oct0 = cta * base + (cta < rem ? cta : rem);
    const int noct = base + (cta < rem ? 1 : 0);
    const bool active = t * 8 < a.D;

    // ---- Algorithm 4 step 1 (optional): RMSNorm of the block input ----
    float x[NB][8];
    load_activations<NB>(x, a.x, a.D, a.batch, a.D, a.g, a.eps, smem);

    // ---- steps 2-10: interlaced gate_up product for rows [16*oct0, 16*(oct0+noct)) ----
    const int row0 = oct0 * 16;
    dot_rows<NB>(a.w_gu, a.D, row0, row0 + noct * 16, x, smem,
                 [&](int row, int b, float v) { s_gu[row - row0][b] = v; });
    __syncthreads();

    // ---- step 11: siLu_Mul (first half of an interlaced block is gate, second half up) ----
    for (int i = t; i < noct * 8 * NB; i += blockDim.x) {
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
    const uint4 *Wd = reinterpret_cast<const uint4 *>(a.w_down) + (size_t)oct0 * 8 * nvec + t;
    const int nj = noct * 8;                                // multiple of 8, hence of U
    if (active) {
        uint4 wa[U], wb[U];
        auto load = [&](uint4 (&w)[U], int j0) {
#pragma unroll
            for (int u = 0; u < U; ++u) w[u] = ldg_stream(Wd + (size_t)(j0 + u) * nvec);
        };
        auto fma_rows = [&](const uint4 (&w)[U], int j0) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float wf[8];
                unpack8(w[u], wf);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const float av = s_act[j0 + u][b];
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[b][i] = fmaf(av, wf[i], acc[b][i]);
                }
            }
        };
        if (nj > 0) load(wa, 0);
        for (int j0 = 0; j0 < nj; j0 += 2 * U) {
            if (j0 + U < nj) load(wb, j0 + U);
            fma_rows(wa, j0);
            if (j0 + U < nj) {
                if (j0 + 2 * U < nj) load(wa, j0 + 2 * U);
                fma_rows(wb, j0 + U);
            }
        }
        // ---- partial sums of all CTAs meet in the FP32 accumulator ----
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
int launch_mlp_nb(Ctx *c, const MlpArgs &a, cudaStream_t st)
{
    constexpr int R = RowsPerGroup<NB>::value;
    const int threads = ((a.D / 8) + 31) / 32 * 32;
    const int nwarps = threads / 32;
    const int n_oct = a.K / 8;
    int grid = c->n_sm;
    if (grid > n_oct) grid = n_oct;
    while ((n_oct + grid - 1) / grid > kMaxOctetsPerCta) grid *= 2;   // tiny GPUs / huge K only
    size_t smem = sizeof(float) * (size_t)(2 * nwarps * R * NB > 32 * NB ? 2 * nwarps * R * NB : 32 * NB);
    ProfScope prof(c, kProfMlp, st);
    if (threads <= 128) mlp_decode_kernel<NB, 128><<<grid, threads, smem, st>>>(a);
    else if (threads <= 256) mlp_decode_kernel<NB, 256><<<grid, threads, smem, st>>>(a);
    else if (threads <= 384) mlp_decode_kernel<NB, 384><<<grid, threads, smem, st>>>(a);
    else if (threads <= 512) mlp_decode_kernel<NB, 512><<<grid, threads, smem, st>>>(a);
    else mlp_decode_kernel<NB, 1024><<<grid, threads, smem, st>>>(a);
    c->launches++;
    FT_CUDA(cudaGetLastError());
    return FASTTPS_OK;
}

}  // namespace

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
