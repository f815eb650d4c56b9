// Fully fused SwiGLU MLP for decode (Algorithm 4 / Eq. 1 / Eq. 31 of the paper).
//
// The paper fuses gate and up into one interlaced Matmul with a siLu_Mul epilogue and
// sends the intermediate through L3 to a separate down projection.  Here the intermediate
// never leaves the SM: a CTA owns a contiguous range of j-octets (8 intermediate columns
// each).  For its range it
//   1. streams one 16-row tile per octet of the packed gate_up matrix (8 gate rows, then the
//      8 matching up rows) and multiplies it with the activations on the tensor cores; the
//      accumulator fragment of a lane holds a gate value and ITS up value (rows g and g + 8),
//   2. applies a = silu(gate) * up and keeps a as a bf16 hi + lo pair in shared memory,
//   3. streams the matching octets of the packed W_down (m16n8k8 fragments: 32 output columns
//      x 8 intermediate columns per 512-byte block) and accumulates y^T[n, b] in registers,
//      each warp owning a fixed set of output columns,
//   4. adds its partial y into an FP32 accumulator in global memory (vector red.add); the
//      CTA that arrives last adds the residual, rounds to bf16 and re-zeroes the accumulator.
// Both weight slices of a CTA are contiguous byte ranges and go through ONE shared-memory
// ring fed by a producer warp, so the W_down octets are already in flight while the gate_up
// reduction and the SiLU step are still running.
#include "mlp_core.cuh"
#include "stream_launch.cuh"

namespace fasttps {

namespace {

template <int IPW, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) mlp_decode_kernel(MlpArgs a)
{
    extern __shared__ __align__(128) unsigned char dsm[];
    __shared__ __align__(16) ActTile s_hi[kMaxOctetsPerCta];   // [octet][batch row][j in octet]
    __shared__ __align__(16) ActTile s_lo[kMaxOctetsPerCta];
    __shared__ int s_last;

    const int t = threadIdx.x;
    const StreamSmemLayout lay = stream_smem_layout(a.D);
    const int nw = lay.nw, nct = nw * 32;
    float *smem_part = reinterpret_cast<float *>(dsm + lay.part_off);
    float *smem_red = reinterpret_cast<float *>(dsm + lay.red_off);

    const int n_oct = a.K >> 3;
    const int base = n_oct / gridDim.x, rem = n_oct % gridDim.x;
    const int cta = blockIdx.x;
    const int oct0 = cta * base + (cta < rem ? cta : rem);
    const int noct = base + (cta < rem ? 1 : 0);
    const size_t gu_tile_bytes = (size_t)a.D * 32;      // 16 rows x D
    const size_t dn_oct_bytes = (size_t)a.D * 16;       // 8 rows x D

    // both weight slices of this CTA, back to back through one ring
    WeightRing ring;
    ring.init(dsm + lay.ring_off, reinterpret_cast<uint64_t *>(dsm + lay.bar_off),
              reinterpret_cast<int *>(dsm + lay.abort_off), lay.nslot, lay.slot_bytes, nw,
              reinterpret_cast<const unsigned char *>(a.w_gu) + (size_t)oct0 * gu_tile_bytes, (long long)noct * gu_tile_bytes,
              reinterpret_cast<const unsigned char *>(a.w_down) + (size_t)oct0 * dn_oct_bytes, (long long)noct * dn_oct_bytes);
    __syncthreads();
    if (t >= nct) {
        if (t == nct) ring.produce();
        return;
    }

    // everything below reads what the previous kernel wrote, or writes what it may still read
    pdl_wait();
    pdl_launch_dependents();

    // ---- Algorithm 4 step 1 (optional): RMSNorm of the block input, as MMA B fragments ----
    uint32_t bf[IPW][4];
    load_b_frags<IPW>(bf, a.x, a.D, a.batch, a.D, nw, a.g, a.eps, smem_red);

    // ---- steps 2-11: interlaced gate_up product, then siLu_Mul on the finished sums ----
    bool ok = mlp_gate_up_phase<IPW>(ring, 0, noct, nw, bf, smem_part, s_hi, s_lo);
    if (!ok) {
        if (t == 0) atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT);
        return;
    }
    named_bar_sync(1, nct);

    // ---- steps 13-15: down projection of this CTA's slice of the intermediate ----
    float acc[IPW][2][4];
#pragma unroll
    for (int i = 0; i < IPW; ++i)
#pragma unroll
        for (int m = 0; m < 2; ++m)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][m][e] = 0.f;
    mlp_down_phase<IPW>(ring, ring.pieces0, noct, nw, s_hi, s_lo, acc, ok);
    if (!named_bar_and(1, nct, ok)) {                       // also: every warp is done with the ring
        if (t == 0) atomicOr(a.status, FASTTPS_DEV_WAIT_TIMEOUT);
        return;
    }
    // ---- partial y -> shared memory -> vector red.add ----
    mlp_scatter_add<IPW>(acc, a.acc, a.batch, a.D, nw);
    __threadfence();
    named_bar_sync(1, nct);
    if (t == 0) s_last = (atomicAdd(a.ticket, 1) == (int)gridDim.x - 1);
    named_bar_sync(1, nct);
    if (!s_last) return;
    __threadfence();
    // last CTA: y (+ residual) -> bf16, accumulator back to zero for the next call
    const int nvec8 = a.batch * (a.D >> 3);
    for (int idx = t; idx < nvec8; idx += nct) {
        float *src = a.acc + (size_t)idx * 8;
        float4 y0, y1;
        asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(y0.x), "=f"(y0.y), "=f"(y0.z), "=f"(y0.w) : "l"(src));
        asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(y1.x), "=f"(y1.y), "=f"(y1.z), "=f"(y1.w) : "l"(src + 4));
        float r[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (a.res) unpack8(*reinterpret_cast<const uint4 *>(a.res + (size_t)idx * 8), r);
        uint4 o;
        o.x = pack2(y0.x + r[0], y0.y + r[1]);
        o.y = pack2(y0.z + r[2], y0.w + r[3]);
        o.z = pack2(y1.x + r[4], y1.y + r[5]);
        o.w = pack2(y1.z + r[6], y1.w + r[7]);
        *reinterpret_cast<uint4 *>(a.out + (size_t)idx * 8) = o;
        *reinterpret_cast<float4 *>(src) = make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4 *>(src + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (t == 0) *a.ticket = 0;
}

}  // namespace

int configure_mlp_kernels()
{
    FT_CUDA(allow_big_smem(mlp_decode_kernel<4, 416>));
    FT_CUDA(allow_big_smem(mlp_decode_kernel<4, 800>));
    FT_CUDA(allow_big_smem(mlp_decode_kernel<8, 416>));
    FT_CUDA(allow_big_smem(mlp_decode_kernel<8, 544>));
    FT_CUDA(allow_big_smem(mlp_decode_kernel<8, 800>));
    return FASTTPS_OK;
}

static int launch_mlp_tile(Ctx *c, const MlpArgs &a, cudaStream_t st)
{
    const StreamSmemLayout lay = stream_smem_layout(a.D);
    if (lay.nw < 1 || lay.nslot < 2) return FASTTPS_INVALID_ARG;
    const int threads = (lay.nw + 1) * 32;
    const int n_oct = a.K / 8;
    int grid = c->n_sm;
    if (grid > n_oct) grid = n_oct;
    while ((n_oct + grid - 1) / grid > kMaxOctetsPerCta) grid *= 2;   // tiny GPUs / huge K only
    ProfScope prof(c, kProfMlp, st);
    int rc;
    if (lay.ipw == 8)
        // 17 warps (hidden 4096: 16 consumer warps) get a register budget of their own: under the 800-thread bound a
        // thread has 72 registers and the tile loops spill
        rc = threads <= 416   ? launch_stream_kernel(mlp_decode_kernel<8, 416>, grid, threads, lay.total, st, &a)
             : threads <= 544 ? launch_stream_kernel(mlp_decode_kernel<8, 544>, grid, threads, lay.total, st, &a)
                              : launch_stream_kernel(mlp_decode_kernel<8, 800>, grid, threads, lay.total, st, &a);
    else
        rc = threads <= 416 ? launch_stream_kernel(mlp_decode_kernel<4, 416>, grid, threads, lay.total, st, &a)
                            : launch_stream_kernel(mlp_decode_kernel<4, 800>, grid, threads, lay.total, st, &a);
    c->launches++;
    return rc;
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
        const int rc = launch_mlp_tile(c, a, st);
        if (rc != FASTTPS_OK) return rc;
    }
    return FASTTPS_OK;
}

}  // namespace fasttps
