// The NON-fused token phase of the paper's starting point (Algorithm 1 "Standard Attention Implementation",
// Algorithm 2 "Standard MLP Implementation"), one plain kernel per operator, every intermediate through device
// memory, the KV cache updated by a Concat into a new buffer.  Comparison arm only: see include/fasttps_baseline.h.
// The kernels are straightforward but not naive (16-byte loads, a warp per output row in the projections, a lane
// group per cache row in the attention products), so that the measured gap is the cost of NOT fusing.
#include <cmath>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/fasttps_baseline.h"
#include "common.cuh"

namespace fasttps {

namespace {

// ---- Algorithm 1, Step 1: RoPE of one tensor [B, H, d] at the positions pos[b] (half-split pairing) ----
__global__ void base_rope_kernel(const __nv_bfloat16 *x, __nv_bfloat16 *y, const int32_t *pos, int H, int d, float theta)
{
    const int b = blockIdx.y, half = d >> 1;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;          // (h, i)
    if (idx >= H * half) return;
    const int h = idx / half, i = idx - h * half;
    const double ang = (double)pos[b] * pow((double)theta, -2.0 * (double)i / (double)d);
    const float c = (float)cos(ang), s = (float)sin(ang);
    const size_t o = ((size_t)b * H + h) * d;
    const float x0 = __bfloat162float(x[o + i]), x1 = __bfloat162float(x[o + i + half]);
    y[o + i] = __float2bfloat16_rn(__fsub_rn(__fmul_rn(x0, c), __fmul_rn(x1, s)));
    y[o + i + half] = __float2bfloat16_rn(__fadd_rn(__fmul_rn(x1, c), __fmul_rn(x0, s)));
}

// ---- Step 2: Transpose [B, N, H, d] -> [B, H, N, d]; with N = 1 new token the element order is unchanged ----
__global__ void base_transpose_kernel(const uint4 *x, uint4 *y, size_t nvec)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nvec) y[i] = x[i];
}

// ---- Step 3: Concat: cat[b, h, 0..L_b) = cache[b, h, 0..L_b), cat[b, h, L_b] = new[b, h] ----
__global__ void base_concat_kernel(const __nv_bfloat16 *cache, const __nv_bfloat16 *nw, __nv_bfloat16 *cat,
                                   const int32_t *seq_lens, int H, int max_seq, int cat_seq, int d)
{
    const int bh = blockIdx.y, b = bh / H, L = seq_lens[b];
    const int vpr = d >> 3;                                            // 16-byte vectors per row
    const size_t total = (size_t)(L + 1) * vpr;
    const uint4 *src = reinterpret_cast<const uint4 *>(cache + (size_t)bh * max_seq * d);
    const uint4 *srcn = reinterpret_cast<const uint4 *>(nw + (size_t)bh * d);
    uint4 *dst = reinterpret_cast<uint4 *>(cat + (size_t)bh * cat_seq * d);
    for (size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += (size_t)gridDim.x * blockDim.x)
        dst[v] = v < (size_t)L * vpr ? src[v] : srcn[v - (size_t)L * vpr];
}

// ---- Step 4: S[b, hq, j] = q . K[b, hk, j] / sqrt(d), j = 0 .. L_b; four lanes per row ----
__global__ void base_qk_kernel(const __nv_bfloat16 *q, const __nv_bfloat16 *kcat, float *s, const int32_t *seq_lens,
                               int Hq, int Hkv, int cat_seq, int d)
{
    const int bh = blockIdx.y, b = bh / Hq, hq = bh - b * Hq, hk = hq / (Hq / Hkv), L = seq_lens[b];
    const int lane = threadIdx.x & 31, sub = lane & 3;
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 2;
    const int epl = d >> 2;                                            // elements per lane
    float acc = 0.f;
    if (row <= L) {
        const __nv_bfloat16 *kr = kcat + (((size_t)b * Hkv + hk) * cat_seq + row) * d + sub * epl;
        const __nv_bfloat16 *qr = q + ((size_t)b * Hq + hq) * d + sub * epl;
        for (int i = 0; i < epl; i += 8) {
            float kf[8], qf[8];
            unpack8(*reinterpret_cast<const uint4 *>(kr + i), kf);
            unpack8(*reinterpret_cast<const uint4 *>(qr + i), qf);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc = fmaf(kf[e], qf[e], acc);
        }
    }
    acc += __shfl_xor_sync(kFull, acc, 1);
    acc += __shfl_xor_sync(kFull, acc, 2);
    if (row <= L && sub == 0) s[(size_t)bh * cat_seq + row] = acc / sqrtf((float)d);
}

// ---- Step 5: P = softmax(S) over j = 0 .. L_b; one CTA per (b, hq) ----
__global__ void base_softmax_kernel(const float *s, float *p, const int32_t *seq_lens, int Hq, int cat_seq)
{
    __shared__ float red[32];
    const int bh = blockIdx.x, b = bh / Hq, n = seq_lens[b] + 1;
    const float *sr = s + (size_t)bh * cat_seq;
    float *pr = p + (size_t)bh * cat_seq;
    const int t = threadIdx.x, lane = t & 31, w = t >> 5, nw = blockDim.x >> 5;
    float m = -INFINITY;
    for (int j = t; j < n; j += blockDim.x) m = fmaxf(m, sr[j]);
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, o));
    if (lane == 0) red[w] = m;
    __syncthreads();
    m = -INFINITY;
    for (int i = 0; i < nw; ++i) m = fmaxf(m, red[i]);
    __syncthreads();
    float sum = 0.f;
    for (int j = t; j < n; j += blockDim.x) sum += expf(sr[j] - m);
    sum = warp_sum(sum);
    if (lane == 0) red[w] = sum;
    __syncthreads();
    sum = 0.f;
    for (int i = 0; i < nw; ++i) sum += red[i];
    for (int j = t; j < n; j += blockDim.x) pr[j] = expf(sr[j] - m) / sum;
}

// ---- Step 6: O[b, hq, c] = sum_j P[j] V[b, hk, j, c]; one CTA per (b, hq); a thread owns one 16-byte vector of the
// row and every (blockDim / vectors-per-row)-th row, four rows in flight ----
__global__ void base_pv_kernel(const float *p, const __nv_bfloat16 *vcat, __nv_bfloat16 *out, const int32_t *seq_lens,
                               int Hq, int Hkv, int cat_seq, int d)
{
    extern __shared__ float part[];                                    // [row lanes][d]
    const int bh = blockIdx.x, b = bh / Hq, hq = bh - b * Hq, hk = hq / (Hq / Hkv), n = seq_lens[b] + 1;
    const int t = threadIdx.x, vpr = d >> 3, rpp = blockDim.x / vpr;   // rows per pass
    const int r = t / vpr, v = t - r * vpr;
    const float *pr = p + (size_t)bh * cat_seq;
    const __nv_bfloat16 *vb = vcat + ((size_t)b * Hkv + hk) * (size_t)cat_seq * d + v * 8;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (r < rpp) {
        int j = r;
        for (; j + 3 * rpp < n; j += 4 * rpp) {
            uint4 q4[4];
            float pj[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                q4[u] = ldg_stream(vb + (size_t)(j + u * rpp) * d);
                pj[u] = pr[j + u * rpp];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float f[8];
                unpack8(q4[u], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = fmaf(pj[u], f[e], acc[e]);
            }
        }
        for (; j < n; j += rpp) {
            float f[8];
            unpack8(ldg_stream(vb + (size_t)j * d), f);
            const float pj = pr[j];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(pj, f[e], acc[e]);
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) part[r * d + v * 8 + e] = acc[e];
    }
    __syncthreads();
    for (int c = t; c < d; c += blockDim.x) {
        float o = 0.f;
        for (int i = 0; i < rpp; ++i) o += part[i * d + c];
        out[((size_t)b * Hq + hq) * d + c] = __float2bfloat16_rn(o);
    }
}

// ---- Algorithm 2: projections with one warp per output row of the transposed matrix W^T [n_out][n_in]; NB batch
// rows share every weight vector, four weight vectors in flight per lane ----
template <int NB>
__global__ void base_gemv_kernel(const __nv_bfloat16 *x, const __nv_bfloat16 *wt, __nv_bfloat16 *y, int batch, int n_in, int n_out)
{
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (row >= n_out) return;
    const __nv_bfloat16 *wr = wt + (size_t)row * n_in;
    for (int b0 = 0; b0 < batch; b0 += NB) {                           // more rows than NB: the weights come from the L2 again
        float acc[NB];
#pragma unroll
        for (int bb = 0; bb < NB; ++bb) acc[bb] = 0.f;
        for (int k0 = lane * 8; k0 < n_in; k0 += 4 * 256) {
            uint4 wv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) wv[u] = k0 + u * 256 < n_in ? ldg_stream(wr + k0 + u * 256) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int k = k0 + u * 256;
                if (k >= n_in) break;
                float wf[8];
                unpack8(wv[u], wf);
#pragma unroll
                for (int bb = 0; bb < NB; ++bb) {
                    if (b0 + bb < batch) {
                        float xf[8];
                        unpack8(*reinterpret_cast<const uint4 *>(x + (size_t)(b0 + bb) * n_in + k), xf);
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[bb] = fmaf(wf[e], xf[e], acc[bb]);
                    }
                }
            }
        }
#pragma unroll
        for (int bb = 0; bb < NB; ++bb) {
            const float vsum = warp_sum(acc[bb]);
            if (lane == 0 && b0 + bb < batch) y[(size_t)(b0 + bb) * n_out + row] = __float2bfloat16_rn(vsum);
        }
    }
}

static void launch_base_gemv(const __nv_bfloat16 *x, const __nv_bfloat16 *wt, __nv_bfloat16 *y, int batch, int n_in, int n_out,
                             cudaStream_t st)
{
    const int grid = (n_out + 7) / 8;
    if (batch == 1) base_gemv_kernel<1><<<grid, 256, 0, st>>>(x, wt, y, batch, n_in, n_out);
    else if (batch <= 4) base_gemv_kernel<4><<<grid, 256, 0, st>>>(x, wt, y, batch, n_in, n_out);
    else base_gemv_kernel<8><<<grid, 256, 0, st>>>(x, wt, y, batch, n_in, n_out);
}

__global__ void base_silu_kernel(const __nv_bfloat16 *g, __nv_bfloat16 *s, size_t n)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { const float v = __bfloat162float(g[i]); s[i] = __float2bfloat16_rn(v / (1.f + expf(-v))); }
}

__global__ void base_mul_kernel(const __nv_bfloat16 *a, const __nv_bfloat16 *b, __nv_bfloat16 *m, size_t n)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) m[i] = __float2bfloat16_rn(__bfloat162float(a[i]) * __bfloat162float(b[i]));
}

// brackets each launch with events when the caller wants per-operator times
struct LaunchTimer {
    cudaStream_t st; float *out; int n = 0; cudaEvent_t ev[2 * 16];
    LaunchTimer(cudaStream_t s, float *o, int count) : st(s), out(o)
    {
        if (out) for (int i = 0; i < 2 * count; ++i) cudaEventCreate(&ev[i]);
    }
    void before() { if (out) cudaEventRecord(ev[2 * n], st); }
    void after() { if (out) cudaEventRecord(ev[2 * n + 1], st); ++n; }
    int finish()
    {
        if (!out) return FASTTPS_OK;
        FT_CUDA(cudaStreamSynchronize(st));
        for (int i = 0; i < n; ++i) {
            float ms = 0.f;
            FT_CUDA(cudaEventElapsedTime(&ms, ev[2 * i], ev[2 * i + 1]));
            out[i] = ms * 1000.f;
        }
        for (int i = 0; i < 2 * n; ++i) cudaEventDestroy(ev[i]);
        return FASTTPS_OK;
    }
};

inline bool al16(const void *p) { return p && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

}  // namespace fasttps

using namespace fasttps;

extern "C" int fasttps_baseline_attn(const fasttps_baseline_attn_shape *sh, const fasttps_baseline_attn_buffers *bf,
                                     const void *q, const void *k_new, const void *v_new, const void *k_cache,
                                     const void *v_cache, const int32_t *pos, const int32_t *seq_lens, void *out,
                                     float *launch_us, void *stream)
{
    if (!sh || !bf || !pos || !seq_lens) return FASTTPS_INVALID_ARG;
    const int B = sh->batch, Hq = sh->n_q_heads, Hkv = sh->n_kv_heads, d = sh->head_dim;
    if (B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv || d < 32 || d > 128 || d % 32 || sh->cat_seq < 1 || sh->max_seq < 1)
        return FASTTPS_INVALID_ARG;
    if (!al16(q) || !al16(k_new) || !al16(v_new) || !al16(k_cache) || !al16(v_cache) || !al16(out) || !al16(bf->q_rope) ||
        !al16(bf->k_rope) || !al16(bf->q_trans) || !al16(bf->k_trans) || !al16(bf->v_trans) || !al16(bf->k_cat) ||
        !al16(bf->v_cat) || !bf->s || !bf->p)
        return FASTTPS_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto B16 = [](const void *p) { return static_cast<const __nv_bfloat16 *>(p); };
    auto M16 = [](void *p) { return static_cast<__nv_bfloat16 *>(p); };
    LaunchTimer tm(st, launch_us, 10);
    const int half = d / 2;
    // Step 1: RoPE, one operator call per tensor
    tm.before(); base_rope_kernel<<<dim3((Hq * half + 127) / 128, B), 128, 0, st>>>(B16(q), M16(bf->q_rope), pos, Hq, d, sh->rope_theta); tm.after();
    tm.before(); base_rope_kernel<<<dim3((Hkv * half + 127) / 128, B), 128, 0, st>>>(B16(k_new), M16(bf->k_rope), pos, Hkv, d, sh->rope_theta); tm.after();
    // Step 2: Transpose of Q_rope, K_rope, V
    const size_t nq = (size_t)B * Hq * d / 8, nk = (size_t)B * Hkv * d / 8;
    tm.before(); base_transpose_kernel<<<(unsigned)((nq + 255) / 256), 256, 0, st>>>(static_cast<const uint4 *>(bf->q_rope), static_cast<uint4 *>(bf->q_trans), nq); tm.after();
    tm.before(); base_transpose_kernel<<<(unsigned)((nk + 255) / 256), 256, 0, st>>>(static_cast<const uint4 *>(bf->k_rope), static_cast<uint4 *>(bf->k_trans), nk); tm.after();
    tm.before(); base_transpose_kernel<<<(unsigned)((nk + 255) / 256), 256, 0, st>>>(static_cast<const uint4 *>(v_new), static_cast<uint4 *>(bf->v_trans), nk); tm.after();
    // Step 3: Concat of K and of V into new buffers
    const dim3 cgrid(64, B * Hkv);
    tm.before(); base_concat_kernel<<<cgrid, 256, 0, st>>>(B16(k_cache), B16(bf->k_trans), M16(bf->k_cat), seq_lens, Hkv, sh->max_seq, sh->cat_seq, d); tm.after();
    tm.before(); base_concat_kernel<<<cgrid, 256, 0, st>>>(B16(v_cache), B16(bf->v_trans), M16(bf->v_cat), seq_lens, Hkv, sh->max_seq, sh->cat_seq, d); tm.after();
    // Steps 4-6
    tm.before(); base_qk_kernel<<<dim3((sh->cat_seq * 4 + 255) / 256, B * Hq), 256, 0, st>>>(B16(bf->q_trans), B16(bf->k_cat), bf->s, seq_lens, Hq, Hkv, sh->cat_seq, d); tm.after();
    tm.before(); base_softmax_kernel<<<B * Hq, 256, 0, st>>>(bf->s, bf->p, seq_lens, Hq, sh->cat_seq); tm.after();
    const int pv_threads = 512, pv_rpp = pv_threads / (d / 8);
    tm.before(); base_pv_kernel<<<B * Hq, pv_threads, (size_t)pv_rpp * d * sizeof(float), st>>>(bf->p, B16(bf->v_cat), M16(out), seq_lens, Hq, Hkv, sh->cat_seq, d); tm.after();
    FT_CUDA(cudaGetLastError());
    return tm.finish();
}

extern "C" int fasttps_baseline_mlp(int batch, int hidden, int inter, const fasttps_baseline_mlp_buffers *bf, const void *x,
                                    const void *wt_gate, const void *wt_up, const void *wt_down, void *out, float *launch_us,
                                    void *stream)
{
    if (!bf || batch < 1 || hidden < 8 || inter < 8 || hidden % 8 || inter % 8) return FASTTPS_INVALID_ARG;
    if (!al16(x) || !al16(wt_gate) || !al16(wt_up) || !al16(wt_down) || !al16(out) || !al16(bf->h_g) || !al16(bf->h_s) ||
        !al16(bf->h_u) || !al16(bf->h_m))
        return FASTTPS_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto B16 = [](const void *p) { return static_cast<const __nv_bfloat16 *>(p); };
    auto M16 = [](void *p) { return static_cast<__nv_bfloat16 *>(p); };
    LaunchTimer tm(st, launch_us, 5);
    const size_t n = (size_t)batch * inter;
    const unsigned eg = (unsigned)((n + 255) / 256);
    tm.before(); launch_base_gemv(B16(x), B16(wt_gate), M16(bf->h_g), batch, hidden, inter, st); tm.after();
    tm.before(); base_silu_kernel<<<eg, 256, 0, st>>>(B16(bf->h_g), M16(bf->h_s), n); tm.after();
    tm.before(); launch_base_gemv(B16(x), B16(wt_up), M16(bf->h_u), batch, hidden, inter, st); tm.after();
    tm.before(); base_mul_kernel<<<eg, 256, 0, st>>>(B16(bf->h_u), B16(bf->h_s), M16(bf->h_m), n); tm.after();
    tm.before(); launch_base_gemv(B16(bf->h_m), B16(wt_down), M16(out), batch, inter, hidden, st); tm.after();
    FT_CUDA(cudaGetLastError());
    return tm.finish();
}
