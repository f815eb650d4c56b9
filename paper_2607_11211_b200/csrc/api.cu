// C ABI of the FastTPS decode library: context, argument checks and the launch chains.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

namespace fasttps {

static thread_local char g_last_error[512] = "";

void set_last_error(cudaError_t e, const char *where)
{
    snprintf(g_last_error, sizeof g_last_error, "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
}

void set_last_error_text(const char *msg) { snprintf(g_last_error, sizeof g_last_error, "%s", msg); }

bool pdl_enabled()
{
    static const bool on = [] {
        const char *e = getenv("FASTTPS_PDL");
        return !(e && e[0] == '0');
    }();
    return on;
}

static bool aligned16(const void *p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static bool config_ok(const fasttps_config &f)
{
    if (f.hidden <= 0 || f.hidden > 6144 || !reduction_length_ok(f.hidden)) return false;
    if (f.head_dim != 32 && f.head_dim != 64 && f.head_dim != 96 && f.head_dim != 128) return false;
    if (f.n_q_heads <= 0 || f.n_kv_heads <= 0 || f.n_q_heads % f.n_kv_heads) return false;
    if (f.n_q_heads * f.head_dim > 6144 || !reduction_length_ok(f.n_q_heads * f.head_dim)) return false;
    if (f.inter <= 0 || f.inter % 8) return false;
    if (f.vocab < 0 || f.n_layers < 0 || f.max_batch < 1 || f.max_seq < 1) return false;
    if (!(f.rms_eps >= 0.f) || !(f.rope_theta > 0.f)) return false;
    return true;
}

template <class T>
static cudaError_t dev_alloc(T **p, size_t n, bool zero)
{
    cudaError_t e = cudaMalloc(reinterpret_cast<void **>(p), n * sizeof(T) ? n * sizeof(T) : 16);
    if (e == cudaSuccess && zero) e = cudaMemset(*p, 0, n * sizeof(T) ? n * sizeof(T) : 16);
    return e;
}

static void free_all(Ctx *c)
{
    cudaFree(c->cos_tab); cudaFree(c->sin_tab); cudaFree(c->attn_part); cudaFree(c->attn_ticket);
    cudaFree(c->mlp_acc); cudaFree(c->mlp_ticket); cudaFree(c->amax_val); cudaFree(c->amax_idx);
    cudaFree(c->amax_ticket); cudaFree(c->status); cudaFree(c->qkv); cudaFree(c->attn_out);
    cudaFree(c->h); cudaFree(c->xa); cudaFree(c->xb); cudaFree(c->logits); cudaFree(c->tok); cudaFree(c->tok2);
    if (c->pinned_tok) cudaFreeHost(c->pinned_tok);
    cudaFree(c->grid_bar); cudaFree(c->hacc);
    cudaFree(c->wide_n); cudaFree(c->wide_a_hi); cudaFree(c->wide_a_lo);
    if (c->prof_ev) {
        for (int i = 0; i < 2 * kProfMax; ++i) if (c->prof_ev[i]) cudaEventDestroy(c->prof_ev[i]);
        delete[] c->prof_ev;
    }
    delete[] c->prof_cls;
}

}  // namespace fasttps

using namespace fasttps;

extern "C" {

int fasttps_create(fasttps_ctx **out, const fasttps_config *cfg)
{
    if (!out || !cfg || !config_ok(*cfg)) return FASTTPS_INVALID_ARG;
    *out = nullptr;
    int ndev = 0;
    FT_CUDA(cudaGetDeviceCount(&ndev));
    if (cfg->device < 0 || cfg->device >= ndev) return FASTTPS_INVALID_ARG;
    FT_CUDA(cudaSetDevice(cfg->device));
    Ctx *c = new (std::nothrow) Ctx();
    if (!c) return FASTTPS_OUT_OF_MEMORY;
    memset(c, 0, sizeof *c);
    c->cfg = *cfg;
    FT_CUDA(cudaGetDeviceProperties(&c->prop, cfg->device));
    c->n_sm = c->prop.multiProcessorCount;
    {
        const char *e = getenv("FASTTPS_STEP_KERNEL");
        c->opt_step_kernel = (e && *e) ? atoi(e) != 0 : 1;
    }
    c->opt_gqa_share = 1;
    {
        int rc = configure_attn_kernels();
        if (rc == FASTTPS_OK) rc = configure_linear_kernels();
        if (rc == FASTTPS_OK) rc = configure_mlp_kernels();
        if (rc == FASTTPS_OK) rc = configure_wide_kernels();
        if (rc != FASTTPS_OK) { delete c; return rc; }
    }

    const fasttps_config &f = c->cfg;
    const size_t B = f.max_batch, D = f.hidden, half = f.head_dim / 2;
    const size_t nq = (size_t)f.n_q_heads * f.head_dim, nqkv = nq + 2 * (size_t)f.n_kv_heads * f.head_dim;
    cudaError_t e = cudaSuccess;
    auto A = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
    A(dev_alloc(&c->cos_tab, (size_t)f.max_seq * half, false));
    A(dev_alloc(&c->sin_tab, (size_t)f.max_seq * half, false));
    A(dev_alloc(&c->attn_part, B * f.n_q_heads * kMaxSplits * (f.head_dim + 4), true));
    A(dev_alloc(&c->attn_ticket, B * f.n_q_heads, true));
    A(dev_alloc(&c->mlp_acc, 2 * B * D, true));
    A(dev_alloc(&c->grid_bar, kGridBarWords, true));
    A(dev_alloc(&c->hacc, 2 * B * D, true));
    A(dev_alloc(&c->mlp_ticket, 1, true));
    A(dev_alloc(&c->amax_val, (size_t)kWideMaxB * 1024, true));
    A(dev_alloc(&c->amax_idx, (size_t)kWideMaxB * 1024, true));
    if (f.max_batch > kMaxNB) {
        A(dev_alloc(&c->wide_n, wide_x_elems((int)(nq > D ? nq : D)), true));
        A(dev_alloc(&c->wide_a_hi, wide_a_elems(f.inter), true));
        A(dev_alloc(&c->wide_a_lo, wide_a_elems(f.inter), true));
    }
    A(dev_alloc(&c->amax_ticket, 1, true));
    A(dev_alloc(&c->status, 1, true));
    A(dev_alloc(&c->qkv, B * nqkv, true));
    A(dev_alloc(&c->attn_out, B * nq, true));
    A(dev_alloc(&c->h, B * D, true));
    A(dev_alloc(&c->xa, B * D, true));
    A(dev_alloc(&c->xb, B * D, true));
    A(dev_alloc(&c->logits, B * (size_t)f.vocab, true));
    A(dev_alloc(&c->tok, B, true));
    A(dev_alloc(&c->tok2, B, true));
    if (e == cudaSuccess) e = cudaMallocHost(reinterpret_cast<void **>(&c->pinned_tok), 2 * B * sizeof(int32_t));
    if (e != cudaSuccess) {
        set_last_error(e, "fasttps_create: workspace allocation");
        free_all(c);
        delete c;
        (void)cudaGetLastError();
        return e == cudaErrorMemoryAllocation ? FASTTPS_OUT_OF_MEMORY : FASTTPS_CUDA_ERROR;
    }
    // RoPE table: angle = pos * theta^(-2i/d) in double, cos/sin rounded once to FP32
    std::vector<float> hc((size_t)f.max_seq * half), hs((size_t)f.max_seq * half);
    for (size_t i = 0; i < half; ++i) {
        const double inv_freq = std::pow((double)f.rope_theta, -2.0 * (double)i / (double)f.head_dim);
        for (int p = 0; p < f.max_seq; ++p) {
            const double ang = (double)p * inv_freq;
            hc[(size_t)p * half + i] = (float)std::cos(ang);
            hs[(size_t)p * half + i] = (float)std::sin(ang);
        }
    }
    e = cudaMemcpy(c->cos_tab, hc.data(), hc.size() * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(c->sin_tab, hs.data(), hs.size() * sizeof(float), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        set_last_error(e, "fasttps_create: table upload");
        free_all(c);
        delete c;
        return FASTTPS_CUDA_ERROR;
    }
    *out = reinterpret_cast<fasttps_ctx *>(c);
    return FASTTPS_OK;
}

int fasttps_destroy(fasttps_ctx *ctx)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    cudaSetDevice(c->cfg.device);
    cudaDeviceSynchronize();
    free_all(c);
    delete c;
    return FASTTPS_OK;
}

size_t fasttps_packed_bytes(const fasttps_ctx *ctx, int kind)
{
    if (!ctx) return 0;
    return 2 * packed_elems(reinterpret_cast<const Ctx *>(ctx)->cfg, kind);
}

int fasttps_pack_weight(fasttps_ctx *ctx, int kind, const void *src, void *dst, void *stream)
{
    if (!ctx || !aligned16(src) || !aligned16(dst) || src == dst) return FASTTPS_INVALID_ARG;
    return launch_pack(reinterpret_cast<Ctx *>(ctx), kind, src, dst, false, static_cast<cudaStream_t>(stream));
}

int fasttps_unpack_weight(fasttps_ctx *ctx, int kind, const void *src, void *dst, void *stream)
{
    if (!ctx || !aligned16(src) || !aligned16(dst) || src == dst) return FASTTPS_INVALID_ARG;
    return launch_pack(reinterpret_cast<Ctx *>(ctx), kind, src, dst, true, static_cast<cudaStream_t>(stream));
}

int fasttps_attn_splits(const fasttps_ctx *ctx, int batch)
{
    if (!ctx || batch < 1) return FASTTPS_INVALID_ARG;
    return attn_splits_for(reinterpret_cast<const Ctx *>(ctx), batch);
}

// batch: token rows (sequences x n_new); pos / seq_lens and the caches are per sequence
static int attn_impl(Ctx *c, const __nv_bfloat16 *q, const __nv_bfloat16 *k, const __nv_bfloat16 *v,
                     int q_stride, int kv_stride, void *k_cache, void *v_cache, const int32_t *pos,
                     const int32_t *seq_lens, __nv_bfloat16 *out, int out_stride, int batch, cudaStream_t st, int n_new = 1,
                     int out_chunked = 0, bool fp8 = false, float k_scale = 1.f, float v_scale = 1.f)
{
    const fasttps_config &f = c->cfg;
    AttnArgs a;
    a.q = q; a.k_new = k; a.v_new = v;
    a.q_stride = q_stride; a.kv_stride = kv_stride;
    a.k_cache = static_cast<__nv_bfloat16 *>(k_cache);
    a.v_cache = static_cast<__nv_bfloat16 *>(v_cache);
    a.pos = pos; a.seq_lens = seq_lens;
    a.out = out; a.out_stride = out_stride; a.out_chunked = out_chunked;
    a.batch = batch; a.n_q_heads = f.n_q_heads; a.n_kv_heads = f.n_kv_heads;
    a.head_dim = f.head_dim; a.max_seq = f.max_seq;
    a.n_splits = attn_splits_for(c, batch);
    a.len_add = 0; a.n_new = n_new;
    a.cos_tab = c->cos_tab; a.sin_tab = c->sin_tab;
    a.part = c->attn_part; a.ticket = c->attn_ticket; a.status = c->status;
    a.k_scale = k_scale; a.v_scale = v_scale;
    return launch_attn(c, a, st, fp8);
}

int fasttps_attn_decode(fasttps_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                        void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens,
                        void *out, int batch, void *stream)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (batch < 1 || batch > c->cfg.max_batch) return FASTTPS_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(out) || !pos || !seq_lens)
        return FASTTPS_INVALID_ARG;
    const fasttps_config &f = c->cfg;
    return attn_impl(c, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k_new),
                     static_cast<const __nv_bfloat16 *>(v_new), f.n_q_heads * f.head_dim, f.n_kv_heads * f.head_dim,
                     k_cache, v_cache, pos, seq_lens, static_cast<__nv_bfloat16 *>(out), f.n_q_heads * f.head_dim,
                     batch, static_cast<cudaStream_t>(stream));
}

int fasttps_attn_decode_fp8(fasttps_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                            void *k_cache, void *v_cache, float k_scale, float v_scale, const int32_t *pos,
                            const int32_t *seq_lens, void *out, int batch, void *stream)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (batch < 1 || batch > c->cfg.max_batch) return FASTTPS_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(out) || !pos || !seq_lens)
        return FASTTPS_INVALID_ARG;
    if (!(k_scale > 0.f) || !(v_scale > 0.f) || std::isinf(k_scale) || std::isinf(v_scale)) return FASTTPS_INVALID_ARG;
    const fasttps_config &f = c->cfg;
    return attn_impl(c, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k_new),
                     static_cast<const __nv_bfloat16 *>(v_new), f.n_q_heads * f.head_dim, f.n_kv_heads * f.head_dim,
                     k_cache, v_cache, pos, seq_lens, static_cast<__nv_bfloat16 *>(out), f.n_q_heads * f.head_dim,
                     batch, static_cast<cudaStream_t>(stream), 1, 0, /*fp8=*/true, k_scale, v_scale);
}

// ---- thin-GEMM chain for batches above kMaxNB: every weight is read once for up to kWideMaxB rows ----

static int wide_prep(Ctx *c, const __nv_bfloat16 *x, int x_stride, float *acc, const __nv_bfloat16 *g,
                     __nv_bfloat16 *x_store, __nv_bfloat16 *n_out, int D, int batch, int prof_class, cudaStream_t st)
{
    PrepArgs p;
    p.x = x; p.x_stride = x_stride; p.acc = acc; p.g = g; p.eps = c->cfg.rms_eps;
    p.x_store = x_store; p.n_out = n_out; p.D = D; p.batch = batch;
    return launch_prep_rows(c, p, prof_class, st);
}

// x: chunked activations (c->wide_n)
static WideArgs wide_args(Ctx *c, const __nv_bfloat16 *x, const void *w, int K, int n_out, int batch)
{
    WideArgs a;
    a.x = x; a.w = static_cast<const __nv_bfloat16 *>(w);
    a.K = K; a.n_out = n_out; a.batch = batch; a.epi = kWideStore;
    a.res = nullptr; a.res_stride = 0; a.out_bf16 = nullptr; a.out_f32 = nullptr; a.out_stride = n_out;
    a.pair_rows = 0; a.a_hi = nullptr; a.a_lo = nullptr;
    a.amax_val = c->amax_val; a.amax_idx = c->amax_idx; a.amax_ticket = c->amax_ticket;
    a.next_ids = nullptr; a.adv_pos = nullptr; a.adv_len = nullptr;
    a.status = c->status;
    return a;
}

// x [B][D] (normalised with gain g when given) -> gate_up with siLu_Mul -> down: the sums are left in c->mlp_acc
static int wide_mlp_sums(Ctx *c, const __nv_bfloat16 *x, const __nv_bfloat16 *g, const void *w_gu, const void *w_down,
                         int batch, cudaStream_t st)
{
    const fasttps_config &f = c->cfg;
    // the activations in chunked form, normalised on the way when a gain is given
    int rc = wide_prep(c, x, f.hidden, nullptr, g, nullptr, c->wide_n, f.hidden, batch, kProfMlp, st);
    if (rc) return rc;
    WideArgs a = wide_args(c, c->wide_n, w_gu, f.hidden, 2 * f.inter, batch);
    a.epi = kWideSilu; a.a_hi = c->wide_a_hi; a.a_lo = c->wide_a_lo;
    rc = launch_wide_linear(c, a, kProfMlp, st);
    if (rc) return rc;
    WideDownArgs d;
    d.a_hi = c->wide_a_hi; d.a_lo = c->wide_a_lo;
    d.w = static_cast<const __nv_bfloat16 *>(w_down);
    d.D = f.hidden; d.K = f.inter; d.batch = batch; d.acc = c->mlp_acc; d.status = c->status;
    return launch_wide_down(c, d, st);
}

static bool wide_batch(const Ctx *c, int batch) { return batch > kMaxNB && c->wide_n != nullptr; }

int fasttps_attn_decode_multi(fasttps_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                              void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens,
                              void *out, int batch, int n_new, void *stream)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (batch < 1 || n_new < 1 || n_new > kMaxNB || (long long)batch * n_new > c->cfg.max_batch) return FASTTPS_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(out) || !pos || !seq_lens)
        return FASTTPS_INVALID_ARG;
    const fasttps_config &f = c->cfg;
    return attn_impl(c, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k_new),
                     static_cast<const __nv_bfloat16 *>(v_new), f.n_q_heads * f.head_dim, f.n_kv_heads * f.head_dim,
                     k_cache, v_cache, pos, seq_lens, static_cast<__nv_bfloat16 *>(out), f.n_q_heads * f.head_dim,
                     batch * n_new, static_cast<cudaStream_t>(stream), n_new);
}

static int mlp_impl(Ctx *c, const __nv_bfloat16 *x, const __nv_bfloat16 *g, const void *w_gu, const void *w_down,
                    const __nv_bfloat16 *res, __nv_bfloat16 *out, int batch, cudaStream_t st)
{
    if (wide_batch(c, batch)) {
        const int D = c->cfg.hidden;
        for (int b0 = 0; b0 < batch; b0 += kWideMaxB) {
            const int nb = batch - b0 < kWideMaxB ? batch - b0 : kWideMaxB;
            int rc = wide_mlp_sums(c, x + (size_t)b0 * D, g, w_gu, w_down, nb, st);
            if (rc) return rc;
            // out = bf16(res + sums); the sums go back to zero
            rc = wide_prep(c, res ? res + (size_t)b0 * D : nullptr, D, c->mlp_acc, nullptr, out + (size_t)b0 * D, nullptr, D, nb,
                           kProfMlp, st);
            if (rc) return rc;
        }
        return FASTTPS_OK;
    }
    MlpArgs a;
    a.x = x; a.g = g; a.eps = c->cfg.rms_eps;
    a.w_gu = static_cast<const __nv_bfloat16 *>(w_gu);
    a.w_down = static_cast<const __nv_bfloat16 *>(w_down);
    a.res = res; a.out = out;
    a.D = c->cfg.hidden; a.K = c->cfg.inter; a.batch = batch;
    a.acc = c->mlp_acc; a.ticket = c->mlp_ticket; a.status = c->status;
    return launch_mlp(c, a, st);
}

int fasttps_mlp_decode(fasttps_ctx *ctx, const void *x, const void *w_gate_up, const void *w_down,
                       void *out, int batch, void *stream)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (batch < 1 || batch > c->cfg.max_batch) return FASTTPS_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w_gate_up) || !aligned16(w_down) || !aligned16(out)) return FASTTPS_INVALID_ARG;
    return mlp_impl(c, static_cast<const __nv_bfloat16 *>(x), nullptr, w_gate_up, w_down, nullptr,
                    static_cast<__nv_bfloat16 *>(out), batch, static_cast<cudaStream_t>(stream));
}

static int linear_impl(Ctx *c, int n_in, int n_out, const __nv_bfloat16 *x, int x_stride, const __nv_bfloat16 *g,
                       const void *w, const __nv_bfloat16 *res, int res_stride, __nv_bfloat16 *out_bf16,
                       float *out_f32, int out_stride, int batch, int32_t *next_ids, int32_t *adv_pos,
                       int32_t *adv_len, int prof_class, cudaStream_t st)
{
    if (wide_batch(c, batch)) {
        for (int b0 = 0; b0 < batch; b0 += kWideMaxB) {
            const int nb = batch - b0 < kWideMaxB ? batch - b0 : kWideMaxB;
            // the activations in chunked form; with a gain, RMSNorm on the way (rounded to bf16 like a stored tensor)
            int rc = wide_prep(c, x + (size_t)b0 * x_stride, x_stride, nullptr, g, nullptr, c->wide_n, n_in, nb, prof_class, st);
            if (rc) return rc;
            WideArgs a = wide_args(c, c->wide_n, w, n_in, n_out, nb);
            a.res = res ? res + (size_t)b0 * res_stride : nullptr; a.res_stride = res_stride;
            a.out_bf16 = out_bf16 ? out_bf16 + (size_t)b0 * out_stride : nullptr;
            a.out_f32 = out_f32 ? out_f32 + (size_t)b0 * out_stride : nullptr;
            a.out_stride = out_stride;
            a.pair_rows = prof_class == kProfOproj;
            a.next_ids = next_ids ? next_ids + b0 : nullptr;
            a.adv_pos = adv_pos ? adv_pos + b0 : nullptr;
            a.adv_len = adv_len ? adv_len + b0 : nullptr;
            rc = launch_wide_linear(c, a, prof_class, st);
            if (rc) return rc;
        }
        return FASTTPS_OK;
    }
    LinearArgs a;
    a.prof_class = prof_class;
    a.pair_rows = prof_class == kProfOproj;      // the output projection is the one product over the packed W_o
    a.status = c->status;
    a.x = x; a.x_stride = x_stride; a.g = g; a.eps = c->cfg.rms_eps;
    a.w = static_cast<const __nv_bfloat16 *>(w);
    a.res = res; a.res_stride = res_stride;
    a.out_bf16 = out_bf16; a.out_f32 = out_f32; a.out_stride = out_stride;
    a.n_in = n_in; a.n_out = n_out; a.batch = batch;
    a.amax_val = c->amax_val; a.amax_idx = c->amax_idx; a.amax_ticket = c->amax_ticket;
    a.next_ids = next_ids; a.adv_pos = adv_pos; a.adv_len = adv_len;
    return launch_linear(c, a, st);
}

int fasttps_linear_decode(fasttps_ctx *ctx, int kind, const void *x, const void *g_norm, const void *w,
                          const void *residual, void *out_bf16, float *out_f32, int batch, void *stream)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    const fasttps_config &f = c->cfg;
    if (batch < 1 || batch > f.max_batch) return FASTTPS_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || (g_norm && !aligned16(g_norm)) || (!out_bf16 && !out_f32))
        return FASTTPS_INVALID_ARG;
    int n_in, n_out;
    const int nq = f.n_q_heads * f.head_dim, nkv = f.n_kv_heads * f.head_dim;
    switch (kind) {
    case FASTTPS_W_QKV: n_in = f.hidden; n_out = nq + 2 * nkv; break;
    case FASTTPS_W_O: n_in = nq; n_out = f.hidden; break;
    case FASTTPS_W_LM_HEAD: n_in = f.hidden; n_out = f.vocab; break;
    default: return FASTTPS_INVALID_ARG;
    }
    if (n_out < 1) return FASTTPS_INVALID_ARG;
    return linear_impl(c, n_in, n_out, static_cast<const __nv_bfloat16 *>(x), n_in,
                       static_cast<const __nv_bfloat16 *>(g_norm), w, static_cast<const __nv_bfloat16 *>(residual),
                       n_out, static_cast<__nv_bfloat16 *>(out_bf16), out_f32, n_out, batch, nullptr, nullptr,
                       nullptr, kind == FASTTPS_W_QKV ? kProfQkv : kind == FASTTPS_W_O ? kProfOproj : kProfLmHead,
                       static_cast<cudaStream_t>(stream));
}

// One layer of the thin-GEMM chain for up to kWideMaxB token rows.  The layer input is x_res (+ the FP32 sums `pend`
// still to be folded in, which are cleared); it is materialised in x_store when given (it is the residual of the
// output projection: with pend it must be).  Leaves h in c->h and the MLP sums in c->mlp_acc: the caller's next
// prep folds them in (the input of the next layer, or the layer output).
static int layer_body_wide(Ctx *c, const fasttps_layer_weights &w, const __nv_bfloat16 *x_res, float *pend,
                           __nv_bfloat16 *x_store, void *k_cache, void *v_cache, const int32_t *pos,
                           const int32_t *seq_lens, int batch, int n_new, cudaStream_t st, bool fp8 = false,
                           float k_scale = 1.f, float v_scale = 1.f)
{
    const fasttps_config &f = c->cfg;
    const int D = f.hidden, nq = f.n_q_heads * f.head_dim, nkv = f.n_kv_heads * f.head_dim, nqkv = nq + 2 * nkv;
    const __nv_bfloat16 *resid = x_store ? x_store : x_res;
    // x = x_res + pend (stored), n1 = rmsnorm(x) in chunked form
    int rc = wide_prep(c, x_res, D, pend, static_cast<const __nv_bfloat16 *>(w.g_attn_norm), x_store, c->wide_n, D, batch, kProfQkv, st);
    if (rc) return rc;
    WideArgs a = wide_args(c, c->wide_n, w.w_qkv, D, nqkv, batch);
    a.out_bf16 = c->qkv; a.out_stride = nqkv;
    rc = launch_wide_linear(c, a, kProfQkv, st);
    if (rc) return rc;
    // the attention writes its output straight into the chunked activations of the output projection
    rc = attn_impl(c, c->qkv, c->qkv + nq, c->qkv + nq + nkv, nqkv, nqkv, k_cache, v_cache, pos, seq_lens, c->wide_n, nq,
                   batch, st, n_new, /*out_chunked=*/1, fp8, k_scale, v_scale);
    if (rc) return rc;
    a = wide_args(c, c->wide_n, w.w_o, nq, D, batch);            // h = x + attn . W_o
    a.res = resid; a.res_stride = D; a.out_bf16 = c->h; a.out_stride = D; a.pair_rows = 1;
    rc = launch_wide_linear(c, a, kProfOproj, st);
    if (rc) return rc;
    return wide_mlp_sums(c, c->h, static_cast<const __nv_bfloat16 *>(w.g_mlp_norm), w.w_gate_up, w.w_down, batch, st);
}

// batch: token rows (sequences x n_new)
static int layer_impl(Ctx *c, const fasttps_layer_weights &w, const __nv_bfloat16 *x_in, __nv_bfloat16 *x_out,
                      void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens, int batch,
                      cudaStream_t st, int n_new = 1, bool fp8 = false, float k_scale = 1.f, float v_scale = 1.f)
{
    if (wide_batch(c, batch) && batch <= kWideMaxB) {
        int rc = layer_body_wide(c, w, x_in, nullptr, nullptr, k_cache, v_cache, pos, seq_lens, batch, n_new, st, fp8,
                                 k_scale, v_scale);
        if (rc) return rc;
        // x' = h + MLP sums
        return wide_prep(c, c->h, c->cfg.hidden, c->mlp_acc, nullptr, x_out, nullptr, c->cfg.hidden, batch, kProfMlp, st);
    }
    const fasttps_config &f = c->cfg;
    const int D = f.hidden, nq = f.n_q_heads * f.head_dim, nkv = f.n_kv_heads * f.head_dim, nqkv = nq + 2 * nkv;
    int rc;
    // RMSNorm -> QKV (q | k | v stay in one [B, nqkv] scratch row per sequence)
    rc = linear_impl(c, D, nqkv, x_in, D, static_cast<const __nv_bfloat16 *>(w.g_attn_norm), w.w_qkv, nullptr, 0,
                     c->qkv, nullptr, nqkv, batch, nullptr, nullptr, nullptr, kProfQkv, st);
    if (rc) return rc;
    rc = attn_impl(c, c->qkv, c->qkv + nq, c->qkv + nq + nkv, nqkv, nqkv, k_cache, v_cache, pos, seq_lens,
                   c->attn_out, nq, batch, st, n_new, 0, fp8, k_scale, v_scale);
    if (rc) return rc;
    // h = x + attn . W_o
    rc = linear_impl(c, nq, D, c->attn_out, nq, nullptr, w.w_o, x_in, D, c->h, nullptr, D, batch, nullptr, nullptr,
                     nullptr, kProfOproj, st);
    if (rc) return rc;
    // x' = h + mlp(rmsnorm(h))
    return mlp_impl(c, c->h, static_cast<const __nv_bfloat16 *>(w.g_mlp_norm), w.w_gate_up, w.w_down, c->h, x_out,
                    batch, st);
}

static bool layer_ok(const fasttps_layer_weights *w)
{
    return w && aligned16(w->g_attn_norm) && aligned16(w->w_qkv) && aligned16(w->w_o) && aligned16(w->g_mlp_norm) &&
           aligned16(w->w_gate_up) && aligned16(w->w_down);
}

static int layer_step_impl(Ctx *c, const fasttps_layer_weights &w, const __nv_bfloat16 *x_in, __nv_bfloat16 *x_out,
                           void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens, int batch,
                           cudaStream_t st);

int fasttps_layer_decode(fasttps_ctx *ctx, const fasttps_layer_weights *w, const void *x_in, void *x_out,
                         void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens,
                         int batch, void *stream)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (batch < 1 || batch > c->cfg.max_batch || !layer_ok(w)) return FASTTPS_INVALID_ARG;
    if (!aligned16(x_in) || !aligned16(x_out) || !aligned16(k_cache) || !aligned16(v_cache) || !pos || !seq_lens)
        return FASTTPS_INVALID_ARG;
    if (c->opt_step_kernel != 0 && step_kernel_supported(c, batch, /*layer_mode=*/true))
        return layer_step_impl(c, *w, static_cast<const __nv_bfloat16 *>(x_in), static_cast<__nv_bfloat16 *>(x_out),
                               k_cache, v_cache, pos, seq_lens, batch, static_cast<cudaStream_t>(stream));
    return layer_impl(c, *w, static_cast<const __nv_bfloat16 *>(x_in), static_cast<__nv_bfloat16 *>(x_out), k_cache,
                      v_cache, pos, seq_lens, batch, static_cast<cudaStream_t>(stream));
}

int fasttps_layer_decode_multi(fasttps_ctx *ctx, const fasttps_layer_weights *w, const void *x_in, void *x_out,
                               void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens,
                               int batch, int n_new, void *stream)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (batch < 1 || n_new < 1 || n_new > kMaxNB || (long long)batch * n_new > c->cfg.max_batch || !layer_ok(w))
        return FASTTPS_INVALID_ARG;
    if (!aligned16(x_in) || !aligned16(x_out) || !aligned16(k_cache) || !aligned16(v_cache) || !pos || !seq_lens)
        return FASTTPS_INVALID_ARG;
    if (n_new == 1) return fasttps_layer_decode(ctx, w, x_in, x_out, k_cache, v_cache, pos, seq_lens, batch, stream);
    // the projections and the MLP see batch * n_new token rows; only the attention tells the tokens of a sequence apart
    return layer_impl(c, *w, static_cast<const __nv_bfloat16 *>(x_in), static_cast<__nv_bfloat16 *>(x_out), k_cache,
                      v_cache, pos, seq_lens, batch * n_new, static_cast<cudaStream_t>(stream), n_new);
}

int fasttps_layer_decode_fp8(fasttps_ctx *ctx, const fasttps_layer_weights *w, const void *x_in, void *x_out,
                             void *k_cache, void *v_cache, float k_scale, float v_scale, const int32_t *pos,
                             const int32_t *seq_lens, int batch, void *stream)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (batch < 1 || batch > c->cfg.max_batch || batch > kWideMaxB || !layer_ok(w)) return FASTTPS_INVALID_ARG;
    if (!aligned16(x_in) || !aligned16(x_out) || !aligned16(k_cache) || !aligned16(v_cache) || !pos || !seq_lens)
        return FASTTPS_INVALID_ARG;
    if (!(k_scale > 0.f) || !(v_scale > 0.f) || std::isinf(k_scale) || std::isinf(v_scale)) return FASTTPS_INVALID_ARG;
    // one kernel per product (the persistent layer kernel reads bf16 caches)
    return layer_impl(c, *w, static_cast<const __nv_bfloat16 *>(x_in), static_cast<__nv_bfloat16 *>(x_out), k_cache,
                      v_cache, pos, seq_lens, batch, static_cast<cudaStream_t>(stream), 1, /*fp8=*/true, k_scale, v_scale);
}

static bool use_step_kernel(const Ctx *c, int batch)
{
    return c->opt_step_kernel != 0 && step_kernel_supported(c, batch);
}

int fasttps_set_option(fasttps_ctx *ctx, const char *name, int value)
{
    if (!ctx || !name) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (strcmp(name, "step_kernel") == 0) c->opt_step_kernel = value != 0;
    else if (strcmp(name, "gqa_share") == 0) c->opt_gqa_share = value < 0 ? 0 : (value > 2 ? 2 : value);
    else return FASTTPS_INVALID_ARG;
    return FASTTPS_OK;
}

static int model_args_ok(const Ctx *c, const void *embed, const fasttps_layer_weights *layers, const void *g_final,
                         const void *w_lm_head, void *const *k_caches, void *const *v_caches, const int32_t *token_ids,
                         const int32_t *pos, const int32_t *seq_lens, int batch)
{
    const fasttps_config &f = c->cfg;
    if (batch < 1 || batch > f.max_batch || f.vocab < 1 || f.n_layers < 1) return FASTTPS_INVALID_ARG;
    if (!aligned16(embed) || !layers || !aligned16(g_final) || !aligned16(w_lm_head) || !k_caches || !v_caches ||
        !token_ids || !pos || !seq_lens)
        return FASTTPS_INVALID_ARG;
    for (int l = 0; l < f.n_layers; ++l)
        if (!layer_ok(&layers[l]) || !aligned16(k_caches[l]) || !aligned16(v_caches[l])) return FASTTPS_INVALID_ARG;
    return FASTTPS_OK;
}

// the workspace and shape fields of a step-kernel launch
static void step_args_common(Ctx *c, StepArgs &a, int batch)
{
    const fasttps_config &f = c->cfg;
    a.batch = batch;
    a.D = f.hidden; a.n_q_heads = f.n_q_heads; a.n_kv_heads = f.n_kv_heads; a.head_dim = f.head_dim;
    a.K = f.inter; a.V = f.vocab; a.max_seq = f.max_seq; a.eps = f.rms_eps;
    a.cos_tab = c->cos_tab; a.sin_tab = c->sin_tab;
    a.x0 = c->xa; a.qkv = c->qkv; a.attn_out = c->attn_out; a.h = c->h;
    a.acc = c->mlp_acc; a.hacc = c->hacc; a.attn_part = c->attn_part; a.attn_ticket = c->attn_ticket;
    a.amax_val = c->amax_val; a.amax_idx = c->amax_idx; a.tok = c->tok2;
    a.bar = c->grid_bar; a.status = c->status;
    a.x_out = nullptr;
}

static LayerPtrs layer_ptrs(const fasttps_layer_weights &w, void *k_cache, void *v_cache)
{
    LayerPtrs lp;
    lp.g_attn = static_cast<const __nv_bfloat16 *>(w.g_attn_norm);
    lp.w_qkv = static_cast<const __nv_bfloat16 *>(w.w_qkv);
    lp.w_o = static_cast<const __nv_bfloat16 *>(w.w_o);
    lp.g_mlp = static_cast<const __nv_bfloat16 *>(w.g_mlp_norm);
    lp.w_gu = static_cast<const __nv_bfloat16 *>(w.w_gate_up);
    lp.w_down = static_cast<const __nv_bfloat16 *>(w.w_down);
    lp.k_cache = static_cast<__nv_bfloat16 *>(k_cache);
    lp.v_cache = static_cast<__nv_bfloat16 *>(v_cache);
    return lp;
}

// n_steps consecutive tokens in one launch of the persistent step kernel (batch <= 8)
static int step_impl(Ctx *c, const void *embed, const fasttps_layer_weights *layers, const void *g_final,
                     const void *w_lm_head, void *const *k_caches, void *const *v_caches, const int32_t *token_ids,
                     int32_t *pos, int32_t *seq_lens, float *logits, int32_t *next_ids, int32_t *out_ids, int batch,
                     int n_steps, int advance, cudaStream_t st)
{
    const fasttps_config &f = c->cfg;
    StepArgs a;
    step_args_common(c, a, batch);
    // the layer pointers are launch parameters: a launch keeps the table it was given, whatever later calls pass
    for (int l = 0; l < f.n_layers; ++l) a.layers[l] = layer_ptrs(layers[l], k_caches[l], v_caches[l]);
    a.embed = static_cast<const __nv_bfloat16 *>(embed);
    a.g_final = static_cast<const __nv_bfloat16 *>(g_final);
    a.w_lm = static_cast<const __nv_bfloat16 *>(w_lm_head);
    a.token_ids = token_ids; a.pos = pos; a.seq_lens = seq_lens;
    a.logits = logits; a.next_ids = next_ids; a.out_ids = out_ids;
    a.n_steps = n_steps; a.advance = advance; a.n_layers = f.n_layers;
    return launch_step(c, a, st);
}

// one layer on the caller's activations in one launch of the persistent step kernel (batch <= 8)
static int layer_step_impl(Ctx *c, const fasttps_layer_weights &w, const __nv_bfloat16 *x_in, __nv_bfloat16 *x_out,
                           void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens, int batch,
                           cudaStream_t st)
{
    StepArgs a;
    step_args_common(c, a, batch);
    a.layers[0] = layer_ptrs(w, k_cache, v_cache);
    a.embed = nullptr; a.g_final = nullptr; a.w_lm = nullptr; a.token_ids = nullptr;
    a.pos = const_cast<int32_t *>(pos); a.seq_lens = const_cast<int32_t *>(seq_lens);   // read only: advance is 0
    a.logits = nullptr; a.next_ids = nullptr; a.out_ids = nullptr;
    a.n_steps = 1; a.advance = 0; a.n_layers = 1;
    a.x0 = const_cast<__nv_bfloat16 *>(x_in);            // read only in layer mode
    a.x_out = x_out;
    return launch_layer_step(c, a, st);
}

int fasttps_model_decode(fasttps_ctx *ctx, const void *embed, const fasttps_layer_weights *layers,
                         const void *g_final, const void *w_lm_head,
                         void *const *k_caches, void *const *v_caches,
                         const int32_t *token_ids, int32_t *pos, int32_t *seq_lens,
                         float *logits, int32_t *next_ids, int batch, int advance, void *stream)
{
    if (!ctx || !next_ids) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    const fasttps_config &f = c->cfg;
    int rc = model_args_ok(c, embed, layers, g_final, w_lm_head, k_caches, v_caches, token_ids, pos, seq_lens, batch);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (use_step_kernel(c, batch))
        return step_impl(c, embed, layers, g_final, w_lm_head, k_caches, v_caches, token_ids, pos, seq_lens, logits,
                         next_ids, nullptr, batch, 1, advance, st);
    // larger batches: one kernel per product, chained with programmatic dependent launch
    rc = launch_embed(c, static_cast<const __nv_bfloat16 *>(embed), token_ids, c->xa, batch, st);
    if (rc) return rc;
    if (wide_batch(c, batch) && batch <= kWideMaxB) {
        // thin-GEMM chain: the sums of a layer's MLP are folded into the next layer's input by its first kernel
        for (int l = 0; l < f.n_layers; ++l) {
            rc = layer_body_wide(c, layers[l], l == 0 ? c->xa : c->h, l == 0 ? nullptr : c->mlp_acc, l == 0 ? nullptr : c->xb,
                                 k_caches[l], v_caches[l], pos, seq_lens, batch, 1, st);
            if (rc) return rc;
        }
        // x_L = h + sums, final RMSNorm, logits from the chunked activations
        rc = wide_prep(c, c->h, f.hidden, c->mlp_acc, static_cast<const __nv_bfloat16 *>(g_final), nullptr, c->wide_n, f.hidden,
                       batch, kProfLmHead, st);
        if (rc) return rc;
        WideArgs a = wide_args(c, c->wide_n, w_lm_head, f.hidden, f.vocab, batch);
        a.out_f32 = logits ? logits : c->logits; a.out_stride = f.vocab;
        a.next_ids = next_ids; a.adv_pos = advance ? pos : nullptr; a.adv_len = advance ? seq_lens : nullptr;
        return launch_wide_linear(c, a, kProfLmHead, st);
    }
    __nv_bfloat16 *cur = c->xa, *nxt = c->xb;
    for (int l = 0; l < f.n_layers; ++l) {
        rc = layer_impl(c, layers[l], cur, nxt, k_caches[l], v_caches[l], pos, seq_lens, batch, st);
        if (rc) return rc;
        __nv_bfloat16 *tmp = cur; cur = nxt; nxt = tmp;
    }
    float *lg = logits ? logits : c->logits;
    return linear_impl(c, f.hidden, f.vocab, cur, f.hidden, static_cast<const __nv_bfloat16 *>(g_final), w_lm_head,
                       nullptr, 0, nullptr, lg, f.vocab, batch, next_ids, advance ? pos : nullptr,
                       advance ? seq_lens : nullptr, kProfLmHead, st);
}

int fasttps_model_generate(fasttps_ctx *ctx, const void *embed, const fasttps_layer_weights *layers,
                           const void *g_final, const void *w_lm_head,
                           void *const *k_caches, void *const *v_caches,
                           const int32_t *token_ids, int32_t *pos, int32_t *seq_lens,
                           int32_t *out_ids, int n_steps, int batch, void *stream)
{
    if (!ctx || !out_ids || n_steps < 1) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    int rc = model_args_ok(c, embed, layers, g_final, w_lm_head, k_caches, v_caches, token_ids, pos, seq_lens, batch);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (use_step_kernel(c, batch))
        return step_impl(c, embed, layers, g_final, w_lm_head, k_caches, v_caches, token_ids, pos, seq_lens, nullptr,
                         out_ids + (size_t)(n_steps - 1) * batch, out_ids, batch, n_steps, 1, st);
    for (int s = 0; s < n_steps; ++s) {
        rc = fasttps_model_decode(ctx, embed, layers, g_final, w_lm_head, k_caches, v_caches,
                                  s == 0 ? token_ids : out_ids + (size_t)(s - 1) * batch, pos, seq_lens, nullptr,
                                  out_ids + (size_t)s * batch, batch, 1, stream);
        if (rc) return rc;
    }
    return FASTTPS_OK;
}

int fasttps_model_decode_host(fasttps_ctx *ctx, const void *embed, const fasttps_layer_weights *layers,
                              const void *g_final, const void *w_lm_head,
                              void *const *k_caches, void *const *v_caches,
                              const int32_t *host_token_ids, int32_t *pos, int32_t *seq_lens,
                              int32_t *host_next_ids, int batch, void *stream)
{
    if (!ctx || !host_token_ids || !host_next_ids) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (batch < 1 || batch > c->cfg.max_batch) return FASTTPS_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    memcpy(c->pinned_tok, host_token_ids, sizeof(int32_t) * batch);
    FT_CUDA(cudaMemcpyAsync(c->tok, c->pinned_tok, sizeof(int32_t) * batch, cudaMemcpyHostToDevice, st));
    int rc = fasttps_model_decode(ctx, embed, layers, g_final, w_lm_head, k_caches, v_caches, c->tok, pos, seq_lens,
                                  nullptr, c->tok, batch, 1, stream);
    if (rc) return rc;
    FT_CUDA(cudaMemcpyAsync(c->pinned_tok + c->cfg.max_batch, c->tok, sizeof(int32_t) * batch,
                            cudaMemcpyDeviceToHost, st));
    FT_CUDA(cudaStreamSynchronize(st));
    memcpy(host_next_ids, c->pinned_tok + c->cfg.max_batch, sizeof(int32_t) * batch);
    return FASTTPS_OK;
}

int fasttps_get_status(fasttps_ctx *ctx, uint32_t *host_status)
{
    if (!ctx || !host_status) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    FT_CUDA(cudaDeviceSynchronize());
    FT_CUDA(cudaMemcpy(host_status, c->status, sizeof(uint32_t), cudaMemcpyDeviceToHost));
    FT_CUDA(cudaMemset(c->status, 0, sizeof(uint32_t)));
    if (*host_status & FASTTPS_DEV_WAIT_TIMEOUT) {
        // CTAs that gave up left without taking their tickets and with partial sums already added: everything the
        // kernels expect to find at zero goes back to zero, so that the next call starts clean
        const fasttps_config &f = c->cfg;
        const size_t B = f.max_batch, D = f.hidden;
        FT_CUDA(cudaMemset(c->mlp_acc, 0, 2 * B * D * sizeof(float)));
        FT_CUDA(cudaMemset(c->hacc, 0, 2 * B * D * sizeof(float)));
        FT_CUDA(cudaMemset(c->mlp_ticket, 0, sizeof(int)));
        FT_CUDA(cudaMemset(c->amax_ticket, 0, sizeof(int)));
        FT_CUDA(cudaMemset(c->attn_ticket, 0, B * f.n_q_heads * sizeof(int)));
        FT_CUDA(cudaMemset(c->grid_bar, 0, kGridBarWords * sizeof(unsigned)));
    }
    return FASTTPS_OK;
}

// Test hook: the state an abandoned call leaves behind, made on the host (no kernel is involved, nothing waits or
// faults): partial sums in the accumulators, tickets taken, barrier words counted up, and the time-out bit set.
int fasttps_debug_leave_workspace_dirty(fasttps_ctx *ctx)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    const fasttps_config &f = c->cfg;
    const size_t B = f.max_batch, D = f.hidden;
    FT_CUDA(cudaDeviceSynchronize());
    FT_CUDA(cudaMemset(c->mlp_acc, 0x3f, 2 * B * D * sizeof(float)));          // 0x3f3f3f3f = 0.747 in every sum
    FT_CUDA(cudaMemset(c->hacc, 0x3f, 2 * B * D * sizeof(float)));
    FT_CUDA(cudaMemset(c->mlp_ticket, 0x01, sizeof(int)));
    FT_CUDA(cudaMemset(c->amax_ticket, 0x01, sizeof(int)));
    FT_CUDA(cudaMemset(c->attn_ticket, 0x01, B * f.n_q_heads * sizeof(int)));
    FT_CUDA(cudaMemset(c->grid_bar, 0x01, kGridBarWords * sizeof(unsigned)));
    const uint32_t bit = FASTTPS_DEV_WAIT_TIMEOUT;
    FT_CUDA(cudaMemcpy(c->status, &bit, sizeof(bit), cudaMemcpyHostToDevice));
    return FASTTPS_OK;
}

int fasttps_profile(fasttps_ctx *ctx, int enable)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (enable && !c->prof_ev) {
        c->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfMax]();
        c->prof_cls = new (std::nothrow) unsigned char[kProfMax]();
        if (!c->prof_ev || !c->prof_cls) return FASTTPS_OUT_OF_MEMORY;
        for (int i = 0; i < 2 * kProfMax; ++i) FT_CUDA(cudaEventCreate(&c->prof_ev[i]));
    }
    c->prof_on = enable != 0;
    if (enable) c->prof_n = 0;
    return FASTTPS_OK;
}

int fasttps_profile_read(fasttps_ctx *ctx, double *ms_per_class, uint64_t *launches_per_class)
{
    if (!ctx || !ms_per_class || !launches_per_class) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    for (int k = 0; k < kProfClasses; ++k) { ms_per_class[k] = 0.0; launches_per_class[k] = 0; }
    if (!c->prof_ev) return FASTTPS_OK;
    FT_CUDA(cudaDeviceSynchronize());
    for (int i = 0; i < c->prof_n; ++i) {
        float ms = 0.f;
        FT_CUDA(cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]));
        ms_per_class[c->prof_cls[i]] += ms;
        launches_per_class[c->prof_cls[i]] += 1;
    }
    return FASTTPS_OK;
}

uint64_t fasttps_launch_count(const fasttps_ctx *ctx)
{
    return ctx ? reinterpret_cast<const Ctx *>(ctx)->launches : 0;
}

const char *fasttps_strerror(int code)
{
    switch (code) {
    case FASTTPS_OK: return "ok";
    case FASTTPS_INVALID_ARG: return "invalid argument (null or misaligned pointer, batch out of range, unsupported dims)";
    case FASTTPS_CUDA_ERROR: return "CUDA error (see fasttps_last_error)";
    case FASTTPS_OUT_OF_MEMORY: return "out of device memory";
    default: return "unknown status";
    }
}

const char *fasttps_last_error(void) { return g_last_error; }

}  // extern "C"
