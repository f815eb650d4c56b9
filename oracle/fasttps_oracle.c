/*
 * CPU oracle for the FastTPS token-phase (decode) step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what
 * the decode path computes, written from the paper's definitions.  Only the
 * test-suite, the smoke check and the benchmark's CPU-baseline leg may call
 * it; the product library never does, and the two share no code.
 *
 * What it follows (paper passages):
 *   - SwiGLU MLP                      Eq. 1, Eq. 31 (gate = first half of W_gu)
 *   - static KV cache, in-place append Eq. 2 (address jump), Section 3.1.1
 *   - fused attention step order       Algorithm 3, steps 6-12
 *     (joint RoPE on q,k -> write K row -> QK^T over the cache including the
 *      new row -> softmax -> PV)
 *   - MLP step order                   Algorithm 4 (RMSNorm, gate_up, siLu_Mul, down)
 *   - block structure (norm, QKV, attention, output projection, norm, MLP)
 *                                      Figure 1 caption, Section 2.2, Section 2.3
 *   - the same attention step over a cache of 8-bit (E4M3) codes   Section 6.2 (compatibility with quantisation)
 *
 * Precision model.  Every tensor that crosses one of the three block
 * functions (attention, MLP, layer) is bf16, rounded to nearest even.  Inside
 * a function all reductions are accumulated in double (so the result does not
 * depend on summation order) and softmax/SiLU/RMSNorm are evaluated in
 * double.  The one place that is evaluated in single precision on purpose is
 * RoPE: the rotated key row is persisted in the cache and compared to one
 * bf16 ulp, so its arithmetic is pinned to FP32 with separately rounded
 * products (cos/sin are FP32 values of a double computation).
 *
 * Readings taken where the paper is silent (listed in full in the design
 * document): half-split RoPE pairing (i, i+d/2), theta passed by the caller;
 * scores scaled by 1/sqrt(d); the new token attends to itself; eps inside the
 * square root of RMSNorm; pre-norm residual connections; no biases; lowest
 * index wins an argmax tie.
 *
 * Parity pins: see tests/test_oracle_pins.py (closed forms, invariants,
 * special cases, brute force at tiny sizes against sums expanded in plain
 * Python floats).  Against the authors' own implementation the oracle is
 * "parity unpinned": the paper prints no numeric example of the method.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC -o liboracle.so fasttps_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ bf16 */

float orc_bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* FP32 -> bf16, round to nearest, ties to even.  NaN stays NaN (quiet). */
uint16_t orc_f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u)            /* NaN */
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* double -> bf16 with a single rounding: first squeeze the double into an
 * FP32 with round-to-odd (truncate toward zero, then set the last bit if
 * anything was lost), which keeps enough information for the final RNE. */
uint16_t orc_f64_to_bf16(double x)
{
    if (isnan(x)) return 0x7fc0u;
    float f = (float)x;
    if (isinf(f)) return orc_f32_to_bf16(f);
    if ((double)f != x) {
        if (fabs((double)f) > fabs(x)) f = nextafterf(f, 0.0f);   /* truncate */
        uint32_t u;
        memcpy(&u, &f, 4);
        u |= 1u;                                                  /* sticky  */
        memcpy(&f, &u, 4);
    }
    return orc_f32_to_bf16(f);
}

void orc_f32_to_bf16_array(const float *x, uint16_t *y, size_t n)
{
    for (size_t i = 0; i < n; ++i) y[i] = orc_f32_to_bf16(x[i]);
}

void orc_f64_to_bf16_array(const double *x, uint16_t *y, size_t n)
{
    for (size_t i = 0; i < n; ++i) y[i] = orc_f64_to_bf16(x[i]);
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* --------------------------------------------------------------- RMSNorm */

/* y = x * 1/sqrt(mean(x^2) + eps) * g, per row; Algorithm 4 step 1 / Section 2.3.
 * x [B,D] bf16, g [D] bf16 -> y [B,D] bf16. */
void orc_rmsnorm(const uint16_t *x, const uint16_t *g, uint16_t *y, int B, int D, double eps)
{
    for (int b = 0; b < B; ++b) {
        double ss = 0.0;
        for (int i = 0; i < D; ++i) {
            double v = orc_bf16_to_f32(x[(size_t)b * D + i]);
            ss += v * v;
        }
        double r = 1.0 / sqrt(ss / (double)D + eps);
        for (int i = 0; i < D; ++i) {
            double v = orc_bf16_to_f32(x[(size_t)b * D + i]);
            double gi = orc_bf16_to_f32(g[i]);
            y[(size_t)b * D + i] = orc_f64_to_bf16(v * r * gi);
        }
    }
}

/* ------------------------------------------------------------------ GEMV */

/* y[b,n] = sum_i x[b,i] * W[i,n]; x [B,in] bf16, W [in,out] bf16 row-major,
 * y [B,out] double.  Row vector times matrix: the shapes stated under Eq. 1
 * (h in R^{N x D}, W in R^{D x K}) admit only h.W. */
void orc_gemv(const uint16_t *x, const uint16_t *W, double *y, int B, int in, int out)
{
    const int NB = 256;
    #pragma omp parallel for schedule(static)
    for (int n0 = 0; n0 < out; n0 += NB) {
        int n1 = n0 + NB < out ? n0 + NB : out;
        for (int b = 0; b < B; ++b) {
            double acc[256];
            for (int n = n0; n < n1; ++n) acc[n - n0] = 0.0;
            for (int i = 0; i < in; ++i) {
                double xi = orc_bf16_to_f32(x[(size_t)b * in + i]);
                const uint16_t *row = W + (size_t)i * out;
                for (int n = n0; n < n1; ++n)
                    acc[n - n0] += xi * (double)orc_bf16_to_f32(row[n]);
            }
            for (int n = n0; n < n1; ++n) y[(size_t)b * out + n] = acc[n - n0];
        }
    }
}

/* y[b,v] = sum_i x[b,i] * W[v,i]; W [out,in] row-major (the lm_head layout). */
void orc_gemv_t(const uint16_t *x, const uint16_t *W, double *y, int B, int in, int out)
{
    #pragma omp parallel for schedule(static)
    for (int v = 0; v < out; ++v) {
        const uint16_t *row = W + (size_t)v * in;
        for (int b = 0; b < B; ++b) {
            double acc = 0.0;
            for (int i = 0; i < in; ++i)
                acc += (double)orc_bf16_to_f32(x[(size_t)b * in + i]) * (double)orc_bf16_to_f32(row[i]);
            y[(size_t)b * out + v] = acc;
        }
    }
}

/* ------------------------------------------------------------------ RoPE */

/* Rotary embedding of one head vector v[d] (FP32, in place) at position pos.
 * Pair (i, i+d/2), frequency theta^(-2i/d); Algorithm 3 step 8 applies it to
 * q and k of a head with one shared set of cos/sin values.  FP32 arithmetic
 * with every product and the sum/difference rounded separately. */
void orc_rope(float *v, int d, int pos, double theta)
{
    int half = d / 2;
    for (int i = 0; i < half; ++i) {
        double freq = pow(theta, -2.0 * (double)i / (double)d);
        double ang = (double)pos * freq;
        float c = (float)cos(ang);
        float s = (float)sin(ang);
        float a = v[i], b = v[i + half];
        volatile float ac = a * c, bs = b * s, bc = b * c, as = a * s;
        v[i] = ac - bs;
        v[i + half] = bc + as;
    }
}

/* ------------------------------------------------------- attention decode */

/* Algorithm 3 for one decode step of a batch.
 *   q      [B,Hq,d]  bf16   new query (before RoPE)
 *   k_new  [B,Hkv,d] bf16   new key   (before RoPE)
 *   v_new  [B,Hkv,d] bf16   new value
 *   k_cache, v_cache [B,Hkv,max_seq,d] bf16, modified in place: row
 *          seq_lens[b] of every head receives bf16(rope(k_new)) resp. v_new
 *          (Eq. 2: element offset (b*Hkv+h)*max_seq*d + seq_lens[b]*d)
 *   pos[b]       rotary position of the new token
 *   seq_lens[b]  rows already in the cache (= row written this step)
 *   out    [B,Hq,d]  bf16   attention output over rows 0..seq_lens[b] inclusive
 * Sequences with seq_lens[b] >= max_seq or pos[b] < 0 are skipped entirely.
 * Query head h reads kv head h / (Hq/Hkv) (grouped-query broadcast, Section 4.1). */
void orc_attn_decode(const uint16_t *q, const uint16_t *k_new, const uint16_t *v_new,
                     uint16_t *k_cache, uint16_t *v_cache,
                     const int32_t *pos, const int32_t *seq_lens, uint16_t *out,
                     int B, int Hq, int Hkv, int d, int max_seq, double theta)
{
    int G = Hq / Hkv;
    /* steps 1, 6-9: V row, joint RoPE, K row */
    for (int b = 0; b < B; ++b) {
        int L = seq_lens[b];
        if (L < 0 || L >= max_seq || pos[b] < 0) continue;
        for (int h = 0; h < Hkv; ++h) {
            float kr[1024];
            for (int c = 0; c < d; ++c) kr[c] = orc_bf16_to_f32(k_new[((size_t)b * Hkv + h) * d + c]);
            orc_rope(kr, d, pos[b], theta);
            size_t row = (((size_t)b * Hkv + h) * max_seq + L) * d;
            for (int c = 0; c < d; ++c) {
                k_cache[row + c] = orc_f32_to_bf16(kr[c]);
                v_cache[row + c] = v_new[((size_t)b * Hkv + h) * d + c];
            }
        }
    }
    /* steps 10-12 per query head */
    #pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            int L = seq_lens[b];
            if (L < 0 || L >= max_seq || pos[b] < 0) continue;
            int Nt = L + 1;
            int hk = h / G;
            float qr[1024];
            for (int c = 0; c < d; ++c) qr[c] = orc_bf16_to_f32(q[((size_t)b * Hq + h) * d + c]);
            orc_rope(qr, d, pos[b], theta);
            const uint16_t *Kh = k_cache + ((size_t)b * Hkv + hk) * max_seq * d;
            const uint16_t *Vh = v_cache + ((size_t)b * Hkv + hk) * max_seq * d;
            double *s = (double *)malloc(sizeof(double) * (size_t)Nt);
            double scale = 1.0 / sqrt((double)d);
            double m = -INFINITY;
            for (int j = 0; j < Nt; ++j) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c)
                    acc += (double)qr[c] * (double)orc_bf16_to_f32(Kh[(size_t)j * d + c]);
                s[j] = acc * scale;
                if (s[j] > m) m = s[j];
            }
            double denom = 0.0;
            for (int j = 0; j < Nt; ++j) { s[j] = exp(s[j] - m); denom += s[j]; }
            for (int c = 0; c < d; ++c) {
                double o = 0.0;
                for (int j = 0; j < Nt; ++j)
                    o += (s[j] / denom) * (double)orc_bf16_to_f32(Vh[(size_t)j * d + c]);
                out[((size_t)b * Hq + h) * d + c] = orc_f64_to_bf16(o);
            }
            free(s);
        }
    }
}

/* Algorithm 3 for N new tokens per sequence (the algorithm is written for Q, K, V in R^{B x N x H x d}; the token
 * phase proper is N = 1).  Token j of sequence b has rotary position pos[b] + j and goes into cache row
 * seq_lens[b] + j; it attends rows 0 .. seq_lens[b] + j: everything cached before the step and the new tokens up to
 * and including itself (causal mask inside the chunk).  Written as the masked definition: all N rows are appended
 * first, then every (token, head) takes its softmax over its own prefix of the rows.
 *   q [B,N,Hq,d], k_new, v_new [B,N,Hkv,d], out [B,N,Hq,d]; caches, pos, seq_lens as in orc_attn_decode.
 * A sequence is skipped unless all N rows fit: seq_lens[b] >= 0, seq_lens[b] + N <= max_seq, pos[b] >= 0. */
void orc_attn_decode_multi(const uint16_t *q, const uint16_t *k_new, const uint16_t *v_new,
                           uint16_t *k_cache, uint16_t *v_cache,
                           const int32_t *pos, const int32_t *seq_lens, uint16_t *out,
                           int B, int N, int Hq, int Hkv, int d, int max_seq, double theta)
{
    int G = Hq / Hkv;
    for (int b = 0; b < B; ++b) {
        int L = seq_lens[b];
        if (L < 0 || L + N > max_seq || pos[b] < 0) continue;
        for (int j = 0; j < N; ++j) {
            for (int h = 0; h < Hkv; ++h) {
                float kr[1024];
                size_t src = (((size_t)b * N + j) * Hkv + h) * d;
                for (int c = 0; c < d; ++c) kr[c] = orc_bf16_to_f32(k_new[src + c]);
                orc_rope(kr, d, pos[b] + j, theta);
                size_t row = (((size_t)b * Hkv + h) * max_seq + L + j) * d;
                for (int c = 0; c < d; ++c) {
                    k_cache[row + c] = orc_f32_to_bf16(kr[c]);
                    v_cache[row + c] = v_new[src + c];
                }
            }
        }
    }
    #pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int jh = 0; jh < N * Hq; ++jh) {
            int L = seq_lens[b];
            if (L < 0 || L + N > max_seq || pos[b] < 0) continue;
            int j = jh / Hq, h = jh % Hq, hk = h / G;
            int Nt = L + j + 1;                              /* rows this token may see */
            float qr[1024];
            size_t qo = (((size_t)b * N + j) * Hq + h) * d;
            for (int c = 0; c < d; ++c) qr[c] = orc_bf16_to_f32(q[qo + c]);
            orc_rope(qr, d, pos[b] + j, theta);
            const uint16_t *Kh = k_cache + ((size_t)b * Hkv + hk) * max_seq * d;
            const uint16_t *Vh = v_cache + ((size_t)b * Hkv + hk) * max_seq * d;
            double *s = (double *)malloc(sizeof(double) * (size_t)Nt);
            double scale = 1.0 / sqrt((double)d), m = -INFINITY, denom = 0.0;
            for (int r = 0; r < Nt; ++r) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += (double)qr[c] * (double)orc_bf16_to_f32(Kh[(size_t)r * d + c]);
                s[r] = acc * scale;
                if (s[r] > m) m = s[r];
            }
            for (int r = 0; r < Nt; ++r) { s[r] = exp(s[r] - m); denom += s[r]; }
            for (int c = 0; c < d; ++c) {
                double o = 0.0;
                for (int r = 0; r < Nt; ++r) o += (s[r] / denom) * (double)orc_bf16_to_f32(Vh[(size_t)r * d + c]);
                out[qo + c] = orc_f64_to_bf16(o);
            }
            free(s);
        }
    }
}

/* Softmax probabilities of one (b, query head) after the append has been
 * done, for tests of the row-sum invariant.  p [seq_lens[b]+1] double. */
void orc_attn_probs(const uint16_t *q, const uint16_t *k_cache, int pos, int L,
                    int b, int h, int Hq, int Hkv, int d, int max_seq, double theta, double *p)
{
    int G = Hq / Hkv, hk = h / G, Nt = L + 1;
    float qr[1024];
    for (int c = 0; c < d; ++c) qr[c] = orc_bf16_to_f32(q[((size_t)b * Hq + h) * d + c]);
    orc_rope(qr, d, pos, theta);
    const uint16_t *Kh = k_cache + ((size_t)b * Hkv + hk) * max_seq * d;
    double scale = 1.0 / sqrt((double)d), m = -INFINITY, denom = 0.0;
    for (int j = 0; j < Nt; ++j) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += (double)qr[c] * (double)orc_bf16_to_f32(Kh[(size_t)j * d + c]);
        p[j] = acc * scale;
        if (p[j] > m) m = p[j];
    }
    for (int j = 0; j < Nt; ++j) { p[j] = exp(p[j] - m); denom += p[j]; }
    for (int j = 0; j < Nt; ++j) p[j] /= denom;
}

/* ---------------------------------------------- attention decode, FP8 KV cache */

/* The 8-bit floating-point format E4M3 (the "fn" variant: no infinities) by its definition: bit 7 sign, bits 6..3
 * exponent e (bias 7), bits 2..0 mantissa m.  e = 0: subnormal, m/8 * 2^-6; otherwise (1 + m/8) * 2^(e-7); the
 * pattern e = 15, m = 7 is NaN, so the largest finite value is 1.75 * 2^8 = 448. */
float orc_e4m3_to_f32(uint8_t c)
{
    int e = (c >> 3) & 15, m = c & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    v = e == 0 ? ldexp((double)m / 8.0, -6) : ldexp(1.0 + (double)m / 8.0, e - 7);
    return (float)((c & 0x80) ? -v : v);
}

/* FP32 -> E4M3: the finite code nearest to x, ties to the code with an even mantissa, magnitudes beyond 448
 * saturate to 448 (no code for infinity), NaN gives the NaN code.  Found by looking at all 127 finite magnitudes. */
uint8_t orc_f32_to_e4m3(float x)
{
    uint8_t sign = signbit(x) ? 0x80 : 0x00;
    double a = fabs((double)x), best_d = INFINITY;
    int best = 0;
    if (isnan(x)) return 0x7f;
    for (int c = 0; c <= 0x7e; ++c) {
        double dd = fabs((double)orc_e4m3_to_f32((uint8_t)c) - a);
        if (dd < best_d || (dd == best_d && (c & 1) == 0)) { best_d = dd; best = c; }
    }
    return (uint8_t)(sign | best);
}

/* Algorithm 3 with the cache held in E4M3 (Section 6.2 states that the method composes with quantisation; the
 * paper gives no scheme, so the reading is the plainest one: one FP32 scale per tensor, given by the caller).
 *   stored code = e4m3(value / scale)  (FP32 division, then the rounding above); value read back = code * scale.
 *   k_cache, v_cache [B,Hkv,max_seq,d] uint8 codes, modified in place: row seq_lens[b] of every head receives the
 *   codes of rope(k_new) / k_scale resp. v_new / v_scale.  The new token attends to its own row AS STORED (the
 *   dequantised codes), so that this step and every later step see the same key and value for it.
 * Everything else (shapes, RoPE in FP32, skipping rules, double accumulation, bf16 output) as orc_attn_decode. */
void orc_attn_decode_fp8(const uint16_t *q, const uint16_t *k_new, const uint16_t *v_new,
                         uint8_t *k_cache, uint8_t *v_cache, float k_scale, float v_scale,
                         const int32_t *pos, const int32_t *seq_lens, uint16_t *out,
                         int B, int Hq, int Hkv, int d, int max_seq, double theta)
{
    int G = Hq / Hkv;
    for (int b = 0; b < B; ++b) {
        int L = seq_lens[b];
        if (L < 0 || L >= max_seq || pos[b] < 0) continue;
        for (int h = 0; h < Hkv; ++h) {
            float kr[1024];
            for (int c = 0; c < d; ++c) kr[c] = orc_bf16_to_f32(k_new[((size_t)b * Hkv + h) * d + c]);
            orc_rope(kr, d, pos[b], theta);
            size_t row = (((size_t)b * Hkv + h) * max_seq + L) * d;
            for (int c = 0; c < d; ++c) {
                volatile float ks = kr[c] / k_scale;
                volatile float vs = orc_bf16_to_f32(v_new[((size_t)b * Hkv + h) * d + c]) / v_scale;
                k_cache[row + c] = orc_f32_to_e4m3(ks);
                v_cache[row + c] = orc_f32_to_e4m3(vs);
            }
        }
    }
    #pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            int L = seq_lens[b];
            if (L < 0 || L >= max_seq || pos[b] < 0) continue;
            int Nt = L + 1;
            int hk = h / G;
            float qr[1024];
            for (int c = 0; c < d; ++c) qr[c] = orc_bf16_to_f32(q[((size_t)b * Hq + h) * d + c]);
            orc_rope(qr, d, pos[b], theta);
            const uint8_t *Kh = k_cache + ((size_t)b * Hkv + hk) * max_seq * d;
            const uint8_t *Vh = v_cache + ((size_t)b * Hkv + hk) * max_seq * d;
            double *s = (double *)malloc(sizeof(double) * (size_t)Nt);
            double scale = 1.0 / sqrt((double)d);
            double m = -INFINITY;
            for (int j = 0; j < Nt; ++j) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c)
                    acc += (double)qr[c] * ((double)orc_e4m3_to_f32(Kh[(size_t)j * d + c]) * (double)k_scale);
                s[j] = acc * scale;
                if (s[j] > m) m = s[j];
            }
            double denom = 0.0;
            for (int j = 0; j < Nt; ++j) { s[j] = exp(s[j] - m); denom += s[j]; }
            for (int c = 0; c < d; ++c) {
                double o = 0.0;
                for (int j = 0; j < Nt; ++j)
                    o += (s[j] / denom) * ((double)orc_e4m3_to_f32(Vh[(size_t)j * d + c]) * (double)v_scale);
                out[((size_t)b * Hq + h) * d + c] = orc_f64_to_bf16(o);
            }
            free(s);
        }
    }
}

/* ------------------------------------------------------------- MLP decode */

static double silu(double t) { return t / (1.0 + exp(-t)); }

/* Eq. 1 / Algorithm 4 steps 2-15 without the norm:
 *   y = ( silu(x.W_gate) * (x.W_up) ) . W_down
 * x [B,D] bf16; w_gu [D,2K] bf16, columns [0,K) gate and [K,2K) up;
 * w_down [K,D] bf16; y [B,D] double (caller rounds). */
void orc_mlp_f64(const uint16_t *x, const uint16_t *w_gu, const uint16_t *w_down,
                 double *y, int B, int D, int K)
{
    double *gu = (double *)malloc(sizeof(double) * (size_t)B * 2 * K);
    orc_gemv(x, w_gu, gu, B, D, 2 * K);
    const int NB = 256;
    #pragma omp parallel for schedule(static)
    for (int n0 = 0; n0 < D; n0 += NB) {
        int n1 = n0 + NB < D ? n0 + NB : D;
        for (int b = 0; b < B; ++b) {
            double acc[256];
            for (int n = n0; n < n1; ++n) acc[n - n0] = 0.0;
            for (int k = 0; k < K; ++k) {
                double a = silu(gu[(size_t)b * 2 * K + k]) * gu[(size_t)b * 2 * K + K + k];
                const uint16_t *row = w_down + (size_t)k * D;
                for (int n = n0; n < n1; ++n) acc[n - n0] += a * (double)orc_bf16_to_f32(row[n]);
            }
            for (int n = n0; n < n1; ++n) y[(size_t)b * D + n] = acc[n - n0];
        }
    }
    free(gu);
}

void orc_mlp_decode(const uint16_t *x, const uint16_t *w_gu, const uint16_t *w_down,
                    uint16_t *out, int B, int D, int K)
{
    double *y = (double *)malloc(sizeof(double) * (size_t)B * D);
    orc_mlp_f64(x, w_gu, w_down, y, B, D, K);
    for (size_t i = 0; i < (size_t)B * D; ++i) out[i] = orc_f64_to_bf16(y[i]);
    free(y);
}

/* ----------------------------------------------------------- layer decode */

/* One decoder layer, decode step (Figure 1: attention block then MLP block,
 * with pre-norm residuals):
 *   n1 = bf16(rmsnorm(x, g_attn))
 *   [q|k|v] = bf16(n1 . W_qkv)                    W_qkv [D, (Hq+2Hkv)d]
 *   a  = attn_decode(q, k, v, caches)             (appends to the caches)
 *   h  = bf16(x + a . W_o)                        W_o [Hq d, D]
 *   n2 = bf16(rmsnorm(h, g_mlp))
 *   x' = bf16(h + mlp(n2))
 */
static void layer_decode_n(const uint16_t *g_attn, const uint16_t *w_qkv, const uint16_t *w_o,
                           const uint16_t *g_mlp, const uint16_t *w_gu, const uint16_t *w_down,
                           const uint16_t *x_in, uint16_t *x_out,
                           void *k_cache, void *v_cache,
                           const int32_t *pos, const int32_t *seq_lens,
                           int n_seq, int n_new, int D, int Hq, int Hkv, int d, int K, int max_seq,
                           double eps, double theta, int fp8, float k_scale, float v_scale)
{
    /* B: token rows of the step = sequences x new tokens per sequence; only the attention tells them apart */
    int B = n_seq * n_new;
    int nq = Hq * d, nkv = Hkv * d, nqkv = nq + 2 * nkv;
    uint16_t *n1 = (uint16_t *)malloc(2 * (size_t)B * D);
    double *qkv = (double *)malloc(sizeof(double) * (size_t)B * nqkv);
    uint16_t *qb = (uint16_t *)malloc(2 * (size_t)B * nq);
    uint16_t *kb = (uint16_t *)malloc(2 * (size_t)B * nkv);
    uint16_t *vb = (uint16_t *)malloc(2 * (size_t)B * nkv);
    uint16_t *ab = (uint16_t *)malloc(2 * (size_t)B * nq);
    double *proj = (double *)malloc(sizeof(double) * (size_t)B * D);
    uint16_t *h = (uint16_t *)malloc(2 * (size_t)B * D);
    uint16_t *n2 = (uint16_t *)malloc(2 * (size_t)B * D);
    double *y = (double *)malloc(sizeof(double) * (size_t)B * D);

    orc_rmsnorm(x_in, g_attn, n1, B, D, eps);
    orc_gemv(n1, w_qkv, qkv, B, D, nqkv);
    for (int b = 0; b < B; ++b) {
        for (int i = 0; i < nq; ++i)  qb[(size_t)b * nq + i]  = orc_f64_to_bf16(qkv[(size_t)b * nqkv + i]);
        for (int i = 0; i < nkv; ++i) kb[(size_t)b * nkv + i] = orc_f64_to_bf16(qkv[(size_t)b * nqkv + nq + i]);
        for (int i = 0; i < nkv; ++i) vb[(size_t)b * nkv + i] = orc_f64_to_bf16(qkv[(size_t)b * nqkv + nq + nkv + i]);
    }
    /* a skipped sequence (bad length) leaves its attention output at zero */
    memset(ab, 0, 2 * (size_t)B * nq);
    if (fp8) orc_attn_decode_fp8(qb, kb, vb, (uint8_t *)k_cache, (uint8_t *)v_cache, k_scale, v_scale, pos, seq_lens, ab, B, Hq, Hkv, d, max_seq, theta);
    else if (n_new == 1) orc_attn_decode(qb, kb, vb, (uint16_t *)k_cache, (uint16_t *)v_cache, pos, seq_lens, ab, B, Hq, Hkv, d, max_seq, theta);
    else orc_attn_decode_multi(qb, kb, vb, (uint16_t *)k_cache, (uint16_t *)v_cache, pos, seq_lens, ab, n_seq, n_new, Hq, Hkv, d, max_seq, theta);
    orc_gemv(ab, w_o, proj, B, nq, D);
    for (size_t i = 0; i < (size_t)B * D; ++i)
        h[i] = orc_f64_to_bf16((double)orc_bf16_to_f32(x_in[i]) + proj[i]);
    orc_rmsnorm(h, g_mlp, n2, B, D, eps);
    orc_mlp_f64(n2, w_gu, w_down, y, B, D, K);
    for (size_t i = 0; i < (size_t)B * D; ++i)
        x_out[i] = orc_f64_to_bf16((double)orc_bf16_to_f32(h[i]) + y[i]);

    free(n1); free(qkv); free(qb); free(kb); free(vb); free(ab); free(proj); free(h); free(n2); free(y);
}

void orc_layer_decode(const uint16_t *g_attn, const uint16_t *w_qkv, const uint16_t *w_o,
                      const uint16_t *g_mlp, const uint16_t *w_gu, const uint16_t *w_down,
                      const uint16_t *x_in, uint16_t *x_out,
                      uint16_t *k_cache, uint16_t *v_cache,
                      const int32_t *pos, const int32_t *seq_lens,
                      int B, int D, int Hq, int Hkv, int d, int K, int max_seq,
                      double eps, double theta)
{
    layer_decode_n(g_attn, w_qkv, w_o, g_mlp, w_gu, w_down, x_in, x_out, k_cache, v_cache, pos, seq_lens,
                   B, 1, D, Hq, Hkv, d, K, max_seq, eps, theta, 0, 1.f, 1.f);
}

/* The same layer over caches of E4M3 codes (orc_attn_decode_fp8 in place of orc_attn_decode; everything else,
 * including the bf16 q | k | v handed to the attention, unchanged). */
void orc_layer_decode_fp8(const uint16_t *g_attn, const uint16_t *w_qkv, const uint16_t *w_o,
                          const uint16_t *g_mlp, const uint16_t *w_gu, const uint16_t *w_down,
                          const uint16_t *x_in, uint16_t *x_out,
                          uint8_t *k_cache, uint8_t *v_cache, float k_scale, float v_scale,
                          const int32_t *pos, const int32_t *seq_lens,
                          int B, int D, int Hq, int Hkv, int d, int K, int max_seq,
                          double eps, double theta)
{
    layer_decode_n(g_attn, w_qkv, w_o, g_mlp, w_gu, w_down, x_in, x_out, k_cache, v_cache, pos, seq_lens,
                   B, 1, D, Hq, Hkv, d, K, max_seq, eps, theta, 1, k_scale, v_scale);
}

/* The same layer for N new tokens per sequence: x_in, x_out [B*N, D] (token j of sequence b in row b*N + j);
 * every block but the attention treats the rows alike (Algorithm 4 is written for h_t in R^{N x D}). */
void orc_layer_decode_multi(const uint16_t *g_attn, const uint16_t *w_qkv, const uint16_t *w_o,
                            const uint16_t *g_mlp, const uint16_t *w_gu, const uint16_t *w_down,
                            const uint16_t *x_in, uint16_t *x_out,
                            uint16_t *k_cache, uint16_t *v_cache,
                            const int32_t *pos, const int32_t *seq_lens,
                            int B, int N, int D, int Hq, int Hkv, int d, int K, int max_seq,
                            double eps, double theta)
{
    layer_decode_n(g_attn, w_qkv, w_o, g_mlp, w_gu, w_down, x_in, x_out, k_cache, v_cache, pos, seq_lens,
                   B, N, D, Hq, Hkv, d, K, max_seq, eps, theta, 0, 1.f, 1.f);
}

/* ------------------------------------------------------------ model decode */

/* Embedding gather -> n_layers layers -> final RMSNorm (-> bf16) -> logits
 * (FP32 of a double sum) -> greedy argmax (lowest index on ties).
 * Per-layer tensors are passed as arrays of pointers.  hidden_out (optional,
 * may be NULL) receives the last layer's output [B,D] bf16. */
void orc_model_decode(const uint16_t *embed, int n_layers,
                      const uint16_t *const *g_attn, const uint16_t *const *w_qkv,
                      const uint16_t *const *w_o, const uint16_t *const *g_mlp,
                      const uint16_t *const *w_gu, const uint16_t *const *w_down,
                      const uint16_t *g_final, const uint16_t *w_lm,
                      uint16_t *const *k_caches, uint16_t *const *v_caches,
                      const int32_t *token_ids, const int32_t *pos, const int32_t *seq_lens,
                      float *logits, int32_t *next_ids, uint16_t *hidden_out,
                      int B, int D, int Hq, int Hkv, int d, int K, int V, int max_seq,
                      double eps, double theta)
{
    uint16_t *xa = (uint16_t *)malloc(2 * (size_t)B * D);
    uint16_t *xb = (uint16_t *)malloc(2 * (size_t)B * D);
    for (int b = 0; b < B; ++b)
        memcpy(xa + (size_t)b * D, embed + (size_t)token_ids[b] * D, 2 * (size_t)D);
    for (int l = 0; l < n_layers; ++l) {
        orc_layer_decode(g_attn[l], w_qkv[l], w_o[l], g_mlp[l], w_gu[l], w_down[l],
                         xa, xb, k_caches[l], v_caches[l], pos, seq_lens,
                         B, D, Hq, Hkv, d, K, max_seq, eps, theta);
        uint16_t *t = xa; xa = xb; xb = t;
    }
    if (hidden_out) memcpy(hidden_out, xa, 2 * (size_t)B * D);
    uint16_t *nf = (uint16_t *)malloc(2 * (size_t)B * D);
    double *lg = (double *)malloc(sizeof(double) * (size_t)B * V);
    orc_rmsnorm(xa, g_final, nf, B, D, eps);
    orc_gemv_t(nf, w_lm, lg, B, D, V);
    for (int b = 0; b < B; ++b) {
        int best = 0;
        for (int v = 0; v < V; ++v) {
            float f = (float)lg[(size_t)b * V + v];
            if (logits) logits[(size_t)b * V + v] = f;
            if (f > (float)lg[(size_t)b * V + best]) best = v;
        }
        if (next_ids) next_ids[b] = best;
    }
    free(nf); free(lg); free(xa); free(xb);
}
