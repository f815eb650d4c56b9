/*
 * fasttps_baseline.h -- the NON-fused token phase, as the paper describes the implementation it starts from
 * (Algorithm 1 "Standard Attention Implementation", Algorithm 2 "Standard MLP Implementation", Section 2.2-2.3),
 * restated as plain CUDA kernels on the same GPU: one kernel per operator, every intermediate tensor written to
 * and read back from device memory, and the KV cache updated by a Concat that copies the whole cache into a new
 * buffer.  It exists only as the comparison arm of the paper's own experiments (Section 5.1-5.3: fused against
 * non-fused latency, the share of Concat) -- it is not part of the decode path and nothing in the decode path
 * calls it.  Same conventions as fasttps.h: device pointers, bf16 unless stated, calls only enqueue on `stream`.
 */
#ifndef FASTTPS_BASELINE_H
#define FASTTPS_BASELINE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Shapes of one call. */
typedef struct {
    int batch, n_q_heads, n_kv_heads, head_dim;
    int max_seq;          /* rows per head of the caller's caches [B, H_kv, max_seq, d]            */
    int cat_seq;          /* rows per head of the Concat outputs  [B, H_kv, cat_seq, d], > every length */
    float rope_theta;
} fasttps_baseline_attn_shape;

/* Scratch tensors of Algorithm 1 (caller-allocated, device). */
typedef struct {
    void *q_rope, *k_rope;            /* [B, H_q, d], [B, H_kv, d]      Step 1 outputs                      */
    void *q_trans, *k_trans, *v_trans;/* same shapes                     Step 2 outputs ([B,N,H,d] -> [B,H,N,d], N = 1) */
    void *k_cat, *v_cat;              /* [B, H_kv, cat_seq, d]           Step 3 outputs: the updated caches */
    float *s, *p;                     /* [B, H_q, cat_seq] FP32          Step 4 / Step 5 outputs             */
} fasttps_baseline_attn_buffers;

/* Algorithm 1, Steps 1-6, one kernel launch per operator and tensor (two RoPE, three Transpose, two Concat, QK^T,
 * Softmax, PV: ten launches).  q [B,H_q,d], k_new, v_new [B,H_kv,d]; k_cache, v_cache [B,H_kv,max_seq,d] are READ
 * ONLY here: the updated caches are the Concat outputs k_cat / v_cat (rows 0..seq_lens[b] of every head).
 * pos, seq_lens [B] int32 device.  out [B,H_q,d].  Returns 0 or a negative fasttps_status code.
 * If launch_us is not NULL (HOST array of 10 floats) every launch is bracketed by CUDA events and the call
 * synchronises: launch_us[i] receives the duration of launch i in the order above. */
int fasttps_baseline_attn(const fasttps_baseline_attn_shape *shape, const fasttps_baseline_attn_buffers *buf,
                          const void *q, const void *k_new, const void *v_new, const void *k_cache, const void *v_cache,
                          const int32_t *pos, const int32_t *seq_lens, void *out, float *launch_us, void *stream);

/* Scratch tensors of Algorithm 2 (caller-allocated, device): h_g, h_s, h_u, h_m [B, K] bf16. */
typedef struct {
    void *h_g, *h_s, *h_u, *h_m;
} fasttps_baseline_mlp_buffers;

/* Algorithm 2, Steps 1-5: gate projection, SiLU, up projection, elementwise product, down projection; five
 * launches, every intermediate a bf16 tensor in device memory.  x [B,D]; wt_gate, wt_up [K,D] and wt_down [D,K] are
 * the TRANSPOSED logical matrices, plain row-major (one output per contiguous row; no tiling, no interlacing).
 * out [B,D].  launch_us as above (5 floats). */
int fasttps_baseline_mlp(int batch, int hidden, int inter, const fasttps_baseline_mlp_buffers *buf, const void *x,
                         const void *wt_gate, const void *wt_up, const void *wt_down, void *out, float *launch_us,
                         void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FASTTPS_BASELINE_H */
