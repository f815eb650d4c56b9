/*
 * fasttps.h -- C ABI of the FastTPS decode (token-phase) library for NVIDIA B200 (sm_100a).
 *
 * The library implements one decode step of a decoder-only transformer layer as
 * described by the FastTPS paper: joint RoPE on the new q/k, in-place append of
 * k/v into a preallocated ("static") KV cache, single-query attention over that
 * cache (Algorithm 3 "GKVC & TPSFLAT", Eq. 2), and the fused SwiGLU MLP
 * (Algorithm 4 "MLP Implementation", Eq. 1, Eq. 31), plus the projections and
 * norms that chain them into a layer and a model (Figure 1, Section 2.2, 2.3).
 *
 * Conventions that hold for every entry point
 *   - "device" pointers are CUDA device memory on the context's GPU, owned by the
 *     caller, contiguous, 16-byte aligned.  bf16 unless stated.  Nothing is
 *     retained after the call returns except where stated (packed weights are
 *     read on every call and must stay alive).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *     only enqueue work and return without synchronising.  One context must not be
 *     used from two streams at the same time (its workspace is shared).
 *   - Return value: FASTTPS_OK or a negative fasttps_status code.  Nothing is
 *     thrown across the boundary.  Conditions that only the device can see (a
 *     sequence whose cache is full, a negative position, a bounded wait that ran
 *     out) never trap: the affected sequence is skipped and a bit is set in the
 *     context's device status word, read with fasttps_get_status().
 *   - There is no CPU fallback: every step runs in the library's CUDA kernels.
 */
#ifndef FASTTPS_H
#define FASTTPS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fasttps_ctx fasttps_ctx;

typedef enum {
    FASTTPS_OK = 0,
    FASTTPS_INVALID_ARG = -1,   /* null/misaligned pointer, batch out of range, unsupported dims */
    FASTTPS_CUDA_ERROR = -2,    /* a CUDA runtime call or launch failed; see fasttps_last_error() */
    FASTTPS_OUT_OF_MEMORY = -3  /* workspace allocation failed in fasttps_create() */
} fasttps_status;

/* bits of the device status word */
#define FASTTPS_DEV_CACHE_FULL   1u   /* some seq_lens[b] >= max_seq (or < 0): sequence skipped */
#define FASTTPS_DEV_BAD_POSITION 2u   /* some pos[b] < 0 or >= max_seq: sequence skipped        */
#define FASTTPS_DEV_WAIT_TIMEOUT 4u   /* a bounded wait on an asynchronous copy ran out         */
#define FASTTPS_DEV_BAD_TOKEN    8u   /* a token id outside [0, vocab): row 0 used instead      */

/* Model shape and limits.  Supported: hidden % 8 == 0, hidden <= 6144;
 * head_dim in {32, 64, 96, 128}; n_q_heads % n_kv_heads == 0; inter % 8 == 0;
 * (n_q_heads * head_dim) % 8 == 0 and <= 6144; max_batch >= 1; max_seq >= 1.
 * vocab and n_layers may be 0 when only the block-level calls are used. */
typedef struct {
    int hidden;        /* D                                   */
    int n_q_heads;     /* H_q                                 */
    int n_kv_heads;    /* H_kv (H_q for multi-head attention) */
    int head_dim;      /* d                                   */
    int inter;         /* K, MLP intermediate size            */
    int vocab;         /* V                                   */
    int n_layers;
    int max_batch;     /* largest batch any call will use     */
    int max_seq;       /* N_p + N_r: rows per head in a cache; also the largest position + 1 */
    float rms_eps;
    float rope_theta;
    int device;        /* CUDA device ordinal                 */
} fasttps_config;

/* Packed weights of one layer (device pointers; see the packing calls). */
typedef struct {
    const void *g_attn_norm;  /* [D] bf16 gain of the norm before attention */
    const void *w_qkv;        /* packed FASTTPS_W_QKV     */
    const void *w_o;          /* packed FASTTPS_W_O       */
    const void *g_mlp_norm;   /* [D] bf16 gain of the norm before the MLP   */
    const void *w_gate_up;    /* packed FASTTPS_W_GATE_UP */
    const void *w_down;       /* packed FASTTPS_W_DOWN    */
} fasttps_layer_weights;

typedef enum {
    FASTTPS_W_QKV = 0,      /* logical [D, (H_q + 2 H_kv) d], columns q | k | v, head-major */
    FASTTPS_W_O = 1,        /* logical [H_q d, D]                                           */
    FASTTPS_W_GATE_UP = 2,  /* logical [D, 2K], columns [0,K) gate and [K,2K) up            */
    FASTTPS_W_DOWN = 3,     /* logical [K, D]                                               */
    FASTTPS_W_LM_HEAD = 4   /* logical [V, D]                                               */
} fasttps_weight_kind;

/* Create a context: validates cfg, selects cfg->device, allocates the workspace
 * (split-KV partials, FP32 accumulators, tickets, activation scratch for the
 * layer/model chains, the RoPE cos/sin table, the status word) and builds the
 * cos/sin table on the host in double precision.  The only call that allocates
 * or synchronises besides fasttps_destroy/get_status/model_decode_host. */
int fasttps_create(fasttps_ctx **out, const fasttps_config *cfg);
int fasttps_destroy(fasttps_ctx *ctx);

/* One-time weight packing, outside the decode path: the offline re-layout of
 * Section 3.2 item 1 ("interlaced layout of gate-up weights").  `src` is the
 * logical row-major bf16 matrix described at fasttps_weight_kind, `dst` a
 * device buffer of fasttps_packed_bytes(kind) bytes.  Packed layouts (bf16):
 *   QKV, LM_HEAD: the transposed matrix W^T [out, in], with `out` padded up to a
 *            multiple of 16 by zero rows, cut into tiles of 16 output rows x 32 inputs;
 *            a tile is stored row-major (1 KB), tiles are ordered by (row tile, input
 *            block), so that the share of a CTA -- a run of row tiles -- is one contiguous
 *            byte range and one tile is the A operand of two tensor-core instructions;
 *   O:       the same tiling, with the 16 rows of a tile paired: row r < 8 of row tile J is output
 *            column 16J + 2r, row r + 8 is column 16J + 2r + 1, so that the two sums a thread of the
 *            tensor-core product holds for a batch row are neighbours (one 8-byte reduction);
 *   GATE_UP: the same tiling of a [2K, D] matrix whose rows are interlaced in blocks of
 *            8: for j-octet J the rows 16J..16J+7 are gate columns 8J..8J+7 and
 *            16J+8..16J+15 the matching up columns, so a gate value and its up value
 *            come out of the same tile;
 *   DOWN:    for every j-octet J (8 rows of the logical [K, D] matrix) and block of 32
 *            output columns one 512-byte block holding W_down[8J..8J+7, 32c..32c+31] in
 *            the register order of two m16n8k8 A operands whose rows are assigned to the
 *            output columns so that a thread's four results are four consecutive columns
 *            (one 16-byte reduction); blocks ordered by (J, c), so a CTA's octets are again
 *            one contiguous byte range.
 * Limits: D and H_q d multiples of 128 up to 3072 or multiples of 256 from 2048 to 6144;
 * K a multiple of 8. */
size_t fasttps_packed_bytes(const fasttps_ctx *ctx, int kind);
int fasttps_pack_weight(fasttps_ctx *ctx, int kind, const void *src, void *dst, void *stream);
/* Inverse of fasttps_pack_weight (for round-trip checks). */
int fasttps_unpack_weight(fasttps_ctx *ctx, int kind, const void *src_packed, void *dst_logical, void *stream);

/* Algorithm 3 (GKVC & TPSFLAT), one decode step for `batch` sequences.
 *   q [B,H_q,d], k_new [B,H_kv,d], v_new [B,H_kv,d]   (before RoPE)
 *   k_cache, v_cache [B,H_kv,max_seq,d]   in/out: row seq_lens[b] of every head
 *       receives bf16(rope(k_new)) resp. v_new -- exactly B*H_kv runs of d
 *       elements at element offset (b*H_kv+h)*max_seq*d + seq_lens[b]*d (Eq. 2);
 *       no other element is written and none is re-loaded to be moved.
 *   pos [B] int32 device: rotary position of the new token.
 *   seq_lens [B] int32 device: rows already cached (N_p) = the row written now.
 *   out [B,H_q,d]: softmax(q' K^T / sqrt(d)) V over rows 0..seq_lens[b] inclusive.
 * Query head h uses kv head h / (H_q/H_kv) (Section 4.1).  With 2 to 16 query heads per kv head every
 * cached row is read once for its whole group and the two products run on the tensor cores (FP32
 * accumulation): there the rotated q and the softmax weights enter the products as pairs of bf16 numbers
 * (value = hi + lo), or rounded to bf16 once with option "gqa_share" 2; with one query head per kv head, more
 * than 16, or option "gqa_share" 0, both stay FP32.  Neither pos nor seq_lens is advanced. */
int fasttps_attn_decode(fasttps_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                        void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens,
                        void *out, int batch, void *stream);

/* Algorithm 3 with N = n_new new tokens per sequence (the algorithm takes Q, K, V in R^{B x N x H x d}; speculative
 * verification, chunked decode), 1 <= n_new <= 8, batch * n_new <= max_batch:
 *   q [B,N,H_q,d], k_new, v_new [B,N,H_kv,d], out [B,N,H_q,d]; caches, pos, seq_lens [B] as above.
 * Token j of sequence b is rotated at position pos[b] + j, goes into row seq_lens[b] + j of every head (B*N*H_kv
 * runs of d elements are written, nothing else) and attends rows 0 .. seq_lens[b] + j: the cached rows and the new
 * tokens up to and including itself (causal inside the chunk).  While n_new * (H_q / H_kv) <= 16 the new tokens of a
 * sequence (times the query heads of a kv head) share ONE pass over the cached rows, on the tensor cores as described
 * above; otherwise, and with option "gqa_share" 0, the cached rows are streamed once per new token and query head in
 * FP32.  The new rows are scored from shared memory either way.  A sequence whose n_new rows do not all fit
 * (seq_lens[b] + n_new > max_seq) is skipped and reported. */
int fasttps_attn_decode_multi(fasttps_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                              void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens,
                              void *out, int batch, int n_new, void *stream);

/* Algorithm 4 steps 2-15 / Eq. 1: out = (silu(x W_gate) * (x W_up)) W_down.
 *   x [B,D]; w_gate_up, w_down packed; out [B,D].  The gate_up products, the
 *   SiLU*mul result and the down-projection partial sums stay on chip; partial
 *   sums of the CTAs meet in an FP32 accumulator of the workspace. */
int fasttps_mlp_decode(fasttps_ctx *ctx, const void *x, const void *w_gate_up, const void *w_down,
                       void *out, int batch, void *stream);

/* Variant of fasttps_mlp_decode that keeps its scratch out of the workspace and allocates nothing.  The paper has
 * no counterpart: the arithmetic and the kernel are those of fasttps_mlp_decode; only the scratch of
 * the kernel (the FP32 accumulator of batch x hidden partial sums and its arrival counter) lives in a
 * fixed array in the library's own device data segment instead of the context workspace.  It is for
 * callers that may not allocate device memory where they call (a frozen memory pool, an allocator
 * lock held elsewhere) and do not want to depend on a workspace they did not size.
 *   Limits: batch <= 8 and hidden <= 6144 (192 KB of accumulator); larger requests return
 *   FASTTPS_INVALID_ARG with a message in fasttps_last_error() and launch nothing.
 *   Set-up: the first call on a device looks the array's address up once (this may load the module);
 *   make it during initialisation, before capturing a stream.  No call allocates or frees.
 *   Every call clears the counter and the accumulator rows it uses, on `stream`, before the kernel.
 *   The context still supplies the model shape and its device status word (a bounded wait that ran out is
 *   reported there), and the call must be made with the context's device current: the array is per device,
 *   and a call made with another device current returns FASTTPS_INVALID_ARG.
 *   The array is one per device and process: calls that overlap in time (other streams or threads)
 *   race on it; calls on one stream are ordered. */
int fasttps_mlp_decode_static(fasttps_ctx *ctx, const void *x, const void *w_gate_up, const void *w_down,
                              void *out, int batch, void *stream);

/* Algorithm 3 over a KV cache of 8-bit floating-point codes (E4M3: 4 exponent bits, bias 7, 3 mantissa bits, no
 * infinities, largest value 448), the quantised cache the paper names as compatible (Section 6.2); one FP32 scale per
 * tensor, given by the caller:
 *   k_cache, v_cache [B,H_kv,max_seq,d] uint8 device, updated in place: row seq_lens[b] of every head receives the
 *       codes of rope(k_new) / k_scale resp. v_new / v_scale (FP32 division, round to nearest even, magnitudes
 *       beyond 448 saturate): B*H_kv runs of d BYTES, nothing else is written.  A stored code c stands for c * scale.
 *   q, k_new, v_new, pos, seq_lens, out as in fasttps_attn_decode (bf16).  The new token attends its own row as
 *       stored (the dequantised codes).  k_scale, v_scale > 0 and finite, else FASTTPS_INVALID_ARG.
 * Every cached row is read once for all query heads of its kv head (1 to 16 of them, else FASTTPS_INVALID_ARG); the
 * codes are widened to fp16 in registers (exact) and the two products run on the tensor cores with the rotated q and
 * the softmax weights as fp16 hi + lo pairs, FP32 accumulation. */
int fasttps_attn_decode_fp8(fasttps_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                            void *k_cache, void *v_cache, float k_scale, float v_scale, const int32_t *pos,
                            const int32_t *seq_lens, void *out, int batch, void *stream);

/* Building block of the chain (QKV, output projection, lm_head; Figure 1):
 *   out[b,n] = (g_norm ? rmsnorm(x[b], g_norm) : x[b]) . W[n,:] (+ residual[b,n])
 *   x [B,in]; w packed [out,in]; residual [B,out] or NULL; out_bf16 [B,out] or NULL;
 *   out_f32 [B,out] float or NULL (at least one output).  in = D for QKV/LM_HEAD,
 *   H_q d for O.  The normalised input is rounded to bf16 before the product. */
int fasttps_linear_decode(fasttps_ctx *ctx, int kind, const void *x, const void *g_norm, const void *w,
                          const void *residual, void *out_bf16, float *out_f32, int batch, void *stream);

/* One decoder layer: RMSNorm -> QKV -> attn_decode -> o_proj (+x) -> RMSNorm -> MLP (+h).
 *   x_in [B,D], x_out [B,D] (may alias x_in); caches, pos, seq_lens as in
 *   fasttps_attn_decode (caches of THIS layer).
 * For batch <= 8 (and n_q_heads * head_dim == hidden, n_q_heads <= 128 and <= the number of SMs) the layer
 * is ONE cooperative launch of the persistent kernel described at fasttps_model_decode, restricted to one
 * layer: the three products share one shared-memory ring and meet at grid-wide barriers; otherwise (and with
 * option "step_kernel" 0) it is one kernel per product, chained with programmatic dependent launch. */
int fasttps_layer_decode(fasttps_ctx *ctx, const fasttps_layer_weights *w, const void *x_in, void *x_out,
                         void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens,
                         int batch, void *stream);

/* The same layer over caches of E4M3 codes (fasttps_attn_decode_fp8 in place of fasttps_attn_decode; Section 6.2):
 * k_cache, v_cache uint8 [B,H_kv,max_seq,d], one scale per tensor; batch <= 32.  Runs one kernel per product (the
 * persistent layer kernel reads bf16 caches).  1 to 16 query heads per kv head, else FASTTPS_INVALID_ARG. */
int fasttps_layer_decode_fp8(fasttps_ctx *ctx, const fasttps_layer_weights *w, const void *x_in, void *x_out,
                             void *k_cache, void *v_cache, float k_scale, float v_scale, const int32_t *pos,
                             const int32_t *seq_lens, int batch, void *stream);

/* The same layer for n_new tokens per sequence (Algorithm 3 and Algorithm 4 for general N): x_in, x_out
 * [B * n_new, D], token j of sequence b in row b * n_new + j; pos, seq_lens [B]; 1 <= n_new <= 8 and
 * batch * n_new <= max_batch.  The projections and the MLP treat the token rows alike; the attention is
 * fasttps_attn_decode_multi.  Runs one kernel per product. */
int fasttps_layer_decode_multi(fasttps_ctx *ctx, const fasttps_layer_weights *w, const void *x_in, void *x_out,
                               void *k_cache, void *v_cache, const int32_t *pos, const int32_t *seq_lens,
                               int batch, int n_new, void *stream);

/* Whole stack, one token per sequence: embedding gather -> n_layers layers ->
 * final RMSNorm -> logits -> greedy argmax (lowest index on ties).
 *   embed [V,D]; layers: HOST array [n_layers]; g_final [D]; w_lm_head packed;
 *   k_caches, v_caches: HOST arrays [n_layers] of device cache pointers;
 *   token_ids [B] int32 device; pos, seq_lens [B] int32 device, each advanced by
 *   one at the end of the step iff advance != 0;
 *   logits [B,V] float device or NULL (an internal buffer is used);
 *   next_ids [B] int32 device (may be the same buffer as token_ids).
 * For batch <= 8 (and n_q_heads * head_dim == hidden, n_q_heads <= 128 and <= the number of SMs,
 * n_layers <= 48) the whole step is ONE cooperative
 * launch of a persistent kernel (one CTA per SM, grid-wide barriers between the products,
 * weights and K/V streamed ahead through shared memory across all boundaries); larger
 * batches run one kernel per product, chained with programmatic dependent launch.  The
 * layer pointers are copied into the launch parameters at the call: the host arrays may be
 * reused or changed as soon as the call returns, and calls that pass different tables (other
 * caches, other weights) may follow one another on the stream without synchronising. */
int fasttps_model_decode(fasttps_ctx *ctx, const void *embed, const fasttps_layer_weights *layers,
                         const void *g_final, const void *w_lm_head,
                         void *const *k_caches, void *const *v_caches,
                         const int32_t *token_ids, int32_t *pos, int32_t *seq_lens,
                         float *logits, int32_t *next_ids, int batch, int advance, void *stream);

/* Greedy decode of n_steps consecutive tokens per sequence without returning to the host:
 * step 0 consumes token_ids [B], every later step the argmax of the step before it.
 *   out_ids [n_steps, B] int32 device: the token chosen at every step;
 *   pos, seq_lens are advanced by n_steps (sequences that would outgrow max_seq are
 *   reported in the status word and stop contributing at that point).
 * For batch <= 8 all steps run inside one launch of the persistent kernel, so the weight
 * stream never stops between tokens. */
int fasttps_model_generate(fasttps_ctx *ctx, const void *embed, const fasttps_layer_weights *layers,
                           const void *g_final, const void *w_lm_head,
                           void *const *k_caches, void *const *v_caches,
                           const int32_t *token_ids, int32_t *pos, int32_t *seq_lens,
                           int32_t *out_ids, int n_steps, int batch, void *stream);

/* End-to-end variant with HOST token buffers: copies host_token_ids [B] to the
 * device, runs fasttps_model_decode(advance = 1) on `stream`, copies next ids
 * back into host_next_ids [B] and synchronises the stream.  pos/seq_lens stay
 * on the device. */
int fasttps_model_decode_host(fasttps_ctx *ctx, const void *embed, const fasttps_layer_weights *layers,
                              const void *g_final, const void *w_lm_head,
                              void *const *k_caches, void *const *v_caches,
                              const int32_t *host_token_ids, int32_t *pos, int32_t *seq_lens,
                              int32_t *host_next_ids, int batch, void *stream);

/* Tuning switches of a context (host side, take effect at the next call):
 *   "step_kernel" 0/1  route model and layer calls with batch <= 8 through the persistent step kernel
 *                      (default: environment variable FASTTPS_STEP_KERNEL, else 1).
 *   "gqa_share" 0/1    fasttps_attn_decode and the per-product chain read every cached K/V row once for
 *                      the whole group of query heads that shares it (Section 4.1; groups of 2 to 16)
 *                      instead of once per query head (default 1; 0 is the comparison point).
 * Unknown names return FASTTPS_INVALID_ARG. */
int fasttps_set_option(fasttps_ctx *ctx, const char *name, int value);

/* Synchronises the device and returns the status word (then clears it).  If the word reports a bounded wait
 * that ran out, the workspace's accumulators, tickets and barrier words are cleared as well: the kernels of the
 * abandoned call left them in an unknown state, and the next call must find them at zero. */
int fasttps_get_status(fasttps_ctx *ctx, uint32_t *host_status);
/* Test hook: puts the workspace into the state an abandoned call leaves behind -- garbage in the accumulators,
 * tickets and barrier words, the FASTTPS_DEV_WAIT_TIMEOUT bit set -- with host-side memsets only (no kernel runs,
 * nothing waits).  The next fasttps_get_status() must report the bit and make the context usable again. */
int fasttps_debug_leave_workspace_dirty(fasttps_ctx *ctx);
/* Optional per-launch timing for benchmarks: while enabled, every kernel launch of this
 * context is bracketed by CUDA events on its stream (up to 8192 launches; not usable during
 * stream capture).  fasttps_profile_read() synchronises and sums the elapsed time and the
 * launch count per kernel class into arrays of FASTTPS_PROFILE_CLASSES entries, in the order
 * qkv projection, attention, output projection, fused MLP, lm_head, embedding gather,
 * persistent step kernel. */
#define FASTTPS_PROFILE_CLASSES 7
int fasttps_profile(fasttps_ctx *ctx, int enable);
int fasttps_profile_read(fasttps_ctx *ctx, double *ms_per_class, uint64_t *launches_per_class);
/* Number of kernels this context has launched so far (host counter). */
uint64_t fasttps_launch_count(const fasttps_ctx *ctx);
/* Number of CTAs the attention kernel is launched with for this batch (how many of them take part is decided
 * on the device from the lengths; for tests/benchmarks). */
int fasttps_attn_splits(const fasttps_ctx *ctx, int batch);
/* Diagnostic, host only (no context, no CUDA call; no counterpart in the paper): how the persistent step kernel
 * cuts the cached rows of one query head, all sequences of the batch end to end plus one new row each (Algorithm 3
 * over a ragged batch), into shares for the group_size CTAs of the head in decode step `step` of a launch.
 * seq_lens, pos: HOST arrays of `batch` (<= 8) entries, as passed to fasttps_model_decode.  For share g,
 * nseg_out[g] segments are written to seg_out[(g * 8 + j) * 5 + 0..4] = sequence, first row, end row (exclusive; row
 * seq_len is the new row), first share that holds rows of that sequence, number of shares that do.  Returns the
 * number of shares in use (<= group_size; 0 if no sequence is valid), or a negative FASTTPS error code. */
int fasttps_attention_shares(const int32_t *seq_lens, const int32_t *pos, int batch, int max_seq, int step,
                             int group_size, int32_t *seg_out, int32_t *nseg_out);
/* Diagnostic, host only (no context, no CUDA call; no counterpart in the paper): how the stand-alone attention
 * kernel cuts the flattened row space -- for every sequence and head (K/V heads on grouped-query shapes with up to
 * 16 query heads per K/V head, query heads otherwise) the cached rows plus the new row -- into shares for n_cta
 * CTAs.  seq_lens, pos: HOST arrays of `batch` entries.  Writes up to max_segs segments, in CTA order, as
 * seg_out[7 i + 0..6] = CTA, sequence, head, first row, end row (exclusive; row seq_len is the new row), first CTA
 * that holds rows of that head, number of CTAs that do (at most 32: a head has that many partial records).
 * Returns the number of segments (which may exceed max_segs), or a negative FASTTPS error code. */
int fasttps_attention_walk(const int32_t *seq_lens, const int32_t *pos, int batch, int heads, int max_seq, int n_cta,
                           int32_t *seg_out, int max_segs);
const char *fasttps_strerror(int code);
/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char *fasttps_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FASTTPS_H */
