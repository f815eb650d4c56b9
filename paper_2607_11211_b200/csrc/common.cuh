// Shared device helpers and the context layout of the FastTPS decode library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fasttps.h"

namespace fasttps {

constexpr int kMaxNB = 8;            // batch rows one weight pass of the register-resident kernels serves
constexpr int kWideMaxB = 32;        // batch rows one weight pass of the thin-GEMM kernels serves (batches above kMaxNB)
constexpr int kMaxSplits = 32;       // split-KV partitions per (sequence, head)
constexpr unsigned kFull = 0xffffffffu;

// ------------------------------------------------------------------ context

struct LayerPtrs;

struct Ctx {
    // persistent step kernel: grid barrier words, FP32 sums of the output projection
    unsigned *grid_bar;
    float *hacc;
    int opt_step_kernel;             // 1: model calls with batch <= 8 use the persistent step kernel
    int opt_gqa_share;               // 1: the attention kernel streams a K/V head once for its group of 2, 4 or 8 query heads
    fasttps_config cfg;
    int n_sm;
    cudaDeviceProp prop;
    // device workspace
    float *cos_tab, *sin_tab;        // [max_seq][d/2]
    float *attn_part;                // [max_batch][Hq][kMaxSplits][d + 2]
    int *attn_ticket;                // [max_batch][Hq]
    float *mlp_acc;                  // [max_batch][D] FP32, kept at zero between calls
    int *mlp_ticket;                 // [1]
    float *amax_val;                 // [max_batch][n_cta] lm_head argmax partials
    int *amax_idx;
    int *amax_ticket;
    uint32_t *status;                // device status word
    // activation scratch of the chains
    __nv_bfloat16 *qkv;              // [max_batch][(Hq+2Hkv) d]
    __nv_bfloat16 *attn_out;         // [max_batch][Hq d]
    __nv_bfloat16 *h;                // [max_batch][D]
    __nv_bfloat16 *xa, *xb;          // [max_batch][D]
    float *logits;                   // [max_batch][V]
    // thin-GEMM path (batches above kMaxNB; allocated when max_batch > kMaxNB)
    __nv_bfloat16 *wide_n;           // chunked [32][max(D, Hq d)] activations of the product to come
    __nv_bfloat16 *wide_a_hi, *wide_a_lo;   // chunked [32][K] MLP intermediate as a bf16 pair
    int32_t *tok;                    // [max_batch] staging for the host-buffer entry point
    int32_t *tok2;                   // [max_batch] current tokens inside the persistent step kernel
    int32_t *pinned_tok;             // pinned host staging [2][max_batch]
    uint64_t launches;
    // optional per-launch timing (CUDA events on the launch stream), off by default
    bool prof_on;
    int prof_n;                      // event pairs used
    cudaEvent_t *prof_ev;            // [2 * kProfMax]
    unsigned char *prof_cls;         // kernel class of each pair
};

constexpr int kProfMax = 8192;
constexpr int kGridBarWords = 256;          // barrier counter, sign-off counter, one group counter per query head (<= 128)
constexpr int kGridBarDoneWord = 32;        // CTAs that have left the launch (on a cache line of its own)
constexpr int kMaxStepLayers = 48;          // layers the persistent step kernel's layer table holds
enum ProfClass { kProfQkv = 0, kProfAttn, kProfOproj, kProfMlp, kProfLmHead, kProfEmbed, kProfStep, kProfClasses };

// Brackets one kernel launch with events when profiling is on.
struct ProfScope {
    Ctx *c; cudaStream_t st; int slot;
    ProfScope(Ctx *c_, int cls, cudaStream_t st_) : c(c_), st(st_), slot(-1)
    {
        if (c->prof_on && c->prof_n < kProfMax) {
            slot = c->prof_n++;
            c->prof_cls[slot] = (unsigned char)cls;
            cudaEventRecord(c->prof_ev[2 * slot], st);
        }
    }
    ~ProfScope() { if (slot >= 0) cudaEventRecord(c->prof_ev[2 * slot + 1], st); }
};

void set_last_error(cudaError_t e, const char *where);
void set_last_error_text(const char *msg);

#define FT_CUDA(call)                                                   \
    do {                                                                \
        cudaError_t e__ = (call);                                       \
        if (e__ != cudaSuccess) {                                       \
            ::fasttps::set_last_error(e__, #call);                      \
            return FASTTPS_CUDA_ERROR;                                  \
        }                                                               \
    } while (0)

// Launch of a decode-path kernel taking one argument struct.  Unless FASTTPS_PDL=0 is set, the
// launch carries the programmatic-stream-serialization attribute: the kernel may start (and
// prefetch weights, which no kernel writes) while its predecessor in the stream drains, and
// orders everything else behind `griddepcontrol.wait`.
bool pdl_enabled();

template <class Args>
static int launch_ex(void (*kernel)(Args), dim3 grid, dim3 block, size_t smem, cudaStream_t st, const Args *a)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    void *params[] = {const_cast<Args *>(a)};
    FT_CUDA(cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(kernel), params));
    return FASTTPS_OK;
}

// --------------------------------------------------------------- bf16 / loads

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// 8 bf16 (one 16-byte vector) -> 8 floats
__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8])
{
    f[0] = bf_lo(v.x); f[1] = bf_hi(v.x);
    f[2] = bf_lo(v.y); f[3] = bf_hi(v.y);
    f[4] = bf_lo(v.z); f[5] = bf_hi(v.z);
    f[6] = bf_lo(v.w); f[7] = bf_hi(v.w);
}

__device__ __forceinline__ uint32_t pack2(float a, float b)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);   // a -> low half, b -> high half
    return *reinterpret_cast<uint32_t *>(&t);
}

__device__ __forceinline__ float bf16_round(float a)
{
    return __bfloat162float(__float2bfloat16_rn(a));
}

// 2^x with the hardware approximation (2 ulp); exp2(-inf) = 0
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// streaming 16-byte load: read-only path, do not keep in L1
__device__ __forceinline__ uint4 ldg_stream(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// L2-coherent loads for data other CTAs produced in this kernel
__device__ __forceinline__ float ld_cg_f32(const float *p)
{
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ int ld_cg_s32(const int *p)
{
    int v;
    asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

__device__ __forceinline__ __nv_bfloat16 ld_cg_bf16(const __nv_bfloat16 *p)
{
    unsigned short v;
    asm volatile("ld.global.cg.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return __ushort_as_bfloat16(v);
}
__device__ __forceinline__ uint4 ld_cg_u4(const void *p)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 ld_cg_f4(const float *p)
{
    float4 v;
    asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void red_add_v2(float *p, float a, float b)
{
    asm volatile("red.global.add.v2.f32 [%0], {%1,%2};" ::"l"(p), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void red_add_v4(float *p, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// Programmatic dependent launch: wait for the producers of this kernel's inputs /
// let the next kernel in the stream start its independent prologue.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ------------------------------------------------------- warp multi-reduction

// Sums V per-lane values over the 32 lanes of a warp with a halving butterfly.
// On return v[0] of lane l holds the full sum of value index
//   which = (l >> (5 - log2 V)) for V <= 32,
// replicated over the lanes that share it.  V is a power of two, 1 <= V <= 32.
template <int V>
__device__ __forceinline__ float warp_multi_reduce(float (&v)[V], int lane)
{
    static_assert(V >= 1 && V <= 32 && (V & (V - 1)) == 0, "V must be a power of two <= 32");
    int s = 16;
#pragma unroll
    for (int n = V; n > 1; n >>= 1, s >>= 1) {
        const int half = n >> 1;
        const bool upper = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < half; ++i) {
            float send = upper ? v[i] : v[i + half];
            float keep = upper ? v[i + half] : v[i];
            v[i] = keep + __shfl_xor_sync(kFull, send, s);
        }
    }
#pragma unroll
    for (; s >= 1; s >>= 1) v[0] += __shfl_xor_sync(kFull, v[0], s);
    return v[0];
}

template <int V>
__device__ __forceinline__ int warp_multi_which(int lane)
{
    int sh = 5;
#pragma unroll
    for (int n = V; n > 1; n >>= 1) --sh;
    return V == 1 ? 0 : (lane >> sh);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) v += __shfl_xor_sync(kFull, v, s);
    return v;
}

// ---------------------------------------------------------------- launchers

struct LinearArgs {
    const __nv_bfloat16 *x;      // [B][in] rows of stride x_stride
    int x_stride;
    const __nv_bfloat16 *g;      // [in] gain or null
    float eps;
    const __nv_bfloat16 *w;      // [out][in]
    const __nv_bfloat16 *res;    // [B][out] (stride res_stride) or null
    int res_stride;
    __nv_bfloat16 *out_bf16;     // [B][out] (stride out_stride) or null
    float *out_f32;              // [B][out] or null
    int out_stride;
    int n_in, n_out, batch;
    // optional greedy argmax over out (lm_head)
    float *amax_val;
    int *amax_idx;
    int *amax_ticket;
    int32_t *next_ids;
    int32_t *adv_pos, *adv_len;  // advanced by one by the argmax finaliser when non-null
    int prof_class;
    int pair_rows;               // packed rows c and c + 8 of a tile are the output columns 2 c and 2 c + 1 (W_o)
    uint32_t *status;
};

struct AttnArgs {
    const __nv_bfloat16 *q, *k_new, *v_new;
    int q_stride, kv_stride;          // elements between consecutive sequences
    __nv_bfloat16 *k_cache, *v_cache;
    const int32_t *pos, *seq_lens;
    __nv_bfloat16 *out;
    int out_stride;
    int out_chunked;                  // 1: `out` is the chunked [32][H_q d] layout of the thin-GEMM path (wide_x_index)
    int batch, n_q_heads, n_kv_heads, head_dim, max_seq, n_splits;
    int len_add;                      // added to every seq_lens / pos entry (step index of a multi-step launch)
    int n_new;                        // new tokens per sequence (1: the decode step).  With n_new > 1 `batch` counts token
                                      // rows (sequence b, token j -> row b * n_new + j of q / k_new / v_new / out) while
                                      // the caches, pos and seq_lens stay per sequence
    const float *cos_tab, *sin_tab;
    float *part;
    int *ticket;
    uint32_t *status;
    float k_scale, v_scale;           // E4M3 caches only (k_cache / v_cache then point at bytes): value = code * scale
};

struct MlpArgs {
    const __nv_bfloat16 *x;      // [B][D]
    const __nv_bfloat16 *g;      // [D] gain or null (norm prologue)
    float eps;
    const __nv_bfloat16 *w_gu;   // packed [2K][D]
    const __nv_bfloat16 *w_down; // [K][D]
    const __nv_bfloat16 *res;    // [B][D] residual or null
    __nv_bfloat16 *out;          // [B][D]
    int D, K, batch;
    float *acc;                  // [B][D] FP32 zero on entry, zero on exit
    int *ticket;
    uint32_t *status;
};

// One layer's packed weights and caches, as the persistent step kernel reads them (device table).
struct LayerPtrs {
    const __nv_bfloat16 *g_attn, *w_qkv, *w_o, *g_mlp, *w_gu, *w_down;
    __nv_bfloat16 *k_cache, *v_cache;
};

struct StepArgs {
    const __nv_bfloat16 *embed;      // [V][D]
    const __nv_bfloat16 *g_final, *w_lm;
    const int32_t *token_ids;        // [B] tokens of the first step
    int32_t *pos, *seq_lens;         // [B]; advanced by n_steps at the end iff advance
    float *logits;                   // [B][V] of the last step, or null
    int32_t *next_ids;               // [B] argmax of the last step
    int32_t *out_ids;                // [n_steps][B] argmax of every step, or null
    int batch, n_steps, advance, n_layers;
    int D, n_q_heads, n_kv_heads, head_dim, K, V, max_seq;
    float eps;
    const float *cos_tab, *sin_tab;
    // workspace
    __nv_bfloat16 *x0, *qkv, *attn_out, *h;
    float *acc;                      // [2][B][D] FP32, zero on entry and on exit
    float *hacc;                     // [2][B][D] FP32 sums of the output projection, zero on entry and on exit
    float *attn_part;
    int *attn_ticket;
    float *amax_val;
    int *amax_idx;
    int32_t *tok;                    // [B] current tokens
    unsigned *bar;                   // [kGridBarWords], zeroed by the host per launch: [0] grid barrier arrivals, [32] CTAs signed off, [64 + h] group arrivals of head h; zero between launches
    uint32_t *status;
    __nv_bfloat16 *x_out;            // layer mode: [B][D] output of the layer (x0 is then its input; may be the same buffer)
    // the layer table travels with the launch (kernel parameter space): nothing to upload, nothing a later call
    // could overwrite while this launch is still queued
    LayerPtrs layers[kMaxStepLayers];
};

// ---- thin-GEMM path (wide.cu) ----
// Activations travel between its kernels in "chunked" form, so that one k chunk of all 32 batch rows is ONE
// contiguous block (one bulk copy into the ring) whose rows already carry the padding that keeps the shared-memory
// loads free of bank conflicts: element (b, k) of a [32][K] tensor sits at ((k / C) * 32 + b) * R + k % C, with
// C = 256, R = 288 for the tiled products and C = 128, R = 136 for the down projection.
constexpr int kWideXChunk = 256, kWideXRow = 288;       // 576 bytes per row: 512 + 64
constexpr int kWideAChunk = 128, kWideARow = 136;       // 272 bytes per row: 256 + 16
__host__ __device__ inline size_t wide_x_elems(int K) { return (size_t)((K + kWideXChunk - 1) / kWideXChunk) * kWideMaxB * kWideXRow; }
__host__ __device__ inline size_t wide_a_elems(int K) { return (size_t)((K + kWideAChunk - 1) / kWideAChunk) * kWideMaxB * kWideARow; }
__host__ __device__ inline size_t wide_x_index(int b, int k) { return ((size_t)(k / kWideXChunk) * kWideMaxB + b) * kWideXRow + k % kWideXChunk; }
__host__ __device__ inline size_t wide_a_index(int b, int k) { return ((size_t)(k / kWideAChunk) * kWideMaxB + b) * kWideARow + k % kWideAChunk; }

enum { kWideStore = 0, kWideSilu = 1 };
struct WideArgs {
    const __nv_bfloat16 *x;      // chunked [32][K] activations (already normalised)
    const __nv_bfloat16 *w;      // tiled [n_out padded to 16][K]
    int K, n_out, batch;
    int epi;                     // kWideStore: out = sums (+ res); kWideSilu: a = silu(gate) * up from interlaced rows
    const __nv_bfloat16 *res;    // [B][n_out] residual or null
    int res_stride;
    __nv_bfloat16 *out_bf16;     // [B][n_out] or null
    float *out_f32;              // [B][n_out] or null
    int out_stride;
    int pair_rows;               // rows c and c + 8 of a tile are the output columns 2 c and 2 c + 1 (W_o)
    __nv_bfloat16 *a_hi, *a_lo;  // kWideSilu: chunked [32][n_out / 2] intermediate, high and low part
    float *amax_val;             // optional greedy argmax over out (lm_head), as in LinearArgs
    int *amax_idx;
    int *amax_ticket;
    int32_t *next_ids;
    int32_t *adv_pos, *adv_len;
    uint32_t *status;
};
struct WideDownArgs {
    const __nv_bfloat16 *a_hi, *a_lo;    // chunked [32][K] intermediate
    const __nv_bfloat16 *w;      // packed W_down (octet blocks)
    int D, K, batch;
    float *acc;                  // [B][D] FP32 sums, added to
    uint32_t *status;
};
struct PrepArgs {
    const __nv_bfloat16 *x;      // [B][D] residual, rows of stride x_stride, or null
    int x_stride;
    float *acc;                  // [B][D] FP32 sums to fold in (then cleared), or null
    const __nv_bfloat16 *g;      // [D] gain: n_out = rmsnorm(x + acc); null: n_out = x + acc
    float eps;
    __nv_bfloat16 *x_store;      // [B][D] receives bf16(x + acc), or null
    __nv_bfloat16 *n_out;        // chunked [32][D] (the activations of the product to come), or null
    int D, batch;
};
int configure_wide_kernels();
int launch_wide_linear(Ctx *c, const WideArgs &a, int prof_class, cudaStream_t st);
int launch_wide_down(Ctx *c, const WideDownArgs &a, cudaStream_t st);
int launch_prep_rows(Ctx *c, const PrepArgs &a, int prof_class, cudaStream_t st);

int launch_linear(Ctx *c, const LinearArgs &a, cudaStream_t st);
bool step_kernel_supported(const Ctx *c, int batch, bool layer_mode = false);
int launch_step(Ctx *c, const StepArgs &a, cudaStream_t st);
int launch_layer_step(Ctx *c, const StepArgs &a, cudaStream_t st);
int launch_attn(Ctx *c, const AttnArgs &a, cudaStream_t st, bool fp8 = false);
int launch_mlp(Ctx *c, const MlpArgs &a, cudaStream_t st);
int launch_embed(Ctx *c, const __nv_bfloat16 *embed, const int32_t *ids, __nv_bfloat16 *x, int batch, cudaStream_t st);
int launch_pack(Ctx *c, int kind, const void *src, void *dst, bool inverse, cudaStream_t st);
int attn_splits_for(const Ctx *c, int batch);
size_t packed_elems(const fasttps_config &f, int kind);
// A reduction length the tensor-core kernels can split over their warps: a multiple of 128,
// at most 3072, or a multiple of 256 from 2048 to 6144.
inline bool reduction_length_ok(int n)
{
    return n > 0 && ((n % 128 == 0 && n / 128 <= 24) || (n >= 2048 && n % 256 == 0 && n / 256 <= 24));
}
int configure_attn_kernels();
int configure_linear_kernels();
int configure_mlp_kernels();

}  // namespace fasttps
