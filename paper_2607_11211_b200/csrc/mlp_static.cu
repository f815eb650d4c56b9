// fasttps_mlp_decode_static: the fused MLP kernel with its scratch memory in a fixed device array of this
// library instead of the context workspace.  The paper has no counterpart; the arithmetic is that of
// fasttps_mlp_decode (Algorithm 4 / Eq. 1), through the very same kernel.
//
// Who needs it: code that must not allocate device memory at the point of the call -- a caller inside a
// region where the allocator is off limits (its memory pool is frozen, or another library holds the
// allocator lock), or one that wants no dependence on the lifetime of a workspace it did not create.  The
// scratch of the MLP kernel is small and bounded (an FP32 accumulator of batch x hidden values plus one
// counter), so it can live in the data segment of the library: the driver places it when the module is
// loaded and it needs no allocation call, neither here nor in the caller.
//
// Rules of use:
//   * batch <= 8 and hidden <= 6144 (192 KB of accumulator); anything larger is rejected, not truncated;
//   * the FIRST call on a device looks the array's address up (cudaGetSymbolAddress, which may load the
//     module) and caches it; make that call during set-up, before any stream capture;
//   * the array is ONE per device and process: two calls that overlap in time (different streams, or
//     different threads) race on it.  Calls on one stream are ordered and safe.
#include <cstdio>
#include <mutex>

#include "common.cuh"

namespace fasttps {

namespace {

constexpr int kStaticMaxBatch = 8;
constexpr int kStaticMaxHidden = 6144;
constexpr size_t kStaticHeadBytes = 256;       // the arrival counter, alone in its 256 bytes
constexpr size_t kStaticAccBytes = (size_t)kStaticMaxBatch * kStaticMaxHidden * sizeof(float);

static __device__ __align__(256) unsigned char g_mlp_static_scratch[kStaticHeadBytes + kStaticAccBytes];

constexpr int kStaticMaxDevices = 64;
std::mutex g_static_mu;
void *g_static_addr[kStaticMaxDevices];        // per device, null until looked up

// Address of the scratch array on the context's device, which must be the current one (looked up once per device).
int static_scratch(int ctx_device, unsigned char **out)
{
    int dev = -1;
    FT_CUDA(cudaGetDevice(&dev));
    if (dev != ctx_device) {
        set_last_error_text("fasttps_mlp_decode_static: the context's device is not the current device");
        return FASTTPS_INVALID_ARG;
    }
    if (dev < 0 || dev >= kStaticMaxDevices) {
        set_last_error_text("fasttps_mlp_decode_static: device ordinal beyond the per-device address table");
        return FASTTPS_INVALID_ARG;
    }
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_addr[dev]) {
        void *p = nullptr;
        FT_CUDA(cudaGetSymbolAddress((void **)&p, g_mlp_static_scratch));
        g_static_addr[dev] = p;
    }
    *out = static_cast<unsigned char *>(g_static_addr[dev]);
    return FASTTPS_OK;
}

}  // namespace

}  // namespace fasttps

using namespace fasttps;

extern "C" int fasttps_mlp_decode_static(fasttps_ctx *ctx, const void *x, const void *w_gate_up, const void *w_down,
                                         void *out, int batch, void *stream)
{
    if (!ctx) return FASTTPS_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    const int D = c->cfg.hidden;
    if (batch < 1 || batch > kStaticMaxBatch || D > kStaticMaxHidden) {
        char msg[256];
        snprintf(msg, sizeof msg,
                 "fasttps_mlp_decode_static: batch %d x hidden %d does not fit the static scratch (batch <= %d, hidden <= %d)",
                 batch, D, kStaticMaxBatch, kStaticMaxHidden);
        set_last_error_text(msg);
        return FASTTPS_INVALID_ARG;
    }
    if (batch > c->cfg.max_batch) return FASTTPS_INVALID_ARG;
    if (!x || !w_gate_up || !w_down || !out) return FASTTPS_INVALID_ARG;
    if (((uintptr_t)x | (uintptr_t)w_gate_up | (uintptr_t)w_down | (uintptr_t)out) & 15) return FASTTPS_INVALID_ARG;

    unsigned char *scratch = nullptr;
    const int rc = static_scratch(c->cfg.device, &scratch);
    if (rc != FASTTPS_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // The kernel expects the counter and the accumulator rows it uses to be zero.  They are cleared on every
    // call, on the caller's stream: an earlier call that was aborted may have left anything behind.
    FT_CUDA(cudaMemsetAsync(scratch, 0, kStaticHeadBytes + (size_t)batch * D * sizeof(float), st));

    MlpArgs a;
    a.x = static_cast<const __nv_bfloat16 *>(x); a.g = nullptr; a.eps = c->cfg.rms_eps;
    a.w_gu = static_cast<const __nv_bfloat16 *>(w_gate_up);
    a.w_down = static_cast<const __nv_bfloat16 *>(w_down);
    a.res = nullptr; a.out = static_cast<__nv_bfloat16 *>(out);
    a.D = D; a.K = c->cfg.inter; a.batch = batch;
    a.ticket = reinterpret_cast<int *>(scratch);
    a.acc = reinterpret_cast<float *>(scratch + kStaticHeadBytes);
    a.status = c->status;
    return launch_mlp(c, a, st);
}
