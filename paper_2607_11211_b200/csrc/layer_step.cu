// Layer mode of the persistent decode-step kernel (step_kernel.cuh): one decoder layer -- RMSNorm, QKV, attention
// (Algorithm 3) with the output projection, RMSNorm, fused MLP (Algorithm 4) -- on the caller's activations in ONE
// cooperative launch, for batches of up to 8 sequences.  The three products share one shared-memory ring, so the
// weights of the next product are in flight while the current one drains; a closing pass writes x_out = h + y.
#include "step_kernel.cuh"

namespace fasttps {

int launch_layer_step(Ctx *c, const StepArgs &a, cudaStream_t st)
{
    const int ipw = warp_split(a.D).ipw;
    const int bc = a.batch == 1 ? 0 : (a.batch == 2 ? 1 : 2);
#define FT_STEP(DHV)                                                                                  \
    case DHV:                                                                                            \
        if (bc == 2) return ipw == 8 ? launch_step_inst<8, DHV, 2, true>(c, a, st) : launch_step_inst<4, DHV, 2, true>(c, a, st); \
        if (bc == 1) return ipw == 8 ? launch_step_inst<8, DHV, 1, true>(c, a, st) : launch_step_inst<4, DHV, 1, true>(c, a, st); \
        return ipw == 8 ? launch_step_inst<8, DHV, 0, true>(c, a, st) : launch_step_inst<4, DHV, 0, true>(c, a, st)
    switch (a.head_dim) {
        FT_STEP(32);
        FT_STEP(64);
        FT_STEP(96);
        FT_STEP(128);
    default: return FASTTPS_INVALID_ARG;
    }
#undef FT_STEP
}

}  // namespace fasttps
