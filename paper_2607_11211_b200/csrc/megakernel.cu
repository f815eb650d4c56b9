// Model mode of the persistent decode-step kernel (step_kernel.cuh): whole decode steps of the stack, from the
// embedding gather to the greedy argmax, for batches of up to 8 sequences.
#include "step_kernel.cuh"

namespace fasttps {

// True when the persistent kernel can serve this model shape and batch.
bool step_kernel_supported(const Ctx *c, int batch, bool layer_mode)
{
    const fasttps_config &f = c->cfg;
    const WarpSplit s = warp_split(f.hidden);
    if (batch < 1 || batch > kMaxNB) return false;
    if (f.n_q_heads * f.head_dim != f.hidden) return false;      // one reduction length for every product
    if (s.nw < 1 || s.nw > 12) return false;
    if (f.n_q_heads > kMaxStepHeads || f.n_q_heads > c->n_sm) return false;   // a group of at least one CTA per query head
    if (layer_mode) return true;                                 // one layer, no embedding, no logits
    if (f.n_layers > kMaxStepLayers || f.vocab < 1 || f.n_layers < 1) return false;
    return true;
}

int launch_step(Ctx *c, const StepArgs &a, cudaStream_t st)
{
    const int ipw = warp_split(a.D).ipw;
    const int bc = a.batch == 1 ? 0 : (a.batch == 2 ? 1 : 2);
#define FT_STEP(DHV)                                                                                  \
    case DHV:                                                                                            \
        if (bc == 2) return ipw == 8 ? launch_step_inst<8, DHV, 2, false>(c, a, st) : launch_step_inst<4, DHV, 2, false>(c, a, st); \
        if (bc == 1) return ipw == 8 ? launch_step_inst<8, DHV, 1, false>(c, a, st) : launch_step_inst<4, DHV, 1, false>(c, a, st); \
        return ipw == 8 ? launch_step_inst<8, DHV, 0, false>(c, a, st) : launch_step_inst<4, DHV, 0, false>(c, a, st)
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

// Diagnostic entry point: the attention shares of one head group, computed on the host by the same code the
// step kernel runs on the device.
extern "C" int fasttps_attention_shares(const int32_t *seq_lens, const int32_t *pos, int batch, int max_seq, int step,
                                        int group_size, int32_t *seg_out, int32_t *nseg_out)
{
    using namespace fasttps;
    if (!seq_lens || !pos || !seg_out || !nseg_out || batch < 1 || batch > kMaxNB || group_size < 1 ||
        group_size > kMaxSplits || max_seq < 1 || step < 0)
        return FASTTPS_INVALID_ARG;
    int mprime = 0;
    for (int gs = 0; gs < group_size; ++gs) {
        GroupSegs segs;
        int ncta[kMaxNB], cuts[kMaxSplits + 1];
        build_attention_shares(seq_lens, pos, max_seq, step, batch, group_size, gs, /*head=*/0, /*in_group=*/true, &segs, ncta,
                               &mprime, cuts);
        nseg_out[gs] = segs.n;
        for (int j = 0; j < segs.n; ++j) {
            int32_t *o = seg_out + ((size_t)gs * kMaxNB + j) * 5;
            o[0] = segs.seg[j].b; o[1] = segs.seg[j].r0; o[2] = segs.seg[j].r1;
            o[3] = segs.seg[j].first_cta; o[4] = segs.seg[j].n_cta;
        }
    }
    return mprime;
}

