// Pieces shared by the persistent decode-step kernels: the grid-wide barrier, the split of work units over
// CTAs, the shared-memory layout, and the attention arguments of a layer.
#pragma once
#include "attn_core.cuh"
#include "mlp_core.cuh"
#include "stream_launch.cuh"

namespace fasttps {

constexpr unsigned long long kGridWaitNanos = 500ull * 1000 * 1000;   // 0.5 s per barrier at most
// Up to 12 consumer warps + the producer warp = 13 warps, so one of the four SM sub-partitions (16 K
// registers each) hosts four warps: 128 registers per thread is the most a CTA of this size can be given.
constexpr int kMegaThreadsMax = 416;
constexpr int kMaxStepHeads = 128;                                     // query heads: one group counter each

static __device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// A CTA that gives up (a bounded wait ran out) adds this instead of 1: the count is then beyond every target, so
// all waiters are released at once and see from the count itself that the launch is being abandoned.
constexpr unsigned kBarAbort = 0x40000000u;

struct GridBarrier {
    unsigned *count;  // arrivals since the launch (zeroed by the host before every launch)
    uint32_t *status; // device status word
    unsigned target;  // arrivals that complete the barrier this CTA waits at next (always < kBarAbort)
    int ncta;
    int *s_go;        // shared-memory word
};

// All consumer threads of every CTA.  `ok` = this thread saw no failed wait.  Returns the same verdict in
// every thread of the grid that gets past it: false means "leave now".  One atomic per CTA and barrier;
// the waiters poll the arrival counter itself, and nothing else is read on the way out.  (Measured against a
// variant in which the last arriver publishes the target in a flag word on another cache line and the waiters
// poll only that: the extra store after the last arrival costs more than the contention it removes, 657 against
// 692 tok/s on the batch-1 stack.)
static __device__ __forceinline__ bool grid_sync(GridBarrier &gb, int nct, bool ok)
{
    const bool all_ok = named_bar_and(1, nct, ok);       // CTA verdict; all global writes of the phase are issued
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(gb.count, all_ok ? 1u : kBarAbort);
        unsigned v;
        unsigned long long t0 = 0;
        for (unsigned it = 1; (v = ld_acquire_u32(gb.count)) < gb.target; ++it) {
            if ((it & 63u) == 0) {                       // now and then: have we waited too long?
                const unsigned long long now = global_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > kGridWaitNanos) { atomicAdd(gb.count, kBarAbort); v = kBarAbort; break; }
            }
        }
        const int go = all_ok && v < kBarAbort;
        if (!go) atomicOr(gb.status, FASTTPS_DEV_WAIT_TIMEOUT);
        *gb.s_go = go;
    }
    named_bar_sync(1, nct);
    gb.target += (unsigned)gb.ncta;
    return *gb.s_go != 0;
}

__host__ __device__ inline void cta_range(int n_units, int cta, int ncta, int &u0, int &n)
{
    const int base = n_units / ncta, rem = n_units % ncta;
    u0 = cta * base + (cta < rem ? cta : rem);
    n = base + (cta < rem ? 1 : 0);
}

struct MegaLayout {
    int nw, ipw, nslot, slot_stride, wpiece;
    size_t ring_off, bar_off, abort_off, part_off, red_off, scratch_off, total;
};

template <int DH>
__host__ __device__ inline MegaLayout mega_layout(int D)
{
    MegaLayout l;
    const WarpSplit s = warp_split(D);
    l.nw = s.nw; l.ipw = s.ipw;
    l.wpiece = kBlocksPerWarpPerSlot * (s.nw > 0 ? s.nw : 1) * kTileBytes;
    l.slot_stride = l.wpiece > AttnTile<DH>::kPieceBytes ? l.wpiece : AttnTile<DH>::kPieceBytes;
    l.nslot = kRingBudget / l.slot_stride;
    l.nslot = l.nslot >= 8 ? 8 : l.nslot >= 4 ? 4 : l.nslot >= 2 ? 2 : l.nslot;   // a power of two (ring indexing by mask and shift)
    l.ring_off = 0;
    l.bar_off = (size_t)l.nslot * l.slot_stride;
    l.abort_off = l.bar_off + 2 * 8 * 8;
    l.part_off = l.abort_off + 16;
    l.red_off = l.part_off + sizeof(float) * 2 * (size_t)s.nw * 128;
    l.scratch_off = (l.red_off + sizeof(float) * (size_t)s.nw * 8 + 15) & ~(size_t)15;
    l.total = l.scratch_off + sizeof(AttnScratch<DH>);
    return l;
}

static __device__ __forceinline__ AttnArgs attn_args_of(const StepArgs &a, const LayerPtrs &lp, int step, int ncta_attn)
{
    AttnArgs aa;
    const int nq = a.n_q_heads * a.head_dim, nkv = a.n_kv_heads * a.head_dim;
    aa.q = a.qkv; aa.k_new = a.qkv + nq; aa.v_new = a.qkv + nq + nkv;
    aa.q_stride = nq + 2 * nkv; aa.kv_stride = nq + 2 * nkv;
    aa.k_cache = lp.k_cache; aa.v_cache = lp.v_cache;
    aa.pos = a.pos; aa.seq_lens = a.seq_lens;
    aa.out = a.attn_out; aa.out_stride = nq; aa.out_chunked = 0;
    aa.batch = a.batch; aa.n_q_heads = a.n_q_heads; aa.n_kv_heads = a.n_kv_heads;
    aa.head_dim = a.head_dim; aa.max_seq = a.max_seq; aa.n_splits = ncta_attn; aa.len_add = step; aa.n_new = 1; aa.k_scale = aa.v_scale = 1.f;
    aa.cos_tab = a.cos_tab; aa.sin_tab = a.sin_tab;
    aa.part = a.attn_part; aa.ticket = a.attn_ticket; aa.status = a.status;
    return aa;
}

}  // namespace fasttps
