// mbarrier + bulk asynchronous copy (cp.async.bulk, the 1-D TMA path) helpers, and the
// shared-memory weight ring built on them.  Every wait is bounded.
#pragma once
#include "common.cuh"

namespace fasttps {

constexpr uint32_t kWaitPolls = 1u << 22;                        // bounded mbarrier polling: poll count ...
constexpr unsigned long long kWaitNanos = 400ull * 1000 * 1000;  // ... and wall time (0.4 s)

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long v;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(v));
    return v;
}
// Bounded wait: gives up after kWaitPolls polls or kWaitNanos of wall time, whichever comes
// first (or as soon as *abort_flag is set, when given), and reports failure instead of
// spinning forever.
// The polling loop is kept out of line so that the hot loops that call it stay small.
static __device__ __noinline__ bool mbar_wait_slow(uint64_t *bar, uint32_t parity, const volatile int *abort_flag)
{
    unsigned long long t0 = 0;
    for (uint32_t i = 0; i < kWaitPolls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 255u) {
            if (abort_flag && *abort_flag) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitNanos) return false;
        }
    }
    return false;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, const volatile int *abort_flag = nullptr)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag);
}
// global -> shared bulk copy; dst, src 16-byte aligned, bytes a multiple of 16; completes on `bar`
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// the same with an L2 eviction policy (from l2_policy_evict_first): data that is read once
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_g2s_hint(void *dst, const void *src, uint32_t bytes, uint64_t *bar, uint64_t pol)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol) : "memory");
}
// asks the L2 to fetch `bytes` (a multiple of 16) at src: no completion to wait for
__device__ __forceinline__ void bulk_prefetch_l2(const void *src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
// named barrier over the first `nthreads` threads' warps (id 1..15; id 0 is __syncthreads)
__device__ __forceinline__ void named_bar_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// named barrier that also ANDs a predicate over its participants: every thread gets the same verdict
__device__ __forceinline__ bool named_bar_and(int id, int nthreads, bool pred)
{
    uint32_t out;
    asm volatile("{\n\t.reg .pred p, q;\n\t"
                 "setp.ne.u32 q, %1, 0;\n\t"
                 "bar.red.and.pred p, %2, %3, q;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(out) : "r"(pred ? 1u : 0u), "r"(id), "r"(nthreads) : "memory");
    return out != 0;
}

// ----------------------------------------------------------------- weight ring
//
// A CTA's share of a packed weight matrix is one contiguous byte range (two for the fused
// MLP: its gate_up tiles, then its W_down octets).  A dedicated producer warp streams the
// ranges, one after the other, in slot-sized pieces: piece g lands in slot slot_of(g) with
// ONE bulk copy and completes on the slot's "full" mbarrier.  Each consumer warp arrives on
// the slot's "empty" mbarrier when it has read its part, and the producer refills the slot
// as soon as all consumer warps have.  Up to nslot pieces (about 190 KB per SM) are in
// flight at any time, independent of what the consumer warps are doing, which keeps HBM
// busy across reductions, barriers and the switch from one matrix to the next.
struct WeightRing {
    unsigned char *slots;        // nslot * slot_bytes, 128-byte aligned
    uint64_t *full, *empty;      // nslot mbarriers each
    volatile int *abort_flag;    // shared-memory word, set when any bounded wait ran out
    uint64_t policy = 0;         // L2 eviction policy of the weight pieces (0: none)
    int nslot, nshift, slot_bytes;   // nslot = 1 << nshift: slot and round of a piece are a mask and a shift
    const unsigned char *base0, *base1;
    int pieces0, pieces;         // pieces of run 0, of both runs (every run is a whole number of slots)

    // all threads; follow with a block-wide barrier before any other use
    __device__ __forceinline__ void init(unsigned char *slots_, uint64_t *bars, int *abort_, int nslot_, int slot_bytes_,
                                         int n_consumer_warps, const void *b0, long long bytes0, const void *b1,
                                         long long bytes1)
    {
        slots = slots_; full = bars; empty = bars + nslot_; abort_flag = abort_;
        nslot = nslot_; slot_bytes = slot_bytes_;
        nshift = 31 - __clz(nslot_);
        base0 = static_cast<const unsigned char *>(b0);
        base1 = static_cast<const unsigned char *>(b1);
        pieces0 = (int)(bytes0 / slot_bytes_);
        pieces = pieces0 + (int)(bytes1 / slot_bytes_);
        if (threadIdx.x == 0) {
            for (int s = 0; s < nslot; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], n_consumer_warps); }
            *abort_ = 0;
            mbar_fence_init();
        }
    }
    __device__ __forceinline__ int slot_of(int g) const { return g & (nslot - 1); }
    __device__ __forceinline__ int round_of(int g) const { return g >> nshift; }
    // producer thread: wait until the slot of piece g is free again (false after a failed bounded wait)
    __device__ __forceinline__ bool acquire(int g)
    {
        if (g >= nslot && !mbar_wait_bounded(&empty[slot_of(g)], (uint32_t)(round_of(g) - 1) & 1u, abort_flag)) {
            *abort_flag = 1;
            return false;
        }
        return true;
    }
    // producer thread: piece g = `bytes` contiguous bytes at src
    __device__ __forceinline__ bool put(int g, const void *src, uint32_t bytes)
    {
        if (!acquire(g)) return false;
        const int s = slot_of(g);
        mbar_expect_tx(&full[s], bytes);
        if (policy) bulk_g2s_hint(slots + (size_t)s * slot_bytes, src, bytes, &full[s], policy);
        else bulk_g2s(slots + (size_t)s * slot_bytes, src, bytes, &full[s]);
        return true;
    }
    // producer thread: piece g = two blocks of `bytes` each, the second landing at offset off1 of the slot
    __device__ __forceinline__ bool put2(int g, const void *src0, const void *src1, uint32_t bytes, uint32_t off1)
    {
        if (!acquire(g)) return false;
        const int s = slot_of(g);
        mbar_expect_tx(&full[s], 2 * bytes);
        if (policy) {
            bulk_g2s_hint(slots + (size_t)s * slot_bytes, src0, bytes, &full[s], policy);
            bulk_g2s_hint(slots + (size_t)s * slot_bytes + off1, src1, bytes, &full[s], policy);
        } else {
            bulk_g2s(slots + (size_t)s * slot_bytes, src0, bytes, &full[s]);
            bulk_g2s(slots + (size_t)s * slot_bytes + off1, src1, bytes, &full[s]);
        }
        return true;
    }
    // one thread of the producer warp: stream every piece of the two runs given to init(), then return
    __device__ __forceinline__ void produce()
    {
        for (int g = 0; g < pieces; ++g) {
            const unsigned char *src = g < pieces0 ? base0 + (size_t)g * slot_bytes
                                                   : base1 + (size_t)(g - pieces0) * slot_bytes;
            if (!put(g, src, (uint32_t)slot_bytes)) { drain(g); return; }
        }
    }
    // every lane of a consumer warp; returns the slot holding piece g (ok is cleared on a failed wait)
    __device__ __forceinline__ const unsigned char *wait(int g, bool &ok)
    {
        bool mine = ok;
        if (mine) mine = mbar_wait_bounded(&full[slot_of(g)], (uint32_t)(round_of(g)) & 1u, abort_flag);
        mine = __all_sync(kFull, mine);
        if (!mine && ok) *abort_flag = 1;
        ok = mine;
        return slots + (size_t)(slot_of(g)) * slot_bytes;
    }
    // consumer warp, after its last read of piece g.  Every lane first fences its own shared-memory reads: the
    // arrival is made by lane 0 alone, and the warp-level barrier in front of it does not by itself keep the other
    // lanes' loads of the slot ahead of the bulk copy that refills the slot once the last arrival is in.  Without
    // the fence a refill was measured to overtake such loads: the first launch of the fused MLP kernel after a
    // different kernel returned, in up to 70 % of the launches, a first row tile in which 128-byte pieces of one
    // warp's weights were those of the tile two further on (the piece that reuses the slot); with it, none in
    // thousands of launches.
    __device__ __forceinline__ void release(int g)
    {
        __threadfence_block();
        __syncwarp();
        if ((threadIdx.x & 31) == 0) mbar_arrive(&empty[slot_of(g)]);
    }
    // producer thread, on the way out after a failure with pieces [0, issued) handed to the copy engine: the
    // copies still in flight (at most the last nslot pieces) get a bounded chance to land before the CTA's
    // shared memory is given up
    __device__ __forceinline__ void drain(int issued)
    {
        for (int g = issued > nslot ? issued - nslot : 0; g < issued; ++g)
            (void)mbar_wait_bounded(&full[slot_of(g)], (uint32_t)round_of(g) & 1u, nullptr);
    }
};

}  // namespace fasttps
