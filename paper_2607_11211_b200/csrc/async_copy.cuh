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
// first, and reports failure instead of spinning forever.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity)
{
    unsigned long long t0 = 0;
    for (uint32_t i = 0; i < kWaitPolls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 255u) {
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitNanos) return false;
        }
    }
    return false;
}
// global -> shared bulk copy; dst, src 16-byte aligned, bytes a multiple of 16; completes on `bar`
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// ----------------------------------------------------------------- weight ring
//
// A CTA's share of a weight matrix is a contiguous run of rows (each row = the n_in weights
// of one output, or one row of W_down).  The ring streams up to two such runs, one after the
// other, as "groups" of R rows: group g lands in slot g % nslot with ONE bulk copy issued by
// thread 0, and completes on the slot's mbarrier.  Up to nslot groups (about 190 KB per SM)
// are in flight at any time, independent of what the consumer warps are doing, which is what
// keeps HBM busy across reductions, barriers and the switch from one matrix to the next.
//
// Protocol: thread 0 calls start() once (after init + __syncthreads), all threads call
// wait(g) before reading group g, and after a block-wide barrier that follows the last read
// of group g thread 0 calls refill(g) to reuse its slot for group g + nslot.
struct WeightRing {
    unsigned char *slots;        // nslot * slot_bytes, 128-byte aligned
    uint64_t *full;              // nslot mbarriers
    int nslot, slot_bytes, row_bytes, rows_per_group;
    const unsigned char *base0, *base1;
    int rows0, rows1;            // rows in each run
    int groups0, groups;         // groups of run 0, of both runs

    __device__ __forceinline__ void init(unsigned char *slots_, uint64_t *full_, int nslot_, int row_bytes_, int R,
                                         const void *b0, int r0, const void *b1, int r1)
    {
        slots = slots_; full = full_; nslot = nslot_; row_bytes = row_bytes_; rows_per_group = R;
        slot_bytes = R * row_bytes_;
        base0 = static_cast<const unsigned char *>(b0); rows0 = r0;
        base1 = static_cast<const unsigned char *>(b1); rows1 = r1;
        groups0 = (r0 + R - 1) / R;
        groups = groups0 + (r1 + R - 1) / R;
        if (threadIdx.x == 0) {
            for (int s = 0; s < nslot; ++s) mbar_init(&full[s], 1);
            mbar_fence_init();
        }
    }
    // thread 0 only
    __device__ __forceinline__ void issue(int g)
    {
        const bool second = g >= groups0;
        const int gl = second ? g - groups0 : g;
        int n = (second ? rows1 : rows0) - gl * rows_per_group;
        n = n < rows_per_group ? n : rows_per_group;
        const uint32_t bytes = (uint32_t)n * (uint32_t)row_bytes;
        uint64_t *bar = &full[g % nslot];
        mbar_expect_tx(bar, bytes);
        bulk_g2s(slots + (size_t)(g % nslot) * slot_bytes, (second ? base1 : base0) + (size_t)gl * slot_bytes, bytes, bar);
    }
    __device__ __forceinline__ void start()
    {
        for (int g = 0; g < groups && g < nslot; ++g) issue(g);
    }
    __device__ __forceinline__ void refill(int g)
    {
        if (g + nslot < groups) issue(g + nslot);
    }
    // all threads; lane 0 polls, the warp shares the verdict
    __device__ __forceinline__ const unsigned char *wait(int g, bool &ok)
    {
        bool mine = true;
        if ((threadIdx.x & 31) == 0) mine = mbar_wait_bounded(&full[g % nslot], (uint32_t)(g / nslot) & 1u);
        mine = __shfl_sync(kFull, mine ? 1 : 0, 0) != 0;
        // every lane observes the (already completed) phase itself, so that its reads of the
        // slot are ordered after the copy; this returns at once
        if (mine) mine = mbar_try_wait(&full[g % nslot], (uint32_t)(g / nslot) & 1u);
        mine = __all_sync(kFull, mine);
        ok = ok && mine;
        return slots + (size_t)(g % nslot) * slot_bytes;
    }
    // thread 0, after a failed wait: give the copies still in flight (groups g .. issued) a bounded chance to land
    __device__ __forceinline__ void drain(int g)
    {
        for (int u = g; u < groups && u < g + nslot; ++u)
            (void)mbar_wait_bounded(&full[u % nslot], (uint32_t)(u / nslot) & 1u);
    }
};

// shared-memory bytes the ring needs for rows of row_bytes, and how many slots fit into `budget`
__host__ __device__ inline int ring_slots_for(int row_bytes, int R, int budget)
{
    int n = budget / (R * row_bytes);
    return n > 8 ? 8 : n;
}

}  // namespace fasttps
