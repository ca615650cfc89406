// Asynchronous-copy helpers for sm_100a: shared-memory transaction barriers
// (mbarrier) and 1-D bulk copies global -> shared issued through the TMA unit
// (cp.async.bulk, no tensor map, every copy for this CTA alone).  Every wait is bounded: it
// gives up after a fixed number of polls and reports that to the caller, so no
// kernel can spin forever on a barrier that never completes.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace rq {

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
}

// Makes freshly initialised barriers visible to the asynchronous proxy; follow
// with a CTA-wide barrier before the first copy is issued.
__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// One plain arrival.
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// One arrival that also announces `bytes` of copy traffic to wait for.
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}

// Poll limit of a barrier wait.  One poll may itself suspend the thread for a
// hardware-defined short time, so the limit is reached only after a time that
// is orders of magnitude beyond any copy's latency.
constexpr int kMbarPollLimit = 1 << 20;
// upper bound (ns) of the time one poll may keep the thread suspended while the phase is pending
constexpr uint32_t kMbarSuspendNs = 2000;

// Wait for the phase with the given parity to complete.  Returns false if the
// poll limit ran out first.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, int limit = kMbarPollLimit)
{
    const uint32_t addr = smem_addr(bar);
    for (int it = 0; it < limit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity), "r"(kMbarSuspendNs)
            : "memory");
        if (done) return true;
    }
    return false;
}

// Bulk copy of `bytes` (a multiple of 16; both addresses 16-byte aligned) from
// global to this CTA's shared memory; completion is counted on `bar`.
__device__ __forceinline__ void bulk_g2s(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_addr(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

// L2 policy for data that is read once: its lines are the first to be replaced, so that a long
// stream does not push the step's small intermediate results (scores, page lists, partial
// outputs) out of L2 before the next kernel reads them.
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// The same copy with an L2 cache policy for the lines it reads.
__device__ __forceinline__ void bulk_g2s_hint(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar,
                                              uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_addr(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
        : "memory");
}

// Start bringing `bytes` (a multiple of 16, from a 16-byte aligned address) of global memory into L2;
// nothing waits for it.
__device__ __forceinline__ void bulk_prefetch_l2(const void *src_gmem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src_gmem), "r"(bytes) : "memory");
}

// Programmatic dependent launch: wait until the kernels this one depends on
// have completed and their writes are visible (no-op without the attribute).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Allow the next kernel in the stream to begin launching.
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint4 lds16(const void *p) { return *reinterpret_cast<const uint4 *>(p); }

// L2 loads that the compiler must issue where they stand (it would otherwise
// move each load next to its first use to save registers, which serialises
// the round trips of a batch of independent loads).
__device__ __forceinline__ float4 ld_cg_now(const float4 *p)
{
    float4 r;
    asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ uint4 ld_cg_now(const uint4 *p)
{
    uint4 r;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ float2 ld_cg_now(const float2 *p)
{
    float2 r;
    asm volatile("ld.global.cg.v2.f32 {%0, %1}, [%2];" : "=f"(r.x), "=f"(r.y) : "l"(p));
    return r;
}

// Flag shared between CTAs: a release store publishes everything the storing thread has
// written (or has observed through a barrier) before it; the acquire load pairs with it.
__device__ __forceinline__ void st_release(int32_t *p, int32_t v)
{
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int32_t ld_acquire(const int32_t *p)
{
    int32_t v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Polling form of the same: a relaxed load does not hold back the thread's later memory
// operations while it is under way; once it has seen the awaited value, the fence makes the
// publisher's earlier writes visible to what follows.
__device__ __forceinline__ int32_t ld_relaxed(const int32_t *p)
{
    int32_t v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void fence_acquire() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
// add with acquire-release ordering at device scope; returns the value before
__device__ __forceinline__ int32_t atom_add_acq_rel(int32_t *p, int32_t v)
{
    int32_t old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
// fire-and-forget increment of a counter in global memory
__device__ __forceinline__ void red_inc(uint32_t *p)
{
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
// Poll limit and pause of a wait for another CTA's flag: 2^22 polls 128 ns apart, about half a second.
constexpr int kFlagPollLimit = 1 << 22;
constexpr unsigned kFlagPollNs = 128;

__device__ __forceinline__ int ld_volatile(const int32_t *p) { return *reinterpret_cast<const volatile int32_t *>(p); }

}  // namespace rq
