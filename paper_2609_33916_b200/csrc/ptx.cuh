// Thin inline-PTX wrappers for the sm_100a features the tensor-core kernels use:
// mbarrier, TMA (cp.async.bulk.tensor; no load is multicast: every CTA fetches its own tiles),
// tcgen05 (TMEM allocation, UMMA, commit, ld/st) and the shared-memory / instruction
// descriptors.  The one multicast form in here is the tcgen05.commit of a CTA pair, which is an
// mbarrier arrival in both CTAs of one cluster on one GPU, not a copy.
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>
#include <cuda/ptx>

#ifndef MOA_SUSPEND_HINT_NS
#define MOA_SUSPEND_HINT_NS 20000u
#endif

namespace moa {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ------------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Programmatic dependent launch.  A kernel launched with the programmatic-stream-serialization attribute may start while
// the kernel before it in the stream is still running; grid_dependency_wait() then blocks until that kernel has completed and
// its memory operations are visible (without the attribute it returns at once).  grid_launch_dependents() tells the
// scheduler that, as far as this CTA is concerned, the next kernel's CTAs may be started (they are, once every CTA of this grid
// has said so or exited, on whatever SM resources are free).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// The suspend-time hint lets the hardware park the waiting thread (no issue slots spent on
// polling) until the phase completes or the hint (nanoseconds) runs out.
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(MOA_SUSPEND_HINT_NS)
        : "memory");
    return ok != 0;
}

// Every wait in the tensor-core kernels is bounded: after about kWaitCycles SM cycles (two
// seconds) the waiter records `code` in the global status word, raises the CTA's
// abort flag so that every other role gives up quickly as well, and returns false.
// The bound is kept as a count of parked waits (each mbarrier.try_wait parks the thread for up to
// MOA_SUSPEND_HINT_NS = 20 us, about 40,000 cycles), not as a clock reading: the wait loop is inlined
// dozens of times per kernel, and the shorter loop made every tensor-core kernel 1-3 % faster.
constexpr long long kWaitCycles = 4000000000LL;

// Non-blocking probe: much cheaper than try_wait when the phase has already completed (try_wait
// is a potentially suspending instruction and costs the caller ~100 cycles even on success).
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          unsigned int *status, uint32_t code, long long limit = kWaitCycles)
{
    if (mbar_test_wait(bar, parity)) return true;
    // limit / 40,000 parked waits (plus a few, so that a tiny limit still waits), checked with the CTA's abort flag
    const uint32_t max_spins = (uint32_t)(limit / 40000LL) + 64u;
#pragma unroll 1
    for (uint32_t spins = 0; spins < max_spins; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    if (status) atomicCAS(status, 0u, code);
    return false;
}

// After a wait has expired the CTA winds down; copies this thread asked for may still be on their way into the
// CTA's shared memory.  ArmCounts remembers how often the thread armed each barrier, and mbar_drain gives the last
// phase armed on each of them a bounded time (about 0.1 s of SM clock) to complete before the thread leaves.
constexpr long long kDrainCycles = 200000000LL;
template <int N>
struct ArmCounts {
    uint32_t n[N];
    __device__ __forceinline__ ArmCounts()
    {
#pragma unroll
        for (int i = 0; i < N; ++i) n[i] = 0;
    }
};
// The same for one barrier that was armed `uses` times (kernels whose producer counts its loads in registers).
__device__ __forceinline__ void mbar_drain_one(uint64_t *bar, int uses)
{
    if (uses <= 0) return;
    const uint32_t parity = (uint32_t)(uses - 1) & 1u;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > kDrainCycles) break;
}
template <int N>
__device__ __forceinline__ void mbar_arm(uint64_t *bars, int idx, uint32_t bytes, ArmCounts<N> &c)
{
    mbar_arrive_expect_tx(bars + idx, bytes);
    ++c.n[idx];
}
template <int N>
__device__ __forceinline__ void mbar_arm(uint64_t *bars, uint64_t *bar, uint32_t bytes, ArmCounts<N> &c)
{
    mbar_arm(bars, (int)(bar - bars), bytes, c);
}
template <int N>
__device__ __noinline__ void mbar_drain(uint64_t *bars, const ArmCounts<N> &c)
{
    for (int i = 0; i < N; ++i) {
        if (c.n[i] == 0) continue;
        const uint32_t parity = (c.n[i] - 1) & 1;
        const long long t0 = clock64();
        while (!mbar_try_wait(bars + i, parity))
            if (clock64() - t0 > kDrainCycles) break;
    }
}

// -------------------------------------------------------------------- fences / proxies
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ----------------------------------------------------------------------------- TMA
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *m)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
// 3-D tiled load: coordinates (x = innermost element index, y = row, z = head)
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *m, uint64_t *bar, int x, int y, int z)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
        : "memory");
}
// 3-D tiled fp32 add-reduce into global memory (rows past the tensor's extent are clipped)
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap *m, const void *src, int x, int y, int z)
{
    asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
// 3-D tiled store of a shared-memory box to global memory (rows past the tensor's extent are clipped)
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *m, const void *src, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
// 3-D tiled prefetch of a box into L2 (no shared-memory destination, nothing to wait for)
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap *m, int x, int y, int z)
{
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
// Untiled copy of `bytes` contiguous bytes (16-byte aligned source, destination and size)
__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// 4-D forms for the caller's tensors: coordinates (x = element, y = row, z = head, w = batch)
__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *m, uint64_t *bar, int x, int y, int z, int w)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w)
        : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap *m, const void *src, int x, int y, int z, int w)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z), "r"(w)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait()
{
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

// ---------------------------------------------------------------------------- TMEM
// One warp allocates; the base address (lane 0, first column) is written to *dst_smem.
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// ---------------------------------------------------------------------------- UMMA
// D[tmem] (+)= A[smem] * B[smem] (umma_ss2) and D[tmem] (+)= A[tmem] * B[smem] (umma_ts2).
// A descriptor is passed as its two 32-bit halves (only the low half, which holds the address
// field, changes between k-steps: one integer add), and the accumulate flag is a compile-time
// choice, so an UMMA costs the issuing thread two or three instructions instead of a dozen.
template <bool kAccumulate>
__device__ __forceinline__ void umma_ss2(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                         uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(kAccumulate ? 1 : 0)
        : "memory");
}
template <bool kAccumulate>
__device__ __forceinline__ void umma_ts2(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(kAccumulate ? 1 : 0)
        : "memory");
}

// Arrive on an mbarrier of this CTA when all previously issued UMMAs have completed.
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// ------------------------------------------------------------------ CTA pairs (cta_group::2)
// Two CTAs of a cluster (ranks 0 and 1) work on one UMMA of M = 256: each holds 128 rows of A, half of
// the N rows of B and 128 lanes x N columns of the accumulator; the CTA of rank 0 issues.  The forms
// below follow the PTX ISA: allocation and deallocation are executed by one warp of EACH CTA; a copy
// may complete its bytes on a barrier of the other CTA (the barrier is named by its shared::cluster
// address); a commit can arrive on the barrier at the same offset in both CTAs (mask 0b11).
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory location in the CTA of rank `rank`
__device__ __forceinline__ uint32_t mapa_u32(uint32_t cta_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(cta_addr), "r"(rank));
    return r;
}
// every thread of every CTA of the cluster (hardware barrier; all threads reach it, also after an expired wait)
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(void *dst, const CUtensorMap *m, uint32_t bar_cluster_addr, int x, int y, int z)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t *dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
template <bool kAccumulate>
__device__ __forceinline__ void umma_ss2_pair(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                              uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(kAccumulate ? 1 : 0)
        : "memory");
}
template <bool kAccumulate>
__device__ __forceinline__ void umma_ts2_pair(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(kAccumulate ? 1 : 0)
        : "memory");
}
// 4-D tiled load of a CTA of a pair: the bytes complete on the barrier named by its shared::cluster address
// (a barrier of either CTA of the pair); no multicast, each CTA fetches what it stages itself
__device__ __forceinline__ void tma_load_4d_pair(void *dst, const CUtensorMap *m, uint32_t bar_cluster_addr, int x, int y,
                                                 int z, int w)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z), "r"(w)
        : "memory");
}
// Arrival on a barrier of any CTA of the cluster that publishes this thread's earlier writes (also those to the other
// CTA's shared memory) to whoever waits on it with cluster scope
__device__ __forceinline__ void mbar_arrive_release_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(MOA_SUSPEND_HINT_NS)
        : "memory");
    return ok != 0;
}
// mbar_wait for a barrier of this CTA on which threads of the other CTA of the pair arrive (cluster-scope acquire)
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag,
                                                  unsigned int *status, uint32_t code, long long limit = kWaitCycles)
{
    if (mbar_test_wait(bar, parity) && mbar_try_wait_cluster(bar, parity)) return true;
    const uint32_t max_spins = (uint32_t)(limit / 40000LL) + 64u;      // bounded like mbar_wait
#pragma unroll 1
    for (uint32_t spins = 0; spins < max_spins; ++spins) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    if (status) atomicCAS(status, 0u, code);
    return false;
}
// Arrival on a barrier of the other CTA of the cluster with no ordering of this thread's other memory accesses (a
// cluster-scope release costs about a thousand cycles; what such an arrival announces here -- TMEM contents after
// tcgen05.wait, shared memory after a proxy fence -- is complete before the instruction is issued)
__device__ __forceinline__ void mbar_arrive_relaxed_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Bulk copy of `bytes` contiguous bytes from this CTA's shared memory into the shared memory of another CTA of the
// cluster; the bytes are counted on an mbarrier of the receiving CTA when they have landed (both destination addresses
// from mapa_u32; 16-byte aligned addresses and size).  The whole transfer runs in the asynchronous proxy, like a TMA load.
__device__ __forceinline__ void bulk_copy_to_cluster(uint32_t dst_cluster_addr, const void *src, uint32_t bytes,
                                                     uint32_t bar_cluster_addr)
{
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster_addr), "r"(smem_u32(src)), "r"(bytes), "r"(bar_cluster_addr)
                 : "memory");
}
// 16-byte store into the shared memory of a CTA of the cluster (address from mapa_u32)
__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(a), "r"(b), "r"(c), "r"(d)
                 : "memory");
}
// generic-proxy writes (also those to another CTA's shared memory) ordered before later async-proxy reads
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Arrive, on the barrier at this offset in BOTH CTAs of the pair, when all previously issued UMMAs have completed.
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((uint16_t)3)
                 : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle.  A tile is stored as rows of 128
// bytes (64 bf16), eight rows forming one 1024-byte swizzle atom; `addr` must keep the
// tile's 1024-byte alignment apart from a K offset inside the first row.
//   K-major operand  (rows = M or N index, the 64 elements of a row run along K):
//       sbo = bytes between 8-row groups (1024 for a dense tile); lbo unused.
//   MN-major operand (rows = K index, the 64 elements of a row run along M or N):
//       sbo = bytes between groups of 8 K-rows (1024); lbo = bytes between
//       consecutive 64-element column blocks.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version for sm_100
    d |= (uint64_t)2 << 61;   // layout: 128-byte swizzle
    return d;
}

// Instruction descriptor for kind::f16 with bf16 inputs and fp32 accumulation.
// a_mn / b_mn: 1 when that operand is MN-major (0 = K-major).
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int M, int N, int a_mn, int b_mn)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ------------------------------------------------------------- TMEM <-> registers
// 32x32b: thread t of warp w accesses lane 32*(w%4)+t; register i <-> column col+i.
template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&r)[N])
{
    cuda::ptx::tcgen05_ld_32x32b(r, taddr);
}
template <int N>
__device__ __forceinline__ void tmem_st(uint32_t taddr, const uint32_t (&r)[N])
{
    cuda::ptx::tcgen05_st_32x32b(taddr, r);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Packed fp32 pairs (sm_100 f32x2 arithmetic): one instruction for two elements.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

}  // namespace ptx
}  // namespace moa
