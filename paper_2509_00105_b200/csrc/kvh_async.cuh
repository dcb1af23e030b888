// Asynchronous-copy and scheduling primitives of sm_100 used by the persistent kernels of this
// library: mbarriers with bounded waits, 1-D bulk copies between global and shared memory, and
// cluster launch control (a running CTA takes over the work of CTAs that have not started yet).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace kvh {

constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s: no wait in a kernel lasts longer
// How long one try_wait may keep its warp suspended in hardware before it reports "not yet": a
// waiting warp then costs a few instructions per microsecond instead of a busy loop that competes
// with the working warps for issue slots.  The wait still ends the moment the phase completes.
constexpr uint32_t kTryWaitHintNs = 20000u;

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_addr(bar)), "r"(parity), "r"(kTryWaitHintNs) : "memory");
    return done != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Wait for a phase of an mbarrier; false if the time limit ran out or the CTA is aborting.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                          unsigned long long limit_ns = kWaitLimitNs)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long start = global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag || global_ns() - start > limit_ns) return false;
    }
}
// The consumer side of a stage hand-over for a group of n_threads threads (whole warps) that take
// every unit together.  Polling an mbarrier costs issue slots for as long as the data is not
// there, and in a kernel that runs at the speed of memory it usually is not there yet: eight
// polling warps spent a quarter of all issued instructions that way.  So only the group's first
// warp polls; the others sleep on a hardware named barrier (bar_id, 1..15), which costs nothing
// while they wait.  The first warp publishes the outcome in verdict[unit & 1] (shared memory)
// before the barrier and every thread takes it from there, so the whole group always agrees on
// whether to go on: a named barrier that some warps have left for good would never open again.
// (Two slots: a warp can be at most one unit behind the first warp, the barrier sees to that.)
// After the barrier every thread tests the mbarrier once itself; the phase is complete and cannot
// be re-armed before this group has released the stage, so the test succeeds at once and serves
// as the thread's own acquire of the bytes the copy wrote.
// False if the wait ran out or the CTA is aborting; the abort flag is raised then.
__device__ __forceinline__ bool group_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                           volatile int *verdict, uint32_t unit, int bar_id, int n_threads,
                                           bool first_warp)
{
    if (first_warp) {
        const bool ok = mbar_wait(bar, parity, abort_flag);
        if ((threadIdx.x & 31) == 0) {
            if (!ok) *abort_flag = 1;
            verdict[unit & 1] = ok ? 1 : 0;
        }
    }
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(n_threads) : "memory");
    const bool ok = verdict[unit & 1] != 0;
    if (ok) (void)mbar_try_wait(bar, parity);
    return ok;
}

// 1-D bulk copy global -> this CTA's shared memory; bytes is a multiple of 16, both ends 16-byte aligned.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

// 1-D bulk copy this CTA's shared memory -> global, tracked by the issuing thread's bulk groups;
// bytes is a multiple of 16, both ends 16-byte aligned.  Shared memory written with ordinary stores
// needs fence_async_smem() (by the writers, before the barrier that precedes the copy) first.
__device__ __forceinline__ void bulk_store(void *dst, const void *src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(smem_addr(src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Wait until all but the newest N bulk groups of this thread have finished READING shared memory
// (their source may be overwritten); the global writes may still be in flight.
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
// Wait until every bulk group of this thread has completed, writes included.
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Makes this thread's ordinary writes to shared memory visible to the asynchronous proxy.
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 2-D tiled TMA load: the box the tensor map describes, with its corner at element (x, y) of the
// tensor, lands packed (row after row) at dst; its full size counts on the mbarrier, rows or columns
// outside the tensor arrive as zeros.  x times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tensor_load_2d(void *dst, const void *tensor_map, int x, int y, uint64_t *bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_addr(dst)), "l"(tensor_map), "r"(x), "r"(y), "r"(smem_addr(bar)) : "memory");
}

// Cluster launch control (sm_100): a running CTA asks the hardware for the index of a CTA of this
// grid that has not started yet and takes over its work; the 16-byte answer arrives in shared
// memory and completes 16 bytes of transaction on the mbarrier.  Dynamic scheduling of a persistent
// kernel without a work counter in global memory.
__device__ __forceinline__ void clc_try_cancel(void *response, uint64_t *bar)
{
    asm volatile("clusterlaunchcontrol.try_cancel.async.shared::cta.mbarrier::complete_tx::bytes.b128 [%0], [%1];"
                 ::"r"(smem_addr(response)), "r"(smem_addr(bar)) : "memory");
}
// Decode an answer: true and the x index of the cancelled CTA, or false if none was left.
__device__ __forceinline__ bool clc_query(const void *response, uint32_t &ctaid_x)
{
    uint32_t valid, x = 0;
    asm volatile(
        "{\n\t.reg .pred p1;\n\t.reg .b128 resp;\n\t"
        "ld.shared.b128 resp, [%2];\n\t"
        "clusterlaunchcontrol.query_cancel.is_canceled.pred.b128 p1, resp;\n\t"
        "selp.u32 %1, 1, 0, p1;\n\t"
        "@p1 clusterlaunchcontrol.query_cancel.get_first_ctaid.v4.b32.b128 {%0, _, _, _}, resp;\n\t}"
        : "+r"(x), "=r"(valid) : "r"(smem_addr(response)) : "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the next answer may overwrite it
    ctaid_x = x;
    return valid != 0;
}

// The tiles a persistent CTA works through, as seen by its producer warp (all 32 lanes call every
// member).  sched 0: blockIdx.x, blockIdx.x + gridDim.x, ...  sched 1: the grid holds one CTA per
// tile; a CTA starts with its own index and then takes over CTAs that have not started yet, asking
// for the next one (ask) before it feeds the current tile so that the answer is there when needed.
struct TileFeed {
    uint4 *response;               // shared: 2 answers
    uint64_t *bar;                 // shared: 2 mbarriers, initialised with count 1
    int sched, lane;
    volatile int *abort_flag;
    uint32_t query = 0;            // answers asked for so far
    bool asked = false;            // one answer still outstanding

    __device__ __forceinline__ void ask()
    {
        if (sched != 1) return;
        if (lane == 0) {
            mbar_arrive_expect_tx(&bar[query & 1], 16);
            clc_try_cancel(&response[query & 1], &bar[query & 1]);
        }
        asked = true;
    }
    // Moves tile_id on.  1: there is a next tile; 0: none left; -1: the wait for the answer ran out.
    __device__ __forceinline__ int next(int64_t &tile_id, int64_t total_tiles)
    {
        if (sched != 1) {
            tile_id += gridDim.x;
            return tile_id < total_tiles ? 1 : 0;
        }
        uint32_t got = 0, id = 0, w = 1;
        if (lane == 0) {
            w = mbar_wait(&bar[query & 1], (query >> 1) & 1, abort_flag);
            if (w) got = clc_query(&response[query & 1], id);
        }
        w = __shfl_sync(0xffffffffu, w, 0);
        got = __shfl_sync(0xffffffffu, got, 0);
        id = __shfl_sync(0xffffffffu, id, 0);
        if (!w) return -1;
        asked = false;
        ++query;
        if (!got) return 0;                              // no CTA left to take over: never ask again
        tile_id = id;
        return tile_id < total_tiles ? 1 : 0;
    }
    // Before the CTA leaves: an answer still on its way has to land (lane 0).
    __device__ __forceinline__ void drain()
    {
        int never = 0;
        if (asked) (void)mbar_wait(&bar[query & 1], (query >> 1) & 1, &never);
    }
};

}  // namespace kvh
