// Test-only translation unit, built into a library of its own (not part of libkvh.so and not
// declared in include/kvh.h).  It runs the bounded barrier wait of the persistent kernels in the
// three ways it can end, without any copy or any other kernel involved:
//   warp 0 waits on a barrier nobody arrives at, with a short limit: the wait runs out, the warp
//          reports KVH_ERR_TIMEOUT and raises the CTA's abort flag (what a kernel's CTA does);
//   warp 1 waits on the same barrier with the library's own limit (2 s) and must leave early,
//          through the abort flag;
//   warp 2 waits on a second barrier that warp 3 arrives at: the wait succeeds.
// Nothing here can hang: every wait is the bounded one under test.
//
// A second entry point, host code only, drives the decode kernel's ring of stage quanta (QuantaRing)
// the way the producer warp does, against a plain occupancy map.
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvh.h"
#include "kvh_async.cuh"
#include "kvh_decode.cuh"
#include "kvh_decode_tma.cuh"

namespace {

using namespace kvh;

// out[2 w] = 1 if warp w's wait succeeded, else 0; out[2 w + 1] = nanoseconds it waited (w = 0..2)
__global__ void bounded_wait_kernel(unsigned long long limit_ns, int32_t *status, int64_t *out)
{
    __shared__ __align__(8) uint64_t never_bar, arrived_bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&never_bar, 1);
        mbar_init(&arrived_bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane != 0) return;
    if (warp == 3) {
        mbar_arrive(&arrived_bar);
        return;
    }
    const unsigned long long t0 = global_ns();
    const bool ok = warp == 0 ? mbar_wait(&never_bar, 0, &abort_flag, limit_ns)
                  : warp == 1 ? mbar_wait(&never_bar, 0, &abort_flag)
                              : mbar_wait(&arrived_bar, 0, &abort_flag, limit_ns);
    const unsigned long long t1 = global_ns();
    if (!ok && warp == 0) {
        report(status, KVH_ERR_TIMEOUT);
        abort_flag = 1;
    }
    out[2 * warp] = ok ? 1 : 0;
    out[2 * warp + 1] = (int64_t)(t1 - t0);
}

}  // namespace

// limit_ns: the short limit (at most 100 ms is accepted).  dev_status [device]: receives the status
// code like any kernel's.  dev_out [device, 6 x int64].  Returns KVH_OK once the launch is enqueued.
extern "C" kvh_status kvh_selftest_bounded_wait(uint64_t limit_ns, int32_t *dev_status, int64_t *dev_out, void *stream)
{
    if (!dev_status || !dev_out || limit_ns == 0 || limit_ns > 100000000ull) return KVH_ERR_INVALID_ARG;
    bounded_wait_kernel<<<1, 128, 0, static_cast<cudaStream_t>(stream)>>>(limit_ns, dev_status, dev_out);
    return cudaGetLastError() == cudaSuccess ? KVH_OK : KVH_ERR_CUDA;
}

// Host only.  Plays the decode producer's part on a ring of n_quanta quanta for n_units units whose
// sizes come from a seeded generator (bits 2, 4, 8, 16 and, rarely, the end marker's 0): before a
// unit is placed the oldest units are taken back until a slot and the quanta are there, exactly as in
// the kernel; now and then further units are taken back first, as consumers that run ahead would
// allow.  An occupancy map checks what the ring's own counters cannot: that a unit's quanta are
// contiguous, inside the ring and free when it gets them.  Returns 0, or the 1-based number of the
// unit at which a check failed (negative: the ring would have had to wait with nothing held).
// max_in_flight [host, may be NULL]: the most units held at once.
extern "C" int64_t kvh_selftest_quanta_ring(int n_quanta, int64_t n_units, uint64_t seed, int *max_in_flight)
{
    if (n_quanta < 6 || n_quanta > kMaxQuanta || n_units < 0) return INT64_MIN;
    QuantaRing ring(n_quanta);
    bool busy[kMaxQuanta] = {};
    int at_of[kSlots] = {}, held_of[kSlots] = {}, need_of[kSlots] = {};
    int64_t tail = 0;
    int most = 0;
    uint64_t x = seed * 0x9E3779B97F4A7C15ull + 1;
    auto rnd = [&]() { x ^= x << 13; x ^= x >> 7; x ^= x << 17; return x; };
    auto take_back = [&](int64_t u) {
        const int s = (int)(u % kSlots);
        for (int q = 0; q < need_of[s]; ++q) busy[at_of[s] + q] = false;
        ring.give_back(held_of[s]);
    };
    const int sizes[4] = {2, 4, 8, 16};
    for (int64_t unit = 0; unit < n_units; ++unit) {
        const int need = rnd() % 97 == 0 ? 0 : unit_quanta(sizes[rnd() % 4]);
        while (tail < unit && rnd() % 3 == 0) take_back(tail++);          // consumers ahead of the producer's needs
        while (unit - tail >= kSlots || !ring.fits(need)) {
            if (tail == unit) return -(unit + 1);
            take_back(tail++);
        }
        const int s = (int)(unit % kSlots);
        int held;
        const int at = ring.take(need, held);
        if (at < 0 || at + need > n_quanta || held < need || ring.free_q < 0 || ring.head < 0 || ring.head >= n_quanta) return unit + 1;
        for (int q = 0; q < need; ++q) {
            if (busy[at + q]) return unit + 1;
            busy[at + q] = true;
        }
        at_of[s] = at; held_of[s] = held; need_of[s] = need;
        if ((int)(unit + 1 - tail) > most) most = (int)(unit + 1 - tail);
    }
    while (tail < n_units) take_back(tail++);
    if (ring.free_q != n_quanta) return n_units + 1;
    for (int q = 0; q < n_quanta; ++q)
        if (busy[q]) return n_units + 1;
    if (max_in_flight) *max_in_flight = most;
    return 0;
}
