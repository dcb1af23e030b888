// Test-only translation unit, built into a library of its own (not part of libkvh.so and not
// declared in include/kvh.h).  It runs the bounded barrier wait of the persistent kernels in the
// three ways it can end, without any copy or any other kernel involved:
//   warp 0 waits on a barrier nobody arrives at, with a short limit: the wait runs out, the warp
//          reports KVH_ERR_TIMEOUT and raises the CTA's abort flag (what a kernel's CTA does);
//   warp 1 waits on the same barrier with the library's own limit (2 s) and must leave early,
//          through the abort flag;
//   warp 2 waits on a second barrier that warp 3 arrives at: the wait succeeds.
// Nothing here can hang: every wait is the bounded one under test.
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvh.h"
#include "kvh_async.cuh"
#include "kvh_decode.cuh"

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
