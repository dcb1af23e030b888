// Benchmark-only translation unit, built into a library of its own (not part of libkvh.so and not
// declared in include/kvh.h): kernels that do no codec work and move bytes at the read : write mix
// of a decode launch.  The benchmark runs them beside the decode kernel to show what the memory
// system gives a plain streaming kernel at that mix (the copy that defines the HBM peak is 1 : 1).
//
//   kind 0  a persistent grid of warps; per unit a warp issues R 16-byte loads per lane from one
//           contiguous stream and 16 16-byte stores per lane to another (8 KiB written per unit)
//   kind 1  bulk copies only: one thread per CTA brings (R/16) x 16 KiB into shared memory with
//           cp.async.bulk and sends 16 KiB from shared memory to global memory with a bulk store,
//           four units in flight; no per-element instruction runs at all
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvh.h"
#include "kvh_async.cuh"

namespace {

using namespace kvh;

constexpr int kWritesPerLane = 16;
constexpr uint32_t kUnitBytes = 32u * kWritesPerLane * 16u;      // 8 KiB written per unit (kind 0)

template <int R>
__global__ void __launch_bounds__(256) ldst_mix_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst,
                                                       uint64_t n_units)
{
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t u = warp; u < n_units; u += n_warps) {
        const uint4 *in = src + u * (uint64_t)(R * 32) + lane;
        uint4 v[R];
#pragma unroll
        for (int j = 0; j < R; ++j) v[j] = __ldcs(in + j * 32);
        uint4 *out = dst + u * (uint64_t)(kWritesPerLane * 32) + lane;
#pragma unroll
        for (int j = 0; j < kWritesPerLane; ++j) {
            const uint4 a = v[j % R];
            out[j * 32] = make_uint4(a.x + j, a.y ^ j, a.z, a.w);
        }
    }
}

constexpr int kBulkStages = 4;
constexpr uint32_t kBulkUnit = 16u * 1024u;                       // bytes written per unit (kind 1)

__global__ void __launch_bounds__(32) bulk_mix_kernel(const uint8_t *__restrict__ src, uint8_t *__restrict__ dst,
                                                      uint64_t n_units, uint32_t in_bytes, int32_t *timed_out)
{
    extern __shared__ __align__(128) uint8_t stages[];
    __shared__ __align__(8) uint64_t full[kBulkStages];
    if (threadIdx.x != 0) return;
    for (int s = 0; s < kBulkStages; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    int abort_flag = 0;
    const uint64_t stride = gridDim.x;
    auto load = [&](uint64_t i) {                        // unit number i of this CTA
        const uint64_t u = blockIdx.x + i * stride;
        if (u >= n_units) return;
        const int s = (int)(i % kBulkStages);
        mbar_arrive_expect_tx(&full[s], in_bytes);
        bulk_load(stages + (size_t)s * kBulkUnit, src + u * in_bytes, in_bytes, &full[s]);
    };
    for (int i = 0; i < kBulkStages; ++i) load(i);
    uint64_t issued = 0;
    for (uint64_t i = 0; blockIdx.x + i * stride < n_units; ++i) {
        const int s = (int)(i % kBulkStages);
        if (!mbar_wait(&full[s], (uint32_t)(i / kBulkStages) & 1, &abort_flag)) {
            atomicMax(timed_out, (int32_t)KVH_ERR_TIMEOUT);
            break;
        }
        const uint64_t u = blockIdx.x + i * stride;
        bulk_store(dst + u * kBulkUnit, stages + (size_t)s * kBulkUnit, kBulkUnit);
        bulk_commit();
        bulk_wait_read<0>();                             // the stage has been read: it may be filled again
        load(i + kBulkStages);
        issued = i + 1 + kBulkStages;
    }
    // loads still in flight land before the CTA leaves; then every store completes
    for (uint64_t i = issued > (uint64_t)kBulkStages ? issued - kBulkStages : 0; blockIdx.x + i * stride < n_units && i < issued; ++i) {
        int never = 0;
        (void)mbar_wait(&full[i % kBulkStages], (uint32_t)(i / kBulkStages) & 1, &never);
    }
    bulk_wait_all();
}

template <int R>
kvh_status launch_ldst(const void *src, void *dst, uint64_t n_units, int sms, cudaStream_t st)
{
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ldst_mix_kernel<R>, 256, 0) != cudaSuccess || per_sm < 1)
        return KVH_ERR_CUDA;
    ldst_mix_kernel<R><<<sms * per_sm, 256, 0, st>>>(static_cast<const uint4 *>(src), static_cast<uint4 *>(dst), n_units);
    return cudaGetLastError() == cudaSuccess ? KVH_OK : KVH_ERR_CUDA;
}

}  // namespace

// kind: 0 or 1 (see above).  src [device, 16-byte aligned]: at least write_bytes * reads16 / 16 bytes;
// dst [device, 16-byte aligned]: write_bytes, a multiple of 16 KiB; reads16 in {16, 9, 5, 3}: 16-byte
// reads per 16 16-byte writes (the decode mixes of levels 0..3).  dev_status [device]: receives
// KVH_ERR_TIMEOUT if a bounded wait inside kind 1 runs out.  Returns once the launch is enqueued.
extern "C" kvh_status kvh_probe_stream_mix(int kind, const void *src, void *dst, uint64_t write_bytes, int reads16,
                                           int32_t *dev_status, void *stream)
{
    if (!src || !dst || !dev_status || write_bytes == 0 || write_bytes % kBulkUnit != 0) return KVH_ERR_INVALID_ARG;
    if (((uintptr_t)src | (uintptr_t)dst) & 15) return KVH_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return KVH_ERR_CUDA;
    if (kind == 0) {
        const uint64_t n_units = write_bytes / kUnitBytes;
        switch (reads16) {
        case 16: return launch_ldst<16>(src, dst, n_units, sms, st);
        case 9: return launch_ldst<9>(src, dst, n_units, sms, st);
        case 5: return launch_ldst<5>(src, dst, n_units, sms, st);
        case 3: return launch_ldst<3>(src, dst, n_units, sms, st);
        default: return KVH_ERR_INVALID_ARG;
        }
    }
    if (kind != 1 || (reads16 != 16 && reads16 != 9 && reads16 != 5 && reads16 != 3)) return KVH_ERR_INVALID_ARG;
    const size_t dyn = (size_t)kBulkStages * kBulkUnit;
    if (cudaFuncSetAttribute(bulk_mix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return KVH_ERR_CUDA;
    bulk_mix_kernel<<<sms * 3, 32, dyn, st>>>(static_cast<const uint8_t *>(src), static_cast<uint8_t *>(dst),
                                              write_bytes / kBulkUnit, kBulkUnit / 16 * (uint32_t)reads16, dev_status);
    return cudaGetLastError() == cudaSuccess ? KVH_OK : KVH_ERR_CUDA;
}
