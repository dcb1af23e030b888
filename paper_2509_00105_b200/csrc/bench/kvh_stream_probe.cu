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
//   kind 2  the decode kernel's own skeleton with the codec taken out: CTAs of a producer warp and 8
//           consumer warps, two shared-memory stages fed by bulk copies, units handed out through
//           cluster launch control, three CTAs per SM; per unit a consumer thread loads 16 bytes from
//           the stage per row and stores them as one 16-byte vector of each of its 16 (or 8) rows of
//           2 KiB, the decode kernel's store pattern, and does nothing else
//   kind 4  kind 2 writing every 32 KiB page (16 rows of 2 KiB, a 16-token page of one plane) to a
//           pseudo-random page of the destination: what a shuffled page table does to the store stream
//   kind 3  kind 1 with its units handed out through cluster launch control instead of a fixed
//           stride (SMs do not all reach memory equally fast, so a fixed stride waits for the slowest)
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


// kind 3: the bulk copies of kind 1, units pulled through cluster launch control.  One warp per CTA;
// lane 0 issues the copies, all lanes take part in the hand-out.
__global__ void __launch_bounds__(32) bulk_mix_clc_kernel(const uint8_t *__restrict__ src, uint8_t *__restrict__ dst,
                                                          uint32_t n_units, uint32_t in_bytes, int32_t *timed_out)
{
    extern __shared__ __align__(128) uint8_t stages[];
    __shared__ __align__(8) uint64_t full[kBulkStages];
    __shared__ __align__(16) uint4 clc_response[2];
    __shared__ __align__(8) uint64_t clc_bar[2];
    __shared__ int abort_flag;
    const int lane = threadIdx.x;
    if (lane == 0) {
        for (int s = 0; s < kBulkStages; ++s) mbar_init(&full[s], 1);
        mbar_init(&clc_bar[0], 1);
        mbar_init(&clc_bar[1], 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    TileFeed feed{clc_response, clc_bar, 1, lane, &abort_flag};
    int64_t next_id = blockIdx.x;                        // the unit to load next, -1: none left
    bool ok = true;
    auto advance = [&]() {                               // all lanes: move next_id on
        if (next_id < 0) return;
        feed.ask();
        const int more = feed.next(next_id, n_units);
        if (more < 0) ok = false;
        if (more <= 0) next_id = -1;
    };
    int64_t held[kBulkStages];                           // the unit in each stage, -1: empty
    uint32_t loads[kBulkStages];                         // copies issued into each stage so far
#pragma unroll
    for (int s = 0; s < kBulkStages; ++s) { held[s] = -1; loads[s] = 0; }
    auto load = [&](int s) {                             // all lanes: put the next unit into stage s
        held[s] = next_id;
        if (next_id < 0) return;
        if (lane == 0) {
            mbar_arrive_expect_tx(&full[s], in_bytes);
            bulk_load(stages + (size_t)s * kBulkUnit, src + (uint64_t)next_id * in_bytes, in_bytes, &full[s]);
        }
        ++loads[s];
        advance();
    };
#pragma unroll
    for (int s = 0; s < kBulkStages; ++s)
        if (ok) load(s);
    while (ok) {
        bool any = false;
#pragma unroll
        for (int s = 0; s < kBulkStages; ++s) {
            if (!ok || held[s] < 0) continue;
            any = true;
            bool w = true;
            if (lane == 0) w = mbar_wait(&full[s], (loads[s] - 1) & 1, &abort_flag);
            w = __shfl_sync(0xffffffffu, w, 0);
            if (!w) { ok = false; break; }
            if (lane == 0) {
                bulk_store(dst + (uint64_t)held[s] * kBulkUnit, stages + (size_t)s * kBulkUnit, kBulkUnit);
                bulk_commit();
                bulk_wait_read<0>();                     // the stage has been read: it may be filled again
            }
            __syncwarp();
            load(s);
        }
        if (!any) break;
    }
    if (lane == 0) {
        if (!ok) {
            atomicMax(timed_out, (int32_t)KVH_ERR_TIMEOUT);
            // copies still in flight land before the CTA leaves
            int never = 0;
            for (int s = 0; s < kBulkStages; ++s)
                if (held[s] >= 0) (void)mbar_wait(&full[s], (loads[s] - 1) & 1, &never);
        }
        feed.drain();
        bulk_wait_all();
    }
}

// ---- kind 2: producer warp + 8 consumer warps over a two-stage ring, no codec work ------------------

constexpr int kRingConsumers = 256;
constexpr int kRingThreads = kRingConsumers + 32;
constexpr int kRingStages = 2;
constexpr uint32_t kRingStageBytes = 36u * 1024u;                 // the decode kernel's stage at 1024 channels
constexpr uint32_t kRingRowBytes = 2048u;                         // a page row of 1024 bf16 channels

// ROWS: rows of 2 KiB a thread writes per unit (16: 64 KiB per unit; 8: 32 KiB, the raw level's half tile)
// SCATTER: the destination's 32 KiB pages are permuted (page i of the sequential order goes to page
// i * 104729 mod n_pages; the multiplier shares no factor with the page counts used here, so this is
// a bijection).
constexpr uint32_t kRingPage = 32u * 1024u;
constexpr uint64_t kRingScatterMul = 104729ull;
template <int ROWS, bool SCATTER>
__global__ void __launch_bounds__(kRingThreads, 3) ring_mix_kernel(const uint8_t *__restrict__ src, uint8_t *__restrict__ dst,
                                                                   uint32_t n_units, uint32_t in_bytes, int32_t *status)
{
    extern __shared__ __align__(128) uint8_t stage_mem[];
    __shared__ __align__(8) uint64_t full_bar[kRingStages];
    __shared__ __align__(8) uint64_t empty_bar[kRingStages];
    __shared__ int64_t unit_of[kRingStages];                      // the stage's unit, -1: no more work
    __shared__ int abort_flag;
    __shared__ int wait_verdict[2];
    __shared__ __align__(16) uint4 clc_response[2];
    __shared__ __align__(8) uint64_t clc_bar[2];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t kUnitWrite = 2u * 128u * ROWS * 16u;       // 2 row groups x 128 vectors x ROWS rows x 16 bytes
    if (threadIdx.x == 0) {
        for (int s = 0; s < kRingStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kRingConsumers / 32);
        }
        mbar_init(&clc_bar[0], 1);
        mbar_init(&clc_bar[1], 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == kRingConsumers / 32) {
        // producer warp: one bulk copy per unit into the next stage
        uint32_t unit = 0;
        bool ok = true;
        auto emit = [&](int64_t id) -> bool {
            const int s = unit % kRingStages;
            if (unit >= (uint32_t)kRingStages) {
                bool w = true;
                if (lane == 0) w = mbar_wait(&empty_bar[s], ((unit / kRingStages) - 1) & 1, &abort_flag);
                if (!__shfl_sync(0xffffffffu, w, 0)) return false;
            }
            if (lane == 0) {
                unit_of[s] = id;
                if (id < 0) {
                    mbar_arrive(&full_bar[s]);
                } else {
                    mbar_arrive_expect_tx(&full_bar[s], in_bytes);
                    bulk_load(stage_mem + (size_t)s * kRingStageBytes, src + (uint64_t)id * in_bytes, in_bytes, &full_bar[s]);
                }
            }
            ++unit;
            return true;
        };
        TileFeed feed{clc_response, clc_bar, 1, lane, &abort_flag};
        int64_t id = blockIdx.x;
        while (ok && id < (int64_t)n_units) {
            feed.ask();
            ok = emit(id);
            if (!ok) break;
            const int more = feed.next(id, n_units);
            if (more < 0) ok = false;
            if (more <= 0) break;
        }
        if (ok) ok = emit(-1);                                   // end marker
        if (!ok && lane == 0) {
            atomicMax(status, (int32_t)KVH_ERR_TIMEOUT);
            abort_flag = 1;
        }
        if (lane == 0) {                                         // leave only after every copy issued has landed
            int never = 0;
            const uint32_t first = unit > (uint32_t)kRingStages ? unit - kRingStages : 0;
            for (uint32_t w = first; w < unit; ++w)
                (void)mbar_wait(&full_bar[w % kRingStages], (w / kRingStages) & 1, &never);
            feed.drain();
        }
    } else {
        const int g = threadIdx.x >> 7, cv = threadIdx.x & 127;   // row group and 16-byte vector within a row
        const uint32_t n_vec = in_bytes / 16u;
        for (uint32_t unit = 0;; ++unit) {
            const int s = unit % kRingStages;
            if (!group_wait(&full_bar[s], (unit / kRingStages) & 1, &abort_flag, wait_verdict, unit, 1, kRingConsumers,
                            warp == 0)) {
                if (threadIdx.x == 0) atomicMax(status, (int32_t)KVH_ERR_TIMEOUT);
                break;
            }
            const int64_t id = unit_of[s];
            if (id < 0) break;
            const uint4 *st = reinterpret_cast<const uint4 *>(stage_mem + (size_t)s * kRingStageBytes);
            uint64_t off = (uint64_t)id * kUnitWrite + (uint64_t)g * ROWS * kRingRowBytes;    // a thread's rows lie in one page
            if (SCATTER) {
                const uint64_t n_pages = (uint64_t)n_units * kUnitWrite / kRingPage;
                off = (off / kRingPage * kRingScatterMul) % n_pages * kRingPage + off % kRingPage;
            }
            uint4 *out = reinterpret_cast<uint4 *>(dst + off) + cv;
            uint32_t v = threadIdx.x;                            // < 256 <= n_vec
#pragma unroll
            for (int k = 0; k < ROWS; ++k) {
                out[k * (kRingRowBytes / 16)] = st[v];
                v += kRingConsumers;
                if (v >= n_vec) v -= n_vec;                  // n_vec >= 768 > 256: one step suffices
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[s]);
        }
    }
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

// kind: 0 .. 4 (see above).  src [device, 16-byte aligned]: at least write_bytes * reads16 / 16 bytes;
// dst [device, 16-byte aligned]: write_bytes, a multiple of 16 KiB; reads16 in {16, 9, 5, 3}: 16-byte
// reads per 16 16-byte writes (the decode mixes of levels 0..3).  dev_status [device]: receives
// KVH_ERR_TIMEOUT if a bounded wait inside kinds 1 to 4 runs out; kinds 2 and 4 want write_bytes to be a
// multiple of 64 KiB.  Returns once the launch is enqueued.
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
    if (kind == 2 || kind == 4) {
        if (reads16 != 16 && reads16 != 9 && reads16 != 5 && reads16 != 3) return KVH_ERR_INVALID_ARG;
        // the raw level is fed in half tiles (32 KiB in, 32 KiB out), the quantised ones in whole tiles
        const bool half = reads16 == 16;
        const uint32_t unit_write = half ? 32u * 1024u : 64u * 1024u;
        if (write_bytes % unit_write != 0 || write_bytes / unit_write > 0x7fffffffull) return KVH_ERR_INVALID_ARG;
        const uint32_t n_units = (uint32_t)(write_bytes / unit_write);
        const uint32_t in_bytes = unit_write / 16u * (uint32_t)reads16;
        const size_t dyn = (size_t)kRingStages * kRingStageBytes;
        const uint64_t n_pages = write_bytes / kRingPage;
        if (kind == 4 && n_pages % kRingScatterMul == 0) return KVH_ERR_INVALID_ARG;   // the multiplier is prime: a bijection otherwise
        auto kernel = kind == 4 ? (half ? ring_mix_kernel<8, true> : ring_mix_kernel<16, true>)
                                : (half ? ring_mix_kernel<8, false> : ring_mix_kernel<16, false>);
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
            return KVH_ERR_CUDA;
        kernel<<<n_units, kRingThreads, dyn, st>>>(static_cast<const uint8_t *>(src), static_cast<uint8_t *>(dst), n_units,
                                                   in_bytes, dev_status);
        return cudaGetLastError() == cudaSuccess ? KVH_OK : KVH_ERR_CUDA;
    }
    if (kind == 3) {
        if (reads16 != 16 && reads16 != 9 && reads16 != 5 && reads16 != 3) return KVH_ERR_INVALID_ARG;
        if (write_bytes / kBulkUnit > 0x7fffffffull) return KVH_ERR_INVALID_ARG;
        const size_t dyn = (size_t)kBulkStages * kBulkUnit;
        if (cudaFuncSetAttribute(bulk_mix_clc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
            return KVH_ERR_CUDA;
        const uint32_t n_units = (uint32_t)(write_bytes / kBulkUnit);
        bulk_mix_clc_kernel<<<n_units, 32, dyn, st>>>(static_cast<const uint8_t *>(src), static_cast<uint8_t *>(dst), n_units,
                                                      kBulkUnit / 16 * (uint32_t)reads16, dev_status);
        return cudaGetLastError() == cudaSuccess ? KVH_OK : KVH_ERR_CUDA;
    }
    if (kind != 1 || (reads16 != 16 && reads16 != 9 && reads16 != 5 && reads16 != 3)) return KVH_ERR_INVALID_ARG;
    const size_t dyn = (size_t)kBulkStages * kBulkUnit;
    if (cudaFuncSetAttribute(bulk_mix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return KVH_ERR_CUDA;
    bulk_mix_kernel<<<sms * 3, 32, dyn, st>>>(static_cast<const uint8_t *>(src), static_cast<uint8_t *>(dst),
                                              write_bytes / kBulkUnit, kBulkUnit / 16 * (uint32_t)reads16, dev_status);
    return cudaGetLastError() == cudaSuccess ? KVH_OK : KVH_ERR_CUDA;
}
