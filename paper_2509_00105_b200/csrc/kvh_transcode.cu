// kvh_transcode: host side (argument checks, choice of the kernel instance, launch).
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "kvh.h"
#include "kvh_host.cuh"
#include "kvh_transcode.cuh"

using namespace kvh;

namespace {

typedef void (*TranscodeKernel)(const TranscodeParams, const int, const int);

template <int C>
TranscodeKernel pick_kernel(int lin, int lout)
{
    if (lin < 0) return transcode_tma_kernel<C, -1, -1>;
    switch (lin * 4 + lout) {
    case 0 * 4 + 1: return transcode_tma_kernel<C, 0, 1>;
    case 0 * 4 + 2: return transcode_tma_kernel<C, 0, 2>;
    case 0 * 4 + 3: return transcode_tma_kernel<C, 0, 3>;
    case 1 * 4 + 2: return transcode_tma_kernel<C, 1, 2>;
    case 1 * 4 + 3: return transcode_tma_kernel<C, 1, 3>;
    case 2 * 4 + 3: return transcode_tma_kernel<C, 2, 3>;
    default: return nullptr;
    }
}

}  // namespace

extern "C" kvh_status kvh_transcode(const void *in_streams, uint64_t in_bytes, const kvh_chunk_desc *in_descs,
                                    void *out_streams, uint64_t out_capacity, const kvh_chunk_desc *out_descs,
                                    int n_chunks, int n_layers, int n_channels, int level_in, int level_out,
                                    int32_t *dev_status, void *stream)
{
    if (!in_streams || !out_streams || !in_descs || !out_descs || n_chunks < 0) return KVH_ERR_INVALID_ARG;
    const kvh_status s = check_shape(0, n_layers, n_channels);
    if (s != KVH_OK) return s;
    if (n_channels > kEncMaxChannels) return KVH_ERR_BAD_SHAPE;      // a tile has to fit a shared-memory stage
    if ((level_in < 0) != (level_out < 0)) return KVH_ERR_BAD_LEVEL;
    if (level_in >= 0 && (level_in >= kNumLevels || level_out >= kNumLevels || level_out <= level_in))
        return KVH_ERR_BAD_LEVEL;
    if (!aligned(in_streams, KVH_SECTION_ALIGN) || !aligned(out_streams, KVH_SECTION_ALIGN) ||
        !aligned(in_descs, 8) || !aligned(out_descs, 8))
        return KVH_ERR_MISALIGNED;
    if (n_chunks == 0) return KVH_OK;
    const unsigned grid = grid_for(n_chunks, n_layers);
    if (grid == 0) return KVH_ERR_BAD_SHAPE;
    TranscodeParams p{};
    p.in = static_cast<const uint8_t *>(in_streams);
    p.in_bytes = in_bytes;
    p.in_descs = in_descs;
    p.out = static_cast<uint8_t *>(out_streams);
    p.out_capacity = out_capacity;
    p.out_descs = out_descs;
    p.l = n_layers; p.c = n_channels;
    p.status = dev_status;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return KVH_ERR_CUDA;
    TranscodeKernel kernel = n_channels == 1024 ? pick_kernel<1024>(level_in, level_out)
                                                : pick_kernel<0>(level_in, level_out);
    if (!kernel) return KVH_ERR_BAD_LEVEL;
    const size_t dyn = (size_t)kEncStages * kEncStageBytes;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return KVH_ERR_CUDA;
    const char *sched_env = getenv("KVH_ENCODE_SCHED");              // static tile stride: a measurement aid
    const int sched = (sched_env && strcmp(sched_env, "static") == 0) ? 0 : 1;
    const unsigned pgrid = sched == 1 ? grid : (grid < (unsigned)sms ? grid : (unsigned)sms);
    kernel<<<pgrid, 32 + kEncGroupThreads, dyn, static_cast<cudaStream_t>(stream)>>>(p, n_chunks, sched);
    return launch_status();
}
