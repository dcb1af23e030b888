// kvh_transcode: host side (argument checks, choice of the kernel instance, launch).
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvh.h"
#include "kvh_host.cuh"
#include "kvh_transcode.cuh"

using namespace kvh;

namespace {

template <int C, typename Chunks>
auto pick_kernel(int lin, int lout) -> void (*)(const TranscodeParams, const int, const int, const Chunks)
{
    if (lin < 0) return transcode_tma_kernel<C, -1, -1, Chunks>;
    switch (lin * 4 + lout) {
    case 0 * 4 + 1: return transcode_tma_kernel<C, 0, 1, Chunks>;
    case 0 * 4 + 2: return transcode_tma_kernel<C, 0, 2, Chunks>;
    case 0 * 4 + 3: return transcode_tma_kernel<C, 0, 3, Chunks>;
    case 1 * 4 + 2: return transcode_tma_kernel<C, 1, 2, Chunks>;
    case 1 * 4 + 3: return transcode_tma_kernel<C, 1, 3, Chunks>;
    case 2 * 4 + 3: return transcode_tma_kernel<C, 2, 3, Chunks>;
    default: return nullptr;
    }
}

template <typename Chunks>
kvh_status launch(const TranscodeParams &p, int lin, int lout, int n_chunks, cudaStream_t st, const Chunks &chunks)
{
    const int64_t tiles = (int64_t)grid_for(n_chunks, p.l) * p.n_blocks / p.tpu;     // one CTA per unit
    if (grid_for(n_chunks, p.l) == 0 || tiles > 0x7fffffffLL) return KVH_ERR_BAD_SHAPE;
    const unsigned grid = (unsigned)tiles;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return KVH_ERR_CUDA;
    auto kernel = p.c == 1024 ? pick_kernel<1024, Chunks>(lin, lout) : pick_kernel<0, Chunks>(lin, lout);
    if (!kernel) return KVH_ERR_BAD_LEVEL;
    const size_t dyn = lin >= 1 ? (size_t)tc_stages<1>() * tc_stage_bytes<1>() : (size_t)tc_stages<0>() * tc_stage_bytes<0>();
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return KVH_ERR_CUDA;
    const int sched = kTileSched;
    const unsigned pgrid = sched == 1 ? grid : (grid < (unsigned)sms ? grid : (unsigned)sms);
    kernel<<<pgrid, 32 + kEncGroupThreads, dyn, st>>>(p, n_chunks, sched, chunks);
    return launch_status();
}

}  // namespace

extern "C" kvh_status kvh_transcode(const void *in_streams, uint64_t in_bytes, const kvh_chunk_desc *in_descs,
                                    void *out_streams, uint64_t out_capacity, const kvh_chunk_desc *out_descs,
                                    const kvh_chunk_desc *in_descs_host, const kvh_chunk_desc *out_descs_host,
                                    int n_chunks, int n_layers, int n_channels, int level_in, int level_out,
                                    int32_t *dev_status, void *stream)
{
    if (!in_streams || !out_streams || !in_descs || !out_descs || n_chunks < 0) return KVH_ERR_INVALID_ARG;
    const kvh_status s = check_shape(0, n_layers, n_channels);
    if (s != KVH_OK) return s;
    if (block_width(n_channels) == 0) return KVH_ERR_BAD_SHAPE;      // a tile of a column block has to fit a stage
    if ((level_in < 0) != (level_out < 0)) return KVH_ERR_BAD_LEVEL;
    if (level_in >= 0 && (level_in >= kNumLevels || level_out >= kNumLevels || level_out <= level_in))
        return KVH_ERR_BAD_LEVEL;
    if (!aligned(in_streams, KVH_SECTION_ALIGN) || !aligned(out_streams, KVH_SECTION_ALIGN) ||
        !aligned(in_descs, 8) || !aligned(out_descs, 8))
        return KVH_ERR_MISALIGNED;
    if (n_chunks == 0) return KVH_OK;
    if (grid_for(n_chunks, n_layers) == 0) return KVH_ERR_BAD_SHAPE;
    TranscodeParams p{};
    p.in = static_cast<const uint8_t *>(in_streams);
    p.in_bytes = in_bytes;
    p.in_descs = in_descs;
    p.out = static_cast<uint8_t *>(out_streams);
    p.out_capacity = out_capacity;
    p.out_descs = out_descs;
    p.l = n_layers; p.c = n_channels;
    p.bw = block_width(n_channels);
    p.n_blocks = n_channels / p.bw;
    p.tpu = p.n_blocks == 1 ? tiles_per_unit(p.bw) : 1;              // narrow rows: several tiles per unit
    p.status = dev_status;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (level_in >= 0 || !in_descs_host || !out_descs_host)
        return launch(p, level_in, level_out, n_chunks, st, AllChunks{});
    // host copies of both descriptor arrays: every pair of levels gets its own specialised launch
    // over the list of its chunks; what fits no pair goes to the general instance, which reports it
    static thread_local ListedChunks list;
    for (int pair = 0; pair <= kNumLevels * kNumLevels; ++pair) {
        const int lin = pair / kNumLevels, lout = pair % kNumLevels;
        const bool rest = pair == kNumLevels * kNumLevels;
        if (!rest && lout <= lin) continue;
        int n = 0;
        for (int i = 0; i <= n_chunks; ++i) {
            if (i < n_chunks) {
                const int a = in_descs_host[i].level, b = out_descs_host[i].level;
                const bool proper = a >= 0 && b < kNumLevels && b > a;
                if (rest ? !proper : (a == lin && b == lout)) list.idx[n++] = (uint32_t)i;
            }
            if (n == kMaxListedChunks || (i == n_chunks && n > 0)) {
                const kvh_status ls = rest ? launch(p, -1, -1, n, st, list) : launch(p, lin, lout, n, st, list);
                if (ls != KVH_OK) return ls;
                n = 0;
            }
        }
    }
    return KVH_OK;
}
