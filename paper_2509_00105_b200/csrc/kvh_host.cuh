// Host-side helpers shared by the translation units that implement the C ABI: argument checks
// and launch bookkeeping.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "kvh.h"
#include "kvh_format.cuh"

namespace kvh {

inline bool aligned(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

inline kvh_status check_shape(int level, int l, int c)
{
    if (level < 0 || level >= kNumLevels) return KVH_ERR_BAD_LEVEL;
    if (l <= 0 || c <= 0 || c % kGroup != 0) return KVH_ERR_BAD_SHAPE;
    return KVH_OK;
}

inline kvh_status check_pool(const kvh_pool *pool)
{
    if (!pool || !pool->base) return KVH_ERR_INVALID_ARG;
    if (pool->n_layers <= 0 || pool->n_channels <= 0 || pool->n_channels % kGroup != 0) return KVH_ERR_BAD_SHAPE;
    if (pool->page_tokens <= 0 || kChunkTokens % pool->page_tokens != 0) return KVH_ERR_BAD_SHAPE;
    if (pool->num_pages <= 0) return KVH_ERR_BAD_SHAPE;
    if (pool->layer_stride < 0 || pool->kv_stride < 0 || pool->page_stride < 0) return KVH_ERR_BAD_SHAPE;
    if (!aligned(pool->base, 16) || pool->layer_stride % 8 || pool->kv_stride % 8 || pool->page_stride % 8)
        return KVH_ERR_MISALIGNED;
    return KVH_OK;
}

// one CTA per (chunk, layer, K|V, tile); 0 if the grid would not fit
inline unsigned grid_for(int64_t n_chunks, int l)
{
    const int64_t g = n_chunks * l * 2 * kTilesPerChunk;
    return (g <= 0 || g > 0x7fffffffLL) ? 0u : (unsigned)g;
}

// Width of the column blocks the TMA-fed kernels cut a row of c channels into: c itself up to 1024,
// else the largest divisor of c that is at most 1024 and a multiple of 128 (every piece a bulk copy
// moves is then a multiple of 16 bytes), or 0 if there is none.
inline int block_width(int c)
{
    if (c <= 1024) return c;
    for (int w = 1024; w >= 128; w -= 128)
        if (c % w == 0) return w;
    return 0;
}

// Tiles of 32 tokens a work unit of the TMA-fed kernels takes when rows are bw channels wide: as
// many (1, 2, 4 or 8, a chunk has 8) as keep a unit within 1024 channels' worth of a tile, so that
// narrow rows still give every consumer thread work and the pipeline units of useful size.
inline int tiles_per_unit(int bw)
{
    int t = 1;
    while (t < kTilesPerChunk && 2 * t * bw <= 1024) t <<= 1;
    return t;
}

inline kvh_status launch_status()
{
    return cudaPeekAtLastError() == cudaSuccess ? KVH_OK : KVH_ERR_CUDA;
}

}  // namespace kvh
