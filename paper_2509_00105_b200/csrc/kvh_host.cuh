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

// Called right after a <<<>>> launch: takes the launch's error (if any) off the runtime's
// per-thread slot, so that it is attributed to this launch and does not stick to later calls.
inline kvh_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? KVH_OK : KVH_ERR_CUDA;
}

// Build variants.  The library proper has no run-time switch between its kernels.  Two further
// builds of the same sources exist for the tests and for the scheduling comparison of the
// benchmark: KVH_VARIANT_DIRECT takes the one-CTA-per-tile kernels wherever they apply (so that
// the tests can check both kernel families on every shape), KVH_VARIANT_STATIC_STRIDE
// walks tiles with a fixed stride instead of pulling them through cluster launch control.
#if defined(KVH_VARIANT_DIRECT)
constexpr bool kPreferDirect = true;
constexpr int kTileSched = 1;
constexpr const char *kBuildVariant = "direct";
#elif defined(KVH_VARIANT_STATIC_STRIDE)
constexpr bool kPreferDirect = false;
constexpr int kTileSched = 0;
constexpr const char *kBuildVariant = "static-stride";
#else
constexpr bool kPreferDirect = false;
constexpr int kTileSched = 1;
constexpr const char *kBuildVariant = "default";
#endif

}  // namespace kvh
