// Host side of the C ABI declared in include/kvh.h: argument validation, size
// arithmetic and kernel launches.  No device memory is allocated here, and the
// only state that survives a call is the per-device address of the fixed staging
// array of kvh_load_host_static.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvh.h"

#include "kvh_decode.cuh"
#include "kvh_decode_tma.cuh"
#include "kvh_encode.cuh"
#include "kvh_encode_tma.cuh"
#include "kvh_format.cuh"
#include "kvh_host.cuh"

using namespace kvh;

namespace {

kvh_status launch_decode(DecodeParams &p, const kvh_pool *pool, int n_chunks, void *stream)
{
    p.pool = static_cast<uint16_t *>(pool->base);
    p.layer_stride = pool->layer_stride;
    p.kv_stride = pool->kv_stride;
    p.page_stride = pool->page_stride;
    p.num_pages = pool->num_pages;
    p.page_tokens = pool->page_tokens;
    p.page_shift = 0;
    while ((1 << p.page_shift) < pool->page_tokens) ++p.page_shift;   // divisors of 256 are powers of two
    p.l = pool->n_layers;
    p.c = pool->n_channels;
    const unsigned grid = grid_for(n_chunks, p.l);
    if (grid == 0) return KVH_ERR_BAD_SHAPE;
    // the persistent TMA kernel needs a column block to fit a shared-memory stage and pages of at
    // least 8 tokens; otherwise (and in the "direct" build) the one-CTA-per-tile kernel runs
    const bool want_tma = !kPreferDirect;
    p.bw = block_width(p.c);                             // rows wider than 1024 channels go in column blocks
    p.n_blocks = p.bw > 0 ? p.c / p.bw : 1;
    const bool small_pages = p.page_tokens < 16;           // a thread's rows may then span several pages
    // narrow rows: several tiles per unit (the instance for small pages keeps one)
    p.tpu = (p.bw > 0 && p.n_blocks == 1 && !small_pages) ? tiles_per_unit(p.bw) : 1;
    const int64_t tiles = (int64_t)grid * p.n_blocks / p.tpu;
    if (want_tma && p.bw > 0 && tiles <= 0x7fffffffLL && p.page_tokens >= 8) {    // a lane per page id of a chunk
        int dev = 0, sms = 0, per_sm = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return KVH_ERR_CUDA;
        // Stage memory per CTA: a ring of quanta of 12 * c bytes, 72 KiB of them when c = 1024, so
        // that three CTAs (24 consumer warps) share an SM.  A unit takes 1, 2 or 3 quanta by its
        // level: 6 units in flight at 2 bits, 3 at 4 bits, 2 at 8 bits or raw.
        const int quanta = ring_quanta(p.bw * p.tpu);
        const size_t dyn = (size_t)quanta * tma_quantum_bytes(p.bw * p.tpu);
        // the instance with the channel count of the Llama-3 shapes compiled in, or the general one
        auto kernel = p.c == 1024 ? (small_pages ? decode_tma_kernel<1024, true> : decode_tma_kernel<1024, false>)
                                  : (small_pages ? decode_tma_kernel<0, true> : decode_tma_kernel<0, false>);
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kTmaThreads, dyn) != cudaSuccess ||
            per_sm < 1)
            return KVH_ERR_CUDA;
        const int sched = kTileSched;
        const int64_t resident = (int64_t)sms * per_sm;
        const unsigned pgrid = sched == 1 ? (unsigned)tiles : (unsigned)(tiles < resident ? tiles : resident);
        kernel<<<pgrid, kTmaThreads, dyn, static_cast<cudaStream_t>(stream)>>>(p, n_chunks, quanta, sched);
        return launch_status();
    }
    decode_kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return launch_status();
}

// Tensor map of the encode source seen as a 2-D tensor [n_layers * 2 * src_N rows][c channels] of
// bf16, with boxes of 256 channels x 32 rows; false if the driver entry point is not to be had.
bool make_kv_map(const EncodeParams &p, CUtensorMap *map)
{
    static PFN_cuTensorMapEncodeTiled encode = [] {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
    }();
    if (!encode) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)p.c, (cuuint64_t)p.l * 2 * (cuuint64_t)p.src_N};
    const cuuint64_t strides[1] = {(cuuint64_t)p.c * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBoxChannels, (cuuint32_t)kTileTokens};
    const cuuint32_t elem[2] = {1, 1};
    if (dims[1] > 0x7fffffffull) return false;           // row coordinates are 32-bit signed
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<uint16_t *>(p.kv), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename Chunks>
kvh_status launch_encode_tma(const EncodeParams &p, int level, unsigned grid, int n_chunks, cudaStream_t st,
                             const Chunks &chunks)
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return KVH_ERR_CUDA;
    const size_t dyn = (size_t)kEncStages * kEncStageBytes;
    void (*kernel)(const EncodeParams, const int, const int, const Chunks, const CUtensorMap);
    CUtensorMap kv_map{};
    // wider rows in blocks of 1024 channels: the instance with the boxed stage; it wants the tensor
    // map unless tokens are gathered from kept runs
    const bool boxed = p.c != 1024 && p.bw == 1024 && (p.n_runs > 0 || make_kv_map(p, &kv_map));
    if (p.boxes && !make_kv_map(p, &kv_map)) return KVH_ERR_CUDA;
    if (p.c == 1024) {
        kernel = level == 0 ? encode_tma_kernel<1024, 0, Chunks> : level == 1 ? encode_tma_kernel<1024, 1, Chunks>
               : level == 2 ? encode_tma_kernel<1024, 2, Chunks> : level == 3 ? encode_tma_kernel<1024, 3, Chunks>
               : encode_tma_kernel<1024, -1, Chunks>;
    } else if (boxed) {
        kernel = level == 0 ? encode_tma_kernel<1024, 0, Chunks, true> : level == 1 ? encode_tma_kernel<1024, 1, Chunks, true>
               : level == 2 ? encode_tma_kernel<1024, 2, Chunks, true> : level == 3 ? encode_tma_kernel<1024, 3, Chunks, true>
               : encode_tma_kernel<1024, -1, Chunks, true>;
    } else {
        kernel = level == 0 ? encode_tma_kernel<0, 0, Chunks> : level == 1 ? encode_tma_kernel<0, 1, Chunks>
               : level == 2 ? encode_tma_kernel<0, 2, Chunks> : level == 3 ? encode_tma_kernel<0, 3, Chunks>
               : encode_tma_kernel<0, -1, Chunks>;
    }
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return KVH_ERR_CUDA;
    const int sched = kTileSched;
    const unsigned pgrid = sched == 1 ? grid : (grid < (unsigned)sms ? grid : (unsigned)sms);
    kernel<<<pgrid, 32 + kEncGroupThreads, dyn, st>>>(p, n_chunks, sched, chunks, kv_map);
    return launch_status();
}

// Encode launch: the persistent TMA-fed kernel when rows are at most 1024 channels wide or divide
// into column blocks, otherwise (and in the "direct" build, token dropping apart) one CTA per tile
// reading global memory directly.
// descs_host (may be nullptr): the caller's host copy of p.descs, indexed like it.  With it the
// chunks of each level go, as index lists in the kernel parameters, to the instance specialised for
// that level; without it one instance that holds all levels takes the chunks in order.
kvh_status launch_encode(const EncodeParams &p, int64_t n_chunks, void *stream,
                         const kvh_chunk_desc *descs_host = nullptr)
{
    const unsigned grid = grid_for(n_chunks, p.l);
    if (grid == 0) return KVH_ERR_BAD_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int bw = block_width(p.c);
    if (bw > 0 && (p.n_runs > 0 || !kPreferDirect)) {
        EncodeParams q = p;
        q.bw = bw;
        q.n_blocks = p.c / bw;
        q.tpu = q.n_blocks == 1 ? tiles_per_unit(bw) : 1;        // narrow rows: several tiles per unit
        // 768, 1280, 1536 ...: neither packed by whole tiles nor blocks of 1024: blocks of 256 channels,
        // 4 tiles per unit, fetched as 2-D boxes (token dropping gathers rows and keeps the row copies)
        CUtensorMap probe;
        if (p.c % kBoxChannels == 0 && p.c % 1024 != 0 && p.c != 256 && p.c != 512 && p.n_runs == 0 &&
            make_kv_map(p, &probe)) {                    // without a tensor map the row copies remain
            q.bw = kBoxChannels;
            q.n_blocks = p.c / kBoxChannels;
            q.tpu = 1024 / kBoxChannels;
            q.boxes = 1;
        }
        auto tiles = [&](int64_t chunks) -> unsigned {   // one CTA per unit and column block; 0 if too many
            const int64_t g = (int64_t)grid_for(chunks, p.l) * q.n_blocks / q.tpu;
            return (grid_for(chunks, p.l) == 0 || g > 0x7fffffffLL) ? 0u : (unsigned)g;
        };
        if (tiles(n_chunks) == 0) return KVH_ERR_BAD_SHAPE;
        const int level = p.descs ? p.hint_level : p.level;
        if (level >= 0 || !descs_host || !p.descs)
            return launch_encode_tma(q, level, tiles(n_chunks), (int)n_chunks, st, AllChunks{});
        static thread_local ListedChunks list;           // 16 KB of parameters, filled per launch
        q.chunk0 = 0;
        for (int lv = 0; lv < kNumLevels; ++lv) {
            q.hint_level = lv;
            int n = 0;
            for (int64_t i = 0; i <= n_chunks; ++i) {
                if (i < n_chunks && descs_host[p.chunk0 + i].level == lv) list.idx[n++] = (uint32_t)(p.chunk0 + i);
                if (n == kMaxListedChunks || (i == n_chunks && n > 0)) {
                    const kvh_status s = launch_encode_tma(q, lv, tiles(n), n, st, list);
                    if (s != KVH_OK) return s;
                    n = 0;
                }
            }
        }
        // descriptors whose level is no level at all go to the general instance, which reports and skips them
        int n = 0;
        for (int64_t i = 0; i < n_chunks && n < kMaxListedChunks; ++i)
            if (descs_host[p.chunk0 + i].level < 0 || descs_host[p.chunk0 + i].level >= kNumLevels)
                list.idx[n++] = (uint32_t)(p.chunk0 + i);
        if (n > 0) {
            q.hint_level = -1;
            return launch_encode_tma(q, -1, tiles(n), n, st, list);
        }
        return KVH_OK;
    }
    encode_kernel<<<grid, kThreads, 0, st>>>(p);
    return launch_status();
}

}  // namespace

extern "C" {

int kvh_format_version(void) { return KVH_FORMAT_VERSION; }
int kvh_num_levels(void) { return kNumLevels; }
const char *kvh_build_variant(void) { return kBuildVariant; }

const char *kvh_status_string(kvh_status s)
{
    switch (s) {
    case KVH_OK: return "ok";
    case KVH_ERR_INVALID_ARG: return "invalid argument";
    case KVH_ERR_BAD_LEVEL: return "level outside 0..3";
    case KVH_ERR_BAD_SHAPE: return "unsupported shape";
    case KVH_ERR_MISALIGNED: return "misaligned pointer, offset or stride";
    case KVH_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case KVH_ERR_PAGE_OOB: return "page id outside the pool";
    case KVH_ERR_CUDA: return "CUDA runtime error";
    case KVH_ERR_TIMEOUT: return "device wait timed out";
    default: return "unknown status";
    }
}

kvh_status kvh_level_info(int level, int *bits, int *group, int *lossless)
{
    if (level < 0 || level >= kNumLevels) return KVH_ERR_BAD_LEVEL;
    if (bits) *bits = level_bits(level);
    if (group) *group = level == 0 ? 0 : kGroup;
    if (lossless) *lossless = level == 0;
    return KVH_OK;
}

kvh_status kvh_level_bytes(int level, int n_layers, int n_channels, int n_tokens, uint64_t *out)
{
    if (!out) return KVH_ERR_INVALID_ARG;
    const kvh_status s = check_shape(level, n_layers, n_channels);
    if (s != KVH_OK) return s;
    if (n_tokens < 1 || n_tokens > kChunkTokens) return KVH_ERR_BAD_SHAPE;
    *out = chunk_bytes(level, n_layers, n_channels, n_tokens);
    return KVH_OK;
}

kvh_status kvh_plan_chunks(int n_layers, int n_channels, int64_t n_tokens, const int32_t *chunk_levels,
                           int level, uint64_t stream_base, int32_t pt_base, int32_t page_tokens,
                           kvh_chunk_desc *descs_out, uint64_t *total_bytes)
{
    if (n_tokens <= 0 || pt_base < 0) return KVH_ERR_INVALID_ARG;
    if (page_tokens <= 0 || kChunkTokens % page_tokens != 0) return KVH_ERR_BAD_SHAPE;
    if (stream_base % KVH_SECTION_ALIGN) return KVH_ERR_MISALIGNED;
    const int64_t n_chunks = (n_tokens + kChunkTokens - 1) / kChunkTokens;
    const int64_t pages_per_chunk = kChunkTokens / page_tokens;
    if (pt_base + n_chunks * pages_per_chunk > 0x7fffffffLL) return KVH_ERR_BAD_SHAPE;
    uint64_t off = stream_base;
    for (int64_t i = 0; i < n_chunks; ++i) {
        const int k = chunk_levels ? chunk_levels[i] : level;
        const kvh_status s = check_shape(k, n_layers, n_channels);
        if (s != KVH_OK) return s;
        const int64_t left = n_tokens - i * kChunkTokens;
        const int n = (int)(left < kChunkTokens ? left : kChunkTokens);
        if (descs_out) {
            descs_out[i].stream_off = off;
            descs_out[i].level = k;
            descs_out[i].n_tok = n;
            descs_out[i].pt_off = (int32_t)(pt_base + i * pages_per_chunk);
            descs_out[i].reserved = 0;
        }
        off += chunk_bytes(k, n_layers, n_channels, n);
    }
    if (total_bytes) *total_bytes = off - stream_base;
    return KVH_OK;
}

kvh_status kvh_encode(const void *kv, int n_layers, int64_t n_tokens, int n_channels, int level,
                      void *out, uint64_t out_capacity, int32_t *dev_status, void *stream)
{
    if (!kv || !out || n_tokens <= 0) return KVH_ERR_INVALID_ARG;
    const kvh_status s = check_shape(level, n_layers, n_channels);
    if (s != KVH_OK) return s;
    if (!aligned(kv, 16) || !aligned(out, KVH_SECTION_ALIGN)) return KVH_ERR_MISALIGNED;
    uint64_t need = 0;
    const kvh_status ps = kvh_plan_chunks(n_layers, n_channels, n_tokens, nullptr, level, 0, 0, 16, nullptr, &need);
    if (ps != KVH_OK) return ps;
    if (need > out_capacity) return KVH_ERR_BUFFER_TOO_SMALL;
    const int64_t n_chunks = (n_tokens + kChunkTokens - 1) / kChunkTokens;
    EncodeParams p{};
    p.kv = static_cast<const uint16_t *>(kv);
    p.l = n_layers; p.c = n_channels; p.N = n_tokens; p.src_N = n_tokens;
    p.descs = nullptr;
    p.level = level;
    p.full_chunk_bytes = chunk_bytes(level, n_layers, n_channels, kChunkTokens);
    p.out = static_cast<uint8_t *>(out);
    p.capacity = out_capacity;
    p.status = dev_status;
    return launch_encode(p, n_chunks, stream);
}

kvh_status kvh_encode_chunks(const void *kv, int n_layers, int64_t n_tokens, int n_channels,
                             const kvh_chunk_desc *descs, const kvh_chunk_desc *descs_host, int n_chunks,
                             void *out, uint64_t out_capacity, int32_t *dev_status, void *stream)
{
    if (!kv || !out || !descs || n_tokens <= 0) return KVH_ERR_INVALID_ARG;
    const kvh_status s = check_shape(0, n_layers, n_channels);
    if (s != KVH_OK) return s;
    if ((int64_t)n_chunks != (n_tokens + kChunkTokens - 1) / kChunkTokens) return KVH_ERR_BAD_SHAPE;
    if (!aligned(kv, 16) || !aligned(out, KVH_SECTION_ALIGN) || !aligned(descs, 8)) return KVH_ERR_MISALIGNED;
    EncodeParams p{};
    p.kv = static_cast<const uint16_t *>(kv);
    p.l = n_layers; p.c = n_channels; p.N = n_tokens; p.src_N = n_tokens;
    p.descs = descs;
    p.hint_level = -1;
    p.out = static_cast<uint8_t *>(out);
    p.capacity = out_capacity;
    p.status = dev_status;
    return launch_encode(p, n_chunks, stream, descs_host);
}

kvh_status kvh_keep_sinks_and_recent(int64_t n_tokens, int64_t n_sink, int64_t n_recent,
                                     kvh_token_run *runs_out, int *n_runs, int64_t *n_kept)
{
    if (!runs_out || !n_runs || n_tokens <= 0 || n_sink < 0 || n_recent < 0) return KVH_ERR_INVALID_ARG;
    int n = 0;
    if (n_sink >= n_tokens || n_recent >= n_tokens - n_sink) {      // the windows meet: nothing is dropped
        runs_out[n++] = kvh_token_run{0, n_tokens};
    } else {
        if (n_sink > 0) runs_out[n++] = kvh_token_run{0, n_sink};
        if (n_recent > 0) runs_out[n++] = kvh_token_run{n_tokens - n_recent, n_recent};
    }
    *n_runs = n;
    if (n_kept) {
        *n_kept = 0;
        for (int r = 0; r < n; ++r) *n_kept += runs_out[r].count;
    }
    return KVH_OK;
}

kvh_status kvh_encode_kept(const void *kv, int n_layers, int64_t n_tokens, int n_channels,
                           const kvh_token_run *runs, int n_runs, const kvh_chunk_desc *descs, int n_chunks,
                           int level, void *out, uint64_t out_capacity, int32_t *dev_status, void *stream)
{
    if (!kv || !out || !runs || n_tokens <= 0 || n_runs <= 0 || n_runs > kMaxKeptRuns || (!descs && level < 0))
        return KVH_ERR_INVALID_ARG;
    const kvh_status s = check_shape(level < 0 ? 0 : level, n_layers, n_channels);
    if (s != KVH_OK) return s;
    if (block_width(n_channels) == 0) return KVH_ERR_BAD_SHAPE;       // the gather is the TMA-fed kernel's
    if (!aligned(kv, 16) || !aligned(out, KVH_SECTION_ALIGN) || !aligned(descs, 8)) return KVH_ERR_MISALIGNED;
    EncodeParams p{};
    int64_t end = 0, kept = 0;
    for (int r = 0; r < n_runs; ++r) {
        if (runs[r].count <= 0 || runs[r].first < end || runs[r].first > n_tokens - runs[r].count)
            return KVH_ERR_INVALID_ARG;
        p.run_first[r] = runs[r].first;
        p.run_pos[r] = kept;
        end = runs[r].first + runs[r].count;
        kept += runs[r].count;
    }
    p.run_pos[n_runs] = kept;
    p.n_runs = n_runs;
    if ((int64_t)n_chunks != (kept + kChunkTokens - 1) / kChunkTokens) return KVH_ERR_BAD_SHAPE;
    p.kv = static_cast<const uint16_t *>(kv);
    p.l = n_layers; p.c = n_channels; p.N = kept; p.src_N = n_tokens;
    p.descs = descs;
    p.hint_level = level < 0 ? -1 : level;
    if (!descs) {                                        // chunks back to back at the one level
        p.level = level;
        p.full_chunk_bytes = chunk_bytes(level, n_layers, n_channels, kChunkTokens);
        uint64_t need = 0;
        const kvh_status ps = kvh_plan_chunks(n_layers, n_channels, kept, nullptr, level, 0, 0, 16, nullptr, &need);
        if (ps != KVH_OK) return ps;
        if (need > out_capacity) return KVH_ERR_BUFFER_TOO_SMALL;
    }
    p.out = static_cast<uint8_t *>(out);
    p.capacity = out_capacity;
    p.status = dev_status;
    return launch_encode(p, n_chunks, stream);
}

kvh_status kvh_decode_to_pages(const void *chunk, int level, int n_tok, const int32_t *page_ids,
                               const kvh_pool *pool, int32_t *dev_status, void *stream)
{
    if (!chunk || !page_ids) return KVH_ERR_INVALID_ARG;
    const kvh_status ps = check_pool(pool);
    if (ps != KVH_OK) return ps;
    const kvh_status s = check_shape(level, pool->n_layers, pool->n_channels);
    if (s != KVH_OK) return s;
    if (n_tok < 1 || n_tok > kChunkTokens) return KVH_ERR_BAD_SHAPE;
    if (!aligned(chunk, KVH_SECTION_ALIGN) || !aligned(page_ids, 4)) return KVH_ERR_MISALIGNED;
    DecodeParams p{};
    p.streams = static_cast<const uint8_t *>(chunk);
    p.streams_bytes = chunk_bytes(level, pool->n_layers, pool->n_channels, n_tok);
    p.descs = nullptr;
    p.single.stream_off = 0;
    p.single.level = level;
    p.single.n_tok = n_tok;
    p.single.pt_off = 0;
    p.page_table = page_ids;
    p.page_table_len = (n_tok + pool->page_tokens - 1) / pool->page_tokens;
    p.status = dev_status;
    return launch_decode(p, pool, 1, stream);
}

kvh_status kvh_decode_batch(const void *streams_base, uint64_t streams_bytes, const kvh_chunk_desc *descs,
                            int n_chunks, const int32_t *page_table, int64_t page_table_len,
                            const kvh_pool *pool, int32_t *dev_status, void *stream)
{
    if (!streams_base || !descs || !page_table || n_chunks < 0 || page_table_len < 0) return KVH_ERR_INVALID_ARG;
    const kvh_status ps = check_pool(pool);
    if (ps != KVH_OK) return ps;
    if (!aligned(streams_base, KVH_SECTION_ALIGN) || !aligned(descs, 8) || !aligned(page_table, 4))
        return KVH_ERR_MISALIGNED;
    if (n_chunks == 0) return KVH_OK;
    DecodeParams p{};
    p.streams = static_cast<const uint8_t *>(streams_base);
    p.streams_bytes = streams_bytes;
    p.descs = descs;
    p.page_table = page_table;
    p.page_table_len = page_table_len;
    p.status = dev_status;
    return launch_decode(p, pool, n_chunks, stream);
}

// ---- host tier ------------------------------------------------------------------------------

namespace {

// Descriptors must tile [first offset, end) without gaps, in order, so a slice of chunks is one
// contiguous byte range on both sides of the PCIe copy.
kvh_status check_contiguous(const kvh_chunk_desc *d, int n, int l, int c, uint64_t capacity)
{
    uint64_t expect = d[0].stream_off;
    for (int i = 0; i < n; ++i) {
        if (d[i].level < 0 || d[i].level >= kNumLevels) return KVH_ERR_BAD_LEVEL;
        if (d[i].n_tok < 1 || d[i].n_tok > kChunkTokens) return KVH_ERR_BAD_SHAPE;
        if (d[i].stream_off % KVH_SECTION_ALIGN) return KVH_ERR_MISALIGNED;
        if (d[i].stream_off != expect) return KVH_ERR_INVALID_ARG;
        expect += chunk_bytes(d[i].level, l, c, d[i].n_tok);
    }
    return expect <= capacity ? KVH_OK : KVH_ERR_BUFFER_TOO_SMALL;
}

struct Slice { int first, count; uint64_t off, bytes; };

// Next slice of chunks starting at `first`: at least one chunk, about slice_bytes long.
Slice next_slice(const kvh_chunk_desc *d, int n, int first, int l, int c, uint64_t slice_bytes)
{
    Slice s{first, 0, d[first].stream_off, 0};
    while (first + s.count < n && (s.count == 0 || s.bytes < slice_bytes)) {
        s.bytes += chunk_bytes(d[first + s.count].level, l, c, d[first + s.count].n_tok);
        ++s.count;
    }
    return s;
}

// Make `waiter` wait for everything enqueued on `signaller` so far.
bool chain(cudaStream_t signaller, cudaStream_t waiter)
{
    cudaEvent_t ev;
    if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return false;
    const bool ok = cudaEventRecord(ev, signaller) == cudaSuccess &&
                    cudaStreamWaitEvent(waiter, ev, 0) == cudaSuccess;
    cudaEventDestroy(ev);            // released once the recorded work completes
    return ok;
}

}  // namespace

kvh_status kvh_load_host(const void *host_streams, void *dev_staging, uint64_t staging_bytes,
                         const kvh_chunk_desc *descs_host, const kvh_chunk_desc *descs_dev, int n_chunks,
                         const int32_t *page_table, int64_t page_table_len, const kvh_pool *pool,
                         int32_t *dev_status, int32_t *host_status, uint64_t slice_bytes,
                         void *copy_stream, void *stream)
{
    if (!host_streams || !dev_staging || !descs_host || !descs_dev || !page_table || n_chunks <= 0 ||
        page_table_len < 0 || !copy_stream || copy_stream == stream || (host_status && !dev_status))
        return KVH_ERR_INVALID_ARG;
    const kvh_status ps = check_pool(pool);
    if (ps != KVH_OK) return ps;
    if (!aligned(dev_staging, KVH_SECTION_ALIGN) || !aligned(descs_dev, 8) || !aligned(page_table, 4))
        return KVH_ERR_MISALIGNED;
    const kvh_status cs = check_contiguous(descs_host, n_chunks, pool->n_layers, pool->n_channels, staging_bytes);
    if (cs != KVH_OK) return cs;
    if (slice_bytes == 0) slice_bytes = 64ull << 20;
    cudaStream_t cp = static_cast<cudaStream_t>(copy_stream), st = static_cast<cudaStream_t>(stream);
    if (!chain(st, cp)) return KVH_ERR_CUDA;          // the staging buffer may still be read by earlier work
    for (int i = 0; i < n_chunks;) {
        const Slice s = next_slice(descs_host, n_chunks, i, pool->n_layers, pool->n_channels, slice_bytes);
        if (cudaMemcpyAsync(static_cast<uint8_t *>(dev_staging) + s.off,
                            static_cast<const uint8_t *>(host_streams) + s.off, s.bytes,
                            cudaMemcpyHostToDevice, cp) != cudaSuccess || !chain(cp, st))
            return KVH_ERR_CUDA;
        DecodeParams p{};
        p.streams = static_cast<const uint8_t *>(dev_staging);
        p.streams_bytes = staging_bytes;
        p.descs = descs_dev + s.first;
        p.page_table = page_table;
        p.page_table_len = page_table_len;
        p.status = dev_status;
        const kvh_status ls = launch_decode(p, pool, s.count, stream);
        if (ls != KVH_OK) return ls;
        i += s.count;
    }
    if (host_status &&
        cudaMemcpyAsync(host_status, dev_status, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return KVH_ERR_CUDA;
    return KVH_OK;
}

kvh_status kvh_store_host(const void *kv, int n_layers, int64_t n_tokens, int n_channels,
                          const kvh_chunk_desc *descs_host, const kvh_chunk_desc *descs_dev, int n_chunks,
                          void *dev_staging, uint64_t staging_bytes, void *host_out, int32_t *dev_status,
                          int32_t *host_status, uint64_t slice_bytes, void *copy_stream, void *stream)
{
    if (!kv || !dev_staging || !host_out || !descs_host || !descs_dev || n_tokens <= 0 || !copy_stream ||
        copy_stream == stream || (host_status && !dev_status))
        return KVH_ERR_INVALID_ARG;
    const kvh_status s0 = check_shape(0, n_layers, n_channels);
    if (s0 != KVH_OK) return s0;
    if ((int64_t)n_chunks != (n_tokens + kChunkTokens - 1) / kChunkTokens) return KVH_ERR_BAD_SHAPE;
    if (!aligned(kv, 16) || !aligned(dev_staging, KVH_SECTION_ALIGN) || !aligned(descs_dev, 8))
        return KVH_ERR_MISALIGNED;
    const kvh_status cs = check_contiguous(descs_host, n_chunks, n_layers, n_channels, staging_bytes);
    if (cs != KVH_OK) return cs;
    if (slice_bytes == 0) slice_bytes = 64ull << 20;
    cudaStream_t cp = static_cast<cudaStream_t>(copy_stream), st = static_cast<cudaStream_t>(stream);
    if (!chain(cp, st)) return KVH_ERR_CUDA;          // earlier copies out of the staging buffer finish first
    for (int i = 0; i < n_chunks;) {
        const Slice s = next_slice(descs_host, n_chunks, i, n_layers, n_channels, slice_bytes);
        EncodeParams p{};
        p.kv = static_cast<const uint16_t *>(kv);
        p.l = n_layers; p.c = n_channels; p.N = n_tokens; p.src_N = n_tokens;
        p.descs = descs_dev;
        p.hint_level = -1;
        p.chunk0 = s.first;
        p.out = static_cast<uint8_t *>(dev_staging);
        p.capacity = staging_bytes;
        p.status = dev_status;
        const kvh_status ls = launch_encode(p, s.count, st, descs_host);
        if (ls != KVH_OK) return ls;
        if (!chain(st, cp) ||
            cudaMemcpyAsync(static_cast<uint8_t *>(host_out) + s.off,
                            static_cast<const uint8_t *>(dev_staging) + s.off, s.bytes,
                            cudaMemcpyDeviceToHost, cp) != cudaSuccess)
            return KVH_ERR_CUDA;
        i += s.count;
    }
    if (host_status) {
        if (cudaMemcpyAsync(host_status, dev_status, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return KVH_ERR_CUDA;
    }
    return chain(cp, st) ? KVH_OK : KVH_ERR_CUDA;     // `stream` completes after the last copy out
}

}  // extern "C"

// ---- host-tier load for callers that cannot allocate device memory --------------------------

namespace {

// Staging area of kvh_load_host_static.  It lives in the library's device image, so every GPU
// that loads the library sets this much memory aside until the process exits.
static __device__ __align__(256) uint8_t g_static_staging[KVH_STATIC_STAGING_BYTES];

constexpr int kMaxDevices = 64;
void *g_static_staging_ptr[kMaxDevices];      // device address of the array, per device; nullptr = not set up

// g_static_staging names a host-side handle here, not device memory: the address a kernel or a
// copy may use comes from cudaGetSymbolAddress, asked once per device with that device current.
kvh_status static_staging_address(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return KVH_ERR_CUDA;
    void *p = __atomic_load_n(&g_static_staging_ptr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_static_staging) != cudaSuccess || !p) return KVH_ERR_CUDA;
        __atomic_store_n(&g_static_staging_ptr[dev], p, __ATOMIC_RELEASE);    // every thread gets the same answer
    }
    *out = p;
    return KVH_OK;
}

}  // namespace

extern "C" kvh_status kvh_load_host_static(const void *host_streams, const kvh_chunk_desc *descs_host,
                                           const kvh_chunk_desc *descs_dev, int n_chunks,
                                           const int32_t *page_table, int64_t page_table_len,
                                           const kvh_pool *pool, int32_t *dev_status, int32_t *host_status,
                                           uint64_t slice_bytes, void *copy_stream, void *stream)
{
    if (!descs_host || n_chunks <= 0) return KVH_ERR_INVALID_ARG;
    const kvh_status ps = check_pool(pool);
    if (ps != KVH_OK) return ps;
    // the stored form must fit the fixed staging area: say so before anything is enqueued
    const kvh_status cs = check_contiguous(descs_host, n_chunks, pool->n_layers, pool->n_channels,
                                           KVH_STATIC_STAGING_BYTES);
    if (cs != KVH_OK) return cs;                // KVH_ERR_BUFFER_TOO_SMALL: beyond KVH_STATIC_STAGING_BYTES
    void *staging = nullptr;
    const kvh_status as = static_staging_address(&staging);
    if (as != KVH_OK) return as;
    return kvh_load_host(host_streams, staging, KVH_STATIC_STAGING_BYTES, descs_host, descs_dev, n_chunks,
                         page_table, page_table_len, pool, dev_status, host_status, slice_bytes, copy_stream,
                         stream);
}
