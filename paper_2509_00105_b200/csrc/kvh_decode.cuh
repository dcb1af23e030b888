// Decode kernels: stored chunk -> bf16 pages of the serving engine's pool.
//
// This is the step that runs on every cache hit before the engine can attend
// over a reused context (the "decompression overhead" of the paper's Estimator
// paragraph).  It is bound by HBM traffic: (b+1)/8 bytes read and 2 bytes
// written per element, so the kernel is organised around full-width coalesced
// 16-byte stores of page rows.
//
// Work decomposition: one CTA per (chunk, layer, K|V, 32-token tile).  A tile is
// one K group of tokens, so a thread that owns 8 channels keeps its 8 (min,
// scale) pairs in registers for the whole tile; for V the 4 threads that share a
// 32-channel group each derive the pair from the same metadata word.
#pragma once

#include "kvh_format.cuh"

namespace kvh {

struct DecodeParams {
    const uint8_t *streams;
    uint64_t streams_bytes;
    const kvh_chunk_desc *descs;      // device array, or nullptr to use `single`
    kvh_chunk_desc single;
    const int32_t *page_table;
    int64_t page_table_len;
    uint16_t *pool;
    int64_t layer_stride, kv_stride, page_stride;
    int32_t num_pages, page_tokens, page_shift, l, c;   // page_tokens == 1 << page_shift
    int32_t bw, n_blocks;             // TMA-fed kernel: channels per column block (c when c <= 1024), blocks per row
    int32_t tpu;                      // TMA-fed kernel: 32-token tiles per work unit (1, 2, 4, 8; 1 unless rows are narrow)
    int32_t *status;
};

__device__ __forceinline__ void report(int32_t *status, int code)
{
    if (status) atomicMax(status, code);
}

// A descriptor is usable when following it keeps every access inside the
// buffers the caller described.  Uniform per CTA.
__device__ __forceinline__ int check_desc(const kvh_chunk_desc &d, int l, int c, uint64_t capacity)
{
    if (d.level < 0 || d.level >= kNumLevels) return KVH_ERR_BAD_LEVEL;
    if (d.n_tok < 1 || d.n_tok > kChunkTokens) return KVH_ERR_BAD_SHAPE;
    if (d.stream_off & (KVH_SECTION_ALIGN - 1)) return KVH_ERR_MISALIGNED;
    const uint64_t need = chunk_bytes(d.level, l, c, d.n_tok);
    if (d.stream_off > capacity || need > capacity - d.stream_off) return KVH_ERR_BUFFER_TOO_SMALL;
    return KVH_OK;
}

template <int BITS>
__device__ __forceinline__ uint4 dequant8(uint64_t codes, const float (&lo)[8], const float (&sc)[8])
{
    constexpr uint32_t mask = (1u << BITS) - 1;
    float f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t q = (uint32_t)(codes >> (BITS * i)) & mask;
        f[i] = __fmaf_rn(small_uint_to_f32(q), sc[i], lo[i]);
    }
    return make_uint4(pack_bf16x2_rn(f[0], f[1]), pack_bf16x2_rn(f[2], f[3]),
                      pack_bf16x2_rn(f[4], f[5]), pack_bf16x2_rn(f[6], f[7]));
}

// 8 consecutive codes of BITS bits, starting at element index e (a multiple of 8)
template <int BITS>
__device__ __forceinline__ uint64_t load_codes8(const uint8_t *codes, uint64_t e)
{
    if constexpr (BITS == 8) return __ldcs(reinterpret_cast<const unsigned long long *>(codes + e));
    if constexpr (BITS == 4) return __ldcs(reinterpret_cast<const unsigned int *>(codes + (e >> 1)));
    if constexpr (BITS == 2) return __ldcs(reinterpret_cast<const unsigned short *>(codes + (e >> 2)));
    return 0;
}

// Destination row of chunk token T for this plane, or nullptr if its page id is out of range.
template <int C = 0>
__device__ __forceinline__ uint16_t *page_row(const DecodeParams &p, int32_t pg, uint16_t *plane, int T)
{
    if ((uint32_t)pg >= (uint32_t)p.num_pages) {
        report(p.status, KVH_ERR_PAGE_OOB);
        return nullptr;
    }
    return plane + (int64_t)pg * p.page_stride + (int64_t)(T & (p.page_tokens - 1)) * (C ? C : p.c);
}

template <int BITS>
__device__ __forceinline__ void decode_tile(const DecodeParams &p, const uint8_t *meta,
                                            const uint8_t *codes, const int32_t *page_ids,
                                            uint16_t *plane, int kv, int tile, int nt)
{
    const int c = p.c;
    const int V8 = c >> 3;                               // 8-channel vectors per token row
    const int cstep = V8 <= kThreads ? V8 : kThreads;     // a multiple of 4: V8 is, and so is kThreads
    const int rpp = V8 <= kThreads ? kThreads / V8 : 1;   // token rows the CTA covers per pass
    const int my_row = threadIdx.x / cstep;
    const int my_cv = threadIdx.x - my_row * cstep;
    if (my_row >= rpp) return;                           // whole quads of lanes leave together
    const int t0 = tile * kTileTokens;
    constexpr int U = 8;                                 // rows in flight per thread
    const int lane = threadIdx.x & 31;
    const uint32_t quad = 0xfu << (lane & ~3);           // the 4 lanes that share a V group

    for (int cv = my_cv; cv < V8; cv += cstep) {
        float lo[8], sc[8];
        if constexpr (BITS < 16) {
            if (kv == 0) {                               // K: metadata row `tile`, my 8 channels
                const uint4 *m = reinterpret_cast<const uint4 *>(meta + 4 * ((uint64_t)tile * c + 8 * cv));
                const uint4 m0 = __ldg(m), m1 = __ldg(m + 1);
                const uint32_t w[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
#pragma unroll
                for (int i = 0; i < 8; ++i) decode_params<BITS>(w[i], lo[i], sc[i]);
            }
        }
        for (int tb = my_row; tb < nt; tb += U * rpp) {
            uint4 raw[U];
            uint64_t cd[U];
            uint32_t vm[U];
            int32_t pg[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int t = tb + u * rpp;
                if (t < nt) {
                    const uint64_t e = (uint64_t)(t0 + t) * c + 8 * cv;
                    pg[u] = __ldg(page_ids + ((t0 + t) >> p.page_shift));
                    if constexpr (BITS == 16) {
                        raw[u] = __ldcs(reinterpret_cast<const uint4 *>(codes + 2 * e));
                    } else {
                        cd[u] = load_codes8<BITS>(codes, e);
                        if (kv == 1)
                            vm[u] = __ldg(reinterpret_cast<const uint32_t *>(meta) +
                                          (uint64_t)(t0 + t) * (c / kGroup) + (cv >> 2));
                    }
                }
            }
            // V: the 4 lanes of a quad share each row's group; each derives the scale of every
            // fourth row and hands it round, so a row costs a quarter of a division per lane
            float vsc[U / 4];
            if constexpr (BITS < 16) {
                if (kv == 1) {
#pragma unroll
                    for (int j = 0; j < U / 4; ++j) {
                        const int u = 4 * j + (lane & 3);
                        float l1;
                        vsc[j] = 0.0f;
                        if (tb + u * rpp < nt) {
                            uint32_t m = vm[4 * j];
                            if ((lane & 3) == 1) m = vm[4 * j + 1];
                            if ((lane & 3) == 2) m = vm[4 * j + 2];
                            if ((lane & 3) == 3) m = vm[4 * j + 3];
                            decode_params<BITS>(m, l1, vsc[j]);
                        }
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int t = tb + u * rpp;
                if (t < nt) {                                // uniform within a quad
                    uint4 v;
                    if constexpr (BITS == 16) {
                        v = raw[u];
                    } else {
                        if (kv == 1) {
                            const float s1 = __shfl_sync(quad, vsc[u >> 2], (lane & ~3) | (u & 3));
                            const float l1 = bf16_lo_to_f32(vm[u]);
#pragma unroll
                            for (int i = 0; i < 8; ++i) { lo[i] = l1; sc[i] = s1; }
                        }
                        v = dequant8<BITS>(cd[u], lo, sc);
                    }
                    uint16_t *row = page_row(p, pg[u], plane, t0 + t);
                    if (row) *reinterpret_cast<uint4 *>(row + 8 * cv) = v;
                }
            }
        }
    }
}

static __global__ void __launch_bounds__(kThreads) decode_kernel(const DecodeParams p)
{
    uint32_t b = blockIdx.x;
    const int tile = b % kTilesPerChunk;  b /= kTilesPerChunk;
    const int kv = b & 1;                 b >>= 1;
    const int layer = b % p.l;
    const int chunk = b / p.l;

    const kvh_chunk_desc d = p.descs ? p.descs[chunk] : p.single;
    int err = check_desc(d, p.l, p.c, p.streams_bytes);
    const int npages = (d.n_tok + p.page_tokens - 1) >> p.page_shift;
    if (err == KVH_OK && (d.pt_off < 0 || (int64_t)d.pt_off + npages > p.page_table_len))
        err = KVH_ERR_BUFFER_TOO_SMALL;
    if (err != KVH_OK) {
        if (threadIdx.x == 0) report(p.status, err);
        return;
    }
    const int nt = min(kTileTokens, d.n_tok - tile * kTileTokens);
    if (nt <= 0) return;

    const LayerLayout L = layer_layout(d.level, p.c, d.n_tok);
    const uint8_t *lay = p.streams + d.stream_off + (uint64_t)layer * L.layer_bytes();
    const uint8_t *meta = lay + L.meta_off(kv);
    const uint8_t *codes = lay + L.codes_off(kv);
    const int32_t *page_ids = p.page_table + d.pt_off;
    uint16_t *plane = p.pool + (int64_t)layer * p.layer_stride + (int64_t)kv * p.kv_stride;

    switch (d.level) {                                    // uniform per CTA
    case 0: decode_tile<16>(p, meta, codes, page_ids, plane, kv, tile, nt); break;
    case 1: decode_tile<8>(p, meta, codes, page_ids, plane, kv, tile, nt); break;
    case 2: decode_tile<4>(p, meta, codes, page_ids, plane, kv, tile, nt); break;
    default: decode_tile<2>(p, meta, codes, page_ids, plane, kv, tile, nt); break;
    }
}

}  // namespace kvh
