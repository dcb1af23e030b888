// Encode kernels: bf16 KV tensor [l][2][N][c] -> stored chunks.
//
// This is what the paper's executor runs when the policy decides to keep an
// entry "in full quality" (level 0) or to compress it (levels 1..3).  One HBM
// pass: a CTA owns one (chunk, layer, K|V, 32-token tile); every thread keeps a
// 4-channel x 32-token column of the tile in registers, so group ranges, codes
// and packing all come from the single read of the tile.
//   K groups run down the column (one channel, 32 tokens): a thread reduces them
//     alone, on order-preserving integer keys.
//   V groups run across 8 neighbouring threads (32 channels, one token): the
//     packed (min key, inverted max key) pair is reduced with three xor-shuffles.
#pragma once

#include "kvh_format.cuh"
#include "kvh_decode.cuh"   // report(), check_desc()

namespace kvh {

struct EncodeParams {
    const uint16_t *kv;            // [l][2][N][c]
    int32_t l, c;
    int64_t N;
    const kvh_chunk_desc *descs;   // device array indexed by chunk, or nullptr for one level throughout
    int32_t chunk0;                // first chunk this launch covers
    int32_t level;                 // used when descs == nullptr
    uint64_t full_chunk_bytes;     // kvh_level_bytes(level, l, c, 256), same case
    uint8_t *out;
    uint64_t capacity;
    int32_t *status;
};

// Zero the alignment padding behind a section's payload (fewer than 128 bytes).
__device__ __forceinline__ void zero_pad(uint8_t *section, uint64_t payload, uint64_t padded)
{
    const uint64_t i = payload + threadIdx.x;
    if (i < padded) section[i] = 0;
}

__device__ __forceinline__ void encode_tile_raw(const uint16_t *src, uint8_t *codes, int c, int t0, int nt)
{
    // the tile's rows are contiguous on both sides: a flat copy of nt*c bf16
    const uint4 *s = reinterpret_cast<const uint4 *>(src);
    uint4 *d = reinterpret_cast<uint4 *>(codes + 2 * (uint64_t)t0 * c);
    const int nvec = nt * (c >> 3);
    int v = threadIdx.x;
    for (; v + 3 * kThreads < nvec; v += 4 * kThreads) {
        const uint4 a = __ldcs(s + v), b = __ldcs(s + v + kThreads);
        const uint4 e = __ldcs(s + v + 2 * kThreads), f = __ldcs(s + v + 3 * kThreads);
        d[v] = a; d[v + kThreads] = b; d[v + 2 * kThreads] = e; d[v + 3 * kThreads] = f;
    }
    for (; v < nvec; v += kThreads) d[v] = __ldcs(s + v);
}

// Store the 4 codes of one thread for one token: 4*BITS bits at element index e (multiple of 4).
template <int BITS>
__device__ __forceinline__ void store_codes4(uint8_t *codes, uint64_t e, uint32_t packed)
{
    if constexpr (BITS == 8) *reinterpret_cast<uint32_t *>(codes + e) = packed;
    if constexpr (BITS == 4) *reinterpret_cast<uint16_t *>(codes + (e >> 1)) = (uint16_t)packed;
    if constexpr (BITS == 2) codes[e >> 2] = (uint8_t)packed;
}

template <int BITS>
__device__ __forceinline__ uint32_t quantise4(uint2 x, const float (&lo)[4], const float (&inv)[4])
{
    return quantise<BITS>(bf16_lo_to_f32(x.x), lo[0], inv[0]) |
           quantise<BITS>(bf16_hi_to_f32(x.x), lo[1], inv[1]) << BITS |
           quantise<BITS>(bf16_lo_to_f32(x.y), lo[2], inv[2]) << (2 * BITS) |
           quantise<BITS>(bf16_hi_to_f32(x.y), lo[3], inv[3]) << (3 * BITS);
}

template <int BITS>
__device__ __forceinline__ void encode_tile_quant(const uint16_t *src, uint8_t *meta, uint8_t *codes,
                                                  int c, int kv, int tile, int nt)
{
    const int C4 = c >> 2;                       // 4-channel columns per row; a multiple of 8
    const int lane = threadIdx.x & 31;
    const int t0 = tile * kTileTokens;
    // warp-uniform trip count: the V path shuffles, so whole warps stay in the loop
    for (int base = threadIdx.x - lane; base < C4; base += kThreads) {
        const bool active = base + lane < C4;
        const int cq = active ? base + lane : C4 - 1;
        uint2 x[kTileTokens];
#pragma unroll
        for (int t = 0; t < kTileTokens; ++t) {
            const int row = t < nt ? t : nt - 1;         // short tile: repeat the last valid row
            x[t] = __ldcs(reinterpret_cast<const uint2 *>(src + (uint64_t)row * c) + cq);
        }
        if (kv == 0) {
            // ---- K: one group per channel, down the column ----
            uint32_t mn01 = 0xffffffffu, mn23 = 0xffffffffu, mx01 = 0, mx23 = 0;
#pragma unroll
            for (int t = 0; t < kTileTokens; ++t) {
                const uint32_t k01 = order_keys2(x[t].x), k23 = order_keys2(x[t].y);
                mn01 = __vminu2(mn01, k01); mx01 = __vmaxu2(mx01, k01);
                mn23 = __vminu2(mn23, k23); mx23 = __vmaxu2(mx23, k23);
            }
            uint32_t m[4];
            m[0] = key_to_bf16(mn01 & 0xffffu) | key_to_bf16(mx01 & 0xffffu) << 16;
            m[1] = key_to_bf16(mn01 >> 16) | key_to_bf16(mx01 >> 16) << 16;
            m[2] = key_to_bf16(mn23 & 0xffffu) | key_to_bf16(mx23 & 0xffffu) << 16;
            m[3] = key_to_bf16(mn23 >> 16) | key_to_bf16(mx23 >> 16) << 16;
            float lo[4], inv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) encode_params<BITS>(m[i], lo[i], inv[i]);
            if (active) {
                *reinterpret_cast<uint4 *>(meta + 4 * ((uint64_t)tile * c + 4 * cq)) =
                    make_uint4(m[0], m[1], m[2], m[3]);
#pragma unroll
                for (int t = 0; t < kTileTokens; ++t)
                    if (t < nt)
                        store_codes4<BITS>(codes, (uint64_t)(t0 + t) * c + 4 * cq,
                                           quantise4<BITS>(x[t], lo, inv));
            }
        } else {
            // ---- V: one group per token and 32 channels = 8 neighbouring lanes ----
#pragma unroll
            for (int t = 0; t < kTileTokens; ++t) {
                const uint32_t k01 = order_keys2(x[t].x), k23 = order_keys2(x[t].y);
                const uint32_t mn2 = __vminu2(k01, k23), mx2 = __vmaxu2(k01, k23);
                // pack (min key, ~max key) so one unsigned halfword-min reduces both
                uint32_t pk = min(mn2 & 0xffffu, mn2 >> 16) |
                              (0xffffu - max(mx2 & 0xffffu, mx2 >> 16)) << 16;
                pk = __vminu2(pk, __shfl_xor_sync(0xffffffffu, pk, 1));
                pk = __vminu2(pk, __shfl_xor_sync(0xffffffffu, pk, 2));
                pk = __vminu2(pk, __shfl_xor_sync(0xffffffffu, pk, 4));
                const uint32_t m = key_to_bf16(pk & 0xffffu) | key_to_bf16(0xffffu - (pk >> 16)) << 16;
                if (active && t < nt) {
                    float l1, i1;
                    encode_params<BITS>(m, l1, i1);
                    const float lo[4] = {l1, l1, l1, l1}, inv[4] = {i1, i1, i1, i1};
                    if ((cq & 7) == 0)
                        reinterpret_cast<uint32_t *>(meta)[(uint64_t)(t0 + t) * (c / kGroup) + (cq >> 3)] = m;
                    store_codes4<BITS>(codes, (uint64_t)(t0 + t) * c + 4 * cq, quantise4<BITS>(x[t], lo, inv));
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 2) encode_kernel(const EncodeParams p)
{
    uint32_t b = blockIdx.x;
    const int tile = b % kTilesPerChunk;  b /= kTilesPerChunk;
    const int kv = b & 1;                 b >>= 1;
    const int layer = b % p.l;
    const int chunk = p.chunk0 + b / p.l;

    const int64_t tok0 = (int64_t)chunk * kChunkTokens;
    const int n_expect = (int)min((int64_t)kChunkTokens, p.N - tok0);
    kvh_chunk_desc d;
    if (p.descs) {
        d = p.descs[chunk];
    } else {
        d.stream_off = (uint64_t)chunk * p.full_chunk_bytes;
        d.level = p.level;
        d.n_tok = n_expect;
    }
    int err = check_desc(d, p.l, p.c, p.capacity);
    if (err == KVH_OK && d.n_tok != n_expect) err = KVH_ERR_BAD_SHAPE;
    if (err != KVH_OK) {
        if (threadIdx.x == 0) report(p.status, err);
        return;
    }
    const int n = d.n_tok;
    const int nt = min(kTileTokens, n - tile * kTileTokens);
    if (nt <= 0) return;

    const LayerLayout L = layer_layout(d.level, p.c, n);
    uint8_t *lay = p.out + d.stream_off + (uint64_t)layer * L.layer_bytes();
    uint8_t *meta = lay + L.meta_off(kv);
    uint8_t *codes = lay + L.codes_off(kv);
    const uint16_t *src = p.kv + (((int64_t)layer * 2 + kv) * p.N + tok0 + tile * kTileTokens) * p.c;

    if (tile * kTileTokens + nt == n) {                   // the plane's last tile clears the padding
        zero_pad(codes, L.codes_payload, L.kcodes);
        if (d.level > 0)
            zero_pad(meta, kv ? L.vmeta_payload : L.kmeta_payload, kv ? L.vmeta : L.kmeta);
    }
    switch (d.level) {                                    // uniform per CTA
    case 0: encode_tile_raw(src, codes, p.c, tile * kTileTokens, nt); break;
    case 1: encode_tile_quant<8>(src, meta, codes, p.c, kv, tile, nt); break;
    case 2: encode_tile_quant<4>(src, meta, codes, p.c, kv, tile, nt); break;
    default: encode_tile_quant<2>(src, meta, codes, p.c, kv, tile, nt); break;
    }
}

}  // namespace kvh
