// Encode kernels: bf16 KV tensor [l][2][N][c] -> stored chunks.
//
// This is what the paper's executor runs when the policy decides to keep an
// entry "in full quality" (level 0) or to compress it (levels 1..3).  One HBM
// pass: a CTA owns one (chunk, layer, K|V, 32-token tile) and the group ranges,
// the codes and their packing all come from a single read of the tile.
//   K groups run down a column (one channel, 32 tokens): two threads hold the
//     upper and lower 16 tokens of a 4-channel column in registers and swap their
//     partial ranges through shared memory.
//   V groups run along a row (32 channels, one token): a thread holds 8
//     channels of a row, and the 4 lanes that share a group combine their ranges
//     with two xor-shuffles; each lane derives the reciprocal scale of every
//     fourth row and hands it round.
// Ranges use the packed bf16 min/max instructions, which order -0 below +0 as
// the format's definition does.
#pragma once

#include "kvh_format.cuh"
#include "kvh_decode.cuh"   // report(), check_desc()

namespace kvh {

constexpr int kMaxKeptRuns = KVH_MAX_KEPT_RUNS;

struct EncodeParams {
    const uint16_t *kv;            // [l][2][src_N][c]
    int32_t l, c;
    int64_t N;                     // tokens that get encoded (the kept ones when runs are given)
    int64_t src_N;                 // tokens per plane of kv
    // Token dropping: n_runs > 0 keeps run r = source tokens [run_first[r], run_first[r] + run_pos[r+1]
    // - run_pos[r]) and stores them compacted, so that kept token j of run r is token run_pos[r] + j
    // of the encoded sequence.  n_runs == 0: the encoded sequence is the source itself.
    int32_t n_runs;
    int64_t run_first[kMaxKeptRuns];
    int64_t run_pos[kMaxKeptRuns + 1];
    const kvh_chunk_desc *descs;   // device array indexed by chunk, or nullptr for one level throughout
    int32_t chunk0;                // first chunk this launch covers
    int32_t level;                 // used when descs == nullptr
    int32_t bw, n_blocks;          // TMA-fed kernel: channels per column block (c when c <= 1024) and blocks per row
    int32_t tpu;                   // TMA-fed kernel: 32-token tiles per work unit (1, 2, 4, 8; 1 unless rows are narrow)
    int32_t boxes;                 // TMA-fed kernel: 1 = column blocks of 256 channels fetched as 2-D boxes, a box per tile
    int32_t hint_level;            // >= 0: every chunk has this level (an instance holding only its code runs); -1: any
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

// ---- packed bf16 helpers -------------------------------------------------------------------

__device__ __forceinline__ uint32_t bmin2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("min.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t swap_halves(uint32_t a) { return __byte_perm(a, 0, 0x1032); }

// One element: 2^23 + code, as raw float bits.  Adding 2^23 rounds (x - lo) * inv to an integer,
// ties to even, and leaves it in the low mantissa bits; the product never reaches qmax + 1/2 (it
// is at most qmax * (1 + 2^-22)), so no clamp is needed.
__device__ __forceinline__ uint32_t biased_code(float x, float lo, float inv)
{
    return __float_as_uint(__fadd_rn(__fmul_rn(__fsub_rn(x, lo), inv), 8388608.0f));
}

// Pack 4 biased codes (0x4b000000 + q) of BITS bits: the biases add up to a constant that is
// subtracted once, so no code is masked on its own.  Arithmetic is modulo 2^32.
template <int BITS>
__device__ __forceinline__ uint32_t pack4_biased(uint32_t t0, uint32_t t1, uint32_t t2, uint32_t t3)
{
    constexpr uint32_t bias = 0x4b000000u * (1u + (1u << BITS) + (1u << (2 * BITS)) + (1u << (3 * BITS)));
    return (t0 + (t1 << BITS)) + ((t2 + (t3 << BITS)) << (2 * BITS)) - bias;
}

// bf16 halves of a packed pair as floats; with MASKED the value of a channel whose group is
// stored flat is replaced by 0, which makes (0 - lo) * 0 a zero and the code 0 (x - lo may
// overflow to infinity for such a group, and infinity * 0 would be NaN).
template <bool MASKED>
__device__ __forceinline__ float lo_half(uint32_t pair, uint32_t mask)
{
    const uint32_t v = pair << 16;
    return __uint_as_float(MASKED ? (v & mask) : v);
}
template <bool MASKED>
__device__ __forceinline__ float hi_half(uint32_t pair, uint32_t mask)
{
    return __uint_as_float(MASKED ? (pair & 0xffff0000u & mask) : (pair & 0xffff0000u));
}

// ---- K: one group per channel ----------------------------------------------------------------

constexpr int kHalfRows = kTileTokens / 2;       // rows a thread keeps in registers
constexpr int kColThreads = kThreads / 2;        // 4-channel columns a CTA covers per pass

template <int BITS, bool MASKED>
__device__ __forceinline__ void quantise_column(const uint2 (&x)[kHalfRows], const float (&lo)[4],
                                                const float (&inv)[4], const uint32_t (&mask)[4],
                                                uint8_t *out, uint32_t row_bytes, int rows)
{
#pragma unroll
    for (int t = 0; t < kHalfRows; ++t) {
        if (t < rows) {
            const uint32_t packed = pack4_biased<BITS>(
                biased_code(lo_half<MASKED>(x[t].x, mask[0]), lo[0], inv[0]),
                biased_code(hi_half<MASKED>(x[t].x, mask[1]), lo[1], inv[1]),
                biased_code(lo_half<MASKED>(x[t].y, mask[2]), lo[2], inv[2]),
                biased_code(hi_half<MASKED>(x[t].y, mask[3]), lo[3], inv[3]));
            if constexpr (BITS == 8) *reinterpret_cast<uint32_t *>(out) = packed;
            if constexpr (BITS == 4) *reinterpret_cast<uint16_t *>(out) = (uint16_t)packed;
            if constexpr (BITS == 2) *out = (uint8_t)packed;
            out += row_bytes;
        }
    }
}

// The CTA's two halves of 128 threads take rows 0..15 and 16..31 of a 4-channel column each, so
// a thread keeps 16 rows in registers; the halves swap their partial ranges through shared memory.
template <int BITS>
__device__ __forceinline__ void encode_tile_k(const uint16_t *src, uint8_t *meta, uint8_t *codes,
                                              int c, int tile, int nt, uint4 (*xchg)[kThreads])
{
    const int C4 = c >> 2;                       // 4-channel columns per row
    const int half = threadIdx.x / kColThreads;
    const int col = threadIdx.x - half * kColThreads;
    const int r0 = half * kHalfRows;
    const int rows = max(0, min(kHalfRows, nt - r0));    // rows of mine that exist
    const uint32_t row_bytes = (uint32_t)c * BITS / 8;
    int pass = 0;
    for (int cb = 0; cb < C4; cb += kColThreads, ++pass) {       // same trip count for every thread
        const bool active = cb + col < C4;
        const int cq = active ? cb + col : C4 - 1;
        uint2 x[kHalfRows];
#pragma unroll
        for (int t = 0; t < kHalfRows; ++t) {
            const int row = min(r0 + t, nt - 1);         // rows past the tile repeat its last row
            x[t] = __ldcs(reinterpret_cast<const uint2 *>(src + (uint64_t)row * c) + cq);
        }
        uint32_t mn01 = x[0].x, mn23 = x[0].y, mx01 = x[0].x, mx23 = x[0].y;
#pragma unroll
        for (int t = 1; t < kHalfRows; ++t) {
            mn01 = bmin2(mn01, x[t].x); mx01 = bmax2(mx01, x[t].x);
            mn23 = bmin2(mn23, x[t].y); mx23 = bmax2(mx23, x[t].y);
        }
        xchg[pass & 1][threadIdx.x] = make_uint4(mn01, mn23, mx01, mx23);
        __syncthreads();
        const uint4 o = xchg[pass & 1][threadIdx.x ^ kColThreads];
        mn01 = bmin2(mn01, o.x); mn23 = bmin2(mn23, o.y);
        mx01 = bmax2(mx01, o.z); mx23 = bmax2(mx23, o.w);
        // metadata words: (min | max << 16) per channel
        const uint32_t m[4] = {__byte_perm(mn01, mx01, 0x5410), __byte_perm(mn01, mx01, 0x7632),
                               __byte_perm(mn23, mx23, 0x5410), __byte_perm(mn23, mx23, 0x7632)};
        float lo[4], inv[4];
        uint32_t mask[4];
        bool all_quantised = true;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            encode_params<BITS>(m[i], lo[i], inv[i]);
            mask[i] = inv[i] != 0.0f ? 0xffffffffu : 0u;
            all_quantised = all_quantised && inv[i] != 0.0f;
        }
        if (active) {
            if (half == 0)
                *reinterpret_cast<uint4 *>(meta + 4 * ((uint64_t)tile * c + 4 * cq)) = make_uint4(m[0], m[1], m[2], m[3]);
            uint8_t *out = codes + ((uint64_t)(tile * kTileTokens + r0) * c + 4 * cq) * BITS / 8;
            if (all_quantised) quantise_column<BITS, false>(x, lo, inv, mask, out, row_bytes, rows);
            else quantise_column<BITS, true>(x, lo, inv, mask, out, row_bytes, rows);
        }
    }
}

// ---- V: one group per token and 32 channels --------------------------------------------------

template <int BITS>
__device__ __forceinline__ void encode_tile_v(const uint16_t *src, uint8_t *meta, uint8_t *codes,
                                              int c, int tile, int nt)
{
    const int V8 = c >> 3;                               // 8-channel vectors per row, a multiple of 4
    const int cstep = V8 <= kThreads ? V8 : kThreads;
    const int rpp = V8 <= kThreads ? kThreads / V8 : 1;   // rows the CTA covers per pass
    const int my_row = threadIdx.x / cstep;
    const int my_cv = threadIdx.x - my_row * cstep;
    if (my_row >= rpp) return;                           // whole quads of lanes leave together
    const int lane = threadIdx.x & 31;
    const uint32_t quad = 0xfu << (lane & ~3);           // the 4 lanes that share each group
    const int t0 = tile * kTileTokens;
    const int groups = c / kGroup;
    constexpr int U = 8;                                 // rows in flight per thread

    for (int cv = my_cv; cv < V8; cv += cstep) {
        for (int tb = my_row; tb < nt; tb += U * rpp) {
            uint4 x[U];
            uint32_t m[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int t = tb + u * rpp;
                if (t < nt) x[u] = __ldcs(reinterpret_cast<const uint4 *>(src + (uint64_t)t * c) + cv);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (tb + u * rpp < nt) {                 // the same for the 4 lanes of a quad
                    uint32_t mn = bmin2(bmin2(x[u].x, x[u].y), bmin2(x[u].z, x[u].w));
                    uint32_t mx = bmax2(bmax2(x[u].x, x[u].y), bmax2(x[u].z, x[u].w));
                    mn = bmin2(mn, __shfl_xor_sync(quad, mn, 1));
                    mx = bmax2(mx, __shfl_xor_sync(quad, mx, 1));
                    mn = bmin2(mn, __shfl_xor_sync(quad, mn, 2));
                    mx = bmax2(mx, __shfl_xor_sync(quad, mx, 2));
                    mn = bmin2(mn, swap_halves(mn));
                    mx = bmax2(mx, swap_halves(mx));
                    m[u] = __byte_perm(mn, mx, 0x5410);
                }
            }
            // each lane of a quad divides for every fourth row: a quarter of a division per row
            float mine[U / 4];
#pragma unroll
            for (int j = 0; j < U / 4; ++j) {
                mine[j] = 0.0f;
                if (tb + (4 * j + (lane & 3)) * rpp < nt) {
                    uint32_t w = m[4 * j];
                    if ((lane & 3) == 1) w = m[4 * j + 1];
                    if ((lane & 3) == 2) w = m[4 * j + 2];
                    if ((lane & 3) == 3) w = m[4 * j + 3];
                    float unused;
                    encode_params<BITS>(w, unused, mine[j]);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int t = tb + u * rpp;
                if (t < nt) {
                    const float inv = __shfl_sync(quad, mine[u >> 2], (lane & ~3) | (u & 3));
                    const float lo = bf16_lo_to_f32(m[u]);
                    uint32_t a = 0, b = 0;               // a flat group: every code is 0
                    if (inv != 0.0f) {
                        a = pack4_biased<BITS>(biased_code(lo_half<false>(x[u].x, 0), lo, inv),
                                               biased_code(hi_half<false>(x[u].x, 0), lo, inv),
                                               biased_code(lo_half<false>(x[u].y, 0), lo, inv),
                                               biased_code(hi_half<false>(x[u].y, 0), lo, inv));
                        b = pack4_biased<BITS>(biased_code(lo_half<false>(x[u].z, 0), lo, inv),
                                               biased_code(hi_half<false>(x[u].z, 0), lo, inv),
                                               biased_code(lo_half<false>(x[u].w, 0), lo, inv),
                                               biased_code(hi_half<false>(x[u].w, 0), lo, inv));
                    }
                    const uint64_t e = (uint64_t)(t0 + t) * c + 8 * cv;
                    if constexpr (BITS == 8) *reinterpret_cast<uint2 *>(codes + e) = make_uint2(a, b);
                    if constexpr (BITS == 4)
                        *reinterpret_cast<uint32_t *>(codes + (e >> 1)) = (a & 0xffffu) | (b << 16);
                    if constexpr (BITS == 2)
                        *reinterpret_cast<uint16_t *>(codes + (e >> 2)) = (uint16_t)((a & 0xffu) | (b << 8));
                    if ((cv & 3) == 0)
                        reinterpret_cast<uint32_t *>(meta)[(uint64_t)(t0 + t) * groups + (cv >> 2)] = m[u];
                }
            }
        }
    }
}

static __global__ void __launch_bounds__(kThreads, 2) encode_kernel(const EncodeParams p)
{
    __shared__ uint4 xchg[2][kThreads];                   // K: partial ranges of the two row halves
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
    const uint16_t *src = p.kv + (((int64_t)layer * 2 + kv) * p.src_N + tok0 + tile * kTileTokens) * p.c;

    if (tile * kTileTokens + nt == n) {                   // the plane's last tile clears the padding
        zero_pad(codes, L.codes_payload, L.kcodes);
        if (d.level > 0)
            zero_pad(meta, kv ? L.vmeta_payload : L.kmeta_payload, kv ? L.vmeta : L.kmeta);
    }
    switch (d.level * 2 + kv) {                           // uniform per CTA
    case 0: case 1: encode_tile_raw(src, codes, p.c, tile * kTileTokens, nt); break;
    case 2: encode_tile_k<8>(src, meta, codes, p.c, tile, nt, xchg); break;
    case 3: encode_tile_v<8>(src, meta, codes, p.c, tile, nt); break;
    case 4: encode_tile_k<4>(src, meta, codes, p.c, tile, nt, xchg); break;
    case 5: encode_tile_v<4>(src, meta, codes, p.c, tile, nt); break;
    case 6: encode_tile_k<2>(src, meta, codes, p.c, tile, nt, xchg); break;
    default: encode_tile_v<2>(src, meta, codes, p.c, tile, nt); break;
    }
}

}  // namespace kvh
