// Persistent, TMA-fed encode kernel.
//
// Storing a context is the executor's other direction: the policy has decided to keep an entry
// "in full quality" (level 0) or to compress it (levels 1..3), and the KV tensor has to be turned
// into chunk streams at the speed HBM delivers it (2 bytes read and (b+1)/8 bytes written per
// element).  A 32-token tile of one (layer, K|V) plane is contiguous in the source, so a producer
// warp brings it into a ring of 64 KiB shared-memory stages with one 1-D bulk async copy per tile
// while 8 consumer warps turn the previous tiles into metadata and codes:
//   K (a group = one channel over the tile's 32 tokens): a thread owns 4 channels and keeps all
//     32 rows of them in registers, so ranges, scales and codes need one pass over shared memory
//     and no exchange between threads.
//   V (a group = 32 channels of one token): a thread owns whole groups (64 bytes), again with no
//     exchange.  Neighbouring lanes are 64 bytes apart, so each lane reads its four 16-byte pieces
//     in an order rotated by its lane number (bank conflicts vanish) and rotates the packed codes
//     back in registers before one wide store.
// The three roundings of a code, (x - min) * inv + 2^23, are done two elements at a time with the
// packed binary32 instructions of sm_100 (sub/mul/fma .rn.f32x2: IEEE round-to-nearest on each
// half, no flush to zero), which halves the issue slots the arithmetic takes.  A stage is handed
// back to the producer as soon as its data sits in registers.
//
// Rows wider than 1024 channels are cut into column blocks (RowGeom): blocks of 1024 channels come
// in through 2-D tiled TMA (a tensor map over the source, four boxes of 256 channels x 32 rows per
// tile), other widths and token dropping (kept runs gathered into a compact sequence) through one
// 1-D bulk copy per row issued by the producer's lanes in parallel.
//
// Rows of at most 512 channels: a work unit takes 2, 4 or 8 consecutive tiles of the plane
// (EncodeParams::tpu; they are contiguous in the source), so that a unit still fills a stage and
// every consumer thread has a column of some tile.  Widths that are a multiple of 256 but neither
// one of those nor a multiple of 1024 (768, 1280, 1536 ...) are cut into column blocks of 256
// channels and a unit takes 4 consecutive tiles of one block, each fetched as one 2-D box: in the
// stage that is the layout of a plane 256 channels wide (EncodeParams::boxes).
//
// Tiles are handed out dynamically through cluster launch control, as in the decode kernel.  Every
// wait is bounded: when one runs out the CTA reports KVH_ERR_TIMEOUT, raises its abort flag,
// waits for its copies in flight and leaves.
#pragma once

#include <cuda.h>      // CUtensorMap

#include "kvh_async.cuh"
#include "kvh_encode.cuh"
#include "kvh_format.cuh"

namespace kvh {

constexpr int kEncGroupThreads = 256;                    // consumer threads that share a tile
constexpr int kEncStages = 3;
constexpr uint32_t kEncStageBytes = 2u * kTileTokens * 1024u;   // a 32-token tile at c = 1024
constexpr int kEncMaxChannels = 1024;

// Which chunks a launch covers: chunk0, chunk0 + 1, ... in order, or the ones a list names.  The
// list travels in the kernel's parameters (no device memory), which is what lets the host hand
// each level's chunks of a mixed context to the kernel instance specialised for that level.
constexpr int kMaxListedChunks = 4000;
struct AllChunks {
    __device__ __forceinline__ int chunk(int i, int chunk0) const { return chunk0 + i; }
};
struct ListedChunks {
    uint32_t idx[kMaxListedChunks];
    __device__ __forceinline__ int chunk(int i, int) const { return (int)idx[i]; }
};

struct EncUnit {
    int32_t bits;          // 16, 8, 4, 2; 0 marks the end of the CTA's work
    int32_t kv;            // 0 K, 1 V
    int32_t nt;            // tokens in the unit (1..32 * tpu)
    int32_t tile;          // index within the chunk of the unit's first tile
    int32_t last;          // the plane's last tile clears the sections' padding
    uint32_t meta_payload, meta_padded, codes_payload, codes_padded;
    uint8_t *meta;         // the plane's metadata section in the stream
    uint8_t *codes;        // the plane's code section
    int32_t col0;          // first channel of the tile's column block (0 unless rows are wider than a stage holds)
    int32_t cw;            // channels per row of the block = per stage row
};

// Rows wider than 1024 channels are cut into column blocks of equal width (a divisor of c that is a
// multiple of 128); a tile is then 32 tokens of one block.  In the stage its rows are cw channels
// wide and packed; in the plane (source and stream) rows are cf channels wide and the block starts
// at channel col0.  With the channel count compiled in, all three are constants.
// Blocks of 1024 channels arrive through 2-D tiled TMA as 4 boxes of 256 channels x 32 rows
// (a box dimension is at most 256 elements): the stage is then [box][row][256 channels] (boxed)
// instead of [row][cw channels].
constexpr int kBoxChannels = 256;
constexpr uint32_t kBoxBytes = 2u * kBoxChannels * kTileTokens;      // 16 KiB
struct RowGeom {
    int cw, cf, col0;
    bool boxed;
    // byte offset in the stage of channel ch (a multiple of 4) of row 0, and between rows
    __device__ __forceinline__ uint32_t stage_col(int ch) const
    {
        return boxed ? (uint32_t)(ch / kBoxChannels) * kBoxBytes + 2u * (uint32_t)(ch % kBoxChannels) : 2u * (uint32_t)ch;
    }
    __device__ __forceinline__ uint32_t stage_row_bytes() const { return boxed ? 2u * kBoxChannels : 2u * (uint32_t)cw; }
};
template <int C, bool WIDE = false>
__device__ __forceinline__ RowGeom row_geom(int cw, int cf, int col0)
{
    if constexpr (C != 0 && !WIDE) return RowGeom{C, C, 0, false};        // rows of exactly C channels
    else if constexpr (C != 0) return RowGeom{C, cf, col0, true};         // blocks of C = 1024 channels of wider rows
    else return RowGeom{cw, cf, col0, false};
}

// Both elements of a packed bf16 pair: 2^23 + code as raw float bits (adding 2^23 to
// s = (x - min) * inv leaves rint(s), ties to even, in the low mantissa bits).  With MASKED the value
// of a channel whose group is stored flat is replaced by 0 first, so that its code is 0 even when
// x - min overflows.
// The product must be rounded before 2^23 is added.  The assembler contracts a packed mul followed
// by a packed add into one fused multiply-add even with .rn on both, which skips that rounding and
// moves a code wherever the product rounds to a tie; it does the same to fma(s, 1.0, 2^23) once it
// has folded the literal 1.0 away.  With a multiplier it cannot know, the fma stays: it rounds
// s * 1 + 2^23 once, exactly like an add, and cannot absorb the mul.
__device__ __forceinline__ void biased_pair_f32(f32x2 x, f32x2 lo2, f32x2 inv2, uint32_t &ta, uint32_t &tb)
{
    const f32x2 magic = f2_from_bits(0x4b000000u, 0x4b000000u);
    const f32x2 s = f2_mul(f2_sub(x, lo2), inv2);
    const float one = kRuntimeOne;
    f2_bits(f2_fma(s, f2_make(one, one), magic), ta, tb);
}
template <bool MASKED>
__device__ __forceinline__ void biased_pair(uint32_t w, f32x2 lo2, f32x2 inv2, uint32_t mask_a, uint32_t mask_b,
                                            uint32_t &ta, uint32_t &tb)
{
    uint32_t a = w << 16, b = w & 0xffff0000u;
    if (MASKED) { a &= mask_a; b &= mask_b; }
    biased_pair_f32(f2_from_bits(a, b), lo2, inv2, ta, tb);
}

// Four biased codes (0x4b000000 + q) into the low 4 * BITS bits.  For 2 and 4 bits the biases end
// up above the field and the caller's narrow store (or a byte permute) drops them.
template <int BITS>
__device__ __forceinline__ uint32_t pack4_low(uint32_t t0, uint32_t t1, uint32_t t2, uint32_t t3)
{
    if constexpr (BITS == 8) {
        return __byte_perm(__byte_perm(t0, t1, 0x0040), __byte_perm(t2, t3, 0x0040), 0x5410);
    } else {
        return (t0 + (t1 << BITS)) + ((t2 + (t3 << BITS)) << (2 * BITS));
    }
}

// Hand a stage back to the producer: every lane's reads of it are done.
__device__ __forceinline__ void enc_release(uint64_t *empty_bar)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(empty_bar);
}

// ---- level 0: the tile's rows as they are ------------------------------------------------------

template <int C>
__device__ __forceinline__ void enc_consume_raw(const uint8_t *st, RowGeom g, int tid, uint64_t *empty_bar,
                                                int nt, int tile, uint8_t *codes_sec)
{
    const int vpr = g.cw >> 3;                            // 16-byte vectors per stage row
    const int nvec = nt * vpr;
    const uint4 *src = reinterpret_cast<const uint4 *>(st);
    uint8_t *dst = codes_sec + 2 * ((size_t)tile * kTileTokens * g.cf + g.col0);
    const bool packed = g.cw == g.cf;                     // the tile's rows are contiguous in the stream too
    constexpr int U = 8;
    const int iters = (nvec + kEncGroupThreads * U - 1) / (kEncGroupThreads * U);     // the same for every thread
    for (int it = 0; it < iters; ++it) {
        const int v0 = it * kEncGroupThreads * U + tid;
        uint4 x[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = v0 + k * kEncGroupThreads;
            if (v < nvec) {
                if (g.boxed) {
                    const int row = v / vpr;
                    x[k] = *reinterpret_cast<const uint4 *>(st + g.stage_col(8 * (v - row * vpr)) + row * g.stage_row_bytes());
                } else {
                    x[k] = src[v];
                }
            }
        }
        if (it == iters - 1) enc_release(empty_bar);
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = v0 + k * kEncGroupThreads;
            if (v < nvec) {
                size_t off = 16 * (size_t)v;
                if (!packed) {
                    const int row = v / vpr;
                    off = 2 * (size_t)row * g.cf + 16 * (size_t)(v - row * vpr);
                }
                __stcs(reinterpret_cast<uint4 *>(dst + off), x[k]);
            }
        }
    }
}

// ---- K: one group per channel -------------------------------------------------------------------

// Codes of one row of a 4-channel column, stored with the width the level needs.
template <int BITS>
__device__ __forceinline__ void store_codes4(uint32_t packed, uint8_t *o)
{
    if constexpr (BITS == 8) *reinterpret_cast<uint32_t *>(o) = packed;
    if constexpr (BITS == 4) *reinterpret_cast<uint16_t *>(o) = (uint16_t)packed;
    if constexpr (BITS == 2) *o = (uint8_t)packed;
}
template <int BITS, bool MASKED>
__device__ __forceinline__ void enc_store_row_k(uint2 x, f32x2 lo_a, f32x2 lo_b, f32x2 inv_a, f32x2 inv_b,
                                                const uint32_t (&mask)[4], uint8_t *o)
{
    uint32_t t0, t1, t2, t3;
    biased_pair<MASKED>(x.x, lo_a, inv_a, mask[0], mask[1], t0, t1);
    biased_pair<MASKED>(x.y, lo_b, inv_b, mask[2], mask[3], t2, t3);
    store_codes4<BITS>(pack4_low<BITS>(t0, t1, t2, t3), o);
}
// The same for a row given as four binary32 values (two pairs) that are exact in bf16; a channel
// stored flat has inv = 0 and must not hold a value whose distance from min overflows.
template <int BITS>
__device__ __forceinline__ void enc_store_row_k_f32(f32x2 xa, f32x2 xb, f32x2 lo_a, f32x2 lo_b, f32x2 inv_a, f32x2 inv_b,
                                                    uint8_t *o)
{
    uint32_t t0, t1, t2, t3;
    biased_pair_f32(xa, lo_a, inv_a, t0, t1);
    biased_pair_f32(xb, lo_b, inv_b, t2, t3);
    store_codes4<BITS>(pack4_low<BITS>(t0, t1, t2, t3), o);
}

// Metadata words (min | max << 16) of 4 channels from their packed ranges, and what follows
// from them; returns whether every one of the 4 groups is quantised (none stored flat).
template <int BITS>
__device__ __forceinline__ bool enc_params_k(uint32_t mn01, uint32_t mn23, uint32_t mx01, uint32_t mx23,
                                             uint4 *meta_out, float (&lo)[4], float (&inv)[4], uint32_t (&mask)[4])
{
    const uint32_t m[4] = {__byte_perm(mn01, mx01, 0x5410), __byte_perm(mn01, mx01, 0x7632),
                           __byte_perm(mn23, mx23, 0x5410), __byte_perm(mn23, mx23, 0x7632)};
    bool all_quantised = true;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        encode_params<BITS>(m[i], lo[i], inv[i]);
        mask[i] = inv[i] != 0.0f ? 0xffffffffu : 0u;
        all_quantised = all_quantised && inv[i] != 0.0f;
    }
    *meta_out = make_uint4(m[0], m[1], m[2], m[3]);
    return all_quantised;
}

// Where the metadata words and the first row's codes of 4-channel column cq of a tile go.
template <int BITS>
__device__ __forceinline__ void enc_k_out(RowGeom g, int cq, int tile, uint8_t *meta_sec, uint8_t *codes_sec,
                                          uint4 *&meta_out, uint8_t *&codes_out, uint32_t &row_bytes)
{
    const size_t ch = (size_t)g.col0 + 4 * (size_t)cq;   // the column's first channel within the plane
    meta_out = reinterpret_cast<uint4 *>(meta_sec + 4 * ((size_t)tile * g.cf + ch));
    codes_out = codes_sec + ((size_t)tile * kTileTokens * g.cf + ch) * BITS / 8;
    row_bytes = (uint32_t)g.cf * BITS / 8;
}

// A full tile of K once its 32 rows of the thread's 4 channels (column cq) sit in registers:
// ranges, metadata, codes.
template <int BITS>
__device__ __forceinline__ void enc_process_k(uint2 (&x)[kTileTokens], RowGeom g, int cq, int tile,
                                              uint8_t *meta_sec, uint8_t *codes_sec)
{
    uint32_t mn01 = x[0].x, mn23 = x[0].y, mx01 = x[0].x, mx23 = x[0].y;
#pragma unroll
    for (int t = 1; t < kTileTokens; ++t) {
        mn01 = bmin2(mn01, x[t].x); mx01 = bmax2(mx01, x[t].x);
        mn23 = bmin2(mn23, x[t].y); mx23 = bmax2(mx23, x[t].y);
    }
    uint4 *meta_out;
    uint8_t *out;
    uint32_t row_bytes;
    enc_k_out<BITS>(g, cq, tile, meta_sec, codes_sec, meta_out, out, row_bytes);
    float lo[4], inv[4];
    uint32_t mask[4];
    const bool all_quantised = enc_params_k<BITS>(mn01, mn23, mx01, mx23, meta_out, lo, inv, mask);
    if (!all_quantised) {
        // a channel stored flat: its values become 0 so that (0 - min) * 0 is a zero and the code 0
        // (x - min may overflow for such a group, and infinity * 0 would be NaN)
        const uint32_t k01 = (mask[0] & 0xffffu) | (mask[1] & 0xffff0000u);
        const uint32_t k23 = (mask[2] & 0xffffu) | (mask[3] & 0xffff0000u);
#pragma unroll
        for (int t = 0; t < kTileTokens; ++t) { x[t].x &= k01; x[t].y &= k23; }
    }
    const f32x2 lo_a = f2_make(lo[0], lo[1]), lo_b = f2_make(lo[2], lo[3]);
    const f32x2 inv_a = f2_make(inv[0], inv[1]), inv_b = f2_make(inv[2], inv[3]);
#pragma unroll
    for (int t = 0; t < kTileTokens; ++t)
        enc_store_row_k<BITS, false>(x[t], lo_a, lo_b, inv_a, inv_b, mask, out + (size_t)t * row_bytes);
}

// Full tiles (nt = 32, or a multiple of 32 when a unit holds several tiles of narrow rows): a thread
// takes 4 channels of one tile, all 32 rows of them in registers, one pass over shared memory.
template <int BITS>
__device__ __forceinline__ void enc_consume_k(const uint8_t *st, RowGeom g, int tid, uint64_t *empty_bar,
                                              int nt, int tile, uint8_t *meta_sec, uint8_t *codes_sec)
{
    const int C4 = g.cw >> 2;                            // 4-channel columns per stage row, <= 256
    const int sub = C4 >= kEncGroupThreads ? 0 : tid / C4;      // which of the unit's tiles
    const bool active = sub * kTileTokens < nt;
    const int cq = active ? tid - sub * C4 : 0;
    const uint32_t rs = g.stage_row_bytes();
    const uint8_t *col = st + g.stage_col(4 * cq) + (active ? sub : 0) * kTileTokens * rs;
    uint2 x[kTileTokens];
#pragma unroll
    for (int t = 0; t < kTileTokens; ++t) x[t] = *reinterpret_cast<const uint2 *>(col + t * rs);
    enc_release(empty_bar);
    if (active) enc_process_k<BITS>(x, g, cq, tile + sub, meta_sec, codes_sec);
}

// A chunk's end that is not a whole number of tiles: rare, so two plain passes over the rows.
// row(t) returns row t of the thread's 4 channels (column cq) as two packed bf16 pairs.
template <int BITS, typename RowFn>
__device__ __forceinline__ void enc_k_short(RowFn row, RowGeom g, int cq, int nt, int tile,
                                            uint8_t *meta_sec, uint8_t *codes_sec)
{
    const uint2 x0 = row(0);
    uint32_t mn01 = x0.x, mn23 = x0.y, mx01 = mn01, mx23 = mn23;
#pragma unroll 1
    for (int t = 1; t < nt; ++t) {
        const uint2 x = row(t);
        mn01 = bmin2(mn01, x.x); mx01 = bmax2(mx01, x.x);
        mn23 = bmin2(mn23, x.y); mx23 = bmax2(mx23, x.y);
    }
    uint4 *meta_out;
    uint8_t *out;
    uint32_t row_bytes;
    enc_k_out<BITS>(g, cq, tile, meta_sec, codes_sec, meta_out, out, row_bytes);
    float lo[4], inv[4];
    uint32_t mask[4];
    (void)enc_params_k<BITS>(mn01, mn23, mx01, mx23, meta_out, lo, inv, mask);
    const f32x2 lo_a = f2_make(lo[0], lo[1]), lo_b = f2_make(lo[2], lo[3]);
    const f32x2 inv_a = f2_make(inv[0], inv[1]), inv_b = f2_make(inv[2], inv[3]);
#pragma unroll 1
    for (int t = 0; t < nt; ++t)
        enc_store_row_k<BITS, true>(row(t), lo_a, lo_b, inv_a, inv_b, mask, out + (size_t)t * row_bytes);
}

template <int BITS>
__device__ __noinline__ void enc_consume_k_short(const uint8_t *st, RowGeom g, int tid, uint64_t *empty_bar,
                                                 int nt, int tile, uint8_t *meta_sec, uint8_t *codes_sec)
{
    const int C4 = g.cw >> 2;
    const int sub = tid / C4;                            // which of the unit's tiles
    const int nt_sub = min(kTileTokens, nt - sub * kTileTokens);
    if (nt_sub > 0) {
        const int cq = tid - sub * C4;
        const uint32_t rs = g.stage_row_bytes();
        const uint8_t *col = st + g.stage_col(4 * cq) + sub * kTileTokens * rs;
        enc_k_short<BITS>([&](int t) { return *reinterpret_cast<const uint2 *>(col + t * rs); }, g, cq, nt_sub,
                          tile + sub, meta_sec, codes_sec);
    }
    enc_release(empty_bar);
}

// ---- V: one group per token and 32 channels ---------------------------------------------------

// p[j] holds the piece with number (j + rot) & 3; put piece k into p[k].
template <int W>
__device__ __forceinline__ void enc_unrotate(uint32_t (&p)[4][W], int rot)
{
    const bool r1 = rot & 1, r2 = rot & 2;
    uint32_t q[4][W];
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int w = 0; w < W; ++w) q[k][w] = r1 ? p[(k + 3) & 3][w] : p[k][w];
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int w = 0; w < W; ++w) p[k][w] = r2 ? q[(k + 2) & 3][w] : q[k][w];
}

// Metadata word (min | max << 16) of one group given as four 16-byte pieces, in any order.
__device__ __forceinline__ uint32_t enc_range_v(const uint4 (&x)[4])
{
    uint32_t mn = bmin2(bmin2(x[0].x, x[0].y), bmin2(x[0].z, x[0].w));
    uint32_t mx = bmax2(bmax2(x[0].x, x[0].y), bmax2(x[0].z, x[0].w));
#pragma unroll
    for (int j = 1; j < 4; ++j) {
        mn = bmin2(mn, bmin2(bmin2(x[j].x, x[j].y), bmin2(x[j].z, x[j].w)));
        mx = bmax2(mx, bmax2(bmax2(x[j].x, x[j].y), bmax2(x[j].z, x[j].w)));
    }
    mn = bmin2(mn, swap_halves(mn));
    mx = bmax2(mx, swap_halves(mx));
    return __byte_perm(mn, mx, 0x5410);
}

// Code words of one 16-byte piece (8 elements) of a group from their 8 biased codes: W words, 2 at
// 8 bits, else 1 (at 2 bits its low 16 bits count).
template <int BITS, int W>
__device__ __forceinline__ void pack_piece_v(const uint32_t (&t)[8], uint32_t (&w)[W])
{
    const uint32_t a = pack4_low<BITS>(t[0], t[1], t[2], t[3]);
    const uint32_t b = pack4_low<BITS>(t[4], t[5], t[6], t[7]);
    if constexpr (BITS == 8) { w[0] = a; w[1] = b; }
    if constexpr (BITS == 4) w[0] = __byte_perm(a, b, 0x5410);
    if constexpr (BITS == 2) w[0] = __byte_perm(a, b, 0x0040);       // 16 bits; the upper half is dropped later
}
// A piece given as 4 packed bf16 pairs ...
template <int BITS, int W>
__device__ __forceinline__ void enc_piece_v(const uint4 &x, f32x2 lo2, f32x2 inv2, uint32_t (&w)[W])
{
    uint32_t t[8];
    biased_pair<false>(x.x, lo2, inv2, 0, 0, t[0], t[1]);
    biased_pair<false>(x.y, lo2, inv2, 0, 0, t[2], t[3]);
    biased_pair<false>(x.z, lo2, inv2, 0, 0, t[4], t[5]);
    biased_pair<false>(x.w, lo2, inv2, 0, 0, t[6], t[7]);
    pack_piece_v<BITS, W>(t, w);
}
// ... or as 8 binary32 values (4 pairs) that are exact in bf16.
template <int BITS, int W>
__device__ __forceinline__ void enc_piece_v_f32(const f32x2 (&x)[4], f32x2 lo2, f32x2 inv2, uint32_t (&w)[W])
{
    uint32_t t[8];
#pragma unroll
    for (int k = 0; k < 4; ++k) biased_pair_f32(x[k], lo2, inv2, t[2 * k], t[2 * k + 1]);
    pack_piece_v<BITS, W>(t, w);
}

// The four pieces' code words of a group, in piece order, to the stream.
template <int BITS, int W>
__device__ __forceinline__ void enc_store_group_v(const uint32_t (&p)[4][W], uint8_t *codes_out)
{
    if constexpr (BITS == 8) {
        uint4 *o = reinterpret_cast<uint4 *>(codes_out);
        o[0] = make_uint4(p[0][0], p[0][1], p[1][0], p[1][1]);
        o[1] = make_uint4(p[2][0], p[2][1], p[3][0], p[3][1]);
    }
    if constexpr (BITS == 4)
        *reinterpret_cast<uint4 *>(codes_out) = make_uint4(p[0][0], p[1][0], p[2][0], p[3][0]);
    if constexpr (BITS == 2)
        *reinterpret_cast<uint2 *>(codes_out) = make_uint2(__byte_perm(p[0][0], p[1][0], 0x5410),
                                                           __byte_perm(p[2][0], p[3][0], 0x5410));
}

// One group with its metadata word m known: store m and the codes.  x[j] is the 16-byte piece
// number (j + rot) & 3 of the group's 64 bytes (ROTATED), or simply piece j.
template <int BITS, bool ROTATED = true>
__device__ __forceinline__ void enc_group_v(const uint4 (&x)[4], int rot, uint32_t m, uint32_t *meta_out,
                                            uint8_t *codes_out)
{
    *meta_out = m;
    float lo, inv;
    encode_params<BITS>(m, lo, inv);
    constexpr int W = BITS == 8 ? 2 : 1;                 // words a piece's 8 codes take (16 bits used at 2 bits)
    uint32_t p[4][W];
    if (inv != 0.0f) {
        const f32x2 lo2 = f2_make(lo, lo), inv2 = f2_make(inv, inv);
#pragma unroll
        for (int j = 0; j < 4; ++j) enc_piece_v<BITS, W>(x[j], lo2, inv2, p[j]);
        if (ROTATED) enc_unrotate<W>(p, rot);
    } else {                                             // a flat group: every code is 0
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int w = 0; w < W; ++w) p[j][w] = 0;
    }
    enc_store_group_v<BITS, W>(p, codes_out);
}

// Index, within the plane's V sections, of group gs of the tile's stage (stage rows hold cw / 32
// groups, plane rows cf / 32).
__device__ __forceinline__ size_t enc_v_group_index(RowGeom g, int tile, int gs)
{
    const int gpr_w = g.cw >> 5, gpr_f = g.cf >> 5;
    const int row = gs / gpr_w;                          // a shift when the width is compiled in
    return ((size_t)tile * kTileTokens + row) * gpr_f + (g.col0 >> 5) + (gs - row * gpr_w);
}

template <int BITS>
__device__ __forceinline__ void enc_consume_v(const uint8_t *st, RowGeom g, int tid, uint64_t *empty_bar,
                                              int nt, int tile, uint8_t *meta_sec, uint8_t *codes_sec)
{
    const int gpr_w = g.cw >> 5;
    const int ngroups = nt * gpr_w;                      // the tile's groups, in stage order
    const int rot = (tid >> 1) & 3;
    uint32_t off[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) off[j] = (uint32_t)((j + rot) & 3) * 16u;
    uint32_t *meta = reinterpret_cast<uint32_t *>(meta_sec);
    constexpr int U = 2;                                 // groups a thread holds at a time
    const int iters = (ngroups + kEncGroupThreads * U - 1) / (kEncGroupThreads * U);  // the same for every thread
    for (int it = 0; it < iters; ++it) {
        const int g0 = it * kEncGroupThreads * U + tid;
        uint4 x[U][4];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int gs = g0 + k * kEncGroupThreads;
            if (gs < ngroups) {
                const int row = gs / gpr_w;              // boxed: 8 groups per box row
                const uint8_t *grp = g.boxed ? st + g.stage_col(32 * (gs - row * gpr_w)) + row * g.stage_row_bytes()
                                             : st + (size_t)gs * 64;
#pragma unroll
                for (int j = 0; j < 4; ++j) x[k][j] = *reinterpret_cast<const uint4 *>(grp + off[j]);
            }
        }
        if (it == iters - 1) enc_release(empty_bar);
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int gs = g0 + k * kEncGroupThreads;
            if (gs < ngroups) {
                const size_t gi = enc_v_group_index(g, tile, gs);
                enc_group_v<BITS>(x[k], rot, enc_range_v(x[k]), meta + gi, codes_sec + gi * (4 * BITS));
            }
        }
    }
}

// One unit of a known level: K or V (or the raw copy), inlined into the caller.
template <int C, int LEVEL, bool WIDE = false>
__device__ __forceinline__ void enc_consume_level(const EncUnit &u, const uint8_t *st, int c_rt, int tid,
                                                  uint64_t *eb)
{
    const RowGeom g = row_geom<C, WIDE>(u.cw, c_rt, u.col0);
    if constexpr (LEVEL == 0) {
        enc_consume_raw<C>(st, g, tid, eb, u.nt, u.tile, u.codes);
    } else {
        constexpr int BITS = 16 >> LEVEL;
        if (u.kv) enc_consume_v<BITS>(st, g, tid, eb, u.nt, u.tile, u.meta, u.codes);
        else if ((u.nt & (kTileTokens - 1)) == 0) enc_consume_k<BITS>(st, g, tid, eb, u.nt, u.tile, u.meta, u.codes);
        else enc_consume_k_short<BITS>(st, g, tid, eb, u.nt, u.tile, u.meta, u.codes);
    }
}
// The same as a function of its own: a kernel that has to hold all four levels keeps each level's
// registers apart this way (inlined side by side they spill).
template <int C, int LEVEL, bool WIDE>
__device__ __noinline__ void enc_consume_level_call(const EncUnit *u, const uint8_t *st, int c_rt, int tid,
                                                    uint64_t *eb)
{
    enc_consume_level<C, LEVEL, WIDE>(*u, st, c_rt, tid, eb);
}

// LEVEL >= 0: every chunk of the launch has this level (checked by the producer); -1: any mix.
template <int C, int LEVEL, bool WIDE>
__device__ __forceinline__ void enc_dispatch(const EncUnit &u, const uint8_t *st, int c_rt, int tid, uint64_t *eb)
{
    if constexpr (LEVEL >= 0) {
        enc_consume_level<C, LEVEL, WIDE>(u, st, c_rt, tid, eb);
    } else {
        switch (u.bits) {                                // uniform per consumer group
        case 16: enc_consume_level_call<C, 0, WIDE>(&u, st, c_rt, tid, eb); break;
        case 8: enc_consume_level_call<C, 1, WIDE>(&u, st, c_rt, tid, eb); break;
        case 4: enc_consume_level_call<C, 2, WIDE>(&u, st, c_rt, tid, eb); break;
        default: enc_consume_level_call<C, 3, WIDE>(&u, st, c_rt, tid, eb); break;
        }
    }
}

// sched: 0 = each CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ... (grid = resident CTAs);
//        1 = one CTA per tile in the grid, running CTAs pull further tiles through cluster launch control.
// The 8 consumer warps take every unit together: a stage's full barrier is then waited on once per
// phase, which is what lets one parity bit tell the phases apart.
template <int C, int LEVEL, typename Chunks, bool WIDE = false>
__global__ void __launch_bounds__(32 + kEncGroupThreads, 1)
encode_tma_kernel(const EncodeParams p, const int n_chunks, const int sched, const Chunks chunks,
                  const __grid_constant__ CUtensorMap kv_map)
{
    extern __shared__ __align__(128) uint8_t stage_mem[];
    __shared__ __align__(8) uint64_t full_bar[kEncStages];
    __shared__ __align__(8) uint64_t empty_bar[kEncStages];
    __shared__ EncUnit info[kEncStages];
    __shared__ int abort_flag;
    __shared__ __align__(16) uint4 clc_response[2];
    __shared__ __align__(8) uint64_t clc_bar[2];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kProducerWarp = kEncGroupThreads / 32;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kEncStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kEncGroupThreads / 32);
        }
        mbar_init(&clc_bar[0], 1);
        mbar_init(&clc_bar[1], 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == kProducerWarp) {
        // ------------------------------ producer warp ------------------------------
        const int tpu = (C != 0) ? 1 : p.tpu;             // tiles per unit
        const int upc = kTilesPerChunk / tpu;             // units per chunk and plane
        const int64_t total_tiles = (int64_t)n_chunks * p.l * 2 * upc * p.n_blocks;
        uint32_t unit = 0;
        bool ok = true;

        auto acquire = [&]() -> bool {                   // wait until the unit's stage is free
            const int s = unit % kEncStages;
            if (unit < (uint32_t)kEncStages) return true;
            bool w = true;
            if (lane == 0) w = mbar_wait(&empty_bar[s], ((unit / kEncStages) - 1) & 1, &abort_flag);
            return __shfl_sync(0xffffffffu, w, 0);
        };

        auto do_tile = [&](int64_t tile_id) {
            // a tile id fits 32 bits (the host refuses larger launches): unsigned 32-bit divisions
            const uint32_t id = (uint32_t)tile_id;
            const uint32_t nb = (uint32_t)p.n_blocks, units = (uint32_t)upc;
            const int cb = (int)(id % nb);                       // column block, fastest: neighbours share rows
            const uint32_t row_tile = id / nb;
            const int tile = (int)(row_tile % units) * tpu;      // the unit's first tile
            const uint32_t plane_id = row_tile / units;
            const int kv = (int)(plane_id & 1);
            const int layer = (int)((plane_id >> 1) % (uint32_t)p.l);
            const int chunk = chunks.chunk((int)((plane_id >> 1) / (uint32_t)p.l), p.chunk0);
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
            if (err == KVH_OK && LEVEL >= 0 && d.level != LEVEL) err = KVH_ERR_BAD_LEVEL;
            if (err != KVH_OK) {
                if (lane == 0) report(p.status, err);
                return;
            }
            const int n = d.n_tok;
            const int nt = min(kTileTokens * tpu, n - tile * kTileTokens);
            if (nt <= 0) return;
            const LayerLayout L = layer_layout(d.level, p.c, n);
            uint8_t *lay = p.out + d.stream_off + (uint64_t)layer * L.layer_bytes();
            const uint16_t *plane = p.kv + ((int64_t)layer * 2 + kv) * p.src_N * p.c;
            const int64_t j0 = tok0 + tile * kTileTokens;        // the tile's first token in the encoded sequence
            ok = acquire();
            if (!ok) return;
            const int s = unit % kEncStages;
            uint8_t *st = stage_mem + (size_t)s * kEncStageBytes;
            const uint32_t row_bytes = 2u * (uint32_t)p.bw;                     // a multiple of 64
            if (lane == 0) {
                EncUnit &u = info[s];
                u.bits = level_bits(d.level); u.kv = kv; u.nt = nt; u.tile = tile;
                u.last = tile * kTileTokens + nt == n && cb == p.n_blocks - 1;
                u.meta_payload = (uint32_t)(kv ? L.vmeta_payload : L.kmeta_payload);
                u.meta_padded = (uint32_t)(kv ? L.vmeta : L.kmeta);
                u.codes_payload = (uint32_t)L.codes_payload;
                u.codes_padded = (uint32_t)L.kcodes;
                u.meta = lay + L.meta_off(kv);
                u.codes = lay + L.codes_off(kv);
                u.col0 = cb * p.bw; u.cw = p.bw;
                const uint32_t n_boxes = (uint32_t)(nt + kTileTokens - 1) / kTileTokens;
                mbar_arrive_expect_tx(&full_bar[s], WIDE && p.n_runs == 0 ? 4 * kBoxBytes
                                                    : p.boxes            ? n_boxes * kBoxBytes
                                                                         : (uint32_t)nt * row_bytes);
            }
            if (p.n_blocks == 1) {
                if (lane == 0) {
                    if (p.n_runs == 0) {
                        bulk_load(st, plane + j0 * p.c, (uint32_t)nt * row_bytes, &full_bar[s]);
                    } else {
                        // token dropping: the tile's rows come from the kept runs it overlaps, one copy per run
                        for (int r = 0; r < p.n_runs; ++r) {
                            const int64_t a = max(j0, p.run_pos[r]), b = min(j0 + nt, p.run_pos[r + 1]);
                            if (a < b)
                                bulk_load(st + (size_t)(a - j0) * row_bytes,
                                          plane + (p.run_first[r] + (a - p.run_pos[r])) * p.c,
                                          (uint32_t)(b - a) * row_bytes, &full_bar[s]);
                        }
                    }
                }
            } else if (WIDE && p.n_runs == 0) {
                // blocks of 1024 channels of wider rows: 4 boxes of 256 channels x 32 rows through the
                // tensor map of the source seen as [planes * tokens][c]; rows past the tile are loaded too
                // (zeros past the tensor's end) and ignored
                if (lane == 0) {
                    const int row = (int)(((int64_t)layer * 2 + kv) * p.src_N + j0);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        tensor_load_2d(st + k * kBoxBytes, &kv_map, cb * p.bw + k * kBoxChannels, row, &full_bar[s]);
                }
            } else if (!WIDE && p.boxes) {
                // blocks of 256 channels: the unit's tiles, one box of 256 channels x 32 rows each, land one
                // behind the other (rows past the unit's last token are loaded too and ignored)
                const int boxes = (nt + kTileTokens - 1) / kTileTokens;
                __syncwarp();                            // the expectation is posted first
                if (lane < boxes) {
                    const int row = (int)(((int64_t)layer * 2 + kv) * p.src_N + j0) + lane * kTileTokens;
                    tensor_load_2d(st + lane * kBoxBytes, &kv_map, cb * p.bw, row, &full_bar[s]);
                }
            } else {
                // a column block of wide rows: lane r copies row r's piece (the expectation is posted first)
                __syncwarp();
                if (lane < nt) {
                    int64_t tok = j0 + lane;                                    // in the encoded sequence
                    for (int r = 0; r < p.n_runs; ++r)
                        if (tok >= p.run_pos[r] && tok < p.run_pos[r + 1]) { tok = p.run_first[r] + (tok - p.run_pos[r]); break; }
                    const uint16_t *src = plane + tok * p.c + cb * p.bw;
                    if (WIDE) {                                                 // the boxed stage layout, piece by piece
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            bulk_load(st + k * kBoxBytes + (size_t)lane * 2 * kBoxChannels, src + k * kBoxChannels,
                                      2 * kBoxChannels, &full_bar[s]);
                    } else {
                        bulk_load(st + (size_t)lane * row_bytes, src, row_bytes, &full_bar[s]);
                    }
                }
            }
            ++unit;
        };

        TileFeed feed{clc_response, clc_bar, sched, lane, &abort_flag};
        int64_t tile_id = blockIdx.x;
        while (ok && tile_id < total_tiles) {
            feed.ask();                                  // the next tile's index travels while this one streams
            do_tile(tile_id);
            if (!ok) break;
            const int more = feed.next(tile_id, total_tiles);
            if (more < 0) ok = false;
            if (more <= 0) break;
        }
        if (ok) ok = acquire();
        if (ok) {                                        // end marker
            if (lane == 0) {
                info[unit % kEncStages].bits = 0;
                mbar_arrive(&full_bar[unit % kEncStages]);
            }
            ++unit;
        }
        if (!ok && lane == 0) {
            report(p.status, KVH_ERR_TIMEOUT);
            abort_flag = 1;
        }
        // Leave only after every copy issued has landed: a normal run has seen them all consumed;
        // after an abort the last kEncStages units may still be in flight.
        if (lane == 0) {
            int never = 0;                               // the drain ignores the abort flag
            const uint32_t first = unit > (uint32_t)kEncStages ? unit - kEncStages : 0;
            for (uint32_t w = first; w < unit; ++w)
                (void)mbar_wait(&full_bar[w % kEncStages], (w / kEncStages) & 1, &never);
            feed.drain();
        }
    } else {
        // ------------------------------ consumer warps ------------------------------
        const int tid = threadIdx.x;
        for (uint32_t unit = 0;; ++unit) {
            const int s = unit % kEncStages;
            // every warp polls for itself here: the warps of this kernel's one CTA per SM hand their stage
            // back early and drift apart by design, and a barrier per unit (group_wait) would march them
            // in step again (measured: 25 % slower at 4 and 2 bits)
            if (!mbar_wait(&full_bar[s], (unit / kEncStages) & 1, &abort_flag)) {
                report(p.status, KVH_ERR_TIMEOUT);
                abort_flag = 1;
                break;
            }
            const EncUnit u = info[s];
            if (u.bits == 0) break;
            const uint8_t *st = stage_mem + (size_t)s * kEncStageBytes;
            uint64_t *eb = &empty_bar[s];
            if (u.last && tid < KVH_SECTION_ALIGN) {     // the plane's last tile clears the padding
                if (u.codes_payload + tid < u.codes_padded) u.codes[u.codes_payload + tid] = 0;
                if (u.bits < 16 && u.meta_payload + tid < u.meta_padded) u.meta[u.meta_payload + tid] = 0;
            }
            enc_dispatch<C, LEVEL, WIDE>(u, st, p.c, tid, eb);
        }
    }
}

}  // namespace kvh
