// Transcoding kernel: a stored chunk at level m becomes a stored chunk at a coarser level n > m
// without its bf16 values ever touching HBM.
//
// The policy's marginal-utility step may decide to "compress furthermore" an entry that is already
// in storage.  What is stored is all there is to compress, so the result is defined as the
// encoding at level n of the values the level-m chunk decodes to.  Per element the kernel reads
// (b_m + 1)/8 bytes and writes (b_n + 1)/8 bytes; a decode into a bf16 buffer followed by an encode
// would move 4 more.
//
// Structure: the encode kernel's pipeline (shared-memory stages fed by 1-D bulk copies, tiles
// handed out through cluster launch control, 8 consumer warps) with the decode kernel's unpacking
// in front.  A level-0 source is the encoder itself reading the chunk's raw rows.  From a
// quantised source the new range of every group follows from its old metadata (tc_new_meta), so a
// K thread walks the rows of its 4 channels and a V thread its groups, one at a time: dequantise,
// round to bf16, quantise again, store.  Such instances need few registers and two small stages
// and run three CTAs per SM.  They move about one byte per element and are bound by instruction
// issue, not by memory.
#pragma once

#include "kvh_async.cuh"
#include "kvh_decode_tma.cuh"
#include "kvh_encode_tma.cuh"
#include "kvh_format.cuh"

namespace kvh {

struct TranscodeParams {
    const uint8_t *in;
    uint64_t in_bytes;
    const kvh_chunk_desc *in_descs;     // device, n_chunks
    uint8_t *out;
    uint64_t out_capacity;
    const kvh_chunk_desc *out_descs;    // device, n_chunks
    int32_t l, c;
    int32_t bw, n_blocks;               // channels per column block (c when c <= 1024), blocks per row
    int32_t tpu;                        // 32-token tiles per work unit (1, 2, 4, 8; 1 unless rows are narrow)
    int32_t *status;
};

struct TcUnit {
    EncUnit e;             // what the encoder needs (bits = the output level's)
    int32_t bits_in;       // 16, 8, 4, 2
};

// Offset of a unit's metadata in its stage; the codes (or raw rows) start at 0.  c: channels per
// stage row times the tiles a unit holds.
__host__ __device__ __forceinline__ uint32_t tc_meta_off(int c) { return 32u * (uint32_t)c; }

// q_i * 2^pos(i) for the 4 codes of one K row of a 4-channel column: x[0] = elements 0, 1 and
// x[1] = elements 2, 3 (see spread8()).
template <int BITS>
__device__ __forceinline__ void spread4(const uint8_t *src, f32x2 (&x)[2])
{
    constexpr uint32_t magic = 0x4b000000u;
    uint32_t m[4];
    if constexpr (BITS == 2) {
        const uint32_t w = *src;
        m[0] = and_or<0x03u>(w, magic); m[1] = and_or<0x0cu>(w, magic);
        m[2] = and_or<0x30u>(w, magic); m[3] = and_or<0xc0u>(w, magic);
    } else if constexpr (BITS == 4) {
        const uint32_t w = *reinterpret_cast<const uint16_t *>(src);
        m[0] = and_or<0x000fu>(w, magic); m[1] = and_or<0x00f0u>(w, magic);
        m[2] = and_or<0x0f00u>(w, magic); m[3] = and_or<0xf000u>(w, magic);
    } else {
        const uint32_t w = *reinterpret_cast<const uint32_t *>(src);
#pragma unroll
        for (int i = 0; i < 4; ++i) m[i] = __byte_perm(w, magic, 0x7440 + i);
    }
    const f32x2 bias = f2_from_bits(magic, magic);
    x[0] = f2_sub(f2_from_bits(m[0], m[1]), bias);
    x[1] = f2_sub(f2_from_bits(m[2], m[3]), bias);
}

// A decoded group needs no second look to know its range.  Its smallest element had code 0 and its
// largest code qmax (the quantiser maps min to 0 and max to qmax whatever the rounding), and
// decoding is monotone, so the decoded values span exactly [xhat(0), xhat(qmax)] and the metadata
// word of the re-encoded group follows from the old one alone.  That makes every element
// independent: the kernel streams rows instead of holding a tile in registers.
template <int BIN>
__device__ __forceinline__ uint32_t tc_new_meta(uint32_t m, float &lo, float &scale)
{
    decode_params<BIN>(m, lo, scale);
    const float qmax = (float)((1 << BIN) - 1);
    return pack_bf16x2_rn(__fmaf_rn(0.0f, scale, lo), __fmaf_rn(qmax, scale, lo));      // xhat(0) | xhat(qmax) << 16
}

// binary32 value of bf16_rne(x): the conversion of a pair whose other half is zero leaves exactly
// that bit pattern (bf16 in the upper half, zeros below)
__device__ __forceinline__ uint32_t round_to_bf16_bits(float x)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(x), "f"(0.0f));
    return r;
}
__device__ __forceinline__ f32x2 round_to_bf16(f32x2 v)
{
    uint32_t a, b;
    f2_bits(v, a, b);
    return f2_from_bits(round_to_bf16_bits(__uint_as_float(a)), round_to_bf16_bits(__uint_as_float(b)));
}

// One K row of a 4-channel column: unpack, dequantise, round to bf16 (the values stay binary32: no
// packing and unpacking in between), quantise at the new level, store.
template <int BIN, int BOUT>
__device__ __forceinline__ void tc_row_k(const uint8_t *codes, const f32x2 (&lo)[2], const f32x2 (&sc)[2], f32x2 lo_a,
                                         f32x2 lo_b, f32x2 inv_a, f32x2 inv_b, uint8_t *o)
{
    f32x2 q[2];
    spread4<BIN>(codes, q);
    enc_store_row_k_f32<BOUT>(round_to_bf16(f2_fma(q[0], sc[0], lo[0])), round_to_bf16(f2_fma(q[1], sc[1], lo[1])), lo_a, lo_b,
                              inv_a, inv_b, o);
}

// K: a thread owns 4 channels of one of the unit's tiles and walks that tile's rows (any number of
// them; a whole tile's 32 rows unrolled).  A channel stored flat at the new level has inv = 0 and
// decoded values all equal to its min (its old range was below the threshold, or so large that the
// new one overflowed: then its old scale was 0 as well), so value - min is 0 and the code 0 without
// any masking.
template <int BIN, int BOUT>
__device__ __forceinline__ void tc_consume_k(const uint8_t *st, RowGeom g, int tid, uint64_t *empty_bar,
                                             int nt_unit, int tile0, int tpu, uint8_t *meta_sec, uint8_t *codes_sec)
{
    const int c = g.cw;                                  // channels per stage row
    const int C4 = c >> 2;
    const int sub = tid / C4;                            // which of the unit's tiles
    const int nt = min(kTileTokens, nt_unit - sub * kTileTokens);
    if (nt > 0) {
        const int cq = tid - sub * C4;
        const int tile = tile0 + sub;
        const uint4 w4 = *reinterpret_cast<const uint4 *>(st + tc_meta_off(c * tpu) + 4 * (size_t)sub * c + 16 * (size_t)cq);
        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
        float l1[4], s1[4], lo_new[4], inv[4];
        uint32_t m[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            m[i] = tc_new_meta<BIN>(w[i], l1[i], s1[i]);
            if constexpr (BIN != 8) s1[i] = __fmul_rn(s1[i], Pos<BIN>::prescale(i));
            encode_params<BOUT>(m[i], lo_new[i], inv[i]);
        }
        uint4 *meta_out;
        uint8_t *out;
        uint32_t out_bytes;
        enc_k_out<BOUT>(g, cq, tile, meta_sec, codes_sec, meta_out, out, out_bytes);
        *meta_out = make_uint4(m[0], m[1], m[2], m[3]);
        const f32x2 lo[2] = {f2_make(l1[0], l1[1]), f2_make(l1[2], l1[3])};
        const f32x2 sc[2] = {f2_make(s1[0], s1[1]), f2_make(s1[2], s1[3])};
        const f32x2 lo_a = f2_make(lo_new[0], lo_new[1]), lo_b = f2_make(lo_new[2], lo_new[3]);
        const f32x2 inv_a = f2_make(inv[0], inv[1]), inv_b = f2_make(inv[2], inv[3]);
        const uint32_t in_bytes = (uint32_t)c * BIN / 8;
        const uint8_t *src = st + (size_t)sub * kTileTokens * in_bytes + (size_t)cq * BIN / 2;   // 4 codes = BIN / 2 bytes
        if (nt == kTileTokens) {
#pragma unroll
            for (int t = 0; t < kTileTokens; ++t)
                tc_row_k<BIN, BOUT>(src + (size_t)t * in_bytes, lo, sc, lo_a, lo_b, inv_a, inv_b, out + (size_t)t * out_bytes);
        } else {
#pragma unroll 1
            for (int t = 0; t < nt; ++t)
                tc_row_k<BIN, BOUT>(src + (size_t)t * in_bytes, lo, sc, lo_a, lo_b, inv_a, inv_b, out + (size_t)t * out_bytes);
        }
    }
    enc_release(empty_bar);
}

// V: a thread dequantises whole groups (32 codes, one metadata word) and encodes them again.
template <int BIN, int BOUT>
__device__ __forceinline__ void tc_consume_v(const uint8_t *st, RowGeom geom, int tid, uint64_t *empty_bar,
                                             int nt, int tile, int tpu, uint8_t *meta_sec, uint8_t *codes_sec)
{
    const int ngroups = nt * (geom.cw >> 5);             // the unit's groups, in stage order
    const uint32_t *meta_in = reinterpret_cast<const uint32_t *>(st + tc_meta_off(geom.cw * tpu));
    uint32_t *meta = reinterpret_cast<uint32_t *>(meta_sec);
    const f32x2 pre01 = f2_make(Pos<BIN>::prescale(0), Pos<BIN>::prescale(1));
    const f32x2 pre23 = f2_make(Pos<BIN>::prescale(2), Pos<BIN>::prescale(3));
    constexpr int W = BOUT == 8 ? 2 : 1;
#pragma unroll 2
    for (int g = tid; g < ngroups; g += kEncGroupThreads) {
        float l1, s0, lo_new, inv;
        const uint32_t m = tc_new_meta<BIN>(meta_in[g], l1, s0);
        encode_params<BOUT>(m, lo_new, inv);
        const f32x2 ss = f2_make(s0, s0), ll = f2_make(l1, l1);
        f32x2 sa = ss, sb = ss;
        if constexpr (BIN != 8) { sa = f2_mul(ss, pre01); sb = f2_mul(ss, pre23); }     // exact: powers of two
        const f32x2 sc[4] = {sa, sb, sa, sb};
        const f32x2 lo2 = f2_make(lo_new, lo_new), inv2 = f2_make(inv, inv);
        const uint8_t *src = st + (size_t)g * (4 * BIN);  // 32 codes = 4 * BIN bytes
        uint32_t p[4][W];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // a group stored flat at the new level decodes to its min everywhere: value - min = 0, code 0
            f32x2 q[4], x[4];
            spread8<BIN>(src + j * BIN, q);
#pragma unroll
            for (int k = 0; k < 4; ++k) x[k] = round_to_bf16(f2_fma(q[k], sc[k], ll));
            enc_piece_v_f32<BOUT, W>(x, lo2, inv2, p[j]);
        }
        const size_t gi = enc_v_group_index(geom, tile, g);
        meta[gi] = m;
        enc_store_group_v<BOUT, W>(p, codes_sec + gi * (4 * BOUT));
    }
    enc_release(empty_bar);
}

// One unit with both levels known at compile time (LOUT > LIN).
template <int C, int LIN, int LOUT>
__device__ __forceinline__ void tc_consume_levels(const EncUnit &u, const uint8_t *st, int c_rt, int tpu_rt, int tid,
                                                  uint64_t *eb)
{
    if constexpr (LIN == 0) {
        enc_consume_level<C, LOUT>(u, st, c_rt, tid, eb);            // raw rows: the encoder as it is
    } else {
        constexpr int BIN = 16 >> LIN, BOUT = 16 >> LOUT;
        const RowGeom g = row_geom<C>(u.cw, c_rt, u.col0);
        const int tpu = C ? 1 : tpu_rt;
        if (u.kv) tc_consume_v<BIN, BOUT>(st, g, tid, eb, u.nt, u.tile, tpu, u.meta, u.codes);
        else tc_consume_k<BIN, BOUT>(st, g, tid, eb, u.nt, u.tile, tpu, u.meta, u.codes);
    }
}
template <int C, int LIN, int LOUT>
__device__ __noinline__ void tc_consume_levels_call(const EncUnit *u, const uint8_t *st, int c_rt, int tpu_rt, int tid,
                                                    uint64_t *eb)
{
    tc_consume_levels<C, LIN, LOUT>(*u, st, c_rt, tpu_rt, tid, eb);
}

// LIN, LOUT >= 0: every chunk goes from LIN to LOUT (checked by the producer); -1: any mix.
template <int C, int LIN, int LOUT>
__device__ __forceinline__ void tc_dispatch(const TcUnit &u, const uint8_t *st, int c_rt, int tpu_rt, int tid,
                                            uint64_t *eb)
{
    if constexpr (LIN >= 0) {
        tc_consume_levels<C, LIN, LOUT>(u.e, st, c_rt, tpu_rt, tid, eb);
    } else {
        switch (u.bits_in * 16 + u.e.bits) {             // uniform per CTA
        case 16 * 16 + 8: tc_consume_levels_call<C, 0, 1>(&u.e, st, c_rt, tpu_rt, tid, eb); break;
        case 16 * 16 + 4: tc_consume_levels_call<C, 0, 2>(&u.e, st, c_rt, tpu_rt, tid, eb); break;
        case 16 * 16 + 2: tc_consume_levels_call<C, 0, 3>(&u.e, st, c_rt, tpu_rt, tid, eb); break;
        case 8 * 16 + 4: tc_consume_levels_call<C, 1, 2>(&u.e, st, c_rt, tpu_rt, tid, eb); break;
        case 8 * 16 + 2: tc_consume_levels_call<C, 1, 3>(&u.e, st, c_rt, tpu_rt, tid, eb); break;
        default: tc_consume_levels_call<C, 2, 3>(&u.e, st, c_rt, tpu_rt, tid, eb); break;
        }
    }
}

// sched as in the encode kernel.  One CTA per SM: 8 consumer warps and a producer warp.
// Bytes of a stage: a raw tile (64 KiB at c = 1024) when the source may be level 0, else codes of at
// most 8 bits plus metadata (36 KiB); two of those per CTA leave room for three CTAs per SM.
template <int LIN>
__host__ __device__ constexpr uint32_t tc_stage_bytes() { return LIN >= 1 ? 36u * 1024u : kEncStageBytes; }
// Stages per CTA: two of them leave room for three CTAs per SM when the source is quantised.
template <int LIN>
__host__ __device__ constexpr int tc_stages() { return LIN >= 1 ? 2 : kEncStages; }

template <int C, int LIN, int LOUT, typename Chunks>
__global__ void __launch_bounds__(32 + kEncGroupThreads, LIN >= 1 ? 3 : 1)
transcode_tma_kernel(const TranscodeParams p, const int n_chunks, const int sched, const Chunks chunks)
{
    constexpr int kStages = tc_stages<LIN>();
    extern __shared__ __align__(128) uint8_t stage_mem[];
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ TcUnit info[kStages];
    __shared__ int abort_flag;
    __shared__ int wait_verdict[2];
    __shared__ __align__(16) uint4 clc_response[2];
    __shared__ __align__(8) uint64_t clc_bar[2];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kProducerWarp = kEncGroupThreads / 32;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
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
        const int tpu = C ? 1 : p.tpu;                    // tiles per unit
        const int upc = kTilesPerChunk / tpu;             // units per chunk and plane
        const int64_t total_tiles = (int64_t)n_chunks * p.l * 2 * upc * p.n_blocks;
        uint32_t unit = 0;
        bool ok = true;
        int cur_chunk = -1;
        bool valid = false;
        kvh_chunk_desc di{}, dout{};
        LayerLayout Li = layer_layout(0, p.c, 1), Lo = Li;

        auto acquire = [&]() -> bool {                   // wait until the unit's stage is free
            const int s = unit % kStages;
            if (unit < (uint32_t)kStages) return true;
            bool w = true;
            if (lane == 0) w = mbar_wait(&empty_bar[s], ((unit / kStages) - 1) & 1, &abort_flag);
            return __shfl_sync(0xffffffffu, w, 0);
        };

        auto do_tile = [&](int64_t tile_id) {
            // a tile id fits 32 bits (the host refuses larger launches): unsigned 32-bit divisions
            const uint32_t id = (uint32_t)tile_id;
            const uint32_t nb = (uint32_t)p.n_blocks, units = (uint32_t)upc;
            const int cb = (int)(id % nb);                       // column block (rows wider than 1024 channels)
            const uint32_t row_tile = id / nb;
            const int tile = (int)(row_tile % units) * tpu;      // the unit's first tile
            const uint32_t plane_id = row_tile / units;
            const int kv = (int)(plane_id & 1);
            const int layer = (int)((plane_id >> 1) % (uint32_t)p.l);
            const int chunk = chunks.chunk((int)((plane_id >> 1) / (uint32_t)p.l), 0);
            if (chunk != cur_chunk) {
                cur_chunk = chunk;
                di = p.in_descs[chunk];
                dout = p.out_descs[chunk];
                int err = check_desc(di, p.l, p.c, p.in_bytes);
                if (err == KVH_OK) err = check_desc(dout, p.l, p.c, p.out_capacity);
                if (err == KVH_OK && di.n_tok != dout.n_tok) err = KVH_ERR_BAD_SHAPE;
                if (err == KVH_OK && dout.level <= di.level) err = KVH_ERR_BAD_LEVEL;   // only towards coarser levels
                if (err == KVH_OK && LIN >= 0 && (di.level != LIN || dout.level != LOUT)) err = KVH_ERR_BAD_LEVEL;
                valid = err == KVH_OK;
                if (!valid) {
                    if (lane == 0) report(p.status, err);
                } else {
                    Li = layer_layout(di.level, p.c, di.n_tok);
                    Lo = layer_layout(dout.level, p.c, dout.n_tok);
                }
            }
            if (!valid) return;
            const int n = di.n_tok;
            const int t0 = tile * kTileTokens;
            const int nt = min(kTileTokens * tpu, n - t0);
            if (nt <= 0) return;
            const uint8_t *lay_in = p.in + di.stream_off + (uint64_t)layer * Li.layer_bytes();
            uint8_t *lay_out = p.out + dout.stream_off + (uint64_t)layer * Lo.layer_bytes();
            ok = acquire();
            if (!ok) return;
            const int s = unit % kStages;
            uint8_t *st = stage_mem + (size_t)s * tc_stage_bytes<LIN>();
            const bool wide = p.n_blocks > 1;
            const int col0 = cb * p.bw;
            const uint32_t gpr = (uint32_t)p.c / kGroup;         // groups per plane row
            const int b = level_bits(di.level);
            // the block's codes (or raw rows) of row r: row_bytes at csrc + r * row_stride; its metadata: one
            // piece of 4 * bw bytes for K, one piece of bw / 8 bytes per row for V
            const uint8_t *csrc = lay_in + Li.codes_off(kv) + ((uint64_t)t0 * p.c + col0) * b / 8;
            const uint32_t row_bytes = (uint32_t)p.bw * b / 8, row_stride = (uint32_t)p.c * b / 8;
            const uint8_t *meta_in = lay_in + Li.meta_off(kv);
            const uint8_t *msrc = kv == 0 ? meta_in + 4 * ((uint64_t)tile * p.c + col0)
                                          : meta_in + 4 * ((uint64_t)t0 * gpr + col0 / kGroup);
            const uint32_t mrow_bytes = 4u * (p.bw / kGroup), mrow_stride = 4u * gpr;
            if (lane == 0) {
                TcUnit &u = info[s];
                u.bits_in = b;
                u.e.bits = level_bits(dout.level); u.e.kv = kv; u.e.nt = nt; u.e.tile = tile;
                u.e.last = t0 + nt == n && cb == p.n_blocks - 1;
                u.e.meta_payload = (uint32_t)(kv ? Lo.vmeta_payload : Lo.kmeta_payload);
                u.e.meta_padded = (uint32_t)(kv ? Lo.vmeta : Lo.kmeta);
                u.e.codes_payload = (uint32_t)Lo.codes_payload;
                u.e.codes_padded = (uint32_t)Lo.kcodes;
                u.e.meta = lay_out + Lo.meta_off(kv);
                u.e.codes = lay_out + Lo.codes_off(kv);
                u.e.col0 = col0; u.e.cw = p.bw;
                if (!wide) {
                    const uint32_t cbytes = round16((uint32_t)nt * row_bytes);
                    const uint32_t mbytes = di.level == 0 ? 0u
                                          : kv == 0     ? 4u * p.c * ((nt + kTileTokens - 1) / kTileTokens)
                                                        : round16((uint32_t)nt * mrow_bytes);
                    mbar_arrive_expect_tx(&full_bar[s], cbytes + mbytes);
                    bulk_load(st, csrc, cbytes, &full_bar[s]);
                    if (mbytes) bulk_load(st + tc_meta_off(p.bw * tpu), msrc, mbytes, &full_bar[s]);
                } else {
                    const uint32_t mbytes = di.level == 0 ? 0u : kv == 0 ? 4u * p.bw : (uint32_t)nt * mrow_bytes;
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)nt * row_bytes + mbytes);
                    if (di.level != 0 && kv == 0) bulk_load(st + tc_meta_off(p.bw), msrc, 4u * p.bw, &full_bar[s]);
                }
            }
            if (wide) {                                  // lane r copies row r's pieces (the expectation is posted first)
                __syncwarp();
                if (lane < nt) {
                    bulk_load(st + (size_t)lane * row_bytes, csrc + (size_t)lane * row_stride, row_bytes, &full_bar[s]);
                    if (di.level != 0 && kv == 1)
                        bulk_load(st + tc_meta_off(p.bw) + (size_t)lane * mrow_bytes, msrc + (size_t)lane * mrow_stride,
                                  mrow_bytes, &full_bar[s]);
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
                info[unit % kStages].e.bits = 0;
                mbar_arrive(&full_bar[unit % kStages]);
            }
            ++unit;
        }
        if (!ok && lane == 0) {
            report(p.status, KVH_ERR_TIMEOUT);
            abort_flag = 1;
        }
        // Leave only after every copy issued has landed (see the encode kernel).
        if (lane == 0) {
            int never = 0;
            const uint32_t first = unit > (uint32_t)kStages ? unit - kStages : 0;
            for (uint32_t w = first; w < unit; ++w)
                (void)mbar_wait(&full_bar[w % kStages], (w / kStages) & 1, &never);
            feed.drain();
        }
    } else {
        // ------------------------------ consumer warps ------------------------------
        const int tid = threadIdx.x;
        for (uint32_t unit = 0;; ++unit) {
            const int s = unit % kStages;
            // quantised sources: three CTAs per SM, so one polling warp per CTA and a named barrier for the
            // rest (group_wait); a level-0 source is the encoder's one CTA per SM, whose warps drift apart by
            // design and poll for themselves
            bool ready;
            if constexpr (LIN >= 1) {
                ready = group_wait(&full_bar[s], (unit / kStages) & 1, &abort_flag, wait_verdict, unit, 1, kEncGroupThreads,
                                   warp == 0);
            } else {
                ready = mbar_wait(&full_bar[s], (unit / kStages) & 1, &abort_flag);
                if (!ready) abort_flag = 1;
            }
            if (!ready) {
                if (LIN < 1 || tid == 0) report(p.status, KVH_ERR_TIMEOUT);
                break;
            }
            const TcUnit u = info[s];
            if (u.e.bits == 0) break;
            const uint8_t *st = stage_mem + (size_t)s * tc_stage_bytes<LIN>();
            if (u.e.last && tid < KVH_SECTION_ALIGN) {   // the plane's last tile clears the padding
                if (u.e.codes_payload + tid < u.e.codes_padded) u.e.codes[u.e.codes_payload + tid] = 0;
                if (u.e.meta_payload + tid < u.e.meta_padded) u.e.meta[u.e.meta_payload + tid] = 0;
            }
            tc_dispatch<C, LIN, LOUT>(u, st, p.c, p.tpu, tid, &empty_bar[s]);
        }
    }
}

}  // namespace kvh
