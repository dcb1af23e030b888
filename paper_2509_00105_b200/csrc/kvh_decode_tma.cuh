// Persistent, TMA-fed decode kernel (pages of >= 8 tokens; rows of up to 1024 channels, or wider
// rows that divide into equal column blocks, which are fed with one bulk copy per row).
//
// Three CTAs per SM loop over work units.  A producer warp walks the CTA's share of
// (layer, K|V, chunk, 32-token tile) tiles, resolves descriptors and page ids, and streams each
// unit's codes and group metadata from HBM into shared-memory stages with 1-D bulk async copies
// (cp.async.bulk, completion counted on an mbarrier).  Eight consumer warps unpack, dequantise and
// write full 16-byte vectors of page rows, row step by row step in lockstep.  Copies for the next
// units are always in flight while the current one is being expanded, and the kernel runs at the
// speed of its writes (2 of the (b+1)/8 + 2 bytes moved per element).
//
// A unit is a 32-token tile of a quantised plane (32*c*b/8 bytes of codes + 4*c bytes of metadata)
// or one 16-token half of a raw bf16 tile (32*c bytes).  Rows of at most 512 channels would leave
// threads idle and make units small, so there a unit takes 2, 4 or 8 consecutive tiles of the plane
// (DecodeParams::tpu; codes and metadata of consecutive tiles are contiguous in the stream).
//
// Stages are cut from a ring of quanta of 12*c bytes, as many per unit as its level needs: one at
// 2 bits, two at 4 bits, three at 8 bits and for a raw half tile.  With the 72 KiB a CTA has at
// c = 1024 that is 6 units in flight at 2 bits, 3 at 4 bits and 2 at 8 bits or raw, whatever the
// mix of levels in the launch.  The kernel is bound by memory and its CTAs by the latency of their
// copies, so the more bytes a CTA has on their way, the less often its consumers stand idle.
//
// Every wait is bounded: a wait that runs out reports KVH_ERR_TIMEOUT, raises the CTA's abort
// flag and the CTA leaves after its copies in flight have landed.
#pragma once

#include "kvh_async.cuh"
#include "kvh_decode.cuh"
#include "kvh_format.cuh"

namespace kvh {

constexpr int kConsumerThreads = 256;
constexpr int kTmaThreads = kConsumerThreads + 32;      // + one producer warp
constexpr int kSlots = 8;                               // units a CTA can have between producer and consumers
constexpr int kMaxQuanta = 24;
constexpr int kTmaMaxChannels = 1024;

struct UnitInfo {
    int32_t bits;        // 16, 8, 4, 2; 0 marks the end of the CTA's work
    int32_t kv;          // 0 K, 1 V
    int32_t row0;        // first token of the unit within its chunk
    int32_t nrows;       // tokens in the unit (1..32 * tpu)
    int32_t pg[4];       // page ids of the page holding row0 and of the next three (pages hold >= 8 tokens)
    const int32_t *pgs;  // the same and up to 12 more, in shared memory (units of several tiles)
    uint16_t *plane;     // pool + layer*layer_stride + kv*kv_stride
    int32_t col0, cw;    // first channel and width of the unit's column block (0, c unless rows exceed 1024 channels)
    uint32_t st_off;     // where the unit's codes (or raw rows) start in the CTA's stage memory
    uint32_t meta_off;   // its metadata, from there
};

// One quantum of stage memory, for units of c channels (times the tiles a unit holds): the codes of a
// 32-token tile at 2 bits (8*c bytes) and its metadata (4*c bytes).
__host__ __device__ __forceinline__ uint32_t tma_quantum_bytes(int c) { return (12u * (uint32_t)c + 127u) & ~127u; }
// Quanta a unit takes: its codes (bits 2, 4, 8) or raw rows (16: half a tile) plus 4*c bytes of metadata.
__host__ __device__ __forceinline__ int unit_quanta(int bits) { return bits == 0 ? 0 : bits == 2 ? 1 : bits == 4 ? 2 : 3; }
// Quanta of a CTA's ring: what 72 KiB hold (three CTAs per SM), at least the 6 that let any unit in.
__host__ __device__ __forceinline__ int ring_quanta(int c)
{
    const int q = (int)((72u * 1024u) / tma_quantum_bytes(c));
    return q < 6 ? 6 : (q > kMaxQuanta ? kMaxQuanta : q);
}

// The producer's book-keeping of the ring.  Units take their quanta at `head`, in order, as one
// contiguous run: a unit that does not fit before the ring's end starts at 0 and takes the quanta
// left before the end along with it (they come back when it does).  Quanta return in the order
// they were taken (the consumers release units in order), so the free quanta are always the one
// circular run from `head` to the oldest unit still held, and "enough free quanta" is all that has
// to be checked.  With at least 6 quanta and units of at most 3, an empty ring takes any unit.
struct QuantaRing {
    int n_quanta, head, free_q;
    __host__ __device__ explicit QuantaRing(int n) : n_quanta(n), head(0), free_q(n) {}
    // quanta given up before the ring's end so that `need` of them are contiguous
    __host__ __device__ int skipped(int need) const { return head + need > n_quanta ? n_quanta - head : 0; }
    __host__ __device__ bool fits(int need) const { return free_q >= need + skipped(need); }
    // Takes `need` contiguous quanta (fits(need) must hold): returns the index of the first and, in
    // held, how many the unit keeps until it is given back (need + the ones skipped).
    __host__ __device__ int take(int need, int &held)
    {
        const int skip = skipped(need);
        if (skip) head = 0;
        const int at = head;
        head += need;
        if (head == n_quanta) head = 0;
        held = need + skip;
        free_q -= held;
        return at;
    }
    __host__ __device__ void give_back(int held) { free_q += held; }
};
__host__ __device__ __forceinline__ uint32_t round16(uint32_t x) { return (x + 15u) & ~15u; }

// ---- dequantisation of 8 consecutive codes with few instructions per element ----------------
//
// A code is never shifted down to bit 0.  For 2- and 4-bit codes the field is masked in place and
// OR-ed into the mantissa of 2^23 (one logic op), so subtracting 2^23 leaves q * 2^pos exactly;
// the group's scale is pre-multiplied by 2^-pos (exact: a power of two, and scales are >= 2^-108
// or zero), hence fma(q * 2^pos, scale * 2^-pos, lo) has the same exact product, the same single
// rounding and the same result as fma(q, scale, lo).  8-bit codes are placed by a byte permute.
template <int BITS> struct Pos;
template <> struct Pos<2> {      // fields of the low byte of a 16-bit half: bits 0, 2, 4, 6
    static constexpr int kFieldsPerWord = 4;
    __device__ static __forceinline__ float prescale(int i) { return 1.0f / (float)(1 << (2 * (i & 3))); }
};
template <> struct Pos<4> {      // fields of a 16-bit half: bits 0, 4, 8, 12
    static constexpr int kFieldsPerWord = 4;
    __device__ static __forceinline__ float prescale(int i) { return 1.0f / (float)(1 << (4 * (i & 3))); }
};
template <> struct Pos<8> {
    static constexpr int kFieldsPerWord = 4;
    __device__ static __forceinline__ float prescale(int) { return 1.0f; }
};

// (a & mask) | c in one logic instruction (mask an immediate)
template <uint32_t MASK>
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "n"(MASK), "r"(c));
    return d;
}

// q_i * 2^pos(i) as floats, for i = 0..7, from the 8 codes of one thread: x[k] holds elements 2k and
// 2k+1 (the subtraction of 2^23 is exact, two elements per instruction)
template <int BITS>
__device__ __forceinline__ void spread8(const uint8_t *src, f32x2 (&x)[4])
{
    constexpr uint32_t magic = 0x4b000000u;
    uint32_t m[8];
    if constexpr (BITS == 2) {
        // one logic op per code: the field is masked where it stands and lands in the mantissa of 2^23
        const uint32_t w = *reinterpret_cast<const uint16_t *>(src);
        const uint32_t t = w >> 8;
        m[0] = and_or<0x03u>(w, magic); m[1] = and_or<0x0cu>(w, magic);
        m[2] = and_or<0x30u>(w, magic); m[3] = and_or<0xc0u>(w, magic);
        m[4] = and_or<0x03u>(t, magic); m[5] = and_or<0x0cu>(t, magic);
        m[6] = and_or<0x30u>(t, magic); m[7] = and_or<0xc0u>(t, magic);
    } else if constexpr (BITS == 4) {
        const uint32_t w = *reinterpret_cast<const uint32_t *>(src);
        const uint32_t t = w >> 16;
        m[0] = and_or<0x000fu>(w, magic); m[1] = and_or<0x00f0u>(w, magic);
        m[2] = and_or<0x0f00u>(w, magic); m[3] = and_or<0xf000u>(w, magic);
        m[4] = and_or<0x000fu>(t, magic); m[5] = and_or<0x00f0u>(t, magic);
        m[6] = and_or<0x0f00u>(t, magic); m[7] = and_or<0xf000u>(t, magic);
    } else {
        const uint2 w = *reinterpret_cast<const uint2 *>(src);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            m[i] = __byte_perm(w.x, magic, 0x7440 + i);       // bytes: code, 0, 0, 0x4b
            m[i + 4] = __byte_perm(w.y, magic, 0x7440 + i);
        }
    }
    const f32x2 bias = f2_from_bits(magic, magic);
#pragma unroll
    for (int k = 0; k < 4; ++k) x[k] = f2_sub(f2_from_bits(m[2 * k], m[2 * k + 1]), bias);
}

// bf16_rne of x[k] * sc[k] + lo[k] for the 8 elements, one rounding each
__device__ __forceinline__ uint4 fma_pack8(const f32x2 (&x)[4], const f32x2 (&sc)[4], const f32x2 (&lo)[4])
{
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        uint32_t a, b;
        f2_bits(f2_fma(x[k], sc[k], lo[k]), a, b);
        w[k] = pack_bf16x2_rn(__uint_as_float(a), __uint_as_float(b));
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Rows of a unit are dealt to threads in runs of consecutive rows: `rpt` rows per thread (a power of
// two, at most 16: 16 when c = 1024), cut into runs of at most a page, so that a run never straddles
// a page or a tile; `cv` is the thread's 8-channel vector within the row.
struct RowRun {
    int cv, first, count;       // count == 0 for idle threads
    uint16_t *dst;              // first row's destination (already offset by cv), nullptr if none
};
struct RowRuns {
    int cv, g, rpp, len, n;     // thread's vector and row group; row groups; rows per run; runs per thread
};

// SMALLPG: pages may hold fewer tokens than a thread has rows (8-token pages); otherwise a thread
// has one run and a tile at most two pages, which the compiler then knows.
template <int C, bool SMALLPG>
__device__ __forceinline__ RowRuns row_runs(const DecodeParams &p, const UnitInfo &u)
{
    const int V8 = (C ? C : u.cw) >> 3;                   // 16-byte vectors per stage row, <= 128
    RowRuns rr;
    rr.rpp = kConsumerThreads / V8;                       // row groups the CTA holds, >= 2
    int rpt = 1;
    const int unit_rows = kTileTokens * (C ? 1 : p.tpu);
    while (rpt * rr.rpp < unit_rows) rpt <<= 1;           // rows per thread
    rr.len = SMALLPG ? min(rpt, p.page_tokens) : rpt;
    rr.n = SMALLPG ? rpt / rr.len : 1;
    rr.g = threadIdx.x / V8;
    rr.cv = threadIdx.x - rr.g * V8;
    return rr;
}

// Run i of the thread: rows [first, first + count) of the unit.
template <int C, bool SMALLPG>
__device__ __forceinline__ RowRun row_run(const DecodeParams &p, const UnitInfo &u, const RowRuns &rr, int i)
{
    RowRun r;
    r.cv = rr.cv;
    r.first = (i * rr.rpp + rr.g) * rr.len;
    r.count = rr.g < rr.rpp ? max(0, min(rr.len, u.nrows - r.first)) : 0;
    r.dst = nullptr;
    if (r.count > 0) {
        const int T = u.row0 + r.first;
        const int pi = (T >> p.page_shift) - (u.row0 >> p.page_shift);
        int32_t pg;
        if constexpr (C == 0 && !SMALLPG) pg = u.pgs[pi];                   // 0..15: a unit of up to 8 tiles
        else pg = pi == 0 ? u.pg[0] : (!SMALLPG || pi == 1) ? u.pg[1] : pi == 2 ? u.pg[2] : u.pg[3];   // selects keep u in registers
        r.dst = page_row<C>(p, pg, u.plane, T);              // reports an out-of-range page id
        if (r.dst) r.dst += (C ? 0 : u.col0) + 8 * r.cv; else r.count = 0;
    }
    return r;
}

template <int C, bool SMALLPG>
__device__ __forceinline__ void consume_raw(const DecodeParams &p, const UnitInfo &u, const uint8_t *codes)
{
    const int cw = C ? C : u.cw;                          // row width in the stage
    const int sstride = cw >> 3, dstride = (C ? C : p.c) >> 3;    // uint4 per stage row / per page row
    const RowRuns rr = row_runs<C, SMALLPG>(p, u);
    for (int i = 0; i < rr.n; ++i) {
        const RowRun r = row_run<C, SMALLPG>(p, u, rr, i);
        const uint4 *src = reinterpret_cast<const uint4 *>(codes + 2 * ((size_t)r.first * cw + 8 * r.cv));
        uint4 *dst = reinterpret_cast<uint4 *>(r.dst);
#pragma unroll 4
        for (int k = 0; k < r.count; ++k) dst[(size_t)k * dstride] = src[(size_t)k * sstride];
    }
}

template <int BITS, int C, bool SMALLPG>
__device__ __forceinline__ void consume_k(const DecodeParams &p, const UnitInfo &u, const uint8_t *codes,
                                          const uint8_t *meta)
{
    const int c = C ? C : u.cw;                           // row width in the stage
    const int dstride = C ? C : p.c;                      // row width of a page
    const RowRuns rr = row_runs<C, SMALLPG>(p, u);
    if (rr.g >= rr.rpp || rr.g * rr.len >= u.nrows) return;     // no rows: no metadata of a tile to read either
    f32x2 lo[4], sc[4];
    {
        // the thread's rows lie in one tile of the unit: that tile's groups
        const int sub = (C || SMALLPG) ? 0 : (rr.g * rr.len) >> 5;
        const uint4 *m = reinterpret_cast<const uint4 *>(meta + (size_t)sub * 4 * c) + 2 * rr.cv;
        const uint4 m0 = m[0], m1 = m[1];
        const uint32_t w[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
        float l1[8], s1[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            decode_params<BITS>(w[i], l1[i], s1[i]);
            if constexpr (BITS != 8) s1[i] = __fmul_rn(s1[i], Pos<BITS>::prescale(i));
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            lo[k] = f2_make(l1[2 * k], l1[2 * k + 1]);
            sc[k] = f2_make(s1[2 * k], s1[2 * k + 1]);
        }
    }
    const uint32_t row_bytes = (uint32_t)c * BITS / 8;
    for (int i = 0; i < rr.n; ++i) {
        const RowRun r = row_run<C, SMALLPG>(p, u, rr, i);
        const uint8_t *src = codes + (size_t)r.first * row_bytes + (size_t)r.cv * BITS;
        uint16_t *dst = r.dst;
#pragma unroll 4
        for (int k = 0; k < r.count; ++k) {
            f32x2 x[4];
            spread8<BITS>(src, x);
            *reinterpret_cast<uint4 *>(dst) = fma_pack8(x, sc, lo);
            src += row_bytes;
            dst += dstride;
        }
    }
}

template <int BITS, int C, bool SMALLPG>
__device__ __forceinline__ void consume_v(const DecodeParams &p, const UnitInfo &u, const uint8_t *codes,
                                          const uint8_t *meta)
{
    const int c = C ? C : u.cw;                           // row width in the stage
    const int dstride = C ? C : p.c;                      // row width of a page
    const RowRuns rr = row_runs<C, SMALLPG>(p, u);
    const int lane = threadIdx.x & 31;
    const uint32_t quad = 0xfu << (lane & ~3);            // the 4 lanes that share every V group
    const int groups = c / kGroup;
    const uint32_t row_bytes = (uint32_t)c * BITS / 8;
    const f32x2 pre01 = f2_make(Pos<BITS>::prescale(0), Pos<BITS>::prescale(1));
    const f32x2 pre23 = f2_make(Pos<BITS>::prescale(2), Pos<BITS>::prescale(3));
    for (int i = 0; i < rr.n; ++i) {
        const RowRun r = row_run<C, SMALLPG>(p, u, rr, i);
        const uint32_t *mrow = reinterpret_cast<const uint32_t *>(meta) + (size_t)r.first * groups + (r.cv >> 2);
        const uint8_t *src = codes + (size_t)r.first * row_bytes + (size_t)r.cv * BITS;
        uint16_t *dst = r.dst;
        // r.count is the same for the 4 lanes of a quad (they share the row group and the page), so
        // the shuffles below are executed by whole quads
        for (int kb = 0; kb < r.count; kb += 4) {
            // each lane of the quad derives the scale of one of the next 4 rows: a quarter of a
            // division per row and lane
            float mine = 0.0f, unused;
            const int kq = kb + (lane & 3);
            if (kq < r.count) decode_params<BITS>(mrow[(size_t)kq * groups], unused, mine);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (kb + j < r.count) {
                    const float s0 = __shfl_sync(quad, mine, (lane & ~3) | j);
                    const float l1 = bf16_lo_to_f32(mrow[(size_t)(kb + j) * groups]);
                    const f32x2 ss = f2_make(s0, s0);
                    f32x2 sa = ss, sb = ss;                  // at 8 bits a code sits at bit 0: nothing to undo
                    if constexpr (BITS != 8) { sa = f2_mul(ss, pre01); sb = f2_mul(ss, pre23); }   // exact: powers of two
                    const f32x2 ll = f2_make(l1, l1);
                    const f32x2 sc[4] = {sa, sb, sa, sb}, lo[4] = {ll, ll, ll, ll};
                    f32x2 x[4];
                    spread8<BITS>(src, x);
                    *reinterpret_cast<uint4 *>(dst) = fma_pack8(x, sc, lo);
                    src += row_bytes;
                    dst += dstride;
                }
            }
        }
    }
}

// ---- full tiles at a compiled-in row width, pages of at least 16 tokens -----------------------
//
// Nearly every unit is one of these, and for them everything but the data is a constant, so the row
// loop unrolls completely, every shared-memory and global offset is an immediate, and no row needs a
// branch or an address computation.
//
// The order of the stores matters as much as their number.  The 8 warps take the tile's rows in
// steps: at step k the CTA's G row groups (G = 2 at c = 1024) write rows kG .. kG + G - 1, each warp
// 512 contiguous bytes of one of them, so that one step lays down G whole rows, 4 KiB in a piece at
// c = 1024; and a named barrier after every step keeps the warps on the same step.  Memory then sees whole rows arrive together instead of 512-byte pieces of rows that lie
// 2 KiB apart and belong to warps that have drifted apart: measured, the barrier alone shortens
// the launch by 1-2.5 % at 8, 4 and 2 bits (and by more the more often it comes: every 8, 4, 2, 1
// rows), on a kernel that has issue slots to spare.
constexpr int kStepBarrier = 2;                                    // named barrier of the consumers' steps (1: group_wait)
__device__ __forceinline__ void step_barrier()
{
    asm volatile("bar.sync %0, %1;" ::"n"(kStepBarrier), "n"(kConsumerThreads) : "memory");
}

template <int C, int ROWS = kTileTokens>
struct FullTile {
    static constexpr int V8 = C >> 3;                              // 16-byte vectors per row
    static constexpr int G = kConsumerThreads / V8;                // row groups the CTA holds
    static constexpr int kSteps = ROWS / G;                        // rows per thread (16 of a tile at c = 1024)
    static constexpr int kStepsPerPage = 16 / G;                   // steps until the rows reach the unit's next 16 tokens
    static_assert(C % 256 == 0 && kSteps * G == ROWS && kSteps % 4 == 0 && 16 % G == 0, "row width");
    int cv, g;
    uint16_t *dst[ROWS / 16];      // the thread's 8 channels of row g of every 16 tokens of the unit; nullptr: page id out of range
    __device__ __forceinline__ FullTile(const DecodeParams &p, const UnitInfo &u)
    {
        g = threadIdx.x / V8;
        cv = threadIdx.x - g * V8;
#pragma unroll
        for (int h = 0; h < ROWS / 16; ++h) {                      // 16 tokens never straddle a page of >= 16
            const int T = u.row0 + 16 * h + g;
            const int pi = (T >> p.page_shift) - (u.row0 >> p.page_shift);          // 0 or 1
            dst[h] = page_row<C>(p, pi ? u.pg[1] : u.pg[0], u.plane, T);            // reports an out-of-range page id
            if (dst[h]) dst[h] += 8 * cv;
        }
    }
    // row of the unit the thread has at step k, and where it goes
    static __device__ __forceinline__ constexpr int row(int k, int g_) { return k * G + g_; }
    __device__ __forceinline__ uint16_t *out(int k) const
    {
        uint16_t *base = dst[k / kStepsPerPage];
        return base ? base + (k % kStepsPerPage) * G * C : nullptr;
    }
};

template <int C>
__device__ __forceinline__ void consume_raw_full(const DecodeParams &p, const UnitInfo &u, const uint8_t *codes)
{
    // a raw unit is a 16-token half of a tile: rows [0, 16) of the stage
    const FullTile<C, 16> t(p, u);
    constexpr int kSteps = FullTile<C, 16>::kSteps, G = FullTile<C, 16>::G, V8 = FullTile<C, 16>::V8;
    const uint4 *src = reinterpret_cast<const uint4 *>(codes) + (size_t)t.g * V8 + t.cv;
    uint4 v[kSteps];
#pragma unroll
    for (int k = 0; k < kSteps; ++k) v[k] = src[k * G * V8];
#pragma unroll
    for (int k = 0; k < kSteps; ++k) {
        uint16_t *o = t.out(k);
        if (o) *reinterpret_cast<uint4 *>(o) = v[k];
        if (k + 1 < kSteps) step_barrier();
    }
}

template <int BITS, int C>
__device__ __forceinline__ void consume_k_full(const DecodeParams &p, const UnitInfo &u, const uint8_t *codes,
                                               const uint8_t *meta)
{
    const FullTile<C> t(p, u);
    constexpr int kSteps = FullTile<C>::kSteps, G = FullTile<C>::G;
    f32x2 lo[4], sc[4];
    {
        const uint4 *m = reinterpret_cast<const uint4 *>(meta) + 2 * t.cv;
        const uint4 m0 = m[0], m1 = m[1];
        const uint32_t w[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
        float l1[8], s1[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            decode_params<BITS>(w[i], l1[i], s1[i]);
            if constexpr (BITS != 8) s1[i] = __fmul_rn(s1[i], Pos<BITS>::prescale(i));
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            lo[k] = f2_make(l1[2 * k], l1[2 * k + 1]);
            sc[k] = f2_make(s1[2 * k], s1[2 * k + 1]);
        }
    }
    constexpr uint32_t row_bytes = (uint32_t)C * BITS / 8;
    const uint8_t *src = codes + (size_t)t.g * row_bytes + (size_t)t.cv * BITS;
#pragma unroll
    for (int k = 0; k < kSteps; ++k) {
        f32x2 x[4];
        spread8<BITS>(src + k * G * row_bytes, x);
        const uint4 v = fma_pack8(x, sc, lo);
        uint16_t *o = t.out(k);
        if (o) *reinterpret_cast<uint4 *>(o) = v;
        if (k + 1 < kSteps) step_barrier();
    }
}

template <int BITS, int C>
__device__ __forceinline__ void consume_v_full(const DecodeParams &p, const UnitInfo &u, const uint8_t *codes,
                                               const uint8_t *meta)
{
    const FullTile<C> t(p, u);
    constexpr int kSteps = FullTile<C>::kSteps, G = FullTile<C>::G, groups = C / kGroup;
    constexpr uint32_t row_bytes = (uint32_t)C * BITS / 8;
    const int lane = threadIdx.x & 31;
    // the 4 lanes that share every group of this thread's rows each derive the scale of every fourth
    // step's row; all 32 lanes of a warp are here together (a warp's lanes share their rows and pages)
    const uint32_t *mrow = reinterpret_cast<const uint32_t *>(meta) + (size_t)t.g * groups + (t.cv >> 2);
    float mine[kSteps / 4];
#pragma unroll
    for (int i = 0; i < kSteps / 4; ++i) {
        float unused;
        decode_params<BITS>(mrow[((lane & 3) + 4 * i) * G * groups], unused, mine[i]);
    }
    const f32x2 pre01 = f2_make(Pos<BITS>::prescale(0), Pos<BITS>::prescale(1));
    const f32x2 pre23 = f2_make(Pos<BITS>::prescale(2), Pos<BITS>::prescale(3));
    const uint8_t *src = codes + (size_t)t.g * row_bytes + (size_t)t.cv * BITS;
#pragma unroll
    for (int k = 0; k < kSteps; ++k) {
        const float s0 = __shfl_sync(0xffffffffu, mine[k >> 2], (lane & ~3) | (k & 3));
        const float l1 = bf16_lo_to_f32(mrow[k * G * groups]);
        const f32x2 ss = f2_make(s0, s0), ll = f2_make(l1, l1);
        f32x2 sa = ss, sb = ss;
        if constexpr (BITS != 8) { sa = f2_mul(ss, pre01); sb = f2_mul(ss, pre23); }      // exact: powers of two
        const f32x2 sc[4] = {sa, sb, sa, sb}, lo[4] = {ll, ll, ll, ll};
        f32x2 x[4];
        spread8<BITS>(src + k * G * row_bytes, x);
        const uint4 v = fma_pack8(x, sc, lo);
        uint16_t *o = t.out(k);
        if (o) *reinterpret_cast<uint4 *>(o) = v;
        if (k + 1 < kSteps) step_barrier();
    }
}

// sched: 0 = each CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ... (grid = resident CTAs);
//        1 = grid holds one CTA per tile and running CTAs pull further tiles through cluster
//            launch control, so faster SMs take more tiles.
template <int C, bool SMALLPG = false>
__global__ void __launch_bounds__(kTmaThreads, 3) decode_tma_kernel(const DecodeParams p, const int n_chunks,
                                                                 const int n_quanta, const int sched)
{
    extern __shared__ __align__(128) uint8_t stage_mem[];
    __shared__ __align__(8) uint64_t full_bar[kSlots];
    __shared__ __align__(8) uint64_t empty_bar[kSlots];
    __shared__ UnitInfo info[kSlots];
    __shared__ int32_t unit_pg[kSlots][16];
    __shared__ int abort_flag;
    __shared__ int wait_verdict[2];
    __shared__ __align__(16) uint4 clc_response[2];
    __shared__ __align__(8) uint64_t clc_bar[2];

    const int tpu = C ? 1 : p.tpu;                        // tiles per unit
    const uint32_t quantum = tma_quantum_bytes(p.bw * tpu);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kConsumerThreads / 32);
        }
        mbar_init(&clc_bar[0], 1);
        mbar_init(&clc_bar[1], 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == kConsumerThreads / 32) {
        // ------------------------------ producer warp ------------------------------
        const int upc = kTilesPerChunk / tpu;             // units per chunk and plane
        const int64_t total_tiles = (int64_t)n_chunks * p.l * 2 * upc * p.n_blocks;
        int cur_chunk = -1;
        bool valid = false;
        kvh_chunk_desc d = p.single;
        int32_t my_pg = 0;                           // lane j holds page id j of the current chunk
        LayerLayout L = layer_layout(0, p.c, 1);
        uint32_t unit = 0;
        bool ok = true;
        // tail is the oldest unit whose quanta have not been taken back; lane j remembers how many the
        // unit in slot j holds
        QuantaRing ring(n_quanta);
        uint32_t tail = 0;
        int slot_q = 0;

        // One unit.  Contiguous source (rows as wide as the plane): one copy of codes_bytes and one of
        // meta_bytes.  A column block of wider rows (row_stride != 0): lane r copies row r's codes_bytes
        // from codes_src + r * row_stride and, for V, its meta_bytes from meta_src + r * mrow_stride
        // (K metadata is one piece: mrow_stride == 0).
        auto emit = [&](int bits, int kv, int row0, int nrows, uint16_t *plane, int col0, const uint8_t *codes_src,
                        uint32_t codes_bytes, uint32_t row_stride, const uint8_t *meta_src, uint32_t meta_bytes,
                        uint32_t mrow_stride) -> bool {
            const int s = unit % kSlots;
            const int need = unit_quanta(bits);
            while (unit - tail >= (uint32_t)kSlots || !ring.fits(need)) {
                if (tail == unit) return false;              // nothing left to take back: cannot happen (an empty ring holds any unit)
                bool w = true;
                if (lane == 0) w = mbar_wait(&empty_bar[tail % kSlots], (tail / kSlots) & 1, &abort_flag);
                w = __shfl_sync(0xffffffffu, w, 0);
                if (!w) return false;
                ring.give_back(__shfl_sync(0xffffffffu, slot_q, tail % kSlots));
                ++tail;
            }
            int held;
            const uint32_t st_off = (uint32_t)ring.take(need, held) * quantum;
            const uint32_t meta_off = 4u * (uint32_t)(bits == 16 ? 8 : bits) * p.bw * tpu;   // behind a tile's codes
            if (lane == s) slot_q = held;
            const int pidx = row0 >> p.page_shift;
            int32_t pg[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) pg[i] = __shfl_sync(0xffffffffu, my_pg, (pidx + i) & 31);
            const int32_t pg_mine = __shfl_sync(0xffffffffu, my_pg, (pidx + lane) & 31);
            if (lane < 16) unit_pg[s][lane] = pg_mine;
            __syncwarp();                                // lane 0's arrival below publishes these too
            uint8_t *st = stage_mem + st_off;
            const bool strided = row_stride != 0;
            if (lane == 0) {
                UnitInfo &u = info[s];
                u.bits = bits; u.kv = kv; u.row0 = row0; u.nrows = nrows; u.plane = plane;
                u.pg[0] = pg[0]; u.pg[1] = pg[1]; u.pg[2] = pg[2]; u.pg[3] = pg[3];
                u.col0 = col0; u.cw = p.bw;
                u.st_off = st_off; u.meta_off = meta_off;
                if (bits == 0) {
                    mbar_arrive(&full_bar[s]);
                } else if (!strided) {
                    mbar_arrive_expect_tx(&full_bar[s], codes_bytes + meta_bytes);
                    bulk_load(st, codes_src, codes_bytes, &full_bar[s]);
                    if (meta_bytes) bulk_load(st + meta_off, meta_src, meta_bytes, &full_bar[s]);
                } else {
                    const uint32_t meta_total = mrow_stride ? (uint32_t)nrows * meta_bytes : meta_bytes;
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)nrows * codes_bytes + meta_total);
                    if (meta_bytes && !mrow_stride) bulk_load(st + meta_off, meta_src, meta_bytes, &full_bar[s]);
                }
            }
            if (strided && bits != 0) {
                __syncwarp();                            // the expectation is posted before any piece lands
                if (lane < nrows) {
                    bulk_load(st + (size_t)lane * codes_bytes, codes_src + (size_t)lane * row_stride, codes_bytes,
                              &full_bar[s]);
                    if (meta_bytes && mrow_stride)
                        bulk_load(st + meta_off + (size_t)lane * meta_bytes, meta_src + (size_t)lane * mrow_stride,
                                  meta_bytes, &full_bar[s]);
                }
            }
            ++unit;
            return true;
        };

        auto do_tile = [&](int64_t tile_id) {
            // a tile id fits 32 bits (the host refuses larger launches): unsigned 32-bit divisions, and none
            // but the one by the layer count when the row width is compiled in.  The producer's arithmetic
            // is serial code in one warp and sits between a stage coming free and the next copy's start.
            const uint32_t id = (uint32_t)tile_id;
            const uint32_t nb = C ? 1u : (uint32_t)p.n_blocks, units = C ? (uint32_t)kTilesPerChunk : (uint32_t)upc;
            const int cb = (int)(id % nb);                       // column block, fastest: neighbours share page rows
            const uint32_t row_tile = id / nb;
            const int tile = (int)(row_tile % units) * tpu;      // the unit's first tile
            // Order of the tiles: a chunk's tiles, then the chunks, then the (layer, K|V) planes.  CTAs that
            // run side by side thus write into one plane of the pool (pages scattered over 64 MiB, not over
            // the whole pool: the same few translations serve every SM) and read from neighbouring chunks.
            // Rows cut into column blocks keep the order that finishes a chunk's planes first: their producer
            // issues a copy per row and has no time to spare for a new descriptor at every unit (measured:
            // 3-9 % slower plane by plane at 1280, 1536 and 4096 channels).
            const uint32_t t2 = row_tile / units;
            int chunk, kv, layer;
            if (nb == 1) {
                chunk = (int)(t2 % (uint32_t)n_chunks);
                const uint32_t plane_id = t2 / (uint32_t)n_chunks;
                kv = (int)(plane_id & 1);
                layer = (int)(plane_id >> 1);
            } else {
                kv = (int)(t2 & 1);
                layer = (int)((t2 >> 1) % (uint32_t)p.l);
                chunk = (int)((t2 >> 1) / (uint32_t)p.l);
            }
            if (chunk != cur_chunk) {
                cur_chunk = chunk;
                if (p.descs) d = p.descs[chunk];
                int err = check_desc(d, p.l, p.c, p.streams_bytes);
                const int npages = (d.n_tok + p.page_tokens - 1) >> p.page_shift;
                if (err == KVH_OK && (d.pt_off < 0 || (int64_t)d.pt_off + npages > p.page_table_len))
                    err = KVH_ERR_BUFFER_TOO_SMALL;
                valid = err == KVH_OK;
                if (!valid) {
                    if (lane == 0) report(p.status, err);
                } else {
                    my_pg = lane < npages ? __ldg(p.page_table + d.pt_off + lane) : 0;
                    L = layer_layout(d.level, p.c, d.n_tok);
                }
            }
            if (!valid) return;
            const int t0 = tile * kTileTokens;
            const int nt = min(kTileTokens * tpu, d.n_tok - t0);
            if (nt <= 0) return;
            const uint8_t *lay = p.streams + d.stream_off + (uint64_t)layer * L.layer_bytes();
            const uint8_t *meta = lay + L.meta_off(kv);
            const uint8_t *codes = lay + L.codes_off(kv);
            uint16_t *plane = p.pool + (int64_t)layer * p.layer_stride + (int64_t)kv * p.kv_stride;
            const bool wide = p.n_blocks > 1;
            const int col0 = cb * p.bw;
            const uint32_t gpr = (uint32_t)p.c / kGroup;         // groups per plane row
            if (d.level == 0) {
                const int half = 16 * tpu;                       // rows of raw bf16 a stage holds
                for (int h = 0; ok && h < nt; h += half) {
                    const int rows = min(half, nt - h);
                    const uint8_t *src = codes + 2 * ((uint64_t)(t0 + h) * p.c + col0);
                    ok = wide ? emit(16, kv, t0 + h, rows, plane, col0, src, 2u * p.bw, 2u * p.c, nullptr, 0, 0)
                              : emit(16, kv, t0 + h, rows, plane, 0, src, round16(2u * rows * p.c), 0, nullptr, 0, 0);
                }
            } else {
                const int b = level_bits(d.level);
                const uint8_t *csrc = codes + ((uint64_t)t0 * p.c + col0) * b / 8;
                const uint8_t *msrc = kv == 0 ? meta + 4 * ((uint64_t)tile * p.c + col0)
                                              : meta + 4 * ((uint64_t)t0 * gpr + col0 / kGroup);
                if (wide) {
                    ok = kv == 0 ? emit(b, kv, t0, nt, plane, col0, csrc, (uint32_t)p.bw * b / 8, (uint32_t)p.c * b / 8,
                                        msrc, 4u * p.bw, 0)
                                 : emit(b, kv, t0, nt, plane, col0, csrc, (uint32_t)p.bw * b / 8, (uint32_t)p.c * b / 8,
                                        msrc, 4u * (p.bw / kGroup), 4u * gpr);
                } else {
                    const uint32_t cbytes = round16((uint32_t)nt * p.c * b / 8);
                    const uint32_t mbytes = kv == 0 ? 4u * p.c * ((nt + kTileTokens - 1) / kTileTokens) : round16(4u * nt * gpr);
                    ok = emit(b, kv, t0, nt, plane, 0, csrc, cbytes, 0, msrc, mbytes, 0);
                }
            }
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
        if (ok) ok = emit(0, 0, 0, 0, nullptr, 0, nullptr, 0, 0, nullptr, 0, 0);      // end marker
        if (!ok && lane == 0) {
            report(p.status, KVH_ERR_TIMEOUT);
            abort_flag = 1;
        }
        // Leave only after every copy issued has landed: a normal run has seen them all consumed;
        // after an abort the units not taken back yet may still be in flight.
        if (lane == 0) {
            int never = 0;                           // the drain ignores the abort flag
            for (uint32_t w = tail; w < unit; ++w)
                (void)mbar_wait(&full_bar[w % kSlots], (w / kSlots) & 1, &never);
            feed.drain();
        }
    } else {
        // ------------------------------ consumer warps ------------------------------
        for (uint32_t unit = 0;; ++unit) {
            const int s = unit % kSlots;
            if (!group_wait(&full_bar[s], (unit / kSlots) & 1, &abort_flag, wait_verdict, unit, 1, kConsumerThreads, warp == 0)) {
                if (threadIdx.x == 0) report(p.status, KVH_ERR_TIMEOUT);
                break;
            }
            UnitInfo u = info[s];
            if (u.bits == 0) break;
            u.pgs = unit_pg[s];
            const uint8_t *st = stage_mem + u.st_off;
            const uint8_t *mt = st + u.meta_off;
            bool done = false;
            if constexpr (C != 0 && !SMALLPG) {
                // the common case by far: a whole tile (or, raw, a whole 16-token half of one)
                if (u.nrows == (u.bits == 16 ? 16 : kTileTokens)) {
                    switch (u.bits * 2 + u.kv) {              // uniform per CTA
                    case 32: case 33: consume_raw_full<C>(p, u, st); break;
                    case 16: consume_k_full<8, C>(p, u, st, mt); break;
                    case 17: consume_v_full<8, C>(p, u, st, mt); break;
                    case 8: consume_k_full<4, C>(p, u, st, mt); break;
                    case 9: consume_v_full<4, C>(p, u, st, mt); break;
                    case 4: consume_k_full<2, C>(p, u, st, mt); break;
                    default: consume_v_full<2, C>(p, u, st, mt); break;
                    }
                    done = true;
                }
            }
            if (!done)
            switch (u.bits * 2 + u.kv) {                      // uniform per CTA
            case 32: case 33: consume_raw<C, SMALLPG>(p, u, st); break;
            case 16: consume_k<8, C, SMALLPG>(p, u, st, mt); break;
            case 17: consume_v<8, C, SMALLPG>(p, u, st, mt); break;
            case 8: consume_k<4, C, SMALLPG>(p, u, st, mt); break;
            case 9: consume_v<4, C, SMALLPG>(p, u, st, mt); break;
            case 4: consume_k<2, C, SMALLPG>(p, u, st, mt); break;
            default: consume_v<2, C, SMALLPG>(p, u, st, mt); break;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[s]);
        }
    }
}

}  // namespace kvh
