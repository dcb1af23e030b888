/*
 * kvh_oracle.c — CPU oracle for the per-chunk KV-cache codec.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow,
 * single-threaded statement of what the codec computes, written so that a
 * reader can check it against the definition by eye.  Only the tests, the
 * smoke check and the benchmark's cpu-baseline leg may call it; the CUDA
 * library shares no source, header, table or helper with this file and the
 * constants of the format are restated here on purpose.
 *
 * What the paper fixes and this file follows:
 *   - an entry may be stored "in full quality" or compressed at a rate
 *     (Design section, last paragraph; the three per-entry choices);
 *   - the quantisation method is asymmetric group quantisation of the cited
 *     kind, and the one printed width is 2 bits (Preliminary Results,
 *     "Understanding the improvements");
 *   - a rate is a size fraction: size(i) x (m - n) is the space saved
 *     (marginal-utility-drop equation);
 *   - the KV tensor is l layers x {K,V} x N tokens x c channels (notation
 *     macros N, c, l, k).
 * The design section that would define the levels is not part of the paper's
 * text, so the level ladder, group geometry, metadata and bit order below are
 * this library's stated reading of it.  PARITY UNPINNED against the paper's own
 * quantiser parameters (group size, metadata format): nothing printed in the
 * paper can confirm or refute them.  Everything else is pinned by the CPU
 * tests (closed forms, a hand-worked group, invariants, an independent
 * bit-at-a-time brute-force path).
 *
 * Format (one chunk of n <= 256 tokens, c channels, l layers):
 *   level 0        raw bf16, lossless
 *   level 1, 2, 3  b = 8, 4, 2 bit codes, qmax = 2^b - 1
 *   K groups: one channel over 32 consecutive tokens of the chunk (the last
 *             group of a short chunk covers only the valid tokens)
 *   V groups: 32 consecutive channels of one token
 *   metadata per group: u32 = bf16(min) | bf16(max) << 16
 *   per layer: Kmeta | Kcodes | Vmeta | Vcodes, each padded with zero bytes
 *   to a multiple of 128 bytes; layers follow one another.
 *   Kmeta[ceil(n/32)][c], Vmeta[n][c/32]; code of element (t, ch) occupies
 *   bits [b*(t*c+ch), b*(t*c+ch)+b) of its section read as a little-endian
 *   bit string (bit i of the string is bit i%8 of byte i/8).
 *
 * Arithmetic (binary32, round to nearest even, no contraction):
 *   lo = f32(min), hi = f32(max), r = hi - lo
 *   2^-100 <= r <= FLT_MAX: inv = qmax / r, scale = r / qmax;
 *   otherwise (a flat group, a range too small for qmax / r to stay finite,
 *   or a range that overflowed): inv = 0, scale = 0 — every code is 0 and
 *   decodes to min
 *   encode: q = clamp((int) rint((f32(x) - lo) * inv), 0, qmax)
 *   decode: xhat = bf16_rne(fma(f32(q), scale, lo))
 *
 * Build: gcc -std=c99 -O2 -ffp-contract=off -fno-fast-math -shared -fPIC -lm
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define KVO_GROUP 32        /* tokens per K group, channels per V group */
#define KVO_CHUNK 256       /* most tokens in one chunk */
#define KVO_SECTION_ALIGN 128
#define KVO_RANGE_MIN 0x1p-100f   /* smallest group range that is quantised */
#define KVO_RANGE_MAX 0x1.fffffep+127f

/* ---- bf16 <-> binary32, in integer operations -------------------------- */

float kvo_f32_from_bf16(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;   /* bf16 is the top half of a binary32 */
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

uint16_t kvo_bf16_from_f32(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u)      /* NaN stays NaN */
        return (uint16_t)((u >> 16) | 0x0040u);
    /* round to nearest, ties to even, on the 16 discarded bits */
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* Total order on bf16 bit patterns that agrees with numeric order on finite
 * values and puts -0 below +0: negatives are bit-flipped, the rest get the
 * sign bit set. */
uint32_t kvo_order_key(uint16_t h)
{
    return (h & 0x8000u) ? (uint32_t)(uint16_t)~h : (uint32_t)(h | 0x8000u);
}

/* ---- level ladder and sizes ------------------------------------------- */

int kvo_num_levels(void) { return 4; }

/* bits per stored element at a level; -1 for an unknown level */
int kvo_level_bits(int level)
{
    switch (level) {
    case 0: return 16;
    case 1: return 8;
    case 2: return 4;
    case 3: return 2;
    default: return -1;
    }
}

static uint64_t pad_section(uint64_t bytes)
{
    return (bytes + KVO_SECTION_ALIGN - 1) / KVO_SECTION_ALIGN * KVO_SECTION_ALIGN;
}

/* Unpadded byte count of one section of one layer.
 * which: 0 Kmeta, 1 Kcodes, 2 Vmeta, 3 Vcodes. */
uint64_t kvo_section_payload_bytes(int level, int which, int c, int n)
{
    int b = kvo_level_bits(level);
    uint64_t un = (uint64_t)n, uc = (uint64_t)c;
    if (b < 0 || c <= 0 || n <= 0) return 0;
    if (level == 0)
        return (which == 1 || which == 3) ? 2u * un * uc : 0;
    switch (which) {
    case 0: return 4u * uc * ((un + KVO_GROUP - 1) / KVO_GROUP);
    case 2: return 4u * un * (uc / KVO_GROUP);
    case 1:
    case 3: return un * uc * (uint64_t)b / 8u;
    default: return 0;
    }
}

uint64_t kvo_section_bytes(int level, int which, int c, int n)
{
    return pad_section(kvo_section_payload_bytes(level, which, c, n));
}

/* size(i, M, R) of the utility definition for one chunk: stored bytes of n
 * tokens at a level.  0 means invalid arguments. */
uint64_t kvo_level_bytes(int level, int l, int c, int n)
{
    uint64_t per_layer = 0;
    int w;
    if (kvo_level_bits(level) < 0 || l <= 0 || c <= 0 || c % KVO_GROUP != 0 ||
        n <= 0 || n > KVO_CHUNK)
        return 0;
    for (w = 0; w < 4; ++w) per_layer += kvo_section_bytes(level, w, c, n);
    return (uint64_t)l * per_layer;
}

/* ---- the quantiser, one scalar step at a time -------------------------- */

/* min and max of count values x[0], x[stride], ... on the order key */
void kvo_group_range(const uint16_t *x, int count, int64_t stride,
                     uint16_t *mn, uint16_t *mx)
{
    uint16_t lo = x[0], hi = x[0];
    int i;
    for (i = 1; i < count; ++i) {
        uint16_t v = x[(int64_t)i * stride];
        if (kvo_order_key(v) < kvo_order_key(lo)) lo = v;
        if (kvo_order_key(v) > kvo_order_key(hi)) hi = v;
    }
    *mn = lo;
    *mx = hi;
}

static int range_is_quantised(float r)
{
    return r >= KVO_RANGE_MIN && r <= KVO_RANGE_MAX;
}

uint32_t kvo_quantize(uint16_t x, uint16_t mn, uint16_t mx, int bits)
{
    const float qmax = (float)((1 << bits) - 1);
    float lo = kvo_f32_from_bf16(mn);
    float hi = kvo_f32_from_bf16(mx);
    float r = hi - lo;
    float inv, d, s, q;
    if (!range_is_quantised(r)) return 0;     /* inv = 0: every code is 0 */
    inv = qmax / r;
    d = kvo_f32_from_bf16(x) - lo;
    s = d * inv;
    q = rintf(s);                             /* ties to even */
    if (q < 0.0f) q = 0.0f;
    if (q > qmax) q = qmax;
    return (uint32_t)q;
}

uint16_t kvo_dequantize(uint32_t q, uint16_t mn, uint16_t mx, int bits)
{
    const float qmax = (float)((1 << bits) - 1);
    float lo = kvo_f32_from_bf16(mn);
    float hi = kvo_f32_from_bf16(mx);
    float r = hi - lo;
    float scale = range_is_quantised(r) ? r / qmax : 0.0f;
    return kvo_bf16_from_f32(fmaf((float)q, scale, lo));
}

uint32_t kvo_pack_meta(uint16_t mn, uint16_t mx)
{
    return (uint32_t)mn | ((uint32_t)mx << 16);
}

/* ---- the bit string ----------------------------------------------------- */

void kvo_put_code(uint8_t *section, uint64_t index, int bits, uint32_t q)
{
    int i;
    for (i = 0; i < bits; ++i) {
        uint64_t pos = index * (uint64_t)bits + (uint64_t)i;
        if ((q >> i) & 1u) section[pos / 8] |= (uint8_t)(1u << (pos % 8));
    }
}

uint32_t kvo_get_code(const uint8_t *section, uint64_t index, int bits)
{
    uint32_t q = 0;
    int i;
    for (i = 0; i < bits; ++i) {
        uint64_t pos = index * (uint64_t)bits + (uint64_t)i;
        q |= (uint32_t)((section[pos / 8] >> (pos % 8)) & 1u) << i;
    }
    return q;
}

static void put_u32le(uint8_t *p, uint32_t v)
{
    p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8);
    p[2] = (uint8_t)(v >> 16); p[3] = (uint8_t)(v >> 24);
}

static uint32_t get_u32le(const uint8_t *p)
{
    return (uint32_t)p[0] | (uint32_t)p[1] << 8 | (uint32_t)p[2] << 16 |
           (uint32_t)p[3] << 24;
}

static void put_u16le(uint8_t *p, uint16_t v)
{
    p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8);
}

static uint16_t get_u16le(const uint8_t *p)
{
    return (uint16_t)(p[0] | p[1] << 8);
}

/* ---- one chunk ---------------------------------------------------------- */

/* Encode tokens [tok0, tok0+n) of a context kv[l][2][N][c] (bf16 bit
 * patterns) into out, which must hold kvo_level_bytes(level, l, c, n) bytes.
 * Returns 0, or -1 on invalid arguments. */
int kvo_encode_chunk(const uint16_t *kv, int l, int64_t N, int c, int64_t tok0,
                     int n, int level, uint8_t *out)
{
    const int b = kvo_level_bits(level);
    const uint64_t total = kvo_level_bytes(level, l, c, n);
    int layer, kvsel, t, ch;
    if (total == 0 || tok0 < 0 || tok0 + n > N) return -1;
    memset(out, 0, total);                    /* padding bits are zero */
    for (layer = 0; layer < l; ++layer) {
        for (kvsel = 0; kvsel < 2; ++kvsel) {
            const uint16_t *plane =
                kv + (((int64_t)layer * 2 + kvsel) * N + tok0) * c;
            uint8_t *meta = out;
            uint8_t *codes = out + kvo_section_bytes(level, 2 * kvsel, c, n);
            if (level == 0) {
                for (t = 0; t < n; ++t)
                    for (ch = 0; ch < c; ++ch)
                        put_u16le(codes + 2 * ((int64_t)t * c + ch),
                                  plane[(int64_t)t * c + ch]);
            } else if (kvsel == 0) {
                /* K: a group is one channel over up to 32 tokens */
                int g, ngroups = (n + KVO_GROUP - 1) / KVO_GROUP;
                for (g = 0; g < ngroups; ++g) {
                    int t0 = g * KVO_GROUP;
                    int cnt = (n - t0 < KVO_GROUP) ? n - t0 : KVO_GROUP;
                    for (ch = 0; ch < c; ++ch) {
                        uint16_t mn, mx;
                        kvo_group_range(plane + (int64_t)t0 * c + ch, cnt, c,
                                        &mn, &mx);
                        put_u32le(meta + 4 * ((int64_t)g * c + ch),
                                  kvo_pack_meta(mn, mx));
                        for (t = t0; t < t0 + cnt; ++t)
                            kvo_put_code(codes, (uint64_t)t * c + ch, b,
                                         kvo_quantize(plane[(int64_t)t * c + ch],
                                                      mn, mx, b));
                    }
                }
            } else {
                /* V: a group is 32 consecutive channels of one token */
                int g, ngroups = c / KVO_GROUP;
                for (t = 0; t < n; ++t) {
                    for (g = 0; g < ngroups; ++g) {
                        uint16_t mn, mx;
                        const uint16_t *x = plane + (int64_t)t * c + g * KVO_GROUP;
                        kvo_group_range(x, KVO_GROUP, 1, &mn, &mx);
                        put_u32le(meta + 4 * ((int64_t)t * ngroups + g),
                                  kvo_pack_meta(mn, mx));
                        for (ch = 0; ch < KVO_GROUP; ++ch)
                            kvo_put_code(codes,
                                         (uint64_t)t * c + g * KVO_GROUP + ch, b,
                                         kvo_quantize(x[ch], mn, mx, b));
                    }
                }
            }
            out += kvo_section_bytes(level, 2 * kvsel, c, n) +
                   kvo_section_bytes(level, 2 * kvsel + 1, c, n);
        }
    }
    return 0;
}

/* Decode one stored chunk into a paged pool.  Token t of the chunk goes to
 * page page_ids[t / page_tokens], slot t % page_tokens; element address (in
 * bf16 elements) = layer*layer_stride + kvsel*kv_stride + page*page_stride +
 * slot*c + ch.  A page id outside [0, num_pages) is skipped and counted.
 * Returns the number of skipped tokens x planes, or -1 on invalid arguments. */
int kvo_decode_chunk(const uint8_t *chunk, int level, int l, int c, int n,
                     const int32_t *page_ids, uint16_t *pool,
                     int64_t layer_stride, int64_t kv_stride,
                     int64_t page_stride, int32_t num_pages, int page_tokens)
{
    const int b = kvo_level_bits(level);
    int layer, kvsel, t, ch, skipped = 0;
    if (kvo_level_bytes(level, l, c, n) == 0 || page_tokens <= 0) return -1;
    for (layer = 0; layer < l; ++layer) {
        for (kvsel = 0; kvsel < 2; ++kvsel) {
            const uint8_t *meta = chunk;
            const uint8_t *codes = chunk + kvo_section_bytes(level, 2 * kvsel, c, n);
            for (t = 0; t < n; ++t) {
                int32_t page = page_ids[t / page_tokens];
                uint16_t *row;
                if (page < 0 || page >= num_pages) { ++skipped; continue; }
                row = pool + (int64_t)layer * layer_stride +
                      (int64_t)kvsel * kv_stride + (int64_t)page * page_stride +
                      (int64_t)(t % page_tokens) * c;
                for (ch = 0; ch < c; ++ch) {
                    uint64_t idx = (uint64_t)t * c + ch;
                    if (level == 0) {
                        row[ch] = get_u16le(codes + 2 * idx);
                    } else {
                        uint32_t m = (kvsel == 0)
                            ? get_u32le(meta + 4 * ((int64_t)(t / KVO_GROUP) * c + ch))
                            : get_u32le(meta + 4 * ((int64_t)t * (c / KVO_GROUP) +
                                                    ch / KVO_GROUP));
                        row[ch] = kvo_dequantize(kvo_get_code(codes, idx, b),
                                                 (uint16_t)(m & 0xffffu),
                                                 (uint16_t)(m >> 16), b);
                    }
                }
            }
            chunk += kvo_section_bytes(level, 2 * kvsel, c, n) +
                     kvo_section_bytes(level, 2 * kvsel + 1, c, n);
        }
    }
    return skipped;
}
