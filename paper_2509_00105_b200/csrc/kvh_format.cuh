// Byte layout of a stored chunk and the codec's scalar arithmetic, shared by the
// host entry points and the kernels of this library.
//
// The paper leaves the stored form open (it names "full quality" and
// quantisation "to 2 bits"); the layout below is this library's definition and
// is documented in full in include/kvh.h.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "kvh.h"

namespace kvh {

constexpr int kChunkTokens = KVH_CHUNK_TOKENS;
constexpr int kGroup = KVH_GROUP;
constexpr int kTileTokens = 32;                    // one K group of tokens = one work tile
constexpr int kTilesPerChunk = kChunkTokens / kTileTokens;
constexpr int kNumLevels = 4;
constexpr int kThreads = 256;

__host__ __device__ __forceinline__ uint64_t pad_section(uint64_t bytes)
{
    return (bytes + (KVH_SECTION_ALIGN - 1)) & ~uint64_t(KVH_SECTION_ALIGN - 1);
}

__host__ __device__ __forceinline__ int level_bits(int level) { return 16 >> level; }

// Section sizes (padded) of one layer of an n-token chunk.
struct LayerLayout {
    uint64_t kmeta, kcodes, vmeta, vcodes;         // padded byte counts
    uint64_t kmeta_payload, vmeta_payload, codes_payload;
    __host__ __device__ uint64_t layer_bytes() const { return kmeta + kcodes + vmeta + vcodes; }
    // byte offset of the K (kv = 0) or V (kv = 1) metadata section within the layer
    __host__ __device__ uint64_t meta_off(int kv) const { return kv ? kmeta + kcodes : 0; }
    __host__ __device__ uint64_t codes_off(int kv) const { return kv ? kmeta + kcodes + vmeta : kmeta; }
};

__host__ __device__ __forceinline__ LayerLayout layer_layout(int level, int c, int n)
{
    LayerLayout L;
    const uint64_t un = (uint64_t)n, uc = (uint64_t)c;
    if (level == 0) {
        L.kmeta_payload = L.vmeta_payload = 0;
        L.codes_payload = 2 * un * uc;
    } else {
        L.kmeta_payload = 4 * uc * ((un + kGroup - 1) / kGroup);
        L.vmeta_payload = 4 * un * (uc / kGroup);
        L.codes_payload = un * uc * (uint64_t)level_bits(level) / 8;
    }
    L.kmeta = pad_section(L.kmeta_payload);
    L.vmeta = pad_section(L.vmeta_payload);
    L.kcodes = L.vcodes = pad_section(L.codes_payload);
    return L;
}

__host__ __device__ __forceinline__ uint64_t chunk_bytes(int level, int l, int c, int n)
{
    return (uint64_t)l * layer_layout(level, c, n).layer_bytes();
}

#ifdef __CUDACC__
// ---- scalar arithmetic (binary32, round to nearest even, no contraction) -----

constexpr float kRangeMin = 0x1p-100f;             // smaller ranges are stored as flat groups
constexpr float kRangeMax = 3.402823466e+38f;

__device__ __forceinline__ float bf16_lo_to_f32(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16_hi_to_f32(uint32_t pair) { return __uint_as_float(pair & 0xffff0000u); }

// r / qmax for qmax = 3, 15, 255, correctly rounded, in three instructions instead of the division
// routine.  With c = RN(1 / qmax) and q0 = RN(r c), the remainder r - qmax q0 comes out exact from
// one fused multiply-add, and q0 + rem c, rounded once, is the correctly rounded quotient.  The
// sequence equals IEEE division bit for bit on every binary32 r in [2^-100, FLT_MAX] for the three
// divisors (checked exhaustively on the host: tests/test_division_by_constant.py); r outside that
// range never gets here.
template <int BITS>
__device__ __forceinline__ float div_by_qmax(float r)
{
    constexpr float qmax = (float)((1 << BITS) - 1);
    constexpr float c = 1.0f / qmax;
    const float q0 = __fmul_rn(r, c);
    const float rem = __fmaf_rn(-qmax, q0, r);
    return __fmaf_rn(rem, c, q0);
}

// scale = (max - min) / qmax and lo = min for decode, from one metadata word
template <int BITS>
__device__ __forceinline__ void decode_params(uint32_t meta, float &lo, float &scale)
{
    lo = bf16_lo_to_f32(meta);
    const float r = __fsub_rn(bf16_hi_to_f32(meta), lo);
    const bool ok = (r >= kRangeMin) && (r <= kRangeMax);
    scale = ok ? div_by_qmax<BITS>(r) : 0.0f;
}

// inv = qmax / (max - min) for encode
template <int BITS>
__device__ __forceinline__ void encode_params(uint32_t meta, float &lo, float &inv)
{
    lo = bf16_lo_to_f32(meta);
    const float r = __fsub_rn(bf16_hi_to_f32(meta), lo);
    const bool ok = (r >= kRangeMin) && (r <= kRangeMax);
    inv = ok ? __fdiv_rn((float)((1 << BITS) - 1), r) : 0.0f;
}

// float(q) for 0 <= q < 2^23 without the int-to-float unit: 2^23 + q is exact
__device__ __forceinline__ float small_uint_to_f32(uint32_t q)
{
    return __fsub_rn(__uint_as_float(0x4b000000u | q), 8388608.0f);
}

// rint(s) for 0 <= s < 2^22, ties to even: adding 2^23 leaves the integer in the low mantissa
// bits.  A flat or overflowed group has inv = 0; there (x - lo) * 0 is 0, or NaN when x - lo
// overflowed, and the min below turns both into code 0 (a NaN's low mantissa bits are not
// trusted: the caller passes inv so the code is forced to 0).
template <int BITS>
__device__ __forceinline__ uint32_t quantise(float x, float lo, float inv)
{
    const float s = __fmul_rn(__fsub_rn(x, lo), inv);
    const uint32_t q = __float_as_uint(__fadd_rn(s, 8388608.0f)) & 0x7fffffu;
    const uint32_t qc = min(q, (uint32_t)((1 << BITS) - 1));
    return inv == 0.0f ? 0u : qc;
}

__device__ __forceinline__ uint32_t pack_bf16x2_rn(float a, float b)
{
    uint32_t r;      // low half = a, high half = b, both rounded to nearest even
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
    return r;
}

// ---- two binary32 values in one 64-bit register -----------------------------------------------

typedef unsigned long long f32x2;

__device__ __forceinline__ f32x2 f2_from_bits(uint32_t a, uint32_t b)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ f32x2 f2_make(float a, float b) { return f2_from_bits(__float_as_uint(a), __float_as_uint(b)); }
__device__ __forceinline__ void f2_bits(f32x2 v, uint32_t &a, uint32_t &b)
{
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
}
__device__ __forceinline__ f32x2 f2_sub(f32x2 a, f32x2 b)
{
    f32x2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 f2_mul(f32x2 a, f32x2 b)
{
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 f2_fma(f32x2 a, f32x2 b, f32x2 c)
{
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// 1.0f that the compiler cannot see through (constant memory may be rewritten from the host, so
// its value is not known at compile time).  See biased_pair() for what depends on that.
static __constant__ float kRuntimeOne = 1.0f;

// Order-preserving 16-bit keys for two packed bf16: numeric order, -0 below +0.
__device__ __forceinline__ uint32_t order_keys2(uint32_t pair)
{
    const uint32_t neg = (pair >> 15) & 0x00010001u;
    return pair ^ (neg * 0x7fffu | 0x80008000u);
}
// inverse of order_keys2 for one 16-bit key
__device__ __forceinline__ uint32_t key_to_bf16(uint32_t key)
{
    return (key & 0x8000u) ? (key ^ 0x8000u) : (~key & 0xffffu);
}
#endif  // __CUDACC__

}  // namespace kvh
