"""Brute-force second statement of the codec — TEST INFRASTRUCTURE ONLY.

An independent check on ``kvh_oracle.c`` for tiny chunks.  Nothing here reuses
the C oracle: values are exact rationals (``fractions.Fraction``), every
binary32 operation of the format's arithmetic is "compute exactly, then round
to 24 significant bits, ties to even", and the packed sections are built as a
Python list of single bits that is folded into bytes at the end.  Pure-Python
loops: use only for a few thousand elements.

Format and arithmetic restated (levels 0..3 = 16, 8, 4, 2 bits; K groups are
one channel over 32 tokens, V groups 32 channels of one token; metadata
u32 = bf16(min) | bf16(max) << 16; sections Kmeta|Kcodes|Vmeta|Vcodes per
layer, each zero-padded to 128 bytes; r = hi - lo, inv = qmax / r,
scale = r / qmax (both 0 unless 2^-100 <= r <= FLT_MAX); q = clamp(rint((x - lo) * inv));
xhat = bf16(fma(q, scale, lo))).
"""
from __future__ import annotations

from fractions import Fraction

BITS = {0: 16, 1: 8, 2: 4, 3: 2}
RANGE_MIN = Fraction(1, 2 ** 100)
FLT_MAX = Fraction(2 ** 128 - 2 ** 104)


def _quantised(r: Fraction) -> bool:
    return RANGE_MIN <= r <= FLT_MAX      # a rounded range beyond FLT_MAX stands for +inf


# ---- exact values and correctly rounded binary formats ----------------------

def bf16_value(h: int) -> Fraction:
    """Exact value of a finite bf16 bit pattern (sign of zero dropped)."""
    sign = -1 if h & 0x8000 else 1
    e = (h >> 7) & 0xFF
    m = h & 0x7F
    assert e != 0xFF, "non-finite input"
    if e == 0:
        return sign * Fraction(m, 1 << 7) * Fraction(1, 1 << 126)
    return sign * (1 + Fraction(m, 1 << 7)) * (Fraction(2) ** (e - 127))


def _round_half_even(x: Fraction) -> int:
    fl = x.numerator // x.denominator
    rem = x - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        return fl + 1
    return fl


def round_binary(x: Fraction, precision: int, emin: int) -> Fraction:
    """Round x to a binary format with `precision` significant bits and
    smallest normal exponent emin (gradual underflow), ties to even.
    Overflow is not handled: inputs are finite and far from the top."""
    if x == 0:
        return Fraction(0)
    a = abs(x)
    # exponent e with 2^e <= a < 2^(e+1)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    elif Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, emin)
    ulp = Fraction(2) ** (e - (precision - 1))
    r = _round_half_even(a / ulp) * ulp
    return r if x > 0 else -r


def f32(x: Fraction) -> Fraction:
    return round_binary(x, 24, -126)


def bf16_bits(x: Fraction) -> int:
    """Bit pattern of a value that is exactly representable in bf16.  Zero
    maps to +0: the decoder's fma never yields -0 because q*scale >= +0."""
    if x == 0:
        return 0
    sign = 0x8000 if x < 0 else 0
    a = abs(x)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    elif Fraction(2) ** (e + 1) <= a:
        e += 1
    if e < -126:
        m = a / (Fraction(2) ** (-126 - 7))
        assert m.denominator == 1 and m < 128
        return sign | int(m)
    frac = a / (Fraction(2) ** e) - 1
    m = frac * 128
    assert m.denominator == 1 and 0 <= m < 128, "not a bf16 value"
    return sign | ((e + 127) << 7) | int(m)


def to_bf16(x: Fraction) -> int:
    """Round an exact value to bf16 (8 significant bits), ties to even."""
    return bf16_bits(round_binary(x, 8, -126))


def key(h: int) -> int:
    """Rank of a bf16 pattern: numeric order, -0 just below +0."""
    v = bf16_value(h)
    return (v, 0 if (h & 0x8000) else 1)


# ---- the quantiser ------------------------------------------------------------

def group_minmax(vals: list[int]) -> tuple[int, int]:
    return min(vals, key=key), max(vals, key=key)


def quantize(x: int, mn: int, mx: int, bits: int) -> int:
    qmax = (1 << bits) - 1
    lo, hi = bf16_value(mn), bf16_value(mx)
    r = f32(hi - lo)
    inv = f32(Fraction(qmax) / r) if _quantised(r) else Fraction(0)
    d = f32(bf16_value(x) - lo)
    s = f32(d * inv)
    q = _round_half_even(s)
    return max(0, min(qmax, q))


def dequantize(q: int, mn: int, mx: int, bits: int) -> int:
    qmax = (1 << bits) - 1
    lo, hi = bf16_value(mn), bf16_value(mx)
    r = f32(hi - lo)
    scale = f32(r / Fraction(qmax)) if _quantised(r) else Fraction(0)
    return to_bf16(f32(q * scale + lo))         # fma: one rounding to binary32


# ---- sections as lists of bits ------------------------------------------------

def _pad128(nbytes: int) -> int:
    return -(-nbytes // 128) * 128


def _bits_to_bytes(bits: list[int], nbytes: int) -> bytes:
    assert len(bits) <= 8 * nbytes
    bits = bits + [0] * (8 * nbytes - len(bits))
    return bytes(sum(bits[8 * i + j] << j for j in range(8)) for i in range(nbytes))


def _value_bits(v: int, width: int) -> list[int]:
    return [(v >> i) & 1 for i in range(width)]


def encode_chunk(kv, l: int, c: int, tok0: int, n: int, level: int) -> bytes:
    """kv[layer][kvsel][token][channel] -> bf16 bit pattern (any nested indexable)."""
    b = BITS[level]
    out = b""
    for layer in range(l):
        for kvsel in range(2):
            x = [[int(kv[layer][kvsel][tok0 + t][ch]) for ch in range(c)] for t in range(n)]
            if level == 0:
                bits = [bit for t in range(n) for ch in range(c) for bit in _value_bits(x[t][ch], 16)]
                out += _bits_to_bytes(bits, _pad128(2 * n * c))
                continue
            meta_bits: list[int] = []
            code_bits: list[int] = [0] * (n * c * b)
            if kvsel == 0:
                for g in range(-(-n // 32)):
                    toks = range(32 * g, min(n, 32 * g + 32))
                    for ch in range(c):
                        mn, mx = group_minmax([x[t][ch] for t in toks])
                        meta_bits += _value_bits(mn | (mx << 16), 32)
                        for t in toks:
                            pos = b * (t * c + ch)
                            code_bits[pos:pos + b] = _value_bits(quantize(x[t][ch], mn, mx, b), b)
                meta_bytes = 4 * c * -(-n // 32)
            else:
                for t in range(n):
                    for g in range(c // 32):
                        chans = range(32 * g, 32 * g + 32)
                        mn, mx = group_minmax([x[t][ch] for ch in chans])
                        meta_bits += _value_bits(mn | (mx << 16), 32)
                        for ch in chans:
                            pos = b * (t * c + ch)
                            code_bits[pos:pos + b] = _value_bits(quantize(x[t][ch], mn, mx, b), b)
                meta_bytes = 4 * n * (c // 32)
            out += _bits_to_bytes(meta_bits, _pad128(meta_bytes))
            out += _bits_to_bytes(code_bits, _pad128(n * c * b // 8))
    return out


def decode_chunk(chunk: bytes, level: int, l: int, c: int, n: int):
    """Returns out[layer][kvsel][t][ch] = bf16 bit pattern of the decoded chunk."""
    b = BITS[level]
    bits = [(byte >> j) & 1 for byte in chunk for j in range(8)]

    def take(pos: int, width: int) -> int:
        return sum(bits[pos + i] << i for i in range(width))

    out = []
    base = 0                                   # bit position of the current section
    for layer in range(l):
        planes = []
        for kvsel in range(2):
            if level == 0:
                plane = [[take(base + 16 * (t * c + ch), 16) for ch in range(c)] for t in range(n)]
                base += 8 * _pad128(2 * n * c)
            else:
                meta_bytes = 4 * c * -(-n // 32) if kvsel == 0 else 4 * n * (c // 32)
                codes = base + 8 * _pad128(meta_bytes)
                plane = []
                for t in range(n):
                    row = []
                    for ch in range(c):
                        gi = (t // 32) * c + ch if kvsel == 0 else t * (c // 32) + ch // 32
                        m = take(base + 32 * gi, 32)
                        q = take(codes + b * (t * c + ch), b)
                        row.append(dequantize(q, m & 0xFFFF, m >> 16, b))
                    plane.append(row)
                base = codes + 8 * _pad128(n * c * b // 8)
            planes.append(plane)
        out.append(planes)
    return out
