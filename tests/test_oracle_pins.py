"""Pins for the CPU oracle: checks against things other than the oracle itself.

Closed forms for the sizes, the capacity figures the paper prints, a group
worked by hand, library conversions (torch's float32 -> bfloat16), invariants
of the quantiser, exact rational arithmetic, and a brute-force second
implementation on tiny chunks.  No GPU.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import naive
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = v
    return out


def bf16_bits(x) -> np.ndarray:
    """float array -> bf16 bit patterns via torch (a library conversion)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bits_to_f32(h) -> np.ndarray:
    h = np.asarray(h, dtype=np.uint16)
    return (h.astype(np.uint32) << 16).view(np.float32)


# ---- sizes -------------------------------------------------------------------

def test_level_ladder():
    assert oracle.lib().kvo_num_levels() == 4
    assert [oracle.level_bits(k) for k in range(4)] == [16, 8, 4, 2]
    assert oracle.level_bits(4) == -1 and oracle.level_bits(-1) == -1


@pytest.mark.parametrize("l,c", [(32, 1024), (80, 1024), (4, 1024)])
def test_full_chunk_sizes_closed_form(l, c):
    n = 256
    raw = l * 2 * n * c * 2
    assert oracle.level_bytes(0, l, c, n) == raw
    # b code bits + 32 metadata bits per 32 elements = b + 1 bits per element
    for level, b in ((1, 8), (2, 4), (3, 2)):
        assert oracle.level_bytes(level, l, c, n) == l * 2 * n * c * (b + 1) // 8
    ratios = [Fraction(raw, oracle.level_bytes(k, l, c, n)) for k in range(4)]
    assert ratios == [1, Fraction(16, 9), Fraction(16, 5), Fraction(16, 3)]
    # payload alone: 16 -> 2 bits is one eighth (the paper's remark on 2-bit quantisation)
    payload = [oracle.section_payload_bytes(k, 1, c, n) for k in range(4)]
    assert [Fraction(payload[0], p) for p in payload] == [1, 2, 4, 8]


def test_sizes_from_the_definition_for_ragged_chunks():
    def pad(x):
        return -(-x // 128) * 128

    for c in (32, 64, 96, 128, 1024):
        for n in (1, 5, 15, 16, 17, 31, 32, 33, 100, 255, 256):
            assert oracle.level_bytes(0, 3, c, n) == 3 * 2 * pad(2 * n * c)
            for level, b in ((1, 8), (2, 4), (3, 2)):
                kmeta = 4 * c * math.ceil(n / 32)
                vmeta = 4 * n * (c // 32)
                codes = n * c * b // 8
                assert oracle.section_bytes(level, 0, c, n) == pad(kmeta)
                assert oracle.section_bytes(level, 2, c, n) == pad(vmeta)
                assert oracle.section_bytes(level, 1, c, n) == pad(codes)
                assert oracle.level_bytes(level, 3, c, n) == 3 * (pad(kmeta) + pad(vmeta) + 2 * pad(codes))


def test_sizes_strictly_decrease_with_level():
    # a rate is a size fraction: a deeper level must save space (marginal-utility-drop equation)
    for n in (3, 16, 33, 256):
        sizes = [oracle.level_bytes(k, 32, 1024, n) for k in range(4)]
        assert all(a > b for a, b in zip(sizes, sizes[1:])), sizes
    # a K group's metadata (4 bytes per channel) outweighs one or two raw tokens, so a 1- or
    # 2-token tail is not smaller at 8 bits than raw; among the quantised levels order holds
    for n in (1, 2):
        sizes = [oracle.level_bytes(k, 32, 1024, n) for k in range(4)]
        assert sizes[1] > sizes[2] > sizes[3] and sizes[1] >= sizes[0]


def test_invalid_size_arguments():
    assert oracle.level_bytes(4, 1, 32, 1) == 0
    assert oracle.level_bytes(0, 0, 32, 1) == 0
    assert oracle.level_bytes(0, 1, 33, 1) == 0       # c must be a multiple of 32
    assert oracle.level_bytes(0, 1, 32, 0) == 0
    assert oracle.level_bytes(0, 1, 32, 257) == 0


def test_paper_capacity_example():
    g = {k: float(v[0]) for k, v in read_golden("paper_capacity.txt").items()}
    l, c = int(g["model_layers"]), int(g["model_kv_channels"])
    per_token = oracle.level_bytes(0, l, c, 256) / 256
    assert per_token == 327680
    # two 80 GB GPUs + 150 GB of host memory, minus 16-bit weights, hold "500K tokens"
    free_bytes = (g["gpu_memory_gb"] + g["cpu_memory_gb"]) * 1e9 - g["model_params_billion"] * 1e9 * 2
    assert abs(free_bytes / per_token - g["tokens_stored"]) / g["tokens_stored"] < 0.10
    # "millions of tokens" <-> 3 TB of KV
    assert g["agentic_kv_bytes"] / per_token > g["agentic_tokens_at_least"]
    assert g["agentic_kv_bytes"] / per_token < 20e6
    # the 32768-token 70B-shaped context of the benchmark is ~10.7 GB
    assert abs(128 * oracle.level_bytes(0, 80, 1024, 256) / 1e9 - 10.7) < 0.05


# ---- bf16 helpers against torch ------------------------------------------------

def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(1)
    u = rng.integers(0, 2 ** 32, size=20000, dtype=np.uint64).astype(np.uint32)
    # add exact ties and near-ties around them
    base = rng.integers(0, 2 ** 16, size=2000, dtype=np.uint64).astype(np.uint32) << 16
    ties = np.concatenate([base | 0x8000, base | 0x7FFF, base | 0x8001])
    u = np.concatenate([u, ties])
    f = u.view(np.float32)
    f = f[np.isfinite(f)]
    want = bf16_bits(f)
    got = np.array([oracle.bf16_from_f32(float(x)) for x in f], dtype=np.uint16)
    assert np.array_equal(got, want)


def test_bf16_widening_matches_torch():
    h = np.arange(65536, dtype=np.uint16)
    t = torch.from_numpy(h.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([oracle.f32_from_bf16(int(x)) for x in h], dtype=np.float32)
    finite = np.isfinite(t)
    assert np.array_equal(got[finite].view(np.uint32), t[finite].view(np.uint32))


def test_order_key_is_numeric_order_with_signed_zero():
    h = np.arange(65536, dtype=np.uint16)
    f = bits_to_f32(h)
    finite = np.isfinite(f)
    h, f = h[finite], f[finite].astype(np.float64)
    keys = np.array([oracle.order_key(int(x)) for x in h], dtype=np.int64)
    order = np.argsort(keys, kind="stable")
    assert len(np.unique(keys)) == len(keys)
    assert np.all(np.diff(f[order]) >= 0)
    assert oracle.order_key(0x8000) < oracle.order_key(0x0000)      # -0 below +0


# ---- the hand-worked group -------------------------------------------------------

def _hand():
    g = read_golden("hand_group.txt")
    vals = bf16_bits([float(v) for v in g["values"]])
    assert np.array_equal(bits_to_f32(vals), np.array([float(v) for v in g["values"]], dtype=np.float32))
    return g, vals


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_hand_group_scalar_steps(bits):
    g, vals = _hand()
    mn, mx = oracle.group_range(vals)
    assert oracle.pack_meta(mn, mx) == int(g["meta"][0], 16)
    codes = [oracle.quantize(int(v), mn, mx, bits) for v in vals]
    assert codes == [int(x) for x in g[f"codes{bits}"]]
    sec = np.zeros(8, dtype=np.uint8)
    for i, q in enumerate(codes):
        oracle.put_code(sec, i, bits, q)
    want = [int(x, 16) for x in g[f"bytes{bits}"]]
    assert sec[:len(want)].tolist() == want and not sec[len(want):].any()
    assert [oracle.get_code(sec, i, bits) for i in range(6)] == codes
    if f"decoded{bits}" in g:
        dec = [oracle.dequantize(q, mn, mx, bits) for q in codes]
        assert np.array_equal(bits_to_f32(dec), np.array([float(x) for x in g[f"decoded{bits}"]], dtype=np.float32))


@pytest.mark.parametrize("level,bits", [(3, 2), (2, 4)])
def test_hand_group_inside_a_chunk(level, bits):
    """The same six values as (a) channel 5 of a 6-token K plane and (b) the first
    six channels of a V group padded with values inside the range."""
    g, vals = _hand()
    c, n = 32, 6
    kv = np.full((1, 2, n, c), bf16_bits([0.75])[0], dtype=np.uint16)
    kv[0, 0, :, 5] = vals                        # K: a group runs along tokens
    kv[0, 1, 2, :6] = vals                       # V: a group runs along channels
    kv[0, 1, 2, 6:] = bf16_bits(np.linspace(-0.9, 1.9, c - 6))
    s = oracle.encode_chunk(kv, 0, n, level)
    kmeta = s[:128].view(np.uint32)
    assert kmeta[5] == int(g["meta"][0], 16)
    kcodes = s[128:256]
    want = [int(x) for x in g[f"codes{bits}"]]
    assert [oracle.get_code(kcodes, t * c + 5, bits) for t in range(n)] == want
    vmeta = s[256:384].view(np.uint32)
    assert vmeta[2] == int(g["meta"][0], 16)
    vcodes = s[384:512]
    row = 2 * c * bits // 8
    wantb = [int(x, 16) for x in g[f"bytes{bits}"]]
    if bits == 2:   # six 2-bit codes end mid-byte: the upper nibble of byte 1 belongs to channels 6, 7
        assert vcodes[row] == wantb[0] and (vcodes[row + 1] & 0x0F) == wantb[1]
    else:
        assert vcodes[row:row + 3].tolist() == wantb


# ---- lossless level ---------------------------------------------------------------

def test_level0_round_trip_is_identity_on_every_bit_pattern():
    c, n, l = 64, 256, 2
    rng = np.random.default_rng(7)
    kv = rng.integers(0, 65536, size=(l, 2, n, c), dtype=np.uint64).astype(np.uint16)
    kv[0, 0, 0, :4] = [0x0000, 0x8000, 0x0001, 0x8001]     # +-0 and subnormals
    s = oracle.encode_chunk(kv, 0, n, 0)
    assert s.size == l * 2 * n * c * 2
    assert np.array_equal(s.view(np.uint16).reshape(l, 2, n, c), kv)     # raw little-endian bf16
    pool = np.full(l * 2 * 16 * 16 * c, 0xDEAD, dtype=np.uint16)
    ids = np.arange(16, dtype=np.int32)[::-1].copy()
    oracle.decode_chunk(s, 0, l, c, n, ids, pool, 2 * 16 * 16 * c, 16 * 16 * c, 16 * c, 16)
    p = pool.reshape(l, 2, 16, 16, c)
    for pg in range(16):
        assert np.array_equal(p[:, :, ids[pg]], kv[:, :, 16 * pg:16 * pg + 16])


# ---- invariants of the quantiser ----------------------------------------------------

def _random_group(rng, kind):
    if kind == "normal":
        return bf16_bits(rng.normal(size=32) * math.exp(rng.normal() * 2))
    if kind == "flat":
        return np.full(32, bf16_bits([rng.normal()])[0], dtype=np.uint16)
    if kind == "zeros":
        return rng.choice(np.array([0x0000, 0x8000], dtype=np.uint16), size=32)
    if kind == "tiny":
        return rng.integers(0, 0x0100, size=32, dtype=np.uint64).astype(np.uint16)   # subnormals and first normals
    if kind == "small":            # ranges just above the 2^-100 threshold
        return bf16_bits(rng.uniform(1, 4, size=32) * 2.0 ** -100)
    if kind == "huge":             # hi - lo overflows binary32
        return bf16_bits(rng.choice([-3e38, 3e38, 1.0], size=32))
    raise AssertionError(kind)


@pytest.mark.parametrize("kind", ["normal", "flat", "zeros", "tiny", "small", "huge"])
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_group_invariants(kind, bits):
    rng = np.random.default_rng(bits * 100 + len(kind))
    qmax = (1 << bits) - 1
    for _ in range(40):
        x = _random_group(rng, kind)
        mn, mx = oracle.group_range(x)
        xf = bits_to_f32(x).astype(np.float64)
        lo, hi = float(bits_to_f32([mn])[0]), float(bits_to_f32([mx])[0])
        assert lo == xf.min() and hi == xf.max()
        q = np.array([oracle.quantize(int(v), mn, mx, bits) for v in x])
        d = bits_to_f32([oracle.dequantize(int(v), mn, mx, bits) for v in q]).astype(np.float64)
        assert q.min() >= 0 and q.max() <= qmax
        # monotone: sorting by value sorts codes and decoded values
        order = np.argsort(xf, kind="stable")
        assert np.all(np.diff(q[order]) >= 0) and np.all(np.diff(d[order]) >= 0)
        # the minimum is code 0 and decodes to itself; a flat group is exact
        assert np.all(q[xf == lo] == 0) and np.all(d[xf == lo] == lo)
        r = hi - lo
        if 2.0 ** -100 <= r <= float(np.finfo(np.float32).max):
            assert np.all(q[xf == hi] == qmax)
        else:                      # flat, too small to quantise, or overflowed: stored as flat
            assert np.all(q == 0) and np.all(d == lo)
            continue
        # error bound: half a step, half a bf16 ulp of the result, and fp32 slack
        ulp = np.where(d == 0, 2.0 ** -133, 2.0 ** (np.floor(np.log2(np.abs(np.where(d == 0, 1, d)))) - 7))
        bound = r / (2 * qmax) + ulp / 2 + r * 2.0 ** -20 + 2.0 ** -140
        assert np.all(np.abs(xf - d) <= bound)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_codes_are_nearest_in_exact_arithmetic_away_from_ties(bits):
    """The fp32 evaluation may differ from exact real arithmetic only when the exact
    scaled value is within fp32 rounding distance of a half-integer."""
    rng = np.random.default_rng(11 + bits)
    qmax = (1 << bits) - 1
    checked = 0
    for _ in range(30):
        x = _random_group(rng, "normal")
        mn, mx = oracle.group_range(x)
        lo, hi = naive.bf16_value(mn), naive.bf16_value(mx)
        for v in x:
            s = (naive.bf16_value(int(v)) - lo) / (hi - lo) * qmax
            frac = s - math.floor(s)
            if abs(frac - Fraction(1, 2)) < Fraction(qmax, 2 ** 20):
                continue
            assert oracle.quantize(int(v), mn, mx, bits) == math.floor(s + Fraction(1, 2))
            checked += 1
    assert checked > 800


def test_rms_error_follows_uniform_quantiser_law():
    """On N(0,1) groups the error of a uniform quantiser is ~ step/sqrt(12)."""
    rng = np.random.default_rng(5)
    rms = {}
    for bits in (2, 4, 8):
        num = den = 0.0
        for _ in range(300):
            x = bf16_bits(rng.normal(size=32))
            mn, mx = oracle.group_range(x)
            xf = bits_to_f32(x).astype(np.float64)
            step = (xf.max() - xf.min()) / ((1 << bits) - 1)
            d = bits_to_f32([oracle.dequantize(oracle.quantize(int(v), mn, mx, bits), mn, mx, bits)
                             for v in x]).astype(np.float64)
            num += np.sum((xf - d) ** 2)
            den += 32 * step ** 2 / 12
        rms[bits] = math.sqrt(num)
        ratio = math.sqrt(num / den)
        # 2- and 4-bit: the law holds; 8-bit: the bf16 output grid adds its own error on top
        assert (0.75 < ratio < 1.15) if bits < 8 else (1.0 < ratio < 3.0), (bits, ratio)
    assert 4.0 < rms[2] / rms[4] < 6.0        # steps differ by 15/3 = 5
    assert 5.0 < rms[4] / rms[8] < 17.0       # 255/15 = 17, reduced by the bf16 floor


# ---- structure of the error (grouping axes) ---------------------------------------------

def test_k_groups_are_per_channel_and_v_groups_per_token():
    l, n, c = 1, 64, 64
    kv = workloads.make_kv(l, n, c, seed=3).view(torch.int16).numpy().view(np.uint16).copy()
    base = {k: oracle.encode_chunk(kv, 0, n, k) for k in (1, 2, 3)}
    # scale one K channel by 8 (exact in bf16): no other K channel's codes or metadata move
    kv2 = kv.copy()
    kv2[0, 0, :, 7] = bf16_bits(bits_to_f32(kv[0, 0, :, 7]) * 8)
    for level, bits in ((1, 8), (2, 4), (3, 2)):
        s1, s2 = base[level], oracle.encode_chunk(kv2, 0, n, level)
        km = oracle.section_bytes(level, 0, c, n)
        kc = oracle.section_bytes(level, 1, c, n)
        m1, m2 = s1[:km].view(np.uint32).reshape(-1, c), s2[:km].view(np.uint32).reshape(-1, c)
        others = [ch for ch in range(c) if ch != 7]
        assert np.array_equal(m1[:, others], m2[:, others]) and not np.array_equal(m1[:, 7], m2[:, 7])
        for t in range(n):
            for ch in range(c):
                q1 = oracle.get_code(s1[km:km + kc], t * c + ch, bits)
                q2 = oracle.get_code(s2[km:km + kc], t * c + ch, bits)
                assert q1 == q2          # scaling by a power of two keeps even channel 7's codes
        assert np.array_equal(s1[km + kc:], s2[km + kc:])      # V untouched
    # scale one V element: only its own (token, 32-channel) group changes
    kv3 = kv.copy()
    kv3[0, 1, 10, 40] = bf16_bits([1000.0])[0]
    s1, s3 = base[3], oracle.encode_chunk(kv3, 0, n, 3)
    off = oracle.section_bytes(3, 0, c, n) + oracle.section_bytes(3, 1, c, n)
    vm = oracle.section_bytes(3, 2, c, n)
    m1, m3 = s1[off:off + vm].view(np.uint32), s3[off:off + vm].view(np.uint32)
    changed = np.nonzero(m1 != m3)[0]
    assert changed.tolist() == [10 * (c // 32) + 1]
    c1, c3 = s1[off + vm:], s3[off + vm:]
    diff = np.nonzero(c1 != c3)[0]
    lo = (10 * c + 32) * 2 // 8
    assert diff.size > 0 and diff.min() >= lo and diff.max() < lo + 32 * 2 // 8


def test_head_sharding_gives_identical_codes():
    """Encoding each 128-channel head on its own yields the same metadata and codes."""
    l, n, c = 2, 40, 256
    kv = workloads.make_kv(l, n, c, seed=9).view(torch.int16).numpy().view(np.uint16).copy()
    for level, bits in ((2, 4), (3, 2)):
        whole = oracle.encode_chunk(kv, 0, n, level)
        for h in range(2):
            part = oracle.encode_chunk(np.ascontiguousarray(kv[..., 128 * h:128 * h + 128]), 0, n, level)
            wl = oracle.level_bytes(level, 1, c, n)
            pl = oracle.level_bytes(level, 1, 128, n)
            for layer in range(l):
                w, p = whole[layer * wl:(layer + 1) * wl], part[layer * pl:(layer + 1) * pl]
                wo = po = 0
                for which in range(4):
                    ws, ps = oracle.section_bytes(level, which, c, n), oracle.section_bytes(level, which, 128, n)
                    wsec, psec = w[wo:wo + ws], p[po:po + ps]
                    wo, po = wo + ws, po + ps
                    if which == 0:      # Kmeta[g][c]
                        a = wsec[:4 * 2 * c].view(np.uint32).reshape(2, c)[:, 128 * h:128 * h + 128]
                        b = psec[:4 * 2 * 128].view(np.uint32).reshape(2, 128)
                        assert np.array_equal(a, b)
                    elif which == 2:    # Vmeta[t][c/32]
                        a = wsec[:4 * n * 8].view(np.uint32).reshape(n, 8)[:, 4 * h:4 * h + 4]
                        b = psec[:4 * n * 4].view(np.uint32).reshape(n, 4)
                        assert np.array_equal(a, b)
                    else:
                        for t in range(0, n, 7):
                            for ch in range(0, 128, 5):
                                assert oracle.get_code(wsec, t * c + 128 * h + ch, bits) == \
                                    oracle.get_code(psec, t * 128 + ch, bits)


def test_padding_is_zero_and_sections_are_aligned():
    l, n, c = 1, 5, 32
    kv = workloads.make_kv(l, n, c, seed=2).view(torch.int16).numpy().view(np.uint16).copy()
    for level in (1, 2, 3):
        s = oracle.encode_chunk(kv, 0, n, level)
        off = 0
        for which in range(4):
            pay = oracle.section_payload_bytes(level, which, c, n)
            tot = oracle.section_bytes(level, which, c, n)
            assert tot % 128 == 0 and off % 128 == 0
            assert not s[off + pay:off + tot].any()
            off += tot
        assert off == s.size


# ---- brute force: the bit-at-a-time rational implementation ---------------------------------

TINY_CASES = [(1, 32, 1), (1, 32, 15), (1, 32, 16), (1, 32, 17), (1, 64, 31), (1, 32, 32), (2, 32, 33), (1, 96, 5)]


@pytest.mark.parametrize("l,c,n", TINY_CASES)
@pytest.mark.parametrize("level", [0, 1, 2, 3])
def test_brute_force_tiny_chunks(l, c, n, level):
    N = n + 3
    kv = workloads.make_kv(l, N, c, seed=100 + n + level).view(torch.int16).numpy().view(np.uint16).copy()
    kv[0, 0, 1, 0] = 0x8000                         # a signed zero and a subnormal in the mix
    kv[0, 1, 1, 1] = 0x0003
    s = oracle.encode_chunk(kv, 2, n, level)
    assert bytes(s) == naive.encode_chunk(kv, l, c, 2, n, level)
    want = np.array(naive.decode_chunk(bytes(s), level, l, c, n), dtype=np.uint16)     # [l][2][n][c]
    npages = (n + 15) // 16
    pool = np.full(l * 2 * npages * 16 * c, 0xDEAD, dtype=np.uint16)
    ids = np.arange(npages, dtype=np.int32)
    oracle.decode_chunk(s, level, l, c, n, ids, pool, 2 * npages * 16 * c, npages * 16 * c, 16 * c, npages)
    got = pool.reshape(l, 2, npages * 16, c)
    assert np.array_equal(got[:, :, :n], want)
    assert np.all(got[:, :, n:] == 0xDEAD)          # slots past the chunk's last token stay untouched


@pytest.mark.parametrize("level,n", [(3, 256), (2, 255)])
def test_brute_force_full_chunk(level, n):
    l, c = 1, 32
    kv = workloads.make_kv(l, 256, c, seed=40 + level).view(torch.int16).numpy().view(np.uint16).copy()
    s = oracle.encode_chunk(kv, 0, n, level)
    assert bytes(s) == naive.encode_chunk(kv, l, c, 0, n, level)


# ---- paged decode: scatter, bounds -------------------------------------------------------------

def test_decode_scatter_and_out_of_range_pages():
    l, c, n = 2, 32, 40
    kv = workloads.make_kv(l, n, c, seed=77).view(torch.int16).numpy().view(np.uint16).copy()
    s = oracle.encode_chunk(kv, 0, n, 0)
    num_pages = 8
    # strided pool with slack between pages, K/V planes and layers
    page_stride, kv_stride = 16 * c + 64, num_pages * (16 * c + 64) + 32
    layer_stride = 2 * kv_stride + 128
    pool = np.full(l * layer_stride, 0xBEEF, dtype=np.uint16)
    ids = np.array([5, 99, 2], dtype=np.int32)       # middle page is out of range
    skipped = oracle.decode_chunk(s, 0, l, c, n, ids, pool, layer_stride, kv_stride, page_stride, num_pages)
    assert skipped == 16 * l * 2
    touched = np.zeros(pool.size, dtype=bool)
    for layer in range(l):
        for kvsel in range(2):
            for t in list(range(0, 16)) + list(range(32, 40)):
                a = layer * layer_stride + kvsel * kv_stride + ids[t // 16] * page_stride + (t % 16) * c
                assert np.array_equal(pool[a:a + c], kv[layer, kvsel, t])
                touched[a:a + c] = True
    assert np.all(pool[~touched] == 0xBEEF)


def test_context_plan_offsets():
    l, c, N = 2, 64, 256 * 2 + 37
    ntoks, levels, offsets = oracle.chunk_plan(N, [3, 0, 2], l, c)
    assert ntoks == [256, 256, 37]
    assert offsets == [0, oracle.level_bytes(3, l, c, 256),
                       oracle.level_bytes(3, l, c, 256) + oracle.level_bytes(0, l, c, 256),
                       oracle.level_bytes(3, l, c, 256) + oracle.level_bytes(0, l, c, 256) + oracle.level_bytes(2, l, c, 37)]
    assert all(o % 128 == 0 for o in offsets)


# ---- token dropping and transcoding (composed from the steps pinned above) -------------------

def _rand_kv(l, N, c, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((l, 2, N, c)).astype(np.float32)
    return np.ascontiguousarray((x.view(np.uint32) >> 16).astype(np.uint16))


def test_kept_runs_of_sinks_and_recent_window():
    assert oracle.keep_sinks_and_recent(1000, 4, 252) == [(0, 4), (748, 252)]
    assert oracle.keep_sinks_and_recent(1000, 0, 10) == [(990, 10)]
    assert oracle.keep_sinks_and_recent(1000, 10, 0) == [(0, 10)]
    assert oracle.keep_sinks_and_recent(100, 60, 40) == [(0, 100)]        # windows meet: nothing dropped
    assert oracle.keep_sinks_and_recent(100, 80, 40) == [(0, 100)]
    with pytest.raises(ValueError):
        oracle.keep_sinks_and_recent(0, 1, 1)


def test_compaction_keeps_exactly_the_kept_tokens_in_order():
    """Token by token: compacted position j holds the j-th kept source token, nothing else."""
    kv = _rand_kv(2, 700, 32, 1)
    runs = [(0, 4), (300, 37), (650, 50)]
    got = oracle.compact_tokens(kv, runs)
    kept = [t for f, n in runs for t in range(f, f + n)]
    assert got.shape == (2, 2, len(kept), 32)
    for j, t in enumerate(kept):
        assert np.array_equal(got[:, :, j], kv[:, :, t])
    for bad in ([(5, 3), (6, 2)], [(10, 0)], [(690, 20)], [(20, 5), (0, 5)]):
        with pytest.raises(ValueError):
            oracle.compact_tokens(kv, bad)


def test_dropping_at_level_0_stores_the_kept_tokens_and_nothing_else():
    l, N, c = 2, 900, 64
    kv = _rand_kv(l, N, c, 2)
    runs = oracle.keep_sinks_and_recent(N, 4, 380)
    stream, offsets = oracle.encode_kept(kv, runs, 0)
    n_kept = 384
    assert len(offsets) == 3 and offsets[-1] == l * 2 * n_kept * c * 2     # size = rate x full size
    assert offsets[-1] * N == oracle.encode_context(kv, 0)[0].size * n_kept
    vals = np.concatenate([oracle.decode_chunk_values(stream[offsets[i]:offsets[i + 1]], 0, l, c, n)
                           for i, n in enumerate((256, 128))], axis=2)
    assert np.array_equal(vals[:, :, :4], kv[:, :, :4])
    assert np.array_equal(vals[:, :, 4:], kv[:, :, N - 380:])


def test_dropping_then_quantising_groups_the_compacted_tokens():
    """K groups run over 32 consecutive *kept* tokens: a group that spans the seam between the
    sink and the recent window takes its range from both sides."""
    l, N, c = 1, 600, 32
    kv = _rand_kv(l, N, c, 3)
    kv[0, 0, 0:4, 0] = 0x4120          # 10.0 in the sinks, channel 0
    kv[0, 0, 400:, 0] = 0xC120         # -10.0 in the recent window
    runs = oracle.keep_sinks_and_recent(N, 4, 200)
    stream, _ = oracle.encode_kept(kv, runs, 3)
    meta0 = int(stream[:4].view(np.uint32)[0])           # K metadata word of channel 0, first group
    assert meta0 == (0xC120 | (0x4120 << 16))
    same = oracle.encode_context(oracle.compact_tokens(kv, runs), 3)[0]
    assert np.array_equal(stream, same)


@pytest.mark.parametrize("level_out", [1, 2, 3])
def test_transcoding_from_full_quality_is_encoding(level_out):
    l, c, n = 2, 64, 77
    kv = _rand_kv(l, n, c, 4)
    raw = oracle.encode_chunk(kv, 0, n, 0)
    assert np.array_equal(oracle.decode_chunk_values(raw, 0, l, c, n), kv)
    assert np.array_equal(oracle.transcode_chunk(raw, 0, level_out, l, c, n), oracle.encode_chunk(kv, 0, n, level_out))


@pytest.mark.parametrize("level_in,level_out", [(1, 2), (1, 3), (2, 3), (2, 2), (3, 1)])
def test_transcoding_against_the_brute_force_path(level_in, level_out):
    """Byte for byte against the exact-arithmetic implementation, composed the same way."""
    l, c, n = 1, 32, 45
    kv = _rand_kv(l, n, c, 5 + level_in)
    s = oracle.encode_chunk(kv, 0, n, level_in)
    got = oracle.transcode_chunk(s, level_in, level_out, l, c, n)
    vals = naive.decode_chunk(bytes(s), level_in, l, c, n)
    want = naive.encode_chunk(vals, l, c, 0, n, level_out)
    assert got.size == oracle.level_bytes(level_out, l, c, n)
    assert bytes(got) == want


def test_transcoding_error_and_range_properties():
    """A transcoded group keeps its minimum exactly, never widens its range, and its values stay
    within half a step of the new level plus half a step of the old one (plus bf16 rounding)."""
    l, c, n = 1, 64, 256
    kv = _rand_kv(l, n, c, 9)
    x = (kv.astype(np.uint32) << 16).view(np.float32)
    s1 = oracle.encode_chunk(kv, 0, n, 1)
    s3 = oracle.transcode_chunk(s1, 1, 3, l, c, n)
    v1 = (oracle.decode_chunk_values(s1, 1, l, c, n).astype(np.uint32) << 16).view(np.float32)
    v3 = (oracle.decode_chunk_values(s3, 3, l, c, n).astype(np.uint32) << 16).view(np.float32)
    k = x[0, 0].reshape(8, 32, c)                        # K groups: [group][token][channel]
    r = k.max(1) - k.min(1)
    k3 = v3[0, 0].reshape(8, 32, c)
    assert np.array_equal(k3.min(1), k.min(1))           # min -> code 0 -> min at both levels
    assert np.all(k3.max(1) <= k.max(1) + 1e-6)
    bound = r[:, None, :] * (0.5 / 255 + 0.5 / 3) + 2.0 ** -7 * np.abs(k).max(1)[:, None, :]
    assert np.all(np.abs(k3 - k) <= bound)
    assert np.abs(v3 - x).mean() > np.abs(v1 - x).mean()  # and it is the coarser of the two


@pytest.mark.parametrize("level", [1, 2, 3])
def test_decoded_group_spans_exactly_the_decodings_of_code_0_and_code_qmax(level):
    """What the transcoding kernel relies on: a group's smallest element has code 0, its largest
    code qmax, and decoding is monotone, so min and max of the decoded group (in the format's
    order, -0 below +0) are dequantize(0) and dequantize(qmax) of the old metadata."""
    bits = 16 >> level
    qmax = (1 << bits) - 1
    rng = np.random.default_rng(level)
    groups = [_rand_kv(1, 32, 32, 40 + level)[0, 0, :, i] for i in range(32)]
    groups += [rng.integers(0, 0x80, 32).astype(np.uint16),                       # subnormals: stored flat
               rng.choice(np.array([0x0000, 0x8000], dtype=np.uint16), 32),       # signed zeros
               rng.choice(np.array([0x7F00, 0xFF00], dtype=np.uint16), 32),       # range overflows
               np.full(32, 0xC000, dtype=np.uint16),
               (rng.integers(0, 200, 32).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)]
    for g in groups:
        g = np.ascontiguousarray(g, dtype=np.uint16)
        mn, mx = oracle.group_range(g)
        dec = np.array([oracle.dequantize(oracle.quantize(int(x), mn, mx, bits), mn, mx, bits) for x in g], dtype=np.uint16)
        dmn, dmx = oracle.group_range(dec)
        assert (dmn, dmx) == (oracle.dequantize(0, mn, mx, bits), oracle.dequantize(qmax, mn, mx, bits))
