"""CPU oracle for the per-chunk KV-cache codec — TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu-baseline leg may import
this package.  It wraps ``kvh_oracle.c`` (plain C, compiled here with gcc) with
numpy-typed helpers and imports nothing from the CUDA package.

bf16 tensors cross this boundary as ``numpy.uint16`` bit patterns; streams as
``numpy.uint8``.  PARITY UNPINNED against the paper's own quantiser parameters
(see the header of ``kvh_oracle.c``); everything else is pinned by the CPU
tests.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "kvh_oracle.c"
_LIB = _HERE / "libkvh_oracle.so"

GROUP = 32
CHUNK = 256
NUM_LEVELS = 4

_CFLAGS = ["-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-Wall",
           "-Wextra", "-shared", "-fPIC"]


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run(["gcc", *_CFLAGS, "-o", str(tmp), str(_SRC), "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(str(build()))
        u8p = ctypes.POINTER(ctypes.c_uint8)
        u16p = ctypes.POINTER(ctypes.c_uint16)
        i32p = ctypes.POINTER(ctypes.c_int32)
        L.kvo_f32_from_bf16.restype = ctypes.c_float
        L.kvo_f32_from_bf16.argtypes = [ctypes.c_uint16]
        L.kvo_bf16_from_f32.restype = ctypes.c_uint16
        L.kvo_bf16_from_f32.argtypes = [ctypes.c_float]
        L.kvo_order_key.restype = ctypes.c_uint32
        L.kvo_order_key.argtypes = [ctypes.c_uint16]
        L.kvo_num_levels.restype = ctypes.c_int
        L.kvo_level_bits.restype = ctypes.c_int
        L.kvo_level_bits.argtypes = [ctypes.c_int]
        for name in ("kvo_section_payload_bytes", "kvo_section_bytes"):
            f = getattr(L, name)
            f.restype = ctypes.c_uint64
            f.argtypes = [ctypes.c_int] * 4
        L.kvo_level_bytes.restype = ctypes.c_uint64
        L.kvo_level_bytes.argtypes = [ctypes.c_int] * 4
        L.kvo_group_range.restype = None
        L.kvo_group_range.argtypes = [u16p, ctypes.c_int, ctypes.c_int64, u16p, u16p]
        L.kvo_quantize.restype = ctypes.c_uint32
        L.kvo_quantize.argtypes = [ctypes.c_uint16, ctypes.c_uint16, ctypes.c_uint16, ctypes.c_int]
        L.kvo_dequantize.restype = ctypes.c_uint16
        L.kvo_dequantize.argtypes = [ctypes.c_uint32, ctypes.c_uint16, ctypes.c_uint16, ctypes.c_int]
        L.kvo_pack_meta.restype = ctypes.c_uint32
        L.kvo_pack_meta.argtypes = [ctypes.c_uint16, ctypes.c_uint16]
        L.kvo_put_code.restype = None
        L.kvo_put_code.argtypes = [u8p, ctypes.c_uint64, ctypes.c_int, ctypes.c_uint32]
        L.kvo_get_code.restype = ctypes.c_uint32
        L.kvo_get_code.argtypes = [u8p, ctypes.c_uint64, ctypes.c_int]
        L.kvo_encode_chunk.restype = ctypes.c_int
        L.kvo_encode_chunk.argtypes = [u16p, ctypes.c_int, ctypes.c_int64, ctypes.c_int,
                                       ctypes.c_int64, ctypes.c_int, ctypes.c_int, u8p]
        L.kvo_decode_chunk.restype = ctypes.c_int
        L.kvo_decode_chunk.argtypes = [u8p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                       i32p, u16p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                       ctypes.c_int32, ctypes.c_int]
        _lib = L
    return _lib


def _p(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


# ---- scalar steps -----------------------------------------------------------

def level_bits(level: int) -> int:
    return lib().kvo_level_bits(level)


def section_bytes(level: int, which: int, c: int, n: int) -> int:
    """Padded size of one section of one layer (0 Kmeta, 1 Kcodes, 2 Vmeta, 3 Vcodes)."""
    return lib().kvo_section_bytes(level, which, c, n)


def section_payload_bytes(level: int, which: int, c: int, n: int) -> int:
    return lib().kvo_section_payload_bytes(level, which, c, n)


def level_bytes(level: int, l: int, c: int, n: int) -> int:
    """Stored bytes of an n-token chunk at a level; 0 for invalid arguments."""
    return lib().kvo_level_bytes(level, l, c, n)


def f32_from_bf16(h: int) -> float:
    return lib().kvo_f32_from_bf16(h)


def bf16_from_f32(f: float) -> int:
    return lib().kvo_bf16_from_f32(f)


def order_key(h: int) -> int:
    return lib().kvo_order_key(h)


def group_range(x: np.ndarray) -> tuple[int, int]:
    x = np.ascontiguousarray(x, dtype=np.uint16)
    mn, mx = ctypes.c_uint16(), ctypes.c_uint16()
    lib().kvo_group_range(_p(x, ctypes.c_uint16), x.size, 1, ctypes.byref(mn), ctypes.byref(mx))
    return mn.value, mx.value


def quantize(x: int, mn: int, mx: int, bits: int) -> int:
    return lib().kvo_quantize(x, mn, mx, bits)


def dequantize(q: int, mn: int, mx: int, bits: int) -> int:
    return lib().kvo_dequantize(q, mn, mx, bits)


def pack_meta(mn: int, mx: int) -> int:
    return lib().kvo_pack_meta(mn, mx)


def put_code(section: np.ndarray, index: int, bits: int, q: int) -> None:
    assert section.dtype == np.uint8 and section.flags.c_contiguous
    lib().kvo_put_code(_p(section, ctypes.c_uint8), index, bits, q)


def get_code(section: np.ndarray, index: int, bits: int) -> int:
    assert section.dtype == np.uint8 and section.flags.c_contiguous
    return lib().kvo_get_code(_p(section, ctypes.c_uint8), index, bits)


# ---- chunk and context level ------------------------------------------------

def encode_chunk(kv: np.ndarray, tok0: int, n: int, level: int) -> np.ndarray:
    """Encode tokens [tok0, tok0+n) of kv[l][2][N][c] (uint16 bf16 bits)."""
    assert kv.dtype == np.uint16 and kv.ndim == 4 and kv.shape[1] == 2 and kv.flags.c_contiguous
    l, _, N, c = kv.shape
    size = level_bytes(level, l, c, n)
    if size == 0:
        raise ValueError("invalid level/shape")
    out = np.empty(size, dtype=np.uint8)
    rc = lib().kvo_encode_chunk(_p(kv, ctypes.c_uint16), l, N, c, tok0, n, level,
                                _p(out, ctypes.c_uint8))
    if rc != 0:
        raise ValueError("kvo_encode_chunk rejected its arguments")
    return out


def chunk_plan(N: int, levels, l: int, c: int) -> tuple[list[int], list[int], list[int]]:
    """Per-chunk (n_tok, level, offset) for a context of N tokens; offsets has nchunks+1 entries."""
    nchunks = (N + CHUNK - 1) // CHUNK
    if isinstance(levels, int):
        levels = [levels] * nchunks
    assert len(levels) == nchunks
    ntoks = [min(CHUNK, N - i * CHUNK) for i in range(nchunks)]
    offsets = [0]
    for n, k in zip(ntoks, levels):
        offsets.append(offsets[-1] + level_bytes(k, l, c, n))
    return ntoks, list(levels), offsets


def encode_context(kv: np.ndarray, levels) -> tuple[np.ndarray, list[int]]:
    """Concatenated chunk streams of a whole context, and the chunk offsets."""
    l, _, N, c = kv.shape
    ntoks, levels, offsets = chunk_plan(N, levels, l, c)
    out = np.empty(offsets[-1], dtype=np.uint8)
    for i, (n, k) in enumerate(zip(ntoks, levels)):
        out[offsets[i]:offsets[i + 1]] = encode_chunk(kv, i * CHUNK, n, k)
    return out, offsets


def decode_chunk(chunk: np.ndarray, level: int, l: int, c: int, n: int, page_ids: np.ndarray,
                 pool: np.ndarray, layer_stride: int, kv_stride: int, page_stride: int,
                 num_pages: int, page_tokens: int = 16) -> int:
    """Decode a chunk into pool (flat uint16, modified in place); returns skipped rows."""
    assert chunk.dtype == np.uint8 and chunk.flags.c_contiguous
    assert pool.dtype == np.uint16 and pool.flags.c_contiguous
    page_ids = np.ascontiguousarray(page_ids, dtype=np.int32)
    assert chunk.size >= level_bytes(level, l, c, n) > 0
    assert page_ids.size >= (n + page_tokens - 1) // page_tokens
    rc = lib().kvo_decode_chunk(_p(chunk, ctypes.c_uint8), level, l, c, n,
                                _p(page_ids, ctypes.c_int32), _p(pool, ctypes.c_uint16),
                                layer_stride, kv_stride, page_stride, num_pages, page_tokens)
    if rc < 0:
        raise ValueError("kvo_decode_chunk rejected its arguments")
    return rc


def decode_context(stream: np.ndarray, offsets, ntoks, levels, l: int, c: int,
                   page_table: np.ndarray, pool: np.ndarray, layer_stride: int, kv_stride: int,
                   page_stride: int, num_pages: int, page_tokens: int = 16) -> int:
    """Decode every chunk of a context; chunk i uses page ids page_table[i*16 : ...]."""
    pages_per_chunk = CHUNK // page_tokens
    skipped = 0
    for i, (n, k) in enumerate(zip(ntoks, levels)):
        skipped += decode_chunk(stream[offsets[i]:offsets[i + 1]], k, l, c, n,
                                page_table[i * pages_per_chunk:], pool, layer_stride,
                                kv_stride, page_stride, num_pages, page_tokens)
    return skipped


# ---- token dropping (the paper's second compression method) -----------------
#
# The paper names token dropping beside quantisation (Introduction: texts that matter only "at
# the beginning and the end" suit it) and cites the attention-sink method for it: the first few
# tokens and a window of the most recent ones are kept, the middle is dropped.  The kept tokens
# are stored compacted, in order, as an ordinary context of n_kept tokens at any level; the rate
# of the method is n_kept / N.  The definition is therefore "encode the compacted tensor".

def keep_sinks_and_recent(N: int, n_sink: int, n_recent: int) -> list[tuple[int, int]]:
    """Kept runs (first token, count) when the first n_sink and the last n_recent tokens of an
    N-token context survive; everything if the two windows meet."""
    if N <= 0 or n_sink < 0 or n_recent < 0:
        raise ValueError("invalid arguments")
    if n_sink + n_recent >= N:
        return [(0, N)]
    runs = []
    if n_sink:
        runs.append((0, n_sink))
    if n_recent:
        runs.append((N - n_recent, n_recent))
    return runs


def compact_tokens(kv: np.ndarray, runs) -> np.ndarray:
    """kv[l][2][N][c] restricted to the kept runs, in order: [l][2][n_kept][c]."""
    prev_end = 0
    for first, count in runs:
        if count <= 0 or first < prev_end or first + count > kv.shape[2]:
            raise ValueError("runs must be ascending, disjoint, non-empty and inside the context")
        prev_end = first + count
    return np.ascontiguousarray(np.concatenate([kv[:, :, f:f + n, :] for f, n in runs], axis=2))


def encode_kept(kv: np.ndarray, runs, levels) -> tuple[np.ndarray, list[int]]:
    """Stored form of a context after token dropping: the chunks of the compacted tensor."""
    return encode_context(compact_tokens(kv, runs), levels)


# ---- transcoding a stored chunk to a lower quality level ---------------------
#
# The policy's marginal-utility step may "compress furthermore" an entry that is already stored.
# What is stored is all there is to compress, so the result is defined as the encoding, at the
# new level, of the values the stored chunk decodes to.

def decode_chunk_values(chunk: np.ndarray, level: int, l: int, c: int, n: int) -> np.ndarray:
    """The bf16 values a stored chunk decodes to, [l][2][n][c] (uint16 bit patterns)."""
    npg = (n + 15) // 16
    pool = np.zeros(l * 2 * npg * 16 * c, dtype=np.uint16)
    skipped = decode_chunk(chunk, level, l, c, n, np.arange(npg, dtype=np.int32), pool,
                           2 * npg * 16 * c, npg * 16 * c, 16 * c, npg)
    assert skipped == 0
    return np.ascontiguousarray(pool.reshape(l, 2, npg * 16, c)[:, :, :n, :])


def transcode_chunk(chunk: np.ndarray, level_in: int, level_out: int, l: int, c: int, n: int) -> np.ndarray:
    """encode(level_out) of decode(level_in) of a stored chunk."""
    return encode_chunk(decode_chunk_values(chunk, level_in, l, c, n), 0, n, level_out)
