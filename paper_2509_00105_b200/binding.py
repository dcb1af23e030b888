"""ctypes binding of the C ABI in include/kvh.h.

Argument marshalling only.  Tensors are passed as raw device pointers and the
work is enqueued on torch's current CUDA stream.  Functions raise ``KvhError``
when the library returns a non-zero status.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from pathlib import Path

import numpy as np
import torch

CHUNK_TOKENS = 256
GROUP = 32
NUM_LEVELS = 4

_LIB_PATH = Path(__file__).resolve().parent / "libkvh.so"
_lib = None


class KvhError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: kvh status {status} ({status_string(status)})")


class ChunkDesc(ctypes.Structure):
    """Mirror of kvh_chunk_desc (24 bytes)."""
    _fields_ = [("stream_off", ctypes.c_uint64), ("level", ctypes.c_int32), ("n_tok", ctypes.c_int32),
                ("pt_off", ctypes.c_int32), ("reserved", ctypes.c_int32)]


DESC_DTYPE = np.dtype([("stream_off", "<u8"), ("level", "<i4"), ("n_tok", "<i4"),
                       ("pt_off", "<i4"), ("reserved", "<i4")])
assert DESC_DTYPE.itemsize == ctypes.sizeof(ChunkDesc) == 24


class _PoolStruct(ctypes.Structure):
    _fields_ = [("base", ctypes.c_void_p), ("layer_stride", ctypes.c_int64), ("kv_stride", ctypes.c_int64),
                ("page_stride", ctypes.c_int64), ("num_pages", ctypes.c_int32), ("page_tokens", ctypes.c_int32),
                ("n_layers", ctypes.c_int32), ("n_channels", ctypes.c_int32)]


def lib() -> ctypes.CDLL:
    """Load libkvh.so (built by ``__graft_entry__.build()``); fails loudly if it is absent."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is not built: run `python -c 'import __graft_entry__ as g; g.build()'` "
                               "at the repository root; this package has no CPU fallback")
        L = ctypes.CDLL(str(_LIB_PATH))
        vp, i32, i64, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint64
        ip = ctypes.POINTER(ctypes.c_int)
        L.kvh_format_version.restype = i32
        L.kvh_num_levels.restype = i32
        L.kvh_status_string.restype = ctypes.c_char_p
        L.kvh_status_string.argtypes = [i32]
        L.kvh_build_variant.restype = ctypes.c_char_p
        L.kvh_level_info.restype = i32
        L.kvh_level_info.argtypes = [i32, ip, ip, ip]
        L.kvh_level_bytes.restype = i32
        L.kvh_level_bytes.argtypes = [i32, i32, i32, i32, ctypes.POINTER(u64)]
        L.kvh_plan_chunks.restype = i32
        L.kvh_plan_chunks.argtypes = [i32, i32, i64, vp, i32, u64, ctypes.c_int32, ctypes.c_int32, vp,
                                      ctypes.POINTER(u64)]
        L.kvh_encode.restype = i32
        L.kvh_encode.argtypes = [vp, i32, i64, i32, i32, vp, u64, vp, vp]
        L.kvh_encode_chunks.restype = i32
        L.kvh_encode_chunks.argtypes = [vp, i32, i64, i32, vp, vp, i32, vp, u64, vp, vp]
        L.kvh_decode_to_pages.restype = i32
        L.kvh_decode_to_pages.argtypes = [vp, i32, i32, vp, ctypes.POINTER(_PoolStruct), vp, vp]
        L.kvh_decode_batch.restype = i32
        L.kvh_decode_batch.argtypes = [vp, u64, vp, i32, vp, i64, ctypes.POINTER(_PoolStruct), vp, vp]
        L.kvh_load_host.restype = i32
        L.kvh_load_host.argtypes = [vp, vp, u64, vp, vp, i32, vp, i64, ctypes.POINTER(_PoolStruct), vp, vp,
                                    u64, vp, vp]
        L.kvh_store_host.restype = i32
        L.kvh_store_host.argtypes = [vp, i32, i64, i32, vp, vp, i32, vp, u64, vp, vp, vp, u64, vp, vp]
        L.kvh_keep_sinks_and_recent.restype = i32
        L.kvh_keep_sinks_and_recent.argtypes = [i64, i64, i64, vp, ip, ctypes.POINTER(i64)]
        L.kvh_encode_kept.restype = i32
        L.kvh_encode_kept.argtypes = [vp, i32, i64, i32, vp, i32, vp, i32, i32, vp, u64, vp, vp]
        L.kvh_transcode.restype = i32
        L.kvh_transcode.argtypes = [vp, u64, vp, vp, u64, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp]
        L.kvh_policy_assign.restype = i32
        L.kvh_policy_assign.argtypes = [vp, vp, vp, i32, vp, vp, ctypes.POINTER(u64), ctypes.POINTER(ctypes.c_double)]
        L.kvh_policy_assign_tiers.restype = i32
        L.kvh_policy_assign_tiers.argtypes = [vp, vp, vp, i32, vp, i32, vp, vp]
        L.kvh_check_page_table.restype = i32
        L.kvh_check_page_table.argtypes = [vp, i64, ctypes.c_int32, ctypes.POINTER(i64)]
        L.kvh_load_host_static.restype = i32
        L.kvh_load_host_static.argtypes = [vp, vp, vp, i32, vp, i64, ctypes.POINTER(_PoolStruct), vp, vp, u64, vp, vp]
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != 0:
        raise KvhError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def format_version() -> int:
    return lib().kvh_format_version()


def build_variant() -> str:
    return lib().kvh_build_variant().decode()


def status_string(status: int) -> str:
    return lib().kvh_status_string(status).decode()


def level_info(level: int) -> tuple[int, int, bool]:
    bits, group, lossless = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    _check(lib().kvh_level_info(level, ctypes.byref(bits), ctypes.byref(group), ctypes.byref(lossless)),
           "kvh_level_info")
    return bits.value, group.value, bool(lossless.value)


def level_bytes(level: int, n_layers: int, n_channels: int, n_tokens: int) -> int:
    out = ctypes.c_uint64()
    _check(lib().kvh_level_bytes(level, n_layers, n_channels, n_tokens, ctypes.byref(out)), "kvh_level_bytes")
    return out.value


def plan_chunks(n_layers: int, n_channels: int, n_tokens: int, levels, stream_base: int = 0,
                pt_base: int = 0, page_tokens: int = 16) -> tuple[np.ndarray, int]:
    """Host layout of a context: (descriptor array of dtype DESC_DTYPE, total stream bytes).
    `levels` is one int for the whole context or a sequence with one level per chunk."""
    n_chunks = (n_tokens + CHUNK_TOKENS - 1) // CHUNK_TOKENS
    descs = np.zeros(max(n_chunks, 0), dtype=DESC_DTYPE)
    total = ctypes.c_uint64()
    if isinstance(levels, (int, np.integer)):
        lv_ptr, level = None, int(levels)
    else:
        lv = np.ascontiguousarray(levels, dtype=np.int32)
        if lv.size != n_chunks:
            raise ValueError(f"need {n_chunks} chunk levels, got {lv.size}")
        lv_ptr, level = lv.ctypes.data, 0
    _check(lib().kvh_plan_chunks(n_layers, n_channels, n_tokens, lv_ptr, level, stream_base, pt_base,
                                 page_tokens, descs.ctypes.data, ctypes.byref(total)), "kvh_plan_chunks")
    return descs, total.value


def descs_to_tensor(descs: np.ndarray, device) -> torch.Tensor:
    """Copy a host descriptor array to the device as a flat uint8 tensor."""
    assert descs.dtype == DESC_DTYPE
    return torch.from_numpy(descs.view(np.uint8).copy()).to(device)


@dataclass
class Pool:
    """The serving engine's paged KV pool: a bf16 tensor [l][2][num_pages][page_tokens][c]
    (any strides for the first three axes; the last two contiguous)."""
    tensor: torch.Tensor

    def __post_init__(self):
        t = self.tensor
        assert t.dtype == torch.bfloat16 and t.dim() == 5 and t.shape[1] == 2
        assert t.stride(4) == 1 and t.stride(3) == t.shape[4]
        self.struct = _PoolStruct(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2), t.shape[2], t.shape[3],
                                  t.shape[0], t.shape[4])

    @classmethod
    def allocate(cls, n_layers: int, num_pages: int, n_channels: int, page_tokens: int = 16,
                 device="cuda") -> "Pool":
        return cls(torch.empty((n_layers, 2, num_pages, page_tokens, n_channels), dtype=torch.bfloat16,
                               device=device))


def _check_kv(kv: torch.Tensor):
    if not (kv.is_cuda and kv.dtype == torch.bfloat16 and kv.dim() == 4 and kv.shape[1] == 2
            and kv.is_contiguous()):
        raise ValueError("kv must be a contiguous CUDA bf16 tensor [l][2][N][c]")
    return kv.shape[0], kv.shape[2], kv.shape[3]


def encode(kv: torch.Tensor, level: int, out: torch.Tensor | None = None,
           dev_status: torch.Tensor | None = None) -> tuple[torch.Tensor, int]:
    """Encode a whole context at one level.  Returns (uint8 stream tensor, bytes used)."""
    l, N, c = _check_kv(kv)
    _, total = plan_chunks(l, c, N, level)
    if out is None:
        out = torch.empty(total, dtype=torch.uint8, device=kv.device)
    _check(lib().kvh_encode(kv.data_ptr(), l, N, c, level, out.data_ptr(), out.numel(), _ptr(dev_status),
                            _stream()), "kvh_encode")
    return out, total


def encode_chunks(kv: torch.Tensor, descs_dev: torch.Tensor, n_chunks: int, out: torch.Tensor,
                  dev_status: torch.Tensor | None = None, descs: np.ndarray | None = None) -> None:
    """Encode a context with one level per chunk; descs_dev is the device copy of plan_chunks()'s
    array.  Passing the host array too (`descs`) lets the library run each level's chunks through
    the kernel specialised for that level."""
    l, N, c = _check_kv(kv)
    host = 0
    if descs is not None:
        assert descs.dtype == DESC_DTYPE and len(descs) == n_chunks and descs.flags.c_contiguous
        host = descs.ctypes.data
    _check(lib().kvh_encode_chunks(kv.data_ptr(), l, N, c, descs_dev.data_ptr(), host, n_chunks, out.data_ptr(),
                                   out.numel(), _ptr(dev_status), _stream()), "kvh_encode_chunks")


def decode_to_pages(chunk: torch.Tensor, level: int, n_tok: int, page_ids: torch.Tensor, pool: Pool,
                    dev_status: torch.Tensor | None = None) -> None:
    """Decode one stored chunk (uint8 CUDA tensor starting at the chunk) into the pool."""
    assert chunk.is_cuda and chunk.dtype == torch.uint8 and page_ids.is_cuda and page_ids.dtype == torch.int32
    need = level_bytes(level, pool.struct.n_layers, pool.struct.n_channels, n_tok)
    if chunk.numel() < need:
        raise KvhError(5, "decode_to_pages")
    if page_ids.numel() < -(-n_tok // pool.struct.page_tokens):
        raise KvhError(5, "decode_to_pages")
    _check(lib().kvh_decode_to_pages(chunk.data_ptr(), level, n_tok, page_ids.data_ptr(),
                                     ctypes.byref(pool.struct), _ptr(dev_status), _stream()),
           "kvh_decode_to_pages")


def decode_batch(streams: torch.Tensor, descs_dev: torch.Tensor, n_chunks: int, page_table: torch.Tensor,
                 pool: Pool, dev_status: torch.Tensor | None = None) -> None:
    """Decode n_chunks stored chunks of mixed levels in one launch."""
    assert streams.is_cuda and streams.dtype == torch.uint8
    assert page_table.is_cuda and page_table.dtype == torch.int32
    assert descs_dev.is_cuda and descs_dev.numel() >= 24 * n_chunks
    _check(lib().kvh_decode_batch(streams.data_ptr(), streams.numel(), descs_dev.data_ptr(), n_chunks,
                                  page_table.data_ptr(), page_table.numel(), ctypes.byref(pool.struct),
                                  _ptr(dev_status), _stream()), "kvh_decode_batch")


def load_host(host_streams: torch.Tensor, staging: torch.Tensor, descs: np.ndarray, descs_dev: torch.Tensor,
              page_table: torch.Tensor, pool: Pool, dev_status: torch.Tensor | None,
              host_status: torch.Tensor | None, copy_stream: torch.cuda.Stream, slice_bytes: int = 0) -> None:
    """Host-tier cache hit: copy the stored chunks from pinned host memory and decode them into the
    pool, slice by slice, the copy on copy_stream overlapping the decode on the current stream."""
    assert host_streams.is_pinned() and host_streams.dtype == torch.uint8 and descs.dtype == DESC_DTYPE
    assert staging.is_cuda and staging.dtype == torch.uint8
    assert host_status is None or (host_status.is_pinned() and host_status.dtype == torch.int32)
    need = int(descs["stream_off"][-1]) + level_bytes(int(descs["level"][-1]), pool.struct.n_layers,
                                                       pool.struct.n_channels, int(descs["n_tok"][-1]))
    if host_streams.numel() < need:
        raise KvhError(5, "load_host")
    _check(lib().kvh_load_host(host_streams.data_ptr(), staging.data_ptr(), staging.numel(), descs.ctypes.data,
                               descs_dev.data_ptr(), len(descs), page_table.data_ptr(), page_table.numel(),
                               ctypes.byref(pool.struct), _ptr(dev_status), _ptr(host_status), slice_bytes,
                               copy_stream.cuda_stream, _stream()), "kvh_load_host")


def store_host(kv: torch.Tensor, descs: np.ndarray, descs_dev: torch.Tensor, staging: torch.Tensor,
               host_out: torch.Tensor, dev_status: torch.Tensor | None, host_status: torch.Tensor | None,
               copy_stream: torch.cuda.Stream, slice_bytes: int = 0) -> None:
    """Store to the host tier: encode the context slice by slice on the current stream and copy
    each slice's streams to pinned host memory on copy_stream."""
    l, N, c = _check_kv(kv)
    assert host_out.is_pinned() and host_out.dtype == torch.uint8 and descs.dtype == DESC_DTYPE
    need = int(descs["stream_off"][-1]) + level_bytes(int(descs["level"][-1]), l, c, int(descs["n_tok"][-1]))
    if host_out.numel() < need:
        raise KvhError(5, "store_host")
    _check(lib().kvh_store_host(kv.data_ptr(), l, N, c, descs.ctypes.data, descs_dev.data_ptr(), len(descs),
                                staging.data_ptr(), staging.numel(), host_out.data_ptr(), _ptr(dev_status),
                                _ptr(host_status), slice_bytes, copy_stream.cuda_stream, _stream()),
           "kvh_store_host")


STATIC_STAGING_BYTES = 64 << 20


def load_host_static(host_streams: torch.Tensor, descs: np.ndarray, descs_dev: torch.Tensor,
                     page_table: torch.Tensor, pool: Pool, dev_status: torch.Tensor | None,
                     host_status: torch.Tensor | None, copy_stream: torch.cuda.Stream, slice_bytes: int = 0) -> None:
    """load_host() for callers that cannot allocate device memory: the chunks are staged in a fixed
    array of STATIC_STAGING_BYTES inside the library instead of a tensor of the caller's.  The
    stream offsets in `descs` must end within that size.  Calls on one device share the array, so
    keep them on one stream (or order them with events)."""
    assert host_streams.is_pinned() and host_streams.dtype == torch.uint8 and descs.dtype == DESC_DTYPE
    assert host_status is None or (host_status.is_pinned() and host_status.dtype == torch.int32)
    need = int(descs["stream_off"][-1]) + level_bytes(int(descs["level"][-1]), pool.struct.n_layers,
                                                       pool.struct.n_channels, int(descs["n_tok"][-1]))
    if host_streams.numel() < need:
        raise KvhError(5, "load_host_static")
    _check(lib().kvh_load_host_static(host_streams.data_ptr(), descs.ctypes.data, descs_dev.data_ptr(), len(descs),
                                      page_table.data_ptr(), page_table.numel(), ctypes.byref(pool.struct),
                                      _ptr(dev_status), _ptr(host_status), slice_bytes, copy_stream.cuda_stream,
                                      _stream()), "kvh_load_host_static")


RUN_DTYPE = np.dtype([("first", "<i8"), ("count", "<i8")])


def keep_sinks_and_recent(n_tokens: int, n_sink: int, n_recent: int) -> tuple[np.ndarray, int]:
    """Kept runs (array of RUN_DTYPE) and the number of kept tokens when the first n_sink and the
    last n_recent tokens of a context survive."""
    runs = np.zeros(2, dtype=RUN_DTYPE)
    n, kept = ctypes.c_int(), ctypes.c_int64()
    _check(lib().kvh_keep_sinks_and_recent(n_tokens, n_sink, n_recent, runs.ctypes.data, ctypes.byref(n),
                                           ctypes.byref(kept)), "kvh_keep_sinks_and_recent")
    return runs[:n.value].copy(), kept.value


def encode_kept(kv: torch.Tensor, runs, descs_dev: torch.Tensor | None, n_chunks: int, out: torch.Tensor,
                dev_status: torch.Tensor | None = None, level: int = -1) -> None:
    """Token dropping: encode only the kept runs of a context, compacted.  descs_dev lays out the
    chunks of the kept sequence (plan_chunks for n_kept tokens); with one level for all chunks pass
    `level` (descs_dev may then be None: chunks back to back) and the specialised kernel runs."""
    l, N, c = _check_kv(kv)
    r = np.ascontiguousarray(np.asarray(runs, dtype=RUN_DTYPE) if not isinstance(runs, np.ndarray) else runs)
    assert r.dtype == RUN_DTYPE
    _check(lib().kvh_encode_kept(kv.data_ptr(), l, N, c, r.ctypes.data, len(r), _ptr(descs_dev), n_chunks, level,
                                 out.data_ptr(), out.numel(), _ptr(dev_status), _stream()), "kvh_encode_kept")


def transcode(in_streams: torch.Tensor, in_descs_dev: torch.Tensor, out_streams: torch.Tensor,
              out_descs_dev: torch.Tensor, n_chunks: int, n_layers: int, n_channels: int,
              level_in: int = -1, level_out: int = -1, dev_status: torch.Tensor | None = None,
              in_descs: np.ndarray | None = None, out_descs: np.ndarray | None = None) -> None:
    """Re-encode stored chunks at a coarser level on the device.  level_in/level_out name the one
    pair of levels all chunks share, or -1/-1 for a mix taken from the descriptors; for a mix the
    host arrays (in_descs, out_descs) let every pair of levels run through its own kernel."""
    assert in_streams.is_cuda and in_streams.dtype == torch.uint8
    assert out_streams.is_cuda and out_streams.dtype == torch.uint8
    assert in_descs_dev.numel() >= 24 * n_chunks and out_descs_dev.numel() >= 24 * n_chunks
    hi = ho = 0
    if in_descs is not None and out_descs is not None:
        assert in_descs.dtype == DESC_DTYPE and out_descs.dtype == DESC_DTYPE
        assert len(in_descs) == len(out_descs) == n_chunks and in_descs.flags.c_contiguous and out_descs.flags.c_contiguous
        hi, ho = in_descs.ctypes.data, out_descs.ctypes.data
    _check(lib().kvh_transcode(in_streams.data_ptr(), in_streams.numel(), in_descs_dev.data_ptr(),
                               out_streams.data_ptr(), out_streams.numel(), out_descs_dev.data_ptr(), hi, ho, n_chunks,
                               n_layers, n_channels, level_in, level_out, _ptr(dev_status), _stream()),
           "kvh_transcode")


OPTION_DTYPE = np.dtype([("size", "<u8"), ("quality", "<f8")])
TIER_DTYPE = np.dtype([("alpha", "<f8"), ("bandwidth", "<f8"), ("capacity", "<u8")])


def _policy_args(freq, options, option_begin):
    f = np.ascontiguousarray(freq, dtype=np.float64)
    o = np.ascontiguousarray(options, dtype=OPTION_DTYPE)
    b = np.ascontiguousarray(option_begin, dtype=np.int32)
    assert b.size == f.size + 1 and b[0] == 0 and b[-1] == o.size
    return f, o, b


def policy_assign(freq, options, option_begin, alpha: float, bandwidth: float, capacity: int):
    """Greedy marginal-utility choice of a stored form per entry for one tier.
    Returns (choice per entry, -1 = evicted; bytes used; total utility)."""
    f, o, b = _policy_args(freq, options, option_begin)
    tier = np.array([(alpha, bandwidth, capacity)], dtype=TIER_DTYPE)
    choice = np.empty(f.size, dtype=np.int32)
    used, total = ctypes.c_uint64(), ctypes.c_double()
    _check(lib().kvh_policy_assign(f.ctypes.data, o.ctypes.data, b.ctypes.data, f.size, tier.ctypes.data,
                                   choice.ctypes.data, ctypes.byref(used), ctypes.byref(total)), "kvh_policy_assign")
    return choice, used.value, total.value


def policy_assign_tiers(freq, options, option_begin, tiers):
    """The same over several tiers, fastest first; tiers: (alpha, bandwidth, capacity) each.
    Returns (tier per entry or -1, choice per entry or -1)."""
    f, o, b = _policy_args(freq, options, option_begin)
    t = np.array([tuple(x) for x in tiers], dtype=TIER_DTYPE)
    tier_out, choice = np.empty(f.size, dtype=np.int32), np.empty(f.size, dtype=np.int32)
    _check(lib().kvh_policy_assign_tiers(f.ctypes.data, o.ctypes.data, b.ctypes.data, f.size, t.ctypes.data, len(t),
                                         tier_out.ctypes.data, choice.ctypes.data), "kvh_policy_assign_tiers")
    return tier_out, choice


def check_page_table(page_table, num_pages: int) -> tuple[int, int]:
    """(status, index of the first offending entry or -1) of a host page table: 0 fine, 6 an id
    outside the pool, 1 an id used twice."""
    t = np.ascontiguousarray(page_table, dtype=np.int32)
    bad = ctypes.c_int64(-1)
    st = lib().kvh_check_page_table(t.ctypes.data, t.size, num_pages, ctypes.byref(bad))
    return st, bad.value
