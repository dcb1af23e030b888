"""B200-native per-chunk KV-cache codec: thin Python binding over the C ABI in include/kvh.h.

Every step of the path runs in the CUDA kernels of ``libkvh.so``; this package
only marshals arguments (tensor pointers, the current CUDA stream).  There is no
CPU fallback: calling into the library without the built extension raises.
"""
from .binding import (  # noqa: F401
    CHUNK_TOKENS, GROUP, NUM_LEVELS, ChunkDesc, KvhError, Pool, decode_batch, decode_to_pages,
    descs_to_tensor, encode, encode_chunks, format_version, build_variant, level_bytes, level_info, lib, load_host,
    load_host_static, plan_chunks, keep_sinks_and_recent, encode_kept, RUN_DTYPE, transcode, check_page_table, policy_assign, policy_assign_tiers, OPTION_DTYPE, TIER_DTYPE, status_string, store_host, STATIC_STAGING_BYTES,
)


def variant(name: str):
    """A second instance of the binding, bound to another build of the same sources: "direct" (the
    one-CTA-per-tile kernels wherever they apply) or "static" (fixed tile stride instead of cluster
    launch control).  The tests use it to check both kernel families on every shape and the
    benchmark to compare the two schedules; the library proper has no run-time switch.  Builds the
    variant if it is missing or stale."""
    import importlib.util
    import sys

    from . import _build, binding
    if name == "default":
        return binding
    if name not in ("direct", "static"):
        raise ValueError(f"unknown build variant {name!r}")
    path = _build.build(variant=name)
    modname = f"{__name__}._binding_{name}"
    if modname in sys.modules:
        return sys.modules[modname]
    spec = importlib.util.spec_from_file_location(modname, binding.__file__)
    mod = importlib.util.module_from_spec(spec)
    sys.modules[modname] = mod
    spec.loader.exec_module(mod)
    mod._LIB_PATH = path
    mod.lib()
    return mod
