"""Build the CUDA library in-tree with nvcc for sm_100a.

Products, all beside this file:
  libkvh.so            the library (csrc/*.cu)
  libkvh_direct.so     the same sources with -DKVH_VARIANT_DIRECT: the one-CTA-per-tile kernels
                       wherever they apply, so that the tests check both kernel families
  libkvh_static.so     the same sources with -DKVH_VARIANT_STATIC_STRIDE: fixed tile stride instead
                       of cluster launch control (the benchmark's scheduling comparison)
  libkvh_selftest.so   csrc/selftest/*.cu: test-only kernels (the bounded wait run to its limit)
  libkvh_probe.so      csrc/bench/*.cu: benchmark-only streaming kernels that do no codec work
"""
from __future__ import annotations

import os
import subprocess
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libkvh.so"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]

VARIANTS = {
    "default": (LIB, CSRC, []),
    "direct": (PKG / "libkvh_direct.so", CSRC, ["-DKVH_VARIANT_DIRECT"]),
    "static": (PKG / "libkvh_static.so", CSRC, ["-DKVH_VARIANT_STATIC_STRIDE"]),
    "selftest": (PKG / "libkvh_selftest.so", CSRC / "selftest", []),
    "probe": (PKG / "libkvh_probe.so", CSRC / "bench", []),
}


def lib_path(variant: str = "default") -> Path:
    return VARIANTS[variant][0]


def sources(variant: str = "default") -> list[Path]:
    return sorted(VARIANTS[variant][1].glob("*.cu"))


def _stale(variant: str) -> bool:
    lib = lib_path(variant)
    if not lib.exists():
        return True
    t = lib.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list((ROOT / "include").glob("*.h"))
    deps += sources(variant)
    return any(d.stat().st_mtime > t for d in deps)


def _start(variant: str, verbose: bool):
    """Start one compiler process per translation unit of a variant; returns [(object, process)]."""
    nvcc = os.environ.get("NVCC", "nvcc")
    objdir = PKG / "_build"
    objdir.mkdir(exist_ok=True)
    common = [nvcc, *NVCC_FLAGS, *VARIANTS[variant][2], f"-I{ROOT / 'include'}", f"-I{CSRC}"]
    if verbose:
        common.insert(1, "-Xptxas=-v")
    jobs = []
    for src in sources(variant):
        obj = objdir / f"{src.stem}.{variant}.{os.getpid()}.o"
        jobs.append((obj, subprocess.Popen([*common, "-c", "-o", str(obj), str(src)])))
    return jobs


def _finish(variant: str, jobs) -> Path:
    nvcc = os.environ.get("NVCC", "nvcc")
    failed = [str(obj) for obj, proc in jobs if proc.wait() != 0]
    if failed:
        raise RuntimeError(f"nvcc failed for {failed}")
    lib = lib_path(variant)
    tmp = lib.with_suffix(f".so.tmp{os.getpid()}")
    subprocess.run([nvcc, "-shared", "-o", str(tmp), *[str(obj) for obj, _ in jobs]], check=True)
    for obj, _ in jobs:
        obj.unlink()
    os.replace(tmp, lib)
    return lib


def build(force: bool = False, verbose: bool = False, variant: str = "default") -> Path:
    """Compile one variant (cross-compiles without a GPU); returns the library's path."""
    if not force and not _stale(variant):
        return lib_path(variant)
    return _finish(variant, _start(variant, verbose))


def build_all(force: bool = False, verbose: bool = False) -> dict[str, Path]:
    """Compile every variant that is missing or stale, all translation units side by side."""
    todo = [v for v in VARIANTS if force or _stale(v)]
    started = {v: _start(v, verbose) for v in todo}
    for v in todo:
        _finish(v, started[v])
    return {v: lib_path(v) for v in VARIANTS}
