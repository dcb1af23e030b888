"""Build the CUDA library in-tree with nvcc for sm_100a."""
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


def sources() -> list[Path]:
    return sorted(CSRC.glob("*.cu"))


def _stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list((ROOT / "include").glob("*.h"))
    return any(d.stat().st_mtime > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile csrc/*.cu into libkvh.so beside this file (cross-compiles without a GPU)."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    objdir = PKG / "_build"
    objdir.mkdir(exist_ok=True)
    common = [nvcc, *NVCC_FLAGS, f"-I{ROOT / 'include'}", f"-I{CSRC}"]
    if verbose:
        common.insert(1, "-Xptxas=-v")
    # one compiler process per translation unit, side by side; then one link
    jobs = []
    for src in sources():
        obj = objdir / (src.stem + f".{os.getpid()}.o")
        jobs.append((obj, subprocess.Popen([*common, "-c", "-o", str(obj), str(src)])))
    failed = [str(obj) for obj, proc in jobs if proc.wait() != 0]
    if failed:
        raise RuntimeError(f"nvcc failed for {failed}")
    tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
    subprocess.run([nvcc, "-shared", "-o", str(tmp), *[str(obj) for obj, _ in jobs]], check=True)
    for obj, _ in jobs:
        obj.unlink()
    os.replace(tmp, LIB)
    return LIB
