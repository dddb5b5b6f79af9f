"""Builds the CUDA library in-tree: nvcc, sm_100a only, one shared object next to the sources."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
LIB = HERE / "libvardrop.so"
SOURCES = ["vardrop_api.cu", "hash.cu", "hash_rows.cu", "select.cu", "attn_fwd.cu", "attn_bwd.cu", "pearson.cu", "gather_rows.cu"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def needs_build() -> bool:
    if not LIB.exists():
        return True
    newest = max(p.stat().st_mtime for p in list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h"))
                 + [HERE.parent / "include" / "vardrop.h"])
    return LIB.stat().st_mtime < newest


def _headers_mtime() -> float:
    return max(p.stat().st_mtime for p in list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h")) + [HERE.parent / "include" / "vardrop.h"])


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compiles every translation unit that is out of date (objects live in _build/, compiled side by side) and links
    the shared object."""
    if not force and not needs_build():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    obj_dir = HERE / "_build"
    obj_dir.mkdir(exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17", "-Xcompiler", "-fPIC"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    hdr = _headers_mtime()

    def compile_one(name: str) -> Path:
        src, obj = CSRC / name, obj_dir / (name + ".o")
        if force or verbose or not obj.exists() or obj.stat().st_mtime < max(src.stat().st_mtime, hdr):
            subprocess.check_call([_nvcc(), *flags, "-c", "-o", str(obj), str(src)])
        return obj

    with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
    subprocess.check_call([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", str(tmp), *[str(o) for o in objs]])
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="-v" in sys.argv)
    print(LIB)
