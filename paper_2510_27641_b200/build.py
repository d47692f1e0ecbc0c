"""Builds libspecattn.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Each source is compiled to an object of its own (in parallel, and only when it or a header
changed), then the objects are linked into the shared library."""
from __future__ import annotations

import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
INCLUDE = PKG.parent / "include"
LIB = PKG / "libspecattn.so"
OBJ = PKG / "_build"
SOURCES = ["api.cu", "select_topp.cu", "sparse_verify.cu"]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "-I", str(INCLUDE), "-I", str(CSRC)]


def _headers() -> list[Path]:
    return list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h")) + list(INCLUDE.glob("*.h"))


def _stale(target: Path, deps: list[Path]) -> bool:
    return not target.exists() or any(d.stat().st_mtime > target.stat().st_mtime for d in deps)


def needs_build() -> bool:
    return _stale(LIB, [CSRC / s for s in SOURCES] + _headers())


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not needs_build():
        return LIB
    OBJ.mkdir(exist_ok=True)
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src: str) -> Path:
        obj = OBJ / (src + ".o")
        if force or verbose or _stale(obj, [CSRC / src] + _headers()):
            subprocess.run(["nvcc", *FLAGS, *extra, "-c", str(CSRC / src), "-o", str(obj)], check=True)
        return obj

    with ThreadPoolExecutor(len(SOURCES)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    subprocess.run(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-Xcompiler", "-fPIC",
                    *[str(o) for o in objs], "-ldl", "-o", str(LIB)], check=True)
    return LIB


if __name__ == "__main__":
    build(force="-f" in sys.argv or "-v" in sys.argv, verbose="-v" in sys.argv)
    print(LIB)
