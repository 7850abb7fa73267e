"""Builds the CUDA library in-tree with nvcc for sm_100a.

    python -m paper_2407_15452_b200.build [--force] [--verbose]

Sources: csrc/*.cu; public header: include/gs.h at the repository root.
Output: paper_2407_15452_b200/libgs_b200.so (objects under _build/).
Also builds the benchmark's own measurement aid, bench_probe.cu at the repository root, into
libbench_probe.so beside it (not part of the library).
"""
from __future__ import annotations

import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
INCLUDE = ROOT / "include"
LIB = PKG / "libgs_b200.so"
OBJ_DIR = ROOT / "_build"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-I", str(INCLUDE), "-I", str(CSRC),
]


def _stale(target: Path, deps) -> bool:
    if not target.exists():
        return True
    t = target.stat().st_mtime
    return any(d.stat().st_mtime > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> Path:
    sources = sorted(CSRC.glob("*.cu"))
    headers = sorted(CSRC.glob("*.cuh")) + sorted(INCLUDE.glob("*.h"))
    OBJ_DIR.mkdir(exist_ok=True)
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src: Path) -> Path:
        obj = OBJ_DIR / (src.stem + ".o")
        if force or _stale(obj, [src] + headers):
            cmd = ["nvcc", *NVCC_FLAGS, *extra, "-c", str(src), "-o", str(obj)]
            r = subprocess.run(cmd, capture_output=True, text=True)
            if verbose or r.returncode != 0:
                sys.stderr.write(r.stdout + r.stderr)
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed on {src.name}")
        return obj

    with ThreadPoolExecutor(max_workers=4) as pool:
        objs = list(pool.map(compile_one, sources))
    if force or _stale(LIB, objs):
        cmd = ["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
               "-o", str(LIB), *map(str, objs)]
        subprocess.run(cmd, check=True)
    return LIB


PROBE_SRC = ROOT / "bench_probe.cu"
PROBE_LIB = ROOT / "libbench_probe.so"


def build_probe(force: bool = False) -> Path:
    """The random-read probe that bench.py --stage walks loads (one file, no dependencies)."""
    if force or _stale(PROBE_LIB, [PROBE_SRC]):
        cmd = ["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
               "-std=c++17", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
               "-o", str(PROBE_LIB), str(PROBE_SRC)]
        subprocess.run(cmd, check=True)
    return PROBE_LIB


if __name__ == "__main__":
    print(build_probe(force="--force" in sys.argv))
    print(build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
