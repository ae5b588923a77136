"""Builds ``libpot_b200.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2507_11959_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
LIB = HERE / "libpot_b200.so"
LIB_CHECKED = HERE / "libpot_b200_checked.so"   # the same sources with -DPOT_CHECKED (device-side index checks)
OBJ_DIR = HERE / "build"
SOURCES = ["api.cu", "quantize.cu", "dequant.cu", "gemv.cu", "gemm.cu", "gemm_prefill.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--use_fast_math=false"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _deps_mtime() -> float:
    files = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [HERE.parent / "include" / "pot.h", Path(__file__)]
    return max(f.stat().st_mtime for f in files)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> Path:
    """Build the library; checked=True builds the variant whose kernels verify their indices before every store,
    atomic and streamed shared-memory read and report a violation through the error words instead of accessing."""
    LIB = LIB_CHECKED if checked else globals()["LIB"]
    OBJ_DIR = HERE / ("build_checked" if checked else "build")
    sources = [s for s in SOURCES if (CSRC / s).exists()]
    if not force and LIB.exists() and LIB.stat().st_mtime >= _deps_mtime():
        return LIB
    OBJ_DIR.mkdir(exist_ok=True)
    nvcc = _nvcc()
    flags = [f for f in NVCC_FLAGS if f != "--use_fast_math=false"] + (["-DPOT_CHECKED"] if checked else [])
    flags += os.environ.get("POT_NVCC_FLAGS", "").split()  # extra compiler flags (experiments)
    if verbose:
        flags += ["-Xptxas", "-v"]

    def compile_one(src: str) -> Path:
        obj = OBJ_DIR / (src + ".o")
        extra = os.environ.get("POT_NVCC_FLAGS_" + src.split(".")[0].upper(), "").split()
        cmd = [nvcc, *flags, *extra, "-c", str(CSRC / src), "-o", str(obj)]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write(f"$ {' '.join(cmd)}\n{r.stdout}{r.stderr}\n")
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(sources))) as ex:
        objs = list(ex.map(compile_one, sources))
    tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
    cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp), *map(str, objs), "-lcuda"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("link failed")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
