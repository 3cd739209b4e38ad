"""Builds libtensair.so (sm_100a only) next to this file with nvcc.

Run as `python -m paper_2211_10280_b200.build [--verbose] [--bounds]`.  With --bounds the checked build is made
instead (-DTENSAIR_BOUNDS: every data-dependent index is compared with its bound on the device) and written to
libtensair_checked.so; the binding loads it when the environment variable TENSAIR_CHECKED is 1.  Sources are compiled in parallel into
`_build/` objects and linked into one shared library; nothing is rebuilt when the sources are older
than the library.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
INCLUDE = HERE.parent / "include"
LIB = HERE / "libtensair.so"
LIB_CHECKED = HERE / "libtensair_checked.so"
OBJ = HERE / "_build"

SOURCES = ["tensair.cu", "schedule.cu", "sampler.cu", "radix_sort.cu", "forward.cu", "message.cu", "apply.cu",
           "static_scratch.cu", "merge.cu", "topk.cu", "alias_build.cu"]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and Path(cand).exists():
            return cand
    raise RuntimeError("nvcc not found; the CUDA library cannot be built")


def _deps():
    return [p for p in list(CSRC.glob("*")) + [INCLUDE / "tensair.h"] if p.is_file()]


def build(force: bool = False, verbose: bool = False, bounds: bool = False) -> Path:
    lib = LIB_CHECKED if bounds else LIB
    objdir = OBJ / "checked" if bounds else OBJ
    newest = max(p.stat().st_mtime for p in _deps())
    if not force and lib.exists() and lib.stat().st_mtime >= newest:
        return lib
    objdir.mkdir(parents=True, exist_ok=True)
    nvcc = _nvcc()
    extra = (["-Xptxas", "-v"] if verbose else []) + (["-DTENSAIR_BOUNDS"] if bounds else [])

    def compile_one(src: str):
        obj = objdir / (src + ".o")
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-I", str(INCLUDE), "-c", str(CSRC / src), "-o", str(obj)]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{res.stdout}\n{res.stderr}")
        if verbose:
            sys.stderr.write(res.stderr)
        return str(obj)

    with ThreadPoolExecutor(max_workers=min(8, len(SOURCES))) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    tmp = lib.with_suffix(f".tmp{os.getpid()}.so")
    subprocess.check_call([nvcc, "-shared", "-o", str(tmp), *objs, "-gencode", "arch=compute_100a,code=sm_100a"])
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, bounds="--bounds" in sys.argv))
