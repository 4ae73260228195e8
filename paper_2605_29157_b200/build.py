"""Builds the in-tree CUDA shared library (sm_100a) with nvcc.

Every source is compiled to an object file of its own (in parallel) and the objects are linked into
`libparallax.so`.  `build(debug_checks=True)` makes `libparallax_debug.so` from the same sources with
`-DPLX_DEBUG_CHECKS`: the kernels then verify every tile coordinate, page id and record index before
using it and report a violation through the status word (PLX_ERR_DEVICE_CHECK) instead of touching
the address.  Set the environment variable PARALLAX_LIBRARY to that file to run through it.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
import tempfile
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
SOURCES = [PKG / "csrc" / "parallax_decode.cu", PKG / "csrc" / "parallax_prefill.cu",
           PKG / "csrc" / "parallax_prepare.cu", PKG / "csrc" / "parallax_backward.cu",
           PKG / "csrc" / "parallax_probe.cu", PKG / "csrc" / "parallax_decode_rows.cu"]
HEADERS = [ROOT / "include" / "parallax.h", ROOT / "include" / "parallax_test_hooks.h",
           PKG / "csrc" / "plx_common.cuh", PKG / "csrc" / "plx_tcgen05.cuh", PKG / "csrc" / "plx_internal.h"]
LIB = PKG / "libparallax.so"
LIB_DEBUG = PKG / "libparallax_debug.so"


def nvcc_flags(verbose: bool = False, debug_checks: bool = False):
    flags = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
             "-Xcompiler", "-fPIC", "-I", str(ROOT / "include"), "-I", str(PKG / "csrc")]
    if verbose:
        flags += ["-Xptxas", "-v"]
    if debug_checks:
        flags += ["-DPLX_DEBUG_CHECKS=1"]
    return flags


def needs_build(lib: Path = LIB) -> bool:
    if not lib.exists():
        return True
    t = lib.stat().st_mtime
    return any(p.stat().st_mtime > t for p in SOURCES + HEADERS + [Path(__file__)])


def build(force: bool = False, verbose: bool = False, debug_checks: bool = False) -> Path:
    lib = LIB_DEBUG if debug_checks else LIB
    if not (force or needs_build(lib)):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = nvcc_flags(verbose, debug_checks)
    work = Path(tempfile.mkdtemp(prefix="plx_build_"))
    try:
        def compile_one(src: Path) -> Path:
            obj = work / (src.stem + ".o")
            subprocess.run([nvcc, *flags, "-c", str(src), "-o", str(obj)], check=True)
            return obj
        with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
            objects = list(pool.map(compile_one, SOURCES))
        tmp = lib.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run([nvcc, "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                        "-o", str(tmp), *[str(o) for o in objects]], check=True)
        os.replace(tmp, lib)
    finally:
        shutil.rmtree(work, ignore_errors=True)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, debug_checks="--debug-checks" in sys.argv))
