"""Builds libws.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2004_13336_b200.build [--force] [--verbose] [--debug]

Each .cu file is compiled to an object in csrc/build/ (in parallel) and the
objects are linked into paper_2004_13336_b200/libws.so.  nvcc cross-compiles
without a GPU.  --debug builds the bounds-checking copy instead
(-DWS_DEBUG_BOUNDS, objects in csrc/build_debug/, libws_debug.so).
"""
from __future__ import annotations

import concurrent.futures as cf
import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
_OBJ = os.path.join(_CSRC, "build")
_OBJ_DEBUG = os.path.join(_CSRC, "build_debug")
LIB_PATH = os.path.join(_PKG, "libws.so")
DEBUG_LIB_PATH = os.path.join(_PKG, "libws_debug.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
    "-I", os.path.join(_ROOT, "include"), "-I", _CSRC,
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _sources():
    return sorted(f for f in os.listdir(_CSRC) if f.endswith(".cu"))


def _headers():
    """Every header a .cu file may include: a change to any of them recompiles every object."""
    hs = [os.path.join(_CSRC, f) for f in sorted(os.listdir(_CSRC)) if f.endswith((".h", ".cuh"))]
    hs.append(os.path.join(_ROOT, "include", "ws.h"))
    return hs


def _deps_mtime() -> float:
    paths = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC) if f.endswith((".cu", ".h", ".cuh"))]
    paths.append(os.path.join(_ROOT, "include", "ws.h"))
    return max(os.path.getmtime(p) for p in paths)


def up_to_date(debug: bool = False) -> bool:
    lib = DEBUG_LIB_PATH if debug else LIB_PATH
    return os.path.exists(lib) and os.path.getmtime(lib) >= _deps_mtime()


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib_path, obj_dir = (DEBUG_LIB_PATH, _OBJ_DEBUG) if debug else (LIB_PATH, _OBJ)
    if not force and up_to_date(debug):
        return lib_path
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()
    extra = ["-Xptxas", "-v"] if verbose else []
    if debug:
        extra.append("-DWS_DEBUG_BOUNDS")
    hdr_mtime = max(os.path.getmtime(h) for h in _headers())

    def compile_one(src: str) -> str:
        obj = os.path.join(obj_dir, src[:-3] + ".o")
        spath = os.path.join(_CSRC, src)
        if (not force and os.path.exists(obj)
                and os.path.getmtime(obj) >= max(os.path.getmtime(spath), hdr_mtime)):
            return obj
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", spath, "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose:
            sys.stderr.write(res.stderr)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed for {src}:\n{res.stdout}\n{res.stderr}")
        return obj

    with cf.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        objs = list(ex.map(compile_one, _sources()))
    cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib_path, *objs]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError(f"link failed:\n{res.stdout}\n{res.stderr}")
    return lib_path


if __name__ == "__main__":
    path = build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv)
    print(path)
