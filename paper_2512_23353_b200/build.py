"""Builds libisopo.so (hand-written CUDA for sm_100a) in-tree with nvcc.

Usage: python -m paper_2512_23353_b200.build [--force] [--debug] [-v]

--debug builds libisopo_debug.so instead: the same sources with -DISOPO_DEBUG, in which every
data-dependent index of the kernels is range-checked before use (a violation skips the access and
sets *info = ISOPO_INFO_BOUNDS | kernel id).  ISOPO_LIB_VARIANT=debug makes the binding load it.
"""

from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
OBJ_DIR = os.path.join(PKG_DIR, "_build")
LIB_PATH = os.path.join(PKG_DIR, "libisopo.so")
DEBUG_LIB_PATH = os.path.join(PKG_DIR, "libisopo_debug.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC,-fvisibility=hidden", "--expt-relaxed-constexpr",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _deps_mtime():
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "isopo.h"), __file__]
    return max(os.path.getmtime(p) for p in paths)


def _compile(src, verbose, debug):
    obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + (".dbg.o" if debug else ".o"))
    cmd = ["nvcc", *NVCC_FLAGS, *(["-DISOPO_DEBUG"] if debug else []), "-c", src, "-o", obj]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
    return obj, r.stderr


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compiles every .cu under csrc/ and links libisopo.so (libisopo_debug.so with `debug`); returns its path."""
    lib_path = DEBUG_LIB_PATH if debug else LIB_PATH
    if not force and os.path.exists(lib_path) and os.path.getmtime(lib_path) >= _deps_mtime():
        return lib_path
    os.makedirs(OBJ_DIR, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=8) as ex:
        results = list(ex.map(lambda s: _compile(s, verbose, debug), _sources()))
    if verbose:
        for _, log in results:
            sys.stderr.write(log)
    cmd = ["nvcc", "-shared", "-o", lib_path, *[o for o, _ in results], "-cudart", "static", "-Xlinker",
           "--exclude-libs=ALL", "-ldl"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
