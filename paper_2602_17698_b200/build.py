"""Builds the C-ABI CUDA library in-tree with nvcc for sm_100a (no JIT cache).

Every `csrc/*.cu` is compiled to its own object (in parallel, only when it or a header changed)
and the objects are linked into `libscalebits.so`; no file uses another file's device symbols,
so no relocatable device code is needed.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libscalebits.so")
LIB_CHECKED = os.path.join(PKG, "libscalebits_checked.so")     # built with -DSB_CHECKED

NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))


def _obj(src: str, tag: str) -> str:
    return os.path.join(OBJ, os.path.splitext(os.path.basename(src))[0] + tag + ".o")


def _newer(path: str, deps) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(d) > t for d in deps)


def stale(lib: str = LIB) -> bool:
    return _newer(lib, sources() + headers())


def build(force: bool = False, verbose: bool = False, defines=(), lib: str = LIB) -> str:
    """Compile and link; `defines` (e.g. ["SB_CHECKED"]) select a variant built into `lib`."""
    if not force and not stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    tag = "".join("_" + d for d in defines)
    dflags = ["-D" + d for d in defines]
    hdrs = headers()

    def compile_one(src: str):
        obj = _obj(src, tag)
        if not force and not _newer(obj, [src] + hdrs):
            return obj, 0, ""
        cmd = [nvcc] + NVCC_FLAGS + dflags + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", obj, src]
        res = subprocess.run(cmd, capture_output=True, text=True)
        return obj, res.returncode, res.stdout + res.stderr

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        results = list(pool.map(compile_one, sources()))
    failed = [r for r in results if r[1] != 0]
    for obj, rc, log in results:
        if log and (verbose or rc != 0):
            sys.stderr.write(log)
    if failed:
        raise RuntimeError("nvcc failed building " + ", ".join(os.path.basename(f[0]) for f in failed))
    cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib] + [r[0] for r in results]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed linking " + os.path.basename(lib))
    return lib


if __name__ == "__main__":
    print(build(force="-f" in sys.argv, verbose="-v" in sys.argv))
