"""Builds ``libmoc.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Every ``csrc/*.cu`` is compiled to an object of its own (in parallel; an object is reused while the
hash of its source, the headers and the flags is unchanged) and the objects are linked into the
shared library.  ``build(debug=True)`` makes ``libmoc_debug.so`` from the same sources with
``-DMOC_DEBUG``: every index a kernel takes from the workspace is checked there before it is used.
"""
from __future__ import annotations

import glob
import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_DIR, "csrc")
LIB = os.path.join(_DIR, "libmoc.so")
LIB_DEBUG = os.path.join(_DIR, "libmoc_debug.so")
INCLUDE = os.path.join(os.path.dirname(_DIR), "include")
OBJ_DIR = os.path.join(_DIR, "_build")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--use_fast_math", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return sorted(glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h")))


def _digest(src: str, flags) -> str:
    h = hashlib.sha1(" ".join(flags).encode())
    for f in [src] + _headers():
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def _source_digest(flags) -> str:
    h = hashlib.sha1(" ".join(flags).encode())
    for f in sources() + _headers():
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def lib_of(debug: bool = False) -> str:
    return LIB_DEBUG if debug else LIB


def stale(debug: bool = False) -> bool:
    lib = lib_of(debug)
    if not os.path.exists(lib):
        return True
    try:
        with open(lib + ".sha1") as f:
            return f.read().strip() != _source_digest(_flags(debug))
    except OSError:
        return True


def _flags(debug: bool):
    return NVCC_FLAGS + (["-DMOC_DEBUG"] if debug else [])


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = lib_of(debug)
    if not force and not stale(debug):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = _flags(debug)
    odir = os.path.join(OBJ_DIR, "debug" if debug else "release")
    os.makedirs(odir, exist_ok=True)

    def compile_one(src):
        obj = os.path.join(odir, os.path.basename(src)[:-3] + ".o")
        want = _digest(src, flags)
        try:
            with open(obj + ".sha1") as f:
                if not force and f.read().strip() == want and os.path.exists(obj):
                    with open(obj + ".log") as lf:
                        return obj, 0, lf.read()
        except OSError:
            pass
        res = subprocess.run([nvcc, *flags, "-I", INCLUDE, "-c", "-o", obj, src], capture_output=True, text=True)
        if res.returncode == 0:
            with open(obj + ".log", "w") as lf:
                lf.write(res.stderr)
            with open(obj + ".sha1", "w") as f:
                f.write(want)
        return obj, res.returncode, res.stdout + res.stderr

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        results = list(pool.map(compile_one, sources()))
    log = "".join(r[2] for r in results)
    if verbose or any(r[1] for r in results):
        sys.stderr.write(log)
    if any(r[1] for r in results):
        raise RuntimeError("nvcc failed building " + os.path.basename(lib))
    tmp = lib + f".{os.getpid()}.tmp"
    res = subprocess.run([nvcc, "-shared", "-o", tmp, *[r[0] for r in results], "-ldl"], capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("link failed building " + os.path.basename(lib))
    if not debug:
        with open(os.path.join(_DIR, "libmoc.ptxas.log"), "w") as f:
            f.write(log)
    os.replace(tmp, lib)
    with open(lib + ".sha1", "w") as f:
        f.write(_source_digest(flags))
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True, debug="--debug" in sys.argv))
