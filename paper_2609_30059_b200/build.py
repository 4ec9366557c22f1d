"""Build libkop.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

`python -m paper_2609_30059_b200.build` compiles every .cu under csrc/ to an object (in parallel)
and links them, together with cuBLAS, into paper_2609_30059_b200/libkop.so. nvcc cross-compiles, so
this works on a machine without a GPU.
"""
from __future__ import annotations

import concurrent.futures
import glob
import hashlib
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libkop.so")
INCLUDE = os.path.join(ROOT, "include")

ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-I" + INCLUDE, "-I" + CSRC] + ARCH


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: libkop cannot be built")
    return exe


def _cuda_lib_dir(nvcc: str) -> str:
    return os.path.join(os.path.dirname(os.path.dirname(os.path.realpath(nvcc))), "lib64")


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + sorted(glob.glob(os.path.join(INCLUDE, "*.h")))


def _fingerprint(flags: list[str], srcs: list[str] | None = None) -> str:
    """Hash of the given sources (default: all), every header and the flags. File times are useless for this:
    a copy of the tree (another machine, a fresh checkout) has new times on unchanged files."""
    h = hashlib.sha256()
    for f in (sources() if srcs is None else srcs) + _headers():
        h.update(os.path.basename(f).encode())
        with open(f, "rb") as fh:
            h.update(fh.read())
    h.update(" ".join(x for x in flags if not x.startswith("-I")).encode())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False, extra_flags: list[str] | None = None,
          out: str | None = None) -> str:
    """Compile and link; returns the path of the shared library."""
    lib = out or LIB
    stamp = lib + ".stamp"
    base_flags = NVCC_FLAGS + (extra_flags or [])
    want = _fingerprint(base_flags)
    if not force and os.path.exists(lib) and os.path.exists(stamp):
        with open(stamp) as fh:
            if fh.read().strip() == want:
                return lib
    nvcc = _nvcc()
    os.makedirs(OBJ, exist_ok=True)
    flags = base_flags + (["-Xptxas", "-v"] if verbose else [])

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJ, os.path.basename(src)[:-3] + (".o" if out is None else f".{os.getpid()}.o"))
        # an object whose source, headers and flags are unchanged is kept (not when forced or verbose)
        ostamp = obj + ".stamp"
        owant = _fingerprint(base_flags, [src])
        if out is None and not force and not verbose and os.path.exists(obj) and os.path.exists(ostamp):
            with open(ostamp) as fh:
                if fh.read().strip() == owant:
                    return obj
        res = subprocess.run([nvcc, *flags, "-c", src, "-o", obj], capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        if out is None:
            with open(ostamp, "w") as fh:
                fh.write(owant + "\n")
        return obj

    with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, len(sources()))) as pool:
        objs = list(pool.map(compile_one, sources()))
    libdir = _cuda_lib_dir(nvcc)
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.run([nvcc, "-shared", *ARCH, "-o", tmp, *objs, "-L" + libdir, "-lcublas", "-lcublasLt",
                    "-Xlinker", "-rpath", "-Xlinker", libdir], check=True)
    os.replace(tmp, lib)
    with open(stamp + f".tmp{os.getpid()}", "w") as fh:
        fh.write(want + "\n")
    os.replace(stamp + f".tmp{os.getpid()}", stamp)
    if out is not None:
        for o in objs:
            os.remove(o)
    return lib


if __name__ == "__main__":
    print(build(force="--incremental" not in sys.argv, verbose="-v" in sys.argv))
