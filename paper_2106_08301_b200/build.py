"""Builds libmwu.so (CUDA, sm_100a) in-tree with nvcc.  No GPU is needed to build.

Every source file is compiled to an object of its own (in parallel, and only when it or a header
changed), then the objects are linked into the shared library."""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libmwu.so")
OBJ_DIR = os.path.join(HERE, "_build")
SOURCES = ["mwu_api.cu", "mwu_project.cu", "mwu_pack.cu", "mwu_gemm.cu", "mwu_gemm2.cu", "mwu_gemm3.cu",
           "mwu_conv.cu", "mwu_nm.cu", "mwu_shapes.cu", "mwu_noalloc.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _sources():
    return [os.path.join(CSRC, s) for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def _headers():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cuh")] + [os.path.join(INCLUDE, "mwu.h")]


def _obj(src: str) -> str:
    return os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def needs_build() -> bool:
    return _stale(LIB, _sources() + _headers())


def _compile(nvcc: str, src: str, verbose: bool):
    cmd = [nvcc] + ARCH + ["-O3", "-lineinfo", "-std=c++17", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC,
                           "-c", src, "-o", _obj(src)]
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    return src, subprocess.run(cmd, capture_output=True, text=True)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    headers = _headers()
    todo = [s for s in _sources() if force or verbose or _stale(_obj(s), [s] + headers)]
    with concurrent.futures.ThreadPoolExecutor(max_workers=max(1, min(len(todo), os.cpu_count() or 1))) as pool:
        for src, res in pool.map(lambda s: _compile(nvcc, s, verbose), todo):
            if res.returncode != 0:
                sys.stderr.write(res.stdout + res.stderr)
                raise RuntimeError(f"nvcc failed on {os.path.basename(src)}")
            if verbose:
                sys.stderr.write(res.stdout + res.stderr)
    link = [nvcc] + ARCH + ["-shared", "-o", LIB] + [_obj(s) for s in _sources()]
    res = subprocess.run(link, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed linking libmwu.so")
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
