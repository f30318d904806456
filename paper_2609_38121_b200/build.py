"""Builds libwushkv.so (sm_100a) in-tree with nvcc.  ``python -m paper_2609_38121_b200.build``.

Every source is compiled to its own object file (in parallel, rebuilt only when it or a header is
newer) and the objects are linked into one shared library.  Extra compiler flags can be passed in
the environment variable WUSHKV_NVCC_FLAGS (they force a full rebuild)."""
from __future__ import annotations

import os
import shlex
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libwushkv.so")
SOURCES = ["api.cu", "transforms_host.cpp", "append.cu", "decode.cu", "decode_static.cu", "prefill.cu", "calibrate.cu", "hessians.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _headers():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))] + \
           [os.path.join(HERE, "..", "include", "wushkv.h")]


def _sources():
    return [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in _sources()] + _headers()
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA source for sm_100a into one shared library; returns its path."""
    extra = shlex.split(os.environ.get("WUSHKV_NVCC_FLAGS", ""))
    if extra:
        force = True
    if not force and not needs_build():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    hdr_time = max(os.path.getmtime(h) for h in _headers())
    base = [_nvcc()] + ARCH + ["-lineinfo", "-O3", "-std=c++17", "-DWUSHKV_BUILD", "-Xcompiler", "-fPIC,-O3"] + extra
    if verbose:
        base += ["-Xptxas", "-v"]

    def compile_one(src):
        path = os.path.join(CSRC, src)
        obj = os.path.join(OBJ, os.path.splitext(src)[0] + ".o")
        if not force and not verbose and os.path.exists(obj) and os.path.getmtime(obj) > max(os.path.getmtime(path), hdr_time):
            return obj, 0, ""
        res = subprocess.run(base + ["-c", path, "-o", obj], capture_output=True, text=True)
        return obj, res.returncode, res.stdout + res.stderr

    with ThreadPoolExecutor(max_workers=8) as pool:
        results = list(pool.map(compile_one, _sources()))
    log = "".join(r[2] for r in results)
    if any(r[1] != 0 for r in results):
        sys.stderr.write(log)
        raise RuntimeError("nvcc failed building libwushkv.so")
    res = subprocess.run([_nvcc()] + ARCH + ["-shared", "-cudart", "shared", "-o", LIB] + [r[0] for r in results],
                         capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(log + res.stdout + res.stderr)
        raise RuntimeError("nvcc failed linking libwushkv.so")
    if verbose:
        sys.stderr.write(log)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
