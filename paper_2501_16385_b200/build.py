"""Builds libfbq.so (CUDA kernels + C ABI) in-tree with nvcc for sm_100a.

Every source file is compiled to an object of its own (in parallel, and only
when it or a header changed), then the objects are linked into the shared
library.  FBQ_EXTRA_NVCC_FLAGS adds compile flags for a build by hand (with
`--force`), e.g. -DFBQ_GEMV_TRACE for the streaming decode kernel's phase marks.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libfbq.so")
SOURCES = ["fbq_api.cu", "fbq_pack.cu", "fbq_generic.cu", "fbq_decode.cu", "fbq_gemv.cu", "fbq_prefill.cu", "fbq_noalloc.cu",
           "fbq_quant.cu", "fbq_reconstruct.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
COMPILE_FLAGS = ARCH + ["-lineinfo", "-O3", "-std=c++17", "-Xptxas=-v", "-Xcompiler", "-fPIC", "-rdc=false"]
LINK_FLAGS = ARCH + ["-shared", "-Xcompiler", "-fPIC", "-cudart", "static"]


def _headers():
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hs.append(os.path.join(HERE, "..", "include", "fbq.h"))
    return hs


def _obj(src: str) -> str:
    return os.path.join(OBJ, os.path.splitext(src)[0] + ".o")


def _stale_obj(src: str, force: bool) -> bool:
    o = _obj(src)
    if force or not os.path.exists(o):
        return True
    t = os.path.getmtime(o)
    return any(os.path.getmtime(d) > t for d in [os.path.join(CSRC, src)] + _headers())


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(HERE, "..", "include", "fbq.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)

    def compile_one(src):
        if not _stale_obj(src, force):
            return src, 0, ""
        tmp = _obj(src) + ".tmp%d" % os.getpid()
        res = subprocess.run([nvcc] + COMPILE_FLAGS + os.environ.get("FBQ_EXTRA_NVCC_FLAGS", "").split() + ["-c", "-o", tmp, os.path.join(CSRC, src)], capture_output=True, text=True)
        if res.returncode == 0:
            os.replace(tmp, _obj(src))
        return src, res.returncode, res.stdout + res.stderr

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 4)) as pool:
        results = list(pool.map(compile_one, SOURCES))
    failed = [r for r in results if r[1] != 0]
    for src, rc, log in results:
        if verbose or rc != 0:
            sys.stderr.write("== %s\n%s" % (src, log))
    if failed:
        raise RuntimeError("nvcc failed compiling " + ", ".join(r[0] for r in failed))
    tmp = LIB + ".tmp%d" % os.getpid()
    res = subprocess.run([nvcc] + LINK_FLAGS + ["-o", tmp] + [_obj(s) for s in SOURCES], capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed linking libfbq.so")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
