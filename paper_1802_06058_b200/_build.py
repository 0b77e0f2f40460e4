"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension).

Every csrc/*.cu is compiled to an object file of its own (in parallel; an object is rebuilt only when its
source, a shared header or the flags changed) and the objects are linked into libvgc.so next to this file."""
from __future__ import annotations

import concurrent.futures
import glob
import hashlib
import os
import subprocess

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
INCLUDE = os.path.join(os.path.dirname(PKG_DIR), "include")
LIB_PATH = os.path.join(PKG_DIR, "libvgc.so")
OBJ_DIR = os.path.join(PKG_DIR, "build")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", INCLUDE]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return sorted(glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h")))


def _newest(paths) -> float:
    return max(os.path.getmtime(p) for p in paths)


def _obj_path(src: str) -> str:
    tag = hashlib.sha1(" ".join(NVCC_FLAGS).encode()).hexdigest()[:8]
    return os.path.join(OBJ_DIR, os.path.splitext(os.path.basename(src))[0] + "." + tag + ".o")


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    return _newest(_sources() + _headers()) > os.path.getmtime(LIB_PATH)


def _compile(nvcc: str, src: str, verbose: bool) -> str:
    obj = _obj_path(src)
    if os.path.exists(obj) and os.path.getmtime(obj) >= _newest([src] + _headers()):
        return obj
    tmp = obj + ".tmp.%d" % os.getpid()
    cmd = [nvcc, *NVCC_FLAGS, "-c", "-o", tmp, src]
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
        print(" ".join(cmd))
    subprocess.run(cmd, check=True)
    os.replace(tmp, obj)
    return obj


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libvgc.so next to this file; returns its path."""
    if not force and not _stale():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    if force:
        for old in glob.glob(os.path.join(OBJ_DIR, "*.o")):
            os.remove(old)
    srcs = _sources()
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(len(srcs), os.cpu_count() or 1)) as pool:
        objs = list(pool.map(lambda s: _compile(nvcc, s, verbose), srcs))
    tmp = LIB_PATH + ".tmp.%d" % os.getpid()
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp, *objs], check=True)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


PROBE_SRC = os.path.join(CSRC, "probe", "mma_rate_probe.cu")
PROBE_LIB_PATH = os.path.join(PKG_DIR, "libvgc_probe.so")


def build_probe() -> str:
    """The tensor-pipe rate probe behind `bench.py --mma-rates`: a measurement aid with a library of its own."""
    if os.path.exists(PROBE_LIB_PATH) and os.path.getmtime(PROBE_LIB_PATH) >= _newest([PROBE_SRC] + _headers()):
        return PROBE_LIB_PATH
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = PROBE_LIB_PATH + ".tmp.%d" % os.getpid()
    subprocess.run([nvcc, *NVCC_FLAGS, "-I", CSRC, "-shared", "-o", tmp, PROBE_SRC], check=True)
    os.replace(tmp, PROBE_LIB_PATH)
    return PROBE_LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
