"""Builds the CUDA shared library (libbtc.so) in-tree with nvcc for sm_100a.

Every translation unit under csrc/ is compiled to an object file of its own (in parallel, and only
when it or a header it includes has changed), then the objects are linked into libbtc.so.
"""
from __future__ import annotations

import concurrent.futures
import os
import re
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libbtc.so")
SOURCES = ["btc_api.cu", "plan.cpp", "skinny_umma.cu", "stream.cu", "peaks.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v",
]


def _extra_flags():
    """Debug switches: BTC_CHECK_OFFSETS=1 in the environment compiles the kernels with a range
    check on every global offset they compute (a violation sets the device error word)."""
    flags = []
    if os.environ.get("BTC_CHECK_OFFSETS") == "1":
        flags.append("-DBTC_CHECK_OFFSETS")
    return flags


def _deps_of(dfile: str):
    try:
        with open(dfile) as f:
            text = f.read().replace("\\\n", " ")
    except OSError:
        return None
    parts = text.split(":", 1)
    return parts[1].split() if len(parts) == 2 else None


def _stale(src: str, obj: str, dfile: str, stamp: str) -> bool:
    if not os.path.exists(obj) or not os.path.exists(stamp):
        return True
    with open(stamp) as f:
        if f.read() != " ".join(NVCC_FLAGS + _extra_flags()):
            return True
    deps = _deps_of(dfile)
    if deps is None:
        return True
    t = os.path.getmtime(obj)
    for d in [src] + deps:
        if not os.path.exists(d) or os.path.getmtime(d) > t:
            return True
    return False


def _compile(nvcc: str, name: str, force: bool):
    src = os.path.join(CSRC, name)
    base = os.path.join(OBJ, re.sub(r"\.(cu|cpp)$", "", name))
    obj, dfile, stamp = base + ".o", base + ".d", base + ".flags"
    if not force and not _stale(src, obj, dfile, stamp):
        return name, 0, "", obj
    flags = NVCC_FLAGS + _extra_flags()
    cmd = [nvcc, *flags, "-MD", "-MF", dfile, "-c", "-o", obj, src]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode == 0:
        with open(stamp, "w") as f:
            f.write(" ".join(flags))
    return name, res.returncode, " ".join(cmd) + "\n" + res.stdout + res.stderr, obj


def build(force: bool = False, verbose: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
        results = list(pool.map(lambda s: _compile(nvcc, s, force), SOURCES))
    log = "".join(r[2] for r in results)
    rebuilt = any(r[2] for r in results)
    if rebuilt:
        with open(os.path.join(HERE, "build.log"), "w") as f:
            f.write(log)
    if any(r[1] != 0 for r in results):
        sys.stderr.write(log)
        raise RuntimeError("nvcc failed building libbtc.so")
    objs = [r[3] for r in results]
    if rebuilt or not os.path.exists(LIB) or any(os.path.getmtime(o) > os.path.getmtime(LIB) for o in objs):
        tmp = LIB + f".tmp{os.getpid()}"
        cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp, *objs, "-lcudart"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError("linking libbtc.so failed")
        os.replace(tmp, LIB)
    if verbose:
        print(log)
    return LIB


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose=True)
