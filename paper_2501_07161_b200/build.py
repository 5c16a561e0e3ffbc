"""Builds libqv2.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libqv2.so")
OBJ_DIR = os.path.join(_HERE, "_build")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
CFLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
          "-Xcompiler", "-fPIC"]
LDFLAGS = ["-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(_HERE, "..", "include", "qv2.h"),
                                                     os.path.abspath(__file__)]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in sources() + _headers())


def _compile(src: str, force: bool, verbose: bool):
    """One translation unit -> object file; skipped when the object is newer than its inputs."""
    obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
    if not force and not verbose and os.path.exists(obj):
        t = os.path.getmtime(obj)
        if all(os.path.getmtime(d) <= t for d in [src] + _headers()):
            return obj, 0, ""
    cmd = [NVCC] + CFLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
    res = subprocess.run(cmd, cwd=_HERE, capture_output=True, text=True)
    return obj, res.returncode, res.stdout + res.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ (in parallel, one object each) and link libqv2.so when it is
    missing or older than a source."""
    if not force and not verbose and not _stale():
        return LIB
    os.makedirs(OBJ_DIR, exist_ok=True)
    srcs = sources()
    with ThreadPoolExecutor(max_workers=min(len(srcs), os.cpu_count() or 1)) as pool:
        done = list(pool.map(lambda s: _compile(s, force, verbose), srcs))
    failed = [d for d in done if d[1] != 0]
    for _, rc, log in done:
        if verbose or rc != 0:
            sys.stderr.write(log)
    if failed:
        raise RuntimeError("nvcc failed building libqv2.so")
    res = subprocess.run([NVCC] + LDFLAGS + ["-o", LIB] + [d[0] for d in done], cwd=_HERE,
                         capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed linking libqv2.so")
    return LIB


PROBES = os.path.join(_HERE, "probes")


def build_probes() -> list:
    """Compile the stand-alone bandwidth probes under probes/ (one executable each, next to its
    source).  They are measurement aids for the profiles, not part of libqv2.so."""
    out = []
    for src in sorted(glob.glob(os.path.join(PROBES, "*.cu"))):
        exe = src[:-3]
        if not os.path.exists(exe) or os.path.getmtime(exe) < os.path.getmtime(src):
            res = subprocess.run([NVCC, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a",
                                  "-lineinfo", "-o", exe, src], cwd=PROBES, capture_output=True, text=True)
            if res.returncode != 0:
                sys.stderr.write(res.stdout + res.stderr)
                raise RuntimeError("nvcc failed building " + src)
        out.append(exe)
    return out


if __name__ == "__main__":
    if "--probes" in sys.argv:
        print("\n".join(build_probes()))
    else:
        print(build(force=True, verbose="-v" in sys.argv))
