"""Builds ``libloki_alloc.so`` in-tree with nvcc for sm_100a.

``python -m paper_2407_03583_b200.build`` (or ``build_library()``) compiles the
CUDA sources under ``csrc/`` in parallel and links the C-ABI shared library next
to this file.  Object files go to ``_build/`` at the repository root.
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
_OBJ = os.path.join(_ROOT, "_build")
LIB_PATH = os.path.join(_PKG, "libloki_alloc.so")
DEBUG_LIB_PATH = os.path.join(_PKG, "libloki_alloc_debug.so")    # the same sources with -DLOKI_DEBUG (bounds-checked kernels)
PROBE_PATH = os.path.join(_ROOT, "fp64_issue_probe")     # measurement aid of bench.py, not part of the library

SOURCES = ["loki_alloc.cu", "loki_kernels_generic.cu", "loki_kernels_direct.cu",
           "loki_alloc_static.cu", "loki_kernels_hoisted.cu", "loki_kernels_hoisted_l1.cu", "loki_kernels_hoisted_l2.cu",
           "loki_kernels_hoisted_l4.cu", "loki_kernels_variant.cu", "loki_route.cu"]
HEADERS = [os.path.join(_CSRC, "loki_internal.h"), os.path.join(_CSRC, "loki_kernels_hoisted_impl.h"),
           os.path.join(_CSRC, "loki_finish.cuh"),
           os.path.join(_ROOT, "include", "loki_alloc.h")]

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC,-ffp-contract=off",
    "-I", os.path.join(_ROOT, "include"), "-I", _CSRC,
]


def _nvcc() -> str:
    cand = os.environ.get("NVCC")
    if cand:
        return cand
    if os.path.exists("/usr/local/cuda/bin/nvcc"):
        return "/usr/local/cuda/bin/nvcc"
    return "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Builds libloki_alloc.so, or with ``debug`` the bounds-checked libloki_alloc_debug.so."""
    obj_dir = os.path.join(_OBJ, "debug") if debug else _OBJ
    lib_path = DEBUG_LIB_PATH if debug else LIB_PATH
    flags = NVCC_FLAGS + (["-DLOKI_DEBUG"] if debug else [])
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()
    # a change of flags invalidates every object
    stamp = os.path.join(obj_dir, "flags.txt")
    sig = hashlib.sha1(" ".join(flags).encode()).hexdigest()
    if not os.path.exists(stamp) or open(stamp).read() != sig:
        force = True
    jobs, objs = [], []
    for src in SOURCES:
        s = os.path.join(_CSRC, src)
        o = os.path.join(obj_dir, src.replace(".cu", ".o"))
        objs.append(o)
        if force or _stale(o, [s] + HEADERS):
            jobs.append([nvcc] + flags + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o])

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))

    with ThreadPoolExecutor(max_workers=max(1, min(os.cpu_count() or 4, 8, len(jobs) or 1))) as ex:
        list(ex.map(run, jobs))
    if jobs or force or _stale(lib_path, objs):
        tmp = lib_path + ".tmp.%d" % os.getpid()
        run([nvcc, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
        os.replace(tmp, lib_path)
    with open(stamp, "w") as f:
        f.write(sig)
    return lib_path


def build_probe(force: bool = False) -> str:
    """Builds the stand-alone FP64 issue-rate probe that sits beside bench.py."""
    src = os.path.join(_ROOT, "fp64_issue_probe.cu")
    if force or _stale(PROBE_PATH, [src]):
        tmp = PROBE_PATH + ".tmp.%d" % os.getpid()
        r = subprocess.run([_nvcc(), "-std=c++17", "-O3", "-lineinfo", "-gencode",
                            "arch=compute_100a,code=sm_100a", "-o", tmp, src], capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("nvcc failed on fp64_issue_probe.cu")
        os.replace(tmp, PROBE_PATH)
    return PROBE_PATH


if __name__ == "__main__":
    build_probe(force="--force" in sys.argv)
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build_library(force="--force" in sys.argv, debug=True))
