"""Build ``libcoopt.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU).

``python -m paper_2602_09323_b200.build`` rebuilds what is older than its sources: every ``.cu`` file
is compiled to an object of its own (in parallel) under ``_build/`` and the objects are linked into
the shared library.  ``--trace`` builds ``libcoopt_trace.so`` instead: the same sources with
``-DCOOPT_TRACE``, whose tcgen05 kernels also write time stamps of their roles into a caller-supplied
buffer (``csrc/coopt_trace.cuh``, read by ``python -m paper_2602_09323_b200.trace``); the ordinary library contains none of that code.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
SRC_DIR = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libcoopt.so")
TRACE_LIB_PATH = os.path.join(PKG_DIR, "libcoopt_trace.so")
BUILD_DIR = os.path.join(PKG_DIR, "_build")
INCLUDE_DIR = os.path.join(os.path.dirname(PKG_DIR), "include")
COMPILE_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr",
]
LINK_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "--shared", "-Xcompiler", "-fPIC", "-cudart", "static"]


def find_nvcc() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: libcoopt.so cannot be built")
    return cand


def sources():
    return sorted(f for f in os.listdir(SRC_DIR) if f.endswith(".cu"))


def _headers():
    hs = [os.path.join(SRC_DIR, f) for f in os.listdir(SRC_DIR) if f.endswith((".cuh", ".h"))]
    hs += [os.path.join(INCLUDE_DIR, f) for f in os.listdir(INCLUDE_DIR) if f.endswith(".h")]
    return hs + [os.path.abspath(__file__)]


def _newer_than(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def needs_build(trace: bool = False) -> bool:
    lib = TRACE_LIB_PATH if trace else LIB_PATH
    return _newer_than(lib, [os.path.join(SRC_DIR, s) for s in sources()] + _headers())


def build(force: bool = False, verbose: bool = False, ptxas_info: bool = False, trace: bool = False) -> str:
    """Compile every CUDA source and link the shared library; returns its path."""
    lib = TRACE_LIB_PATH if trace else LIB_PATH
    if not force and not needs_build(trace):
        return lib
    nvcc = find_nvcc()
    obj_dir = os.path.join(BUILD_DIR, "trace" if trace else "plain")
    os.makedirs(obj_dir, exist_ok=True)
    headers = _headers()
    flags = COMPILE_FLAGS + (["-DCOOPT_TRACE"] if trace else []) + (["-Xptxas", "-v"] if ptxas_info else [])

    def compile_one(src: str):
        obj = os.path.join(obj_dir, src[:-3] + ".o")
        path = os.path.join(SRC_DIR, src)
        if not (force or ptxas_info) and not _newer_than(obj, [path] + headers):
            return obj, ""
        cmd = [nvcc] + flags + ["-c", path, "-o", obj]
        if verbose:
            print(" ".join(cmd), flush=True)
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed on %s:\n%s%s" % (src, res.stdout, res.stderr))
        return obj, res.stdout + res.stderr

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        results = list(pool.map(compile_one, sources()))
    if verbose or ptxas_info:
        sys.stderr.write("".join(out for _, out in results))
    cmd = [nvcc] + LINK_FLAGS + [obj for obj, _ in results] + ["-o", lib]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True, ptxas_info="--ptxas" in sys.argv, trace="--trace" in sys.argv))
