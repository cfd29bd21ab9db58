"""Builds the C-ABI library ``libjd_b200.so`` in-tree with nvcc for sm_100a.

Usage: ``python -m paper_2501_19309_b200.build [--force] [--verbose] [--stamps]``

``--stamps`` builds ``libjd_b200_stamps.so`` instead: the same sources with ``-DJD_PHASE_STAMPS``, in which the
fused kernel records the global timer at its phase boundaries (read with ``phase_times.py``).
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libjd_b200.so")
LIB_STAMPS = os.path.join(PKG, "libjd_b200_stamps.so")
SOURCES = ["jd_api.cu", "jd_simt.cu", "jd_fused_sm100.cu", "jd_batched_sm100.cu", "jd_static.cu"]
HEADERS = ["jd_common.cuh", "jd_kernels.h", "jd_sm100_ptx.cuh"]


def _nvcc() -> str:
    cand = os.environ.get("NVCC")
    if cand:
        return cand
    return "/usr/local/cuda/bin/nvcc" if os.path.exists("/usr/local/cuda/bin/nvcc") else "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "jd.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, stamps: bool = False) -> str:
    if stamps:
        return _compile(LIB_STAMPS, verbose, ["-DJD_PHASE_STAMPS"])
    if not force and not needs_build():
        return LIB
    return _compile(LIB, verbose, [])


def _compile(out: str, verbose: bool, defines: list) -> str:
    """Compiles the sources to objects side by side (the fused kernel's many instantiations dominate), then links."""
    import tempfile
    from concurrent.futures import ThreadPoolExecutor
    flags = ["-Xcompiler", "-fPIC", "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
             "-I", os.path.join(ROOT, "include"), "-I", CSRC] + defines
    if verbose:
        flags += ["-Xptxas", "-v"]
    with tempfile.TemporaryDirectory() as tmp:
        def one(src: str):
            obj = os.path.join(tmp, os.path.splitext(src)[0] + ".o")
            return obj, subprocess.run([_nvcc(), "-c"] + flags + [os.path.join(CSRC, src), "-o", obj],
                                       capture_output=True, text=True)
        with ThreadPoolExecutor(len(SOURCES)) as ex:
            results = list(ex.map(one, SOURCES))
        log = "".join(p.stdout + p.stderr for _, p in results)
        failed = any(p.returncode != 0 for _, p in results)
        if not failed:
            link = subprocess.run([_nvcc(), "-shared", "-Xcompiler", "-fPIC", "-gencode", "arch=compute_100a,code=sm_100a"] +
                                  [o for o, _ in results] + ["-o", out], capture_output=True, text=True)
            log += link.stdout + link.stderr
            failed = link.returncode != 0
    if verbose or failed:
        sys.stderr.write(log)
    if failed:
        raise RuntimeError("nvcc failed building %s" % out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, stamps="--stamps" in sys.argv))
