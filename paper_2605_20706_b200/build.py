"""Builds the lw shared library (CUDA kernels + C ABI) for sm_100a with nvcc, in-tree.

Usage: python -m paper_2605_20706_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB = os.path.join(HERE, "liblw.so")

SOURCES = ["lw_matvec_stream.cu", "lw_matvec_seq.cu", "lw_matvec_tile.cu", "lw_matvec_mma.cu", "lw_probe.cu", "lw_attn.cu", "lw_api.cu", "lw_hostpipe.cu", "lw_dequant.cu", "lw_matvec_generic.cu", "lw_quantize.cpp"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "lw.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu + the host quantiser into liblw.so (no-op when up to date).  The translation
    units are compiled side by side (one nvcc process each) and linked at the end."""
    if not force and not _stale():
        return LIB
    import shutil
    import tempfile
    from concurrent.futures import ThreadPoolExecutor
    objdir = tempfile.mkdtemp(prefix="lw_build_")
    try:
        def compile_one(src):
            obj = os.path.join(objdir, os.path.splitext(src)[0] + ".o")
            cmd = [_nvcc(), "-c", *NVCC_FLAGS, "-I", INCLUDE, "-I", CSRC]
            if verbose:
                cmd += ["-Xptxas", "-v"]
            cmd += [os.path.join(CSRC, src), "-o", obj]
            proc = subprocess.run(cmd, capture_output=True, text=True)
            return src, obj, proc
        with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
            results = list(pool.map(compile_one, SOURCES))
        for src, _, proc in results:
            if proc.returncode != 0:
                sys.stderr.write(proc.stdout + proc.stderr)
                raise RuntimeError("nvcc failed on %s" % src)
            if verbose:
                sys.stderr.write(proc.stdout + proc.stderr)
        tmp = LIB + ".tmp.%d" % os.getpid()
        link = subprocess.run([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
                               *[obj for _, obj, _ in results], "-o", tmp], capture_output=True, text=True)
        if link.returncode != 0:
            sys.stderr.write(link.stdout + link.stderr)
            raise RuntimeError("nvcc failed linking liblw.so")
        os.replace(tmp, LIB)
    finally:
        shutil.rmtree(objdir, ignore_errors=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
