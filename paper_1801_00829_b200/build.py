"""Builds csrc/*.cu into libfusedops.so (sm_100a) next to this file.

    python -m paper_1801_00829_b200.build [--force] [--verbose]

nvcc cross-compiles without a GPU.  Objects go to _build/ (not committed); the
shared library stays in the package directory so it travels with the tree.
"""
from __future__ import annotations

import concurrent.futures
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OBJ_DIR = os.path.join(HERE, "_build")
LIB_PATH = os.path.join(HERE, "libfusedops.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v",
    # no implicit multiply-add contraction: every chain step rounds on its own, so
    # specialised and interpreted chains agree bit for bit; fused multiply-adds
    # are written explicitly (fma) where a kernel wants them
    "-fmad=false",
]


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return (_sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h"))
            + glob.glob(os.path.join(INCLUDE, "*.h")))


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(d) > t for d in _deps())


def _compile_one(src: str, verbose: bool) -> str:
    obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
    log = obj + ".log"
    cmd = [_nvcc()] + NVCC_FLAGS + ["-I", INCLUDE, "-I", OBJ_DIR, "-c", src, "-o", obj]
    res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    with open(log, "w") as fh:
        fh.write(res.stdout)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s" % (src, res.stdout[-4000:]))
    if verbose:
        print(res.stdout)
    return obj


# what the run-time specialised kernels are made of: Cell / MAgg, and Outer
JIT_HEADERS = {"jit_source.inc": ["common.cuh", "cell_flat.cuh", "cell_tiles.cuh", "cell_csr.cuh"],
               "jit_source_outer.inc": ["common.cuh", "ptx.cuh", "outer_kernels.cuh"],
               "jit_source_row.inc": ["common.cuh", "ptx.cuh", "row_kernels.cuh"]}


def _write_jit_source() -> None:
    """Embeds the headers the run-time compiled kernels consist of as C++ string
    literals (_build/jit_source*.inc), without their #include / #pragma once lines."""
    for target, names in JIT_HEADERS.items():
        chunks = []
        for name in names:
            with open(os.path.join(CSRC, name)) as fh:
                lines = [l for l in fh.read().splitlines()
                         if not l.lstrip().startswith("#include") and not l.lstrip().startswith("#pragma once")]
            chunks.append("// ---- %s\n" % name + "\n".join(lines) + "\n")
        text = "".join(chunks)
        assert ')FOJIT"' not in text
        out = []
        step = 8000                                   # keep each literal well below compiler limits
        for i in range(0, len(text), step):
            out.append('R"FOJIT(' + text[i:i + step] + ')FOJIT"\n')
        with open(os.path.join(OBJ_DIR, target), "w") as fh:
            fh.write("".join(out))


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile (if needed) and return the path of libfusedops.so."""
    if not force and not is_stale():
        return LIB_PATH
    os.makedirs(OBJ_DIR, exist_ok=True)
    _write_jit_source()
    srcs = _sources()
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, len(srcs))) as pool:
        objs = list(pool.map(lambda s: _compile_one(s, verbose), srcs))
    tmp = LIB_PATH + ".tmp%d" % os.getpid()
    cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs + ["-ldl"]
    res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n%s" % res.stdout[-4000:])
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    path = build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv)
    print(path)
