"""In-tree build of the sm_100a C-ABI library (``libluq_b200.so``) with nvcc.

``python -m paper_2112_10769_b200.build`` compiles the three translation units
and links one shared library next to this file.  nvcc cross-compiles without a
GPU.  The quantizer file is compiled without FMA contraction; nothing is built
with fast-math, flush-to-zero or approximate division.
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libluq_b200.so")
LIB_DEBUG = os.path.join(HERE, "libluq_b200_debug.so")   # the same sources with -DLUQ_DEBUG (bounds-checking build)
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
COMMON = ["-std=c++17", "-O3", "-lineinfo", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"),
          "-I", CSRC, "--expt-relaxed-constexpr",
          "-diag-suppress", "177"]   # 177: a static member that one instantiation of a configuration struct does not use
UNITS = {"quant.cu": ["-fmad=false"], "gemm.cu": [], "api.cu": []}


def _digest(paths, extra=()) -> str:
    """Content hash of the inputs of one build step (a copied tree keeps contents, not timestamps)."""
    h = hashlib.sha256()
    for item in extra:
        h.update(str(item).encode())
    for path in paths:
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _stale(target: str, digest: str) -> bool:
    stamp = target + ".sha"
    if not os.path.exists(target) or not os.path.exists(stamp):
        return True
    with open(stamp) as f:
        return f.read().strip() != digest


def _stamp(target: str, digest: str) -> None:
    with open(target + ".sha", "w") as f:
        f.write(digest)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compiles the library; debug=True compiles the bounds-checking variant (-DLUQ_DEBUG) next to it."""
    nvcc = os.environ.get("NVCC", "nvcc")
    lib = LIB_DEBUG if debug else LIB
    suffix, define = (".dbg.o", ["-DLUQ_DEBUG"]) if debug else (".o", [])
    headers = [os.path.join(CSRC, "common.cuh"), os.path.join(CSRC, "int4_math.cuh"), os.path.join(ROOT, "include", "luq.h")]
    objs, digests, running = [], [], []
    for name, extra in UNITS.items():
        src = os.path.join(CSRC, name)
        obj = os.path.join(CSRC, name.replace(".cu", suffix))
        objs.append(obj)
        extra = extra + define
        flags = ARCH + COMMON[:5] + extra        # the flags that change the code (not the include paths)
        digest = _digest([src] + headers, flags)
        digests.append(digest)
        if force or _stale(obj, digest):
            cmd = [nvcc] + ARCH + COMMON + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            running.append((subprocess.Popen(cmd), cmd, obj, digest))     # the units compile side by side
    for proc, cmd, obj, digest in running:
        if proc.wait() != 0:
            raise subprocess.CalledProcessError(proc.returncode, cmd)
        _stamp(obj, digest)
    link_digest = _digest([], digests)
    if force or _stale(lib, link_digest):
        subprocess.run([nvcc] + ARCH + ["-shared", "-o", lib] + objs, check=True)
        _stamp(lib, link_digest)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
