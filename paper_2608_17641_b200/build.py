"""Build ``librlcs.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2608_17641_b200.build [--force] [--verbose] [--all-variants]

``--all-variants`` (or RLCS_ALL_VARIANTS=1 in the environment) also compiles the tile shapes that
the kernel selection never returns (tuning history; a 3x larger library and build time).

One object per translation unit, compiled in parallel, then one shared library that exports the
C ABI declared in ``include/rlcs.h``.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "librlcs.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--compress-mode=size",
    "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"),
]


def _sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))


def _deps_mtime():
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "rlcs.h"), __file__]
    return max(os.path.getmtime(f) for f in files)


def build(force: bool = False, verbose: bool = False, all_variants: bool | None = None) -> str:
    if all_variants is None:
        all_variants = os.environ.get("RLCS_ALL_VARIANTS", "0") not in ("", "0")
    flags = ["-DRLCS_ALL_VARIANTS"] if all_variants else []
    stamp = os.path.join(OBJ, "flags.txt")
    same_flags = os.path.exists(stamp) and open(stamp).read() == " ".join(flags)
    if not force and same_flags and os.path.exists(LIB) and os.path.getmtime(LIB) >= _deps_mtime():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    extra = flags + (["-Xptxas", "-v"] if verbose else [])

    def compile_one(src):
        obj = os.path.join(OBJ, src[:-3] + ".o")
        cmd = ["nvcc", *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{res.stdout}\n{res.stderr}")
        if verbose:
            sys.stderr.write(res.stderr)
        return obj

    with ThreadPoolExecutor(max(1, min(len(_sources()), os.cpu_count() or 4))) as ex:
        objs = list(ex.map(compile_one, _sources()))
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.check_call(["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp, *objs])
    os.replace(tmp, LIB)
    with open(stamp, "w") as fh:
        fh.write(" ".join(flags))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv,
                all_variants=True if "--all-variants" in sys.argv else None))
