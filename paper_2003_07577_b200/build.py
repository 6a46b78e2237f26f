"""Builds libebs.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Every translation unit under csrc/ is compiled to an object file in parallel and the objects
are linked into ``paper_2003_07577_b200/libebs.so``.  Nothing is cached outside the tree.
``build(checked=True)`` builds the range-checked variant of the same sources (``-DEBS_CHECKED``,
objects under ``build_checked/``) into ``libebs_checked.so``.
"""
from __future__ import annotations

import concurrent.futures
import glob
import os
import re
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libebs.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


_INCLUDE = re.compile(r'^\s*#\s*include\s+"([^"]+)"', re.M)


def _deps(path: str, seen: set) -> set:
    """The file and every project header it includes, transitively (headers live in csrc/ and include/)."""
    if path in seen:
        return seen
    seen.add(path)
    with open(path) as f:
        for name in _INCLUDE.findall(f.read()):
            for d in (CSRC, os.path.join(ROOT, "include")):
                cand = os.path.join(d, name)
                if os.path.exists(cand):
                    _deps(cand, seen)
    return seen


LIB_CHECKED = os.path.join(PKG, "libebs_checked.so")


def _compile(src: str, verbose: bool, checked: bool = False) -> str:
    obj = os.path.join(OBJ + ("_checked" if checked else ""), os.path.basename(src)[:-3] + ".o")
    newest = max(os.path.getmtime(p) for p in _deps(src, set()))
    if os.path.exists(obj) and os.path.getmtime(obj) >= newest:
        return obj
    cmd = ["nvcc"] + NVCC_FLAGS + (["-DEBS_CHECKED"] if checked else []) + (["-Xptxas", "-v"] if verbose else []) + \
          ["-c", src, "-o", obj]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed for {src}:\n{res.stdout}\n{res.stderr}")
    if verbose:
        with open(obj[:-2] + ".ptxas.txt", "w") as f:
            f.write(res.stderr)
    return obj


def build(force: bool = False, verbose: bool = False, jobs: int | None = None, checked: bool = False) -> str:
    obj_dir, lib = OBJ + ("_checked" if checked else ""), (LIB_CHECKED if checked else LIB)
    os.makedirs(obj_dir, exist_ok=True)
    srcs = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    if force:
        for o in glob.glob(os.path.join(obj_dir, "*.o")):
            os.remove(o)
    jobs = jobs or min(len(srcs), os.cpu_count() or 4)
    with concurrent.futures.ThreadPoolExecutor(max_workers=jobs) as ex:
        objs = list(ex.map(lambda s: _compile(s, verbose, checked), srcs))
    if force or not os.path.exists(lib) or any(os.path.getmtime(o) > os.path.getmtime(lib) for o in objs):
        cmd = ["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib] + objs + ["-lcudart"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"link failed:\n{res.stdout}\n{res.stderr}")
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
