"""Builds libbmu.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Every .cu file is compiled to an object of its own (in parallel, re-compiled
only when it or a header is newer) and the objects are linked into the shared
library.  `extra_flags` / `out` / `objdir` give a second build beside the
default one, e.g. the bounds-checked build (-DBMU_BOUNDS_CHECK).
"""
from __future__ import annotations

import glob
import hashlib
import os
import subprocess
import sys
import zlib
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libbmu.so")
# the same library with every id- and offset-derived address checked (-DBMU_BOUNDS_CHECK)
LIB_CHECKED = os.path.join(HERE, "libbmu_checked.so")
OBJDIR = os.path.join(HERE, "build")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def headers():
    return sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + \
        sorted(glob.glob(os.path.join(ROOT, "include", "*.h")))


def fingerprint(extra=()) -> str:
    """Hash of everything a build depends on: sources, headers, flags."""
    h = hashlib.sha256(" ".join([*NVCC_FLAGS, *extra]).encode())
    for p in sources() + headers():
        h.update(os.path.basename(p).encode())
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def up_to_date(lib: str = LIB, extra=()) -> bool:
    """True if `lib` was built from exactly these sources and flags (a stamp file beside the
    library holds the fingerprint; file times do not survive a copy of the tree)."""
    try:
        with open(lib + ".stamp") as f:
            return os.path.exists(lib) and f.read().strip() == fingerprint(extra)
    except OSError:
        return False


def build_library(force: bool = False, verbose: bool = False, extra_flags=(), out: str = LIB,
                  objdir: str = OBJDIR) -> str:
    env_extra = os.environ.get("BMU_EXTRA_NVCC", "").split()
    extra = [*env_extra, *extra_flags]
    if not force and up_to_date(out, extra):
        return out
    nvcc = os.environ.get("NVCC", "nvcc")
    flags = [*extra, *NVCC_FLAGS]
    if extra:                             # objects of another flag set live apart
        objdir = os.path.join(objdir, "x%08x" % (zlib.crc32(" ".join(extra).encode()) & 0xffffffff))
    if verbose:
        flags += ["-Xptxas", "-v"]
    os.makedirs(objdir, exist_ok=True)
    newest_header = max(os.path.getmtime(p) for p in headers())

    def compile_one(src):
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        if (not force and not verbose and os.path.exists(obj)
                and os.path.getmtime(obj) >= max(os.path.getmtime(src), newest_header)):
            return obj
        subprocess.check_call([nvcc, *flags, "-I", os.path.join(ROOT, "include"), "-I", CSRC,
                               "-c", src, "-o", obj])
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, sources()))
    tmp = out + ".tmp%d" % os.getpid()
    subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
                           *objs, "-o", tmp])
    os.replace(tmp, out)
    with open(out + ".stamp", "w") as f:
        f.write(fingerprint(extra) + "\n")
    return out


def build_checked_library(force: bool = False) -> str:
    return build_library(force=force, extra_flags=["-DBMU_BOUNDS_CHECK"], out=LIB_CHECKED)


if __name__ == "__main__":
    print(build_library(force="-f" in sys.argv or "-v" in sys.argv, verbose="-v" in sys.argv))
    if "--checked" in sys.argv:
        print(build_checked_library(force="-f" in sys.argv))
