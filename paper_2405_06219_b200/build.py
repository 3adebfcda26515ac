"""Builds libskvq.so in-tree with nvcc for sm_100a (no JIT cache, no other architecture)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libskvq.so")
LIB_CHECKED = os.path.join(PKG, "libskvq_checked.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "--expt-relaxed-constexpr"]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def build_library(force: bool = False, verbose: bool = False, checked: bool = False, nvtx: bool = False) -> str:
    """Compile every .cu under csrc/ into paper_2405_06219_b200/libskvq.so; with ``checked`` the debugging build
    (-DSKVQ_CHECKED: every index is compared with its buffer's size, violations set SKVQ_STATUS_BOUNDS) into
    libskvq_checked.so.  ``nvtx`` (with force) compiles NVTX ranges around the entry points into the library being built.
    The translation units are compiled side by side (objects under _build/), then linked."""
    lib = LIB_CHECKED if checked else LIB
    if not force and not nvtx and not needs_build(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(ROOT, "_build", "checked" if checked else "plain")
    os.makedirs(objdir, exist_ok=True)
    flags = [f for f in NVCC_FLAGS if f != "-shared"] + ["-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if checked:
        flags += ["-DSKVQ_CHECKED=1"]
    if nvtx:
        flags += ["-DSKVQ_NVTX=1"]
    if verbose:
        flags += ["-Xptxas", "-v"]

    def compile_one(src):
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        subprocess.run([nvcc, *flags, "-c", "-o", obj, src], check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        objs = list(ex.map(compile_one, sources()))
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-Xcompiler", "-fPIC", "-o", lib, *objs], check=True)
    return lib


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
