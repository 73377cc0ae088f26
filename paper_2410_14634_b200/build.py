"""Builds the CUDA library in-tree for sm_100a (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libinvconv_b200.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = glob.glob(os.path.join(CSRC, "*")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def _includes(path: str, seen: set) -> set:
    """Files reachable from `path` through #include "..." (searched in csrc/ and include/)."""
    if path in seen:
        return seen
    seen.add(path)
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if line.startswith('#include "'):
                name = line.split('"')[1]
                for d in (CSRC, os.path.join(ROOT, "include")):
                    cand = os.path.join(d, name)
                    if os.path.exists(cand):
                        _includes(cand, seen)
    return seen


def _object_stale(obj: str, src: str) -> bool:
    if not os.path.exists(obj):
        return True
    t = os.path.getmtime(obj)
    return any(os.path.getmtime(d) > t for d in _includes(src, set()))


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every csrc/*.cu (one object each, in parallel) and link libinvconv_b200.so next to this file."""
    if not force and not _stale():
        return LIB
    objdir = os.path.join(PKG, "build")
    os.makedirs(objdir, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
             "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]
    extra = os.environ.get("INVCONV_NVCC_FLAGS", "").split()     # development builds only
    flags += extra
    procs, objs = [], []
    for src in sources():
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force or extra or _object_stale(obj, src):
            procs.append((src, subprocess.Popen([NVCC, "-c", *flags, src, "-o", obj])))
    failed = [src for src, pr in procs if pr.wait() != 0]
    if failed:
        raise RuntimeError(f"nvcc failed for {failed}")
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.check_call([NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-Xcompiler", "-fPIC", *objs, "-o", tmp])
    os.replace(tmp, LIB)
    return LIB


LIB_DEBUG = os.path.join(PKG, "libinvconv_b200_debug.so")


def build_debug_bounds() -> str:
    """The debug-bounds variant: the tensor-core and flow-step translation units recompiled with
    -DINVCONV_DEBUG_BOUNDS (checked accessors) and linked with the regular objects of the rest."""
    build()
    objdir = os.path.join(PKG, "build")
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC",
             "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-DINVCONV_DEBUG_BOUNDS"]
    procs, objs = [], [os.path.join(objdir, "invconv_lib.o")]
    for name in ("tensor_lib", "flow_step_lib"):
        obj = os.path.join(objdir, name + "_dbg.o")
        objs.append(obj)
        procs.append(subprocess.Popen([NVCC, "-c", *flags, os.path.join(CSRC, name + ".cu"), "-o", obj]))
    if any(pr.wait() != 0 for pr in procs):
        raise RuntimeError("nvcc failed for the debug-bounds build")
    tmp = LIB_DEBUG + f".tmp{os.getpid()}"
    subprocess.check_call([NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-Xcompiler", "-fPIC", *objs, "-o", tmp])
    os.replace(tmp, LIB_DEBUG)
    return LIB_DEBUG


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
    if "--debug-bounds" in sys.argv:
        print(build_debug_bounds())
