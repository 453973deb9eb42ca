"""Builds the C-ABI CUDA library in-tree with nvcc for sm_100a.

Two libraries come out of the same sources:
  libdes.so        the product;
  libdes_debug.so  compiled with -DDES_DEBUG: every gather, scatter and probe checks its index
                   against the table's bounds and raises the table's status word instead of touching
                   memory out of range (the stand-in for a memory checker), and test-only hooks exist.
Every translation unit is compiled to an object of its own (kept under build/, rebuilt only when the
source or a header it includes is newer), so a change to one kernel file recompiles that file only; the
tensor-core GEMM units, which take longest, are shared by both libraries."""
from __future__ import annotations

import glob
import os
import re
import subprocess
import sys
import warnings
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libdes.so")
LIB_DEBUG = os.path.join(HERE, "libdes_debug.so")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _includes(path, seen=None):
    """The local headers a source includes, directly or not."""
    seen = set() if seen is None else seen
    for name in re.findall(r'#include\s+"([^"]+)"', open(path).read()):
        for base in (CSRC, os.path.join(ROOT, "include")):
            p = os.path.join(base, name)
            if os.path.exists(p) and p not in seen:
                seen.add(p)
                _includes(p, seen)
    return seen


def cutlass_include_dirs():
    """The CUTLASS / CuTe header tree that ships inside Python packages of this
    environment (used by the tcgen05 GEMM translation units only)."""
    import importlib.util
    for pkg, sub in (("flashinfer", os.path.join("data", "cutlass")), ("tilelang", os.path.join("3rdparty", "cutlass"))):
        try:
            spec = importlib.util.find_spec(pkg)
        except Exception:
            spec = None
        if spec is None or not spec.submodule_search_locations:
            continue
        base = os.path.join(list(spec.submodule_search_locations)[0], sub)
        inc = os.path.join(base, "include")
        if os.path.exists(os.path.join(inc, "cutlass", "gemm", "collective", "builders", "sm100_umma_builder.inl")):
            dirs = [inc]
            util = os.path.join(base, "tools", "util", "include")
            if os.path.isdir(util):
                dirs.append(util)
            return dirs
    return []


def _is_tc_unit(src):
    return os.path.basename(src).startswith("des_tc_gemm")


def _object_for(src, debug):
    stem = os.path.splitext(os.path.basename(src))[0]
    return os.path.join(OBJ, stem + (".debug.o" if debug and not _is_tc_unit(src) else ".o"))


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    m = os.path.getmtime(target)
    return any(os.path.getmtime(d) > m for d in deps)


def needs_build(debug: bool = False) -> bool:
    lib = LIB_DEBUG if debug else LIB
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(ROOT, "include", "des.h"), __file__]
    return _stale(lib, deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not force and not needs_build(debug):
        return lib
    os.makedirs(OBJ, exist_ok=True)
    # several processes of one job (one per GPU) may get here together: one builds, the others wait and find it done
    import fcntl
    with open(os.path.join(OBJ, ".lock"), "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if not force and not needs_build(debug):
                return lib
            return _build_locked(lib, force, verbose, debug)
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)


def _build_locked(lib, force, verbose, debug):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    base = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
            "--fmad=true", "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC",
            "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        base.insert(1, "-Xptxas=-v")
    cut = cutlass_include_dirs()
    if not cut:
        # no sm100 CUTLASS headers here: the tensor-core GEMM entry points answer "unsupported" and the first
        # dense layer runs on the CUDA-core kernel (des_build_has_tensor_cores() reports it)
        warnings.warn("no sm100 CUTLASS header tree found: building without the tcgen05 GEMM path")
    jobs = []
    for src in sources():
        obj = _object_for(src, debug)
        if not force and not _stale(obj, [src, __file__] + sorted(_includes(src))):
            continue
        cmd = list(base)
        if _is_tc_unit(src):
            cmd += [x for d in cut for x in ("-I", d)] if cut else ["-DDES_NO_CUTLASS"]
        else:
            if not cut:
                cmd += ["-DDES_NO_CUTLASS"]
            if debug:
                cmd += ["-DDES_DEBUG"]
        jobs.append(cmd + ["-c", "-o", obj, src])
    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as ex:
        for rc in ex.map(subprocess.call, jobs):
            if rc != 0:
                raise RuntimeError("nvcc failed")
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", lib] + [_object_for(s, debug) for s in sources()])
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
