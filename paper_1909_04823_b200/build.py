"""Builds libdes.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdes.so")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    m = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(ROOT, "include", "des.h")]
    return any(os.path.getmtime(d) > m for d in deps)


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


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--fmad=true", "--expt-relaxed-constexpr", "--threads", "0", "-Xcompiler", "-fPIC", "-shared",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    cut = cutlass_include_dirs()
    if cut:
        for d in cut:
            cmd += ["-I", d]
    else:   # no sm100 CUTLASS headers here: the tensor-core GEMMs report "unsupported", CUDA-core path is used
        cmd += ["-DDES_NO_CUTLASS"]
    cmd += ["-o", LIB] + sources()
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
