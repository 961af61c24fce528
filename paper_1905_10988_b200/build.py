"""Build libnatcomp.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libnatcomp.so")
LIB_BOUNDS = os.path.join(HERE, "libnatcomp_bounds.so")   # debug build: checked stores

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=false",          # binary32 sums and products must round exactly once, as written
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "--threads", "0",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib=LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [
        os.path.join(HERE, "..", "include", "natcomp.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, bounds: bool = False) -> str:
    """bounds=True builds the debug library (-DNC_BOUNDS): every global store of the C_nat and
    D_nat kernels is checked against the ranges the call may write; a store outside them is
    skipped and counted (nc_debug_bounds_status), never trapped."""
    lib = LIB_BOUNDS if bounds else LIB
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = ([nvcc] + NVCC_FLAGS + (["-DNC_BOUNDS"] if bounds else [])
           + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources())
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv, bounds="--bounds" in sys.argv))
