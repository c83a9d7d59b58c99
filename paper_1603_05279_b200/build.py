"""Builds libxnor.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
LIB = os.path.join(_HERE, "libxnor.so")
LIB_CHECK = os.path.join(_HERE, "libxnor_check.so")     # the same sources with -DXNOR_BOUNDS_CHECK
SOURCES = sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cu")))
HEADERS = sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cuh"))) + \
    sorted(glob.glob(os.path.join(_ROOT, "include", "*.h")))

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(_ROOT, "include")]


def up_to_date(lib=LIB):
    if not os.path.exists(lib):
        return False
    t = os.path.getmtime(lib)
    return all(os.path.getmtime(f) <= t for f in SOURCES + HEADERS)


def build(force=False, verbose=False, bounds_check=False):
    """Builds libxnor.so, or with bounds_check the checking build libxnor_check.so."""
    lib = LIB_CHECK if bounds_check else LIB
    if not force and up_to_date(lib):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-DXNOR_BOUNDS_CHECK"] if bounds_check else []) + \
        (["-Xptxas", "-v"] if verbose else []) + ["-o", lib] + SOURCES
    subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True))
