"""Builds the CUDA library (libga.so) in-tree with nvcc for sm_100a."""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
LIB = os.path.join(_HERE, "libga.so")
SOURCES = [os.path.join(_HERE, "csrc", "ga_api.cu")]
DEPENDS = SOURCES + [os.path.join(_HERE, "csrc", "ga_kernels.cuh"), os.path.join(_HERE, "csrc", "ga_layer_kernels.cuh"), os.path.join(ROOT, "include", "ga.h")]
NVCC_FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include")]


def build(force=False, verbose=False):
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(s) for s in DEPENDS):
        return LIB
    tmp = f"{LIB}.{os.getpid()}.tmp"
    cmd = ["nvcc", *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-o", tmp, *SOURCES]
    try:
        subprocess.check_call(cmd)
    except OSError:   # the compiler itself is missing
        if os.path.exists(LIB) and not force:   # no nvcc here: keep the library that travelled with the tree
            return LIB
        raise
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    build(force=True, verbose="-v" in sys.argv)
    print(LIB)
