"""Builds libccoll.so (the CUDA kernels and their C ABI) in-tree with nvcc for sm_100a.

--fmad=false: the block rules are stated as separately rounded fp32 operations, so no multiply-add may be
fused.  No fast-math, no flush-to-zero.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SOURCES = [os.path.join(CSRC, f) for f in ("ccoll_kernels.cu", "ccoll_api.cu", "ccoll_noalloc.cu")]
HEADERS = [os.path.join(CSRC, f) for f in ("ccoll_kernels.cuh", "ccoll_device_common.cuh", "ccoll_encode.cuh",
                                            "ccoll_decode.cuh")] + [os.path.join(os.path.dirname(HERE), "include", "ccoll.h")]
LIB = os.path.join(HERE, "libccoll.so")

NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "--fmad=false",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; returns its path."""
    if not force and not stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + SOURCES + ["-o", LIB + ".tmp"]
    subprocess.run(cmd, check=True, cwd=HERE)
    os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
