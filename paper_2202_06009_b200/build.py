"""Compile the CUDA sources of this package for sm_100a into libzoa.so (in-tree)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libzoa.so")
SOURCES = ["zoa_kernels.cu", "zoa_pipeline.cu", "zoa_reduce_pipeline.cu", "zoa_server_pipeline.cu", "zoa_api.cu", "zoa_noalloc.cu"]
HEADERS = ["zoa_device.cuh", "zoa_internal.h", "zoa_ring.cuh", os.path.join("..", "..", "include", "zoa.h")]

# The arithmetic contract needs IEEE division and square root, subnormals kept,
# and no contraction of a multiply and an add into one fused operation.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--fmad=false", "--ftz=false", "--prec-div=true", "--prec-sqrt=true",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    cmd = ["nvcc", *NVCC_FLAGS, "-shared", "-o", LIB, *[os.path.join(CSRC, s) for s in SOURCES]]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
