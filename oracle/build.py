"""Compile the CPU oracle (plain C, gcc) into oracle/libzoa_oracle.so.

Test infrastructure: the shared object holds the float and the double build of
zoa_oracle.c side by side (symbols suffixed _f32 / _f64).
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "zoa_oracle.c")
LIB = os.path.join(HERE, "libzoa_oracle.so")

# One IEEE operation per C operation: no contraction into fused multiply-adds,
# no fast-math (which would also flush subnormals), no vectoriser reassociation.
CFLAGS = ["-O2", "-std=c99", "-fPIC", "-ffp-contract=off", "-fno-fast-math",
          "-fno-unsafe-math-optimizations", "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    objs = []
    for real, suffix in (("float", "_f32"), ("double", "_f64")):
        obj = os.path.join(HERE, f"zoa_oracle{suffix}.o")
        subprocess.check_call(["gcc", *CFLAGS, f"-DZO_REAL={real}", f"-DZO_SUFFIX={suffix}",
                               "-c", SRC, "-o", obj])
        objs.append(obj)
    subprocess.check_call(["gcc", "-shared", "-o", LIB, *objs, "-lm"])
    for obj in objs:
        os.remove(obj)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
