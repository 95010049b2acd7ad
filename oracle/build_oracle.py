"""Compile the CPU oracle (test infrastructure) into two shared libraries.

`liboracle_f32.so`: forward pass in fp32 in the canonical operation order.
`liboracle_f64.so`: everything in double (closed-form and finite-difference checks).

-ffp-contract=off keeps the compiler from fusing anything the source does not
fuse; -mfma only lets the explicit fma calls compile to one instruction.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "snn_oracle.c")
FLAGS = ["-O2", "-ftree-vectorize", "-ffp-contract=off", "-fno-fast-math", "-mavx2", "-mfma",
         "-fopenmp", "-shared", "-fPIC", "-std=c11", "-Wall"]


def lib_path(kind: str) -> str:
    return os.path.join(HERE, f"liboracle_{kind}.so")


def build(force: bool = False) -> None:
    for kind, real in (("f32", "float"), ("f64", "double")):
        out = lib_path(kind)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(SRC):
            continue
        cmd = ["gcc", *FLAGS, f"-DREAL={real}", f"-DPFX={kind}", SRC, "-o", out, "-lm"]
        subprocess.run(cmd, check=True)


if __name__ == "__main__":
    build(force="--force" in sys.argv)
    print("built", lib_path("f32"), lib_path("f64"))
