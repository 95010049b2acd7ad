"""Compile the CUDA library (sm_100a only) into paper_2412_11810_b200/libsnnckpt.so."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SOURCES = [os.path.join(CSRC, "snn_api.cu"), os.path.join(CSRC, "schedule.cpp")]
HEADERS = [os.path.join(CSRC, "kernels.cuh"), os.path.join(CSRC, "tma.cuh"), os.path.join(CSRC, "tc_gemm.cuh"), os.path.join(HERE, "..", "include", "snn.h")]
LIB = os.path.join(HERE, "libsnnckpt.so")
LIB_DEBUG = os.path.join(HERE, "libsnnckpt_debug.so")   # the same sources with -DSNN_DEBUG_CHECKS=1 (bounds-checked)
# -fmad=false: nothing is fused unless the source says fmaf; the forward arithmetic that decides
# spikes is written with explicit intrinsics anyway.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-fmad=false",
              "-Xcompiler", "-fPIC", "-shared"]


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    deps = SOURCES + HEADERS
    out = LIB_DEBUG if debug else LIB
    if not force and os.path.exists(out) and all(os.path.getmtime(out) >= os.path.getmtime(d) for d in deps):
        return out
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, *NVCC_FLAGS, *(["-DSNN_DEBUG_CHECKS=1"] if debug else []), *(["-Xptxas", "-v"] if verbose else []),
           *SOURCES, "-o", out, "-ldl"]
    subprocess.run(cmd, check=True)
    return out


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
