"""Compile the CUDA sources into paper_1908_05033_b200/libdsq_b200.so for
sm_100a with nvcc (cross-compiles without a GPU)."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdsq_b200.so")
SOURCES = ["dsq_elementwise.cu", "dsq_dwconv.cu", "dsq_tc.cu", "dsq_conv3.cu", "dsq_gemm8.cu",
           "dsq_soft.cu"]
HEADERS = ["dsq_common.cuh", "dsq_epilogue.cuh", "dsq_ptx.cuh", "dsq_tc_common.cuh",
           "dsq_tc_host.h", "dsq_hooks.h",
           os.path.join("..", "..", "include", "dsq.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo",
              "-std=c++17", "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC",
              "-Xcompiler", "-fvisibility=default", "--fmad=false", "--threads", "0"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + ["-shared", "-o", LIB]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
