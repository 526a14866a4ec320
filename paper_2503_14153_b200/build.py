"""Builds libspec_decode.so (sm_100a) next to the sources with nvcc."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libspec_decode.so")
SOURCES = ["spec_api.cu"]
DEPS = ["spec_api.cu", "common.cuh", "kernels_simple.cuh", "gemm_stream.cuh", "gemm_cluster.cuh", "gemm_wide.cuh", "glue_tc.cuh", "attention_tc.cuh", "attention_umma.cuh", "labels.cuh",
        os.path.join("..", "..", "include", "spec_decode.h")]


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPS if os.path.exists(os.path.join(CSRC, d)))


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "--use_fast_math" if False else "-Xptxas", "-v" if verbose else "-O3",
           "-cudart", "static", "-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed")
    if verbose:
        print(res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
