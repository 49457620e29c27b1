"""Compile the CUDA library in-tree: paper_1611_05402_b200/csrc/libzipml.so (sm_100a only)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(CSRC, "libzipml.so")
SOURCES = ["api.cu", "quantize.cu", "levels.cu", "sgd.cu", "sgd_ring.cu", "sgd_lean.cu", "sgd_cluster.cu", "sgd_stream.cu", "loss.cu"]
HEADERS = ["common.cuh", "internal.h", "sgd_common.cuh", "int_digits.cuh", os.path.join("..", "..", "include", "zipml.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--fmad=true", "-Xcompiler", "-fPIC", "-shared"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", LIB] + [os.path.join(CSRC, f) for f in SOURCES]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
