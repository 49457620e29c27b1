"""Compile the CUDA library in-tree: paper_1611_05402_b200/csrc/libzipml.so (sm_100a only).

Every source is compiled to its own object (in parallel, only when it or a header is newer than
the object) under csrc/_build/, then the objects are linked into the shared library.
"""
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(CSRC, "_build")
LIB = os.path.join(CSRC, "libzipml.so")
SOURCES = ["api.cu", "quantize.cu", "levels.cu", "sgd.cu", "sgd_ring.cu", "sgd_lean.cu", "sgd_cluster.cu", "sgd_stream.cu",
           "sgd_column.cu", "sgd_apply.cu", "shared_base.cu", "poly.cu", "loss.cu"]
HEADERS = ["common.cuh", "internal.h", "sgd_common.cuh", "int_digits.cuh", os.path.join("..", "..", "include", "zipml.h")]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--fmad=true",
         "-Xcompiler", "-fPIC"]


def _mtime(path: str) -> float:
    return os.path.getmtime(path) if os.path.exists(path) else 0.0


def _compile(src: str, verbose: bool) -> None:
    cmd = ["nvcc"] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", os.path.join(CSRC, src), "-o",
                                                                          os.path.join(OBJ, src + ".o")]
    subprocess.run(cmd, check=True)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    newest_header = max(_mtime(os.path.join(CSRC, h)) for h in HEADERS)
    stale = [s for s in SOURCES
             if force or _mtime(os.path.join(OBJ, s + ".o")) < max(_mtime(os.path.join(CSRC, s)), newest_header)]
    if stale:
        with ThreadPoolExecutor(max_workers=min(len(stale), os.cpu_count() or 1)) as pool:
            list(pool.map(lambda s: _compile(s, verbose), stale))
    objects = [os.path.join(OBJ, s + ".o") for s in SOURCES]
    if stale or _mtime(LIB) < max(_mtime(o) for o in objects):
        subprocess.run(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", LIB] + objects,
                       check=True)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force="-f" in sys.argv or "--force" in sys.argv, verbose="-v" in sys.argv))
