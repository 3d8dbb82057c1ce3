"""Compile the CUDA library in-tree: paper_2401_14021_b200/libralm.so (sm_100a only).

`--debug` builds libralm_debug.so beside it with -DRALM_DEBUG_BOUNDS: every index into a global
array that a scan kernel computes is checked against the array's extent (a violation is recorded
in the status word as RALM_ERR_INTERNAL; nothing traps). Point RALM_LIBRARY at that file to run
the tests or the benchmark on it."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libralm.so")
DEBUG_LIB = os.path.join(HERE, "libralm_debug.so")
SOURCES = ["ralm_api.cu", "os3.cpp"]
HEADERS = ["common.cuh", "scan.cuh", "aux_kernels.cuh", os.path.join("..", "..", "include", "ralm.h")]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    paths += [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    return max(os.path.getmtime(p) for p in paths if os.path.exists(p))


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = DEBUG_LIB if debug else LIB
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _newest_source_mtime():
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "--threads", "0"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if debug:
        cmd += ["-DRALM_DEBUG_BOUNDS"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES] + ["-o", tmp, "-lcudart"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
