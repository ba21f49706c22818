"""Builds libcmpq.so (the CUDA library behind include/cmpq.h) in-tree with nvcc for sm_100a."""
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB_PATH = os.path.join(_PKG, "libcmpq.so")
SOURCES = ["api.cu", "stats.cu", "stats_static.cu", "alloc.cu", "lloyd.cu", "lloyd_hist.cu", "outliers.cu", "pack.cu", "matvec.cu"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "--fmad=false", "--cudart", "static", "-I", INCLUDE, "-I", CSRC]


def _newest_source_mtime():
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "cmpq.h")]
    return max(os.path.getmtime(f) for f in files)


def build(force=False, verbose=False):
    """Compile every .cu into one shared library; returns its path."""
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= _newest_source_mtime():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB_PATH + ".tmp%d" % os.getpid()
    extra = os.environ.get("CMPQ_EXTRA_NVCC_FLAGS", "").split()
    cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-shared", "-o", tmp]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
