"""Builds libcmpq.so (the CUDA library behind include/cmpq.h) in-tree with nvcc for sm_100a."""
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB_PATH = os.path.join(_PKG, "libcmpq.so")
SOURCES = ["api.cu", "stats.cu", "stats_static.cu", "alloc.cu", "lloyd.cu", "lloyd_weighted.cu", "lloyd_hist.cu", "outliers.cu", "pack.cu", "matvec.cu", "transpose.cu", "probe.cu", "lut_store.cu"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "--fmad=false", "--cudart", "static", "-I", INCLUDE, "-I", CSRC]


def _headers_mtime():
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    return max(os.path.getmtime(f) for f in files + [os.path.join(INCLUDE, "cmpq.h")])


def build(force=False, verbose=False):
    """Compile every .cu (one object per source under _build/, recompiled only when it or a header changed,
    or when the flags did) and link them into one shared library; returns its path."""
    import hashlib
    from concurrent.futures import ThreadPoolExecutor

    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    extra = os.environ.get("CMPQ_EXTRA_NVCC_FLAGS", "").split()
    flags = NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else [])
    tag = hashlib.sha1(" ".join([nvcc] + flags).encode()).hexdigest()[:10]
    obj_dir = os.path.join(_PKG, "_build")
    os.makedirs(obj_dir, exist_ok=True)
    hdr = _headers_mtime()
    jobs, objects = [], []
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(obj_dir, "%s.%s.o" % (src[:-3], tag))
        objects.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(path), hdr):
            jobs.append((path, obj))

    def compile_one(job):
        tmp = job[1] + ".tmp%d" % os.getpid()
        subprocess.run([nvcc] + flags + ["-c", "-o", tmp, job[0]], check=True)
        os.replace(tmp, job[1])

    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as pool:
            list(pool.map(compile_one, jobs))
    if jobs or not os.path.exists(LIB_PATH) or os.path.getmtime(LIB_PATH) < max(os.path.getmtime(o) for o in objects):
        tmp = LIB_PATH + ".tmp%d" % os.getpid()
        subprocess.run([nvcc, "-shared", "--cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                        "-o", tmp] + objects, check=True)
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
