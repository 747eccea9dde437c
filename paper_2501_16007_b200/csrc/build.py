"""Builds csrc/libtoploc.so for sm_100a with nvcc (cross-compiles without a GPU).

    python -m paper_2501_16007_b200.csrc.build [--force] [--verbose]
"""
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(os.path.dirname(_HERE))
SOURCES = [os.path.join(_HERE, "toploc.cu"), os.path.join(_HERE, "toploc_direct.cu"),
           os.path.join(_HERE, "toploc_producer.cu")]
HEADERS = [os.path.join(_ROOT, "include", "toploc.h"), os.path.join(_ROOT, "include", "toploc_device.cuh"),
           os.path.join(_HERE, "nearest_ratio.cuh")]
LIBRARY = os.path.join(_HERE, "libtoploc.so")


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def build(force=False, verbose=False):
    newest = max(os.path.getmtime(p) for p in SOURCES + HEADERS + [os.path.abspath(__file__)])
    if not force and os.path.exists(LIBRARY) and os.path.getmtime(LIBRARY) >= newest:
        return LIBRARY
    tmp = LIBRARY + ".tmp%d" % os.getpid()
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC",
           "-I", os.path.join(_ROOT, "include")]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += SOURCES + ["-o", tmp]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIBRARY)
    return LIBRARY


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
