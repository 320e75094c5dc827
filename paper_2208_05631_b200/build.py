"""Builds libqasg.so (sm_100a) in-tree with nvcc.  Usable as `python -m paper_2208_05631_b200.build`."""
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "lib", "libqasg.so")
SOURCES = ["qasg_api.cu", "qasg_kernels.cu", "qasg_logreg.cu", "qasg_static.cu", "qasg_optimal.cu", "qasg_touched.cu",
           "qasg_stream.cu"]
HEADERS = [os.path.join(CSRC, "qasg_internal.h"), os.path.join(CSRC, "qasg_device.cuh"),
           os.path.join(os.path.dirname(HERE), "include", "qasg.h")]


def _nvcc():
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libqasg cannot be built")


def is_stale():
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(p) > built for p in deps)


def build_library(force=False, verbose=False):
    """Compiles every CUDA source of the library for sm_100a and links libqasg.so."""
    if not force and not is_stale():
        return LIB
    os.makedirs(os.path.dirname(LIB), exist_ok=True)
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
