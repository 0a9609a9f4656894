"""Compile the CUDA library for sm_100a into the package directory (in-tree libhma.so)."""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhma.so")
TRACE_LIB = os.path.join(HERE, "libhma_trace.so")      # the same sources with -DHMA_TRACE (per-warp timing stamps)


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def stale(lib=LIB):
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(HERE, "..", "include", "hma.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force=False, verbose=False, trace=False, defines=(), out=None):
    """nvcc -> libhma.so (or, with trace=True, libhma_trace.so built with -DHMA_TRACE).  Cross-compiles without a GPU.
    Returns the library path."""
    lib = out or (TRACE_LIB if trace else LIB)
    if not force and not stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-D" + d for d in defines] + (["-DHMA_TRACE"] if trace else [])
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v", "-o", lib] + flags + sources()
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode:
        raise RuntimeError("nvcc failed")
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True, trace="--trace" in sys.argv))
