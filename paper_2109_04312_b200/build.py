"""Build libmate.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libmate.so")
TRACE_LIB = os.path.join(PKG, "libmate_trace.so")   # same sources with -DMATE_TRACE (cycle counters per role)


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        [os.path.join(ROOT, "include", "mate.h")]


def build(force: bool = False, verbose: bool = False, trace: bool = False) -> str:
    """Compiles the library (trace=True: the profiling build with cycle counters, libmate_trace.so,
    which `bench.py --trace` loads; it is a few per cent slower and never the default)."""
    lib = TRACE_LIB if trace else LIB
    if not force and os.path.exists(lib):
        t = os.path.getmtime(lib)
        if all(os.path.getmtime(p) <= t for p in _deps()):
            return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = lib + ".%d.tmp" % os.getpid()
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", tmp] + sources()
    if trace:
        cmd.insert(1, "-DMATE_TRACE")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, trace="--trace" in sys.argv))
