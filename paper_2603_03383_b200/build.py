"""Build the CUDA library (``libmtv.so``) in-tree with nvcc for sm_100a."""
import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libmtv.so")
# Build variants: the library under another name with extra definitions.  "debug_bounds": every index a kernel reads
# from device memory is checked before use (see mtv_debug_bounds_enabled in include/mtv.h).
VARIANTS = {"debug_bounds": (os.path.join(_HERE, "libmtv_debug_bounds.so"), ["-DMTV_DEBUG_BOUNDS"])}
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
         "-Xcompiler", "-fPIC", "-shared", "-x", "cu"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cpp")))


def _stale(lib=LIB):
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(_HERE, "..", "include", "mtv.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, variant: str = "") -> str:
    """Compile every source under csrc/ into one shared object; returns its path."""
    lib, defs = VARIANTS[variant] if variant else (LIB, [])
    if not force and not _stale(lib):
        return lib
    tmp = lib + ".tmp%d" % os.getpid()
    cmd = [NVCC] + FLAGS + defs + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources()
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    import sys
    names = [a for a in sys.argv[1:] if not a.startswith("-")] or [""]
    for name in names:          # e.g. `build.py debug_bounds`; no name = the normal library
        print(build(force=True, verbose="-v" in sys.argv, variant=name))
