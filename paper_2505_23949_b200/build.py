"""Build step: compiles the CUDA sources under ``csrc/`` for sm_100a into the
in-tree shared library ``libtsenor.so`` (C ABI declared in ``include/tsenor.h``)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libtsenor.so")
LIB_BOUNDS = os.path.join(HERE, "libtsenor_bounds.so")   # same sources with -DTSENOR_BOUNDS (checked indices)
SOURCES = ["tsenor_api.cu"]
HEADERS = ["tsenor_device.cuh", os.path.join(ROOT, "include", "tsenor.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared",
]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + [
        h if os.path.isabs(h) else os.path.join(CSRC, h) for h in HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, bounds: bool = False) -> str:
    """Compiles the library; ``bounds=True`` builds the checked flavour (every computed index of the
    loaders, rounding tables and writers is tested, a bad one sets TSENOR_DEV_INTERNAL)."""
    lib = LIB_BOUNDS if bounds else LIB
    if not force and not _stale(lib):
        return lib
    cmd = ["nvcc", *NVCC_FLAGS, "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if bounds:
        cmd += ["-DTSENOR_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", lib] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
    print(build(force=True, verbose="-v" in sys.argv, bounds=True))
