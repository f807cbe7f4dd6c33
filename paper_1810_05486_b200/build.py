"""Compile the CUDA library (C ABI of include/kahan_sgd.h) for sm_100a with nvcc, in-tree."""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIBRARY = os.path.join(_HERE, "libkahan_sgd.so")
SOURCES = [os.path.join(CSRC, "kahan_sgd_api.cu")]
_DEPENDS = SOURCES + [os.path.join(CSRC, "kahan_sgd_ring.cuh"), os.path.join(CSRC, "kahan_sgd_kernels.cuh"),
                      os.path.join(CSRC, "kahan_sgd_momentum_kernels.cuh"),
                      os.path.join(CSRC, "kahan_sgd_adam_kernels.cuh"),
                      os.path.join(CSRC, "kahan_sgd_convert.cuh"),
                      os.path.join(INCLUDE, "kahan_sgd.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--fmad=false",           # the update has no fused multiply-add
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def is_stale() -> bool:
    if not os.path.exists(LIBRARY):
        return True
    built = os.path.getmtime(LIBRARY)
    return any(os.path.getmtime(p) > built for p in _DEPENDS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Build libkahan_sgd.so if missing or older than its sources; return its path."""
    if not force and not is_stale():
        return LIBRARY
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
        ["-I", INCLUDE, "-I", CSRC] + SOURCES + ["-o", LIBRARY + ".tmp"]
    subprocess.run(cmd, check=True)
    os.replace(LIBRARY + ".tmp", LIBRARY)
    return LIBRARY


if __name__ == "__main__":
    print(build(force=True, verbose=True))
