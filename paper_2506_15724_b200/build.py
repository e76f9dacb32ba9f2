"""Builds libmadakv.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libmadakv.so")
PROBE_SRC = os.path.join(HERE, "csrc", "probe", "exp2_roof.cu")
PROBE = os.path.join(HERE, "exp2_roof.bin")  # measures the exp2 roof (see the source); used by bench.py


def sources():
    return sorted(glob.glob(os.path.join(HERE, "csrc", "*.cu")))


def needs_build():
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(HERE, "csrc", "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(f) > t for f in deps)


def build_probe(force=False):
    """The stand-alone exp2-roof probe (a small CUDA program, not part of the library)."""
    if force or not os.path.exists(PROBE) or os.path.getmtime(PROBE) < os.path.getmtime(PROBE_SRC):
        subprocess.check_call(["nvcc", "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
                               "-o", PROBE, PROBE_SRC])
    return PROBE


def build(force=False, verbose=False):
    build_probe(force)
    if not force and not needs_build():
        return LIB
    cmd = [
        "nvcc", "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
        "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(HERE, "csrc"),
        "-o", LIB,
    ] + (["-Xptxas", "-v"] if verbose else []) + sources()
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
