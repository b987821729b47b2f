"""Build the CUDA library in-tree for sm_100a with nvcc (no JIT cache, no torch extension)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libaspd.so")
LIB_DEBUG_BOUNDS = os.path.join(HERE, "libaspd_debug_bounds.so")   # -DASPD_DEBUG_BOUNDS: kernels that check page ids and rows

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(f) > t for f in deps)


def build(force: bool = False, verbose: bool = False, out: str = LIB, defines=()) -> str:
    if not force and out == LIB and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = ([nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + [f"-D{d}" for d in defines]
           + ["-o", out] + sources())
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return out


def build_debug_bounds(force: bool = False) -> str:
    """The checking build, beside the product library (the GPU tests run a subset against it)."""
    if force or not os.path.exists(LIB_DEBUG_BOUNDS) or (os.path.exists(LIB) and os.path.getmtime(LIB_DEBUG_BOUNDS) < os.path.getmtime(LIB)):
        build(force=True, out=LIB_DEBUG_BOUNDS, defines=["ASPD_DEBUG_BOUNDS"])
    return LIB_DEBUG_BOUNDS


def build_probes() -> str:
    """Stand-alone timing probes of the tensor-core kernels' building blocks (csrc/probes/*.cu -> csrc/probes/bin/)."""
    out_dir = os.path.join(CSRC, "probes", "bin")
    os.makedirs(out_dir, exist_ok=True)
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    for src in sorted(glob.glob(os.path.join(CSRC, "probes", "*.cu"))):
        exe = os.path.join(out_dir, os.path.splitext(os.path.basename(src))[0])
        cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
               "-o", exe, src]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return out_dir


if __name__ == "__main__":
    if "--probes" in sys.argv:
        print(build_probes())
        sys.exit(0)
    if "--debug-bounds" in sys.argv:
        print(build_debug_bounds(force=True))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
