"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.environ.get("HVD_B200_LIB") or os.path.join(PKG, "libhvd_b200.so")

NVCC_FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--shared"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, defines=()) -> str:
    """`defines` adds -D flags (compile-time tunables of the kernels)."""
    if os.environ.get("HVD_B200_LIB") and os.path.exists(LIB) and not force:
        return LIB       # an explicitly chosen library is used as it is
    if not (force or stale()):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, *NVCC_FLAGS, "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [f"-D{d}" for d in defines]
    cmd += ["-o", LIB, *sources()]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libhvd_b200.so")
    return LIB


BOUNDS_LIB = os.path.join(PKG, "libhvd_b200_bounds.so")


def build_bounds_checked(force: bool = False) -> str:
    """The same sources with -DHVD_DEBUG_BOUNDS: every index of the lookup, commit and streaming kernels is tested
    before the access, a violation lands in the device status word (hvd_device_status) and the access is
    skipped.  The tests run the edge cases against this library (HVD_B200_LIB selects it)."""
    if not force and os.path.exists(BOUNDS_LIB):
        t = os.path.getmtime(BOUNDS_LIB)
        deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
        if all(os.path.getmtime(d) <= t for d in deps):
            return BOUNDS_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, *NVCC_FLAGS, "-DHVD_DEBUG_BOUNDS", "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", BOUNDS_LIB, *sources()]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libhvd_b200_bounds.so")
    return BOUNDS_LIB


PROBE_SRC = os.path.join(ROOT, "bench_probe.cu")
PROBE_LIB = os.path.join(ROOT, "libbench_probe.so")


def build_bench_probe(force: bool = False) -> str:
    """The benchmark's read-only probe kernel (bench_probe.cu beside bench.py): a library of its own, so that
    the product library exports only the method."""
    if not force and os.path.exists(PROBE_LIB) and os.path.getmtime(PROBE_LIB) >= os.path.getmtime(PROBE_SRC):
        return PROBE_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    res = subprocess.run([nvcc, *NVCC_FLAGS, "-o", PROBE_LIB, PROBE_SRC], capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libbench_probe.so")
    return PROBE_LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
