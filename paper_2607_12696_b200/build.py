"""Build libmoev.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libmoev.so")
# the same sources with -DMOEV_TEST_HOOKS: millisecond wait budgets and a switch that makes bounded device
# waits run out, for the tests of the time-out path; never loaded by the package itself
TEST_LIB = os.path.join(_HERE, "libmoev_testhooks.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(
        os.path.join(_HERE, "..", "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(out: str, defines=(), verbose: bool = False):
    cmd = [NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC"] + ["-D" + d for d in defines] + ["-o", out] + sources() + ["-lcuda"]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ into one shared library (and its test-hook twin); returns the
    library's path."""
    from concurrent.futures import ThreadPoolExecutor
    jobs = []
    with ThreadPoolExecutor(max_workers=2) as pool:
        if force or _stale(TEST_LIB):
            jobs.append(pool.submit(_compile, TEST_LIB, ("MOEV_TEST_HOOKS",)))
        if force or _stale(LIB):
            jobs.append(pool.submit(_compile, LIB, (), verbose))
        for j in jobs:
            j.result()  # raises if a compilation failed
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
