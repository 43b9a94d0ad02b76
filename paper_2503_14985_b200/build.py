"""Builds libmlt.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import re
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libmlt.so")
SOURCES = ["mlt.cu"]
HEADERS = ["ptx.cuh", "gemm.cuh", "mha.cuh", "paged.cuh", os.path.join("..", "..", "include", "mlt.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


# The attention kernel moves registers between its warpgroups (setmaxnreg): 8 softmax warps at 232 and 4 other
# warps at 40 must fit the launch allocation of 384 threads, i.e. ptxas has to assign at least this many per thread.
MHA_MIN_REGISTERS = 168


def check_mha_registers(ptxas_log: str) -> dict:
    """Register counts of the mha_fwd_kernel instantiations in a `-Xptxas -v` log; raises if one is below the budget
    the in-kernel register hand-over needs (launching such a build would wait for registers that never come)."""
    found = {}
    name = None
    for line in ptxas_log.splitlines():
        m = re.search(r"Compiling entry function '(\w+)'", line)
        if m:
            name = m.group(1)
        m = re.search(r"Used (\d+) registers", line)
        if m and name and "mha_fwd_kernel" in name:
            found[name] = int(m.group(1))
            name = None
    low = {k: v for k, v in found.items() if v < MHA_MIN_REGISTERS}
    if low:
        raise RuntimeError(f"attention kernel compiled with fewer than {MHA_MIN_REGISTERS} registers per thread: {low}")
    return found


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the CUDA sources into libmlt.so next to this file; returns its path."""
    if force or is_stale():
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = LIB + f".tmp{os.getpid()}"
        cmd = [nvcc, *NVCC_FLAGS, "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
        if not check_mha_registers(res.stdout + res.stderr):
            raise RuntimeError("no mha_fwd_kernel entry in the ptxas log")
        os.replace(tmp, LIB)
        if verbose:
            print(res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
