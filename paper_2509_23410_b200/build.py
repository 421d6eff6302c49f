"""Builds the CUDA library in-tree: ``libpatch_b200.so`` next to this file (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpatch_b200.so")
LIB_FI = os.path.join(HERE, "libpatch_b200_fi.so")
SOURCES = ["pack.cu", "masks.cu", "gemv.cu", "gemm_decode_sm100.cu", "gemm_decode_cluster_sm100.cu", "gemm_prefill_sm100.cu", "gemm_prefill2_sm100.cu", "gemm_prefill_pair_sm100.cu", "gemm_prefill_pair_mixed_sm100.cu", "gemm_decode_q4_sm100.cu", "api.cu"]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if os.path.isfile(os.path.join(CSRC, f))]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "patch.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, fault_injection: bool = False) -> str:
    """The library; with ``fault_injection`` the test build ``libpatch_b200_fi.so`` (same sources with
    -DPATCH_FAULT_INJECTION: device-side waits give up after 300 us, and the stream-K decode kernel can be told,
    through its status word, to announce bytes that never arrive -- how the tests make a bounded wait run out)."""
    lib = LIB_FI if fault_injection else LIB
    if not (force or _stale(lib)):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "-o", lib]
    if fault_injection:
        cmd += ["-DPATCH_FAULT_INJECTION"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, fault_injection="--fault-injection" in sys.argv))
