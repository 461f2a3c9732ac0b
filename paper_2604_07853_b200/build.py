"""Build libqarl.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libqarl.so")
SOURCES = ["api.cu", "quantize.cu", "permute.cu", "combine.cu", "gemm_sm100.cu", "gemm_decode_sm100.cu", "harness.cu", "linear_static.cu",
           "gemm_w4a16_sm100.cu", "gemm_w4a16_decode_sm100.cu", "api_ext.cu", "api_ep.cu", "gemm_bf16_sm100.cu", "tbpo.cu", "router.cu", "router_fused_sm100.cu", "moe_bwd.cu"]
HEADERS = ["common.cuh", "quant_device.cuh", "w4_dequant.cuh", "ptx_sm100.cuh", "sched.cuh", "api_util.cuh", os.path.join("..", "..", "include", "qarl.h"),
           os.path.join("..", "..", "include", "qarl_harness.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; returns its path."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [nvcc, *NVCC_FLAGS]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES] + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
