"""Build the sm_100a shared library (C ABI, no torch types) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfirp_b200.so")
SOURCES = ["firp_api.cu", "small_kernels.cu", "gemm_tcgen05.cu", "finish_kernels.cu", "attn_tree.cu", "attn_tc.cu", "fused_step.cu",
           "topb_static.cu"]
HEADERS = ["firp_kernels.cuh", "launch_util.cuh", "tc_device.cuh", "finish_device.cuh", "norm_device.cuh", "attn_device.cuh",
           os.path.join("..", "..", "include", "firp.h")]
# -dlcm=cg: plain global loads are cached in L2 only.  Under programmatic dependent launch kernels of
# consecutive steps share an SM; buffers that are rewritten every step (context lengths, tree metadata,
# activations) must never be served from an L1 line another kernel left behind.
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "--use_fast_math", "-Xptxas", "-dlcm=cg", "-shared"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    tmp = LIB + ".%d.tmp" % os.getpid()
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
