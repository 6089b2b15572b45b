"""Build the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libftc.so")
SOURCES = ["ftc_api.cu", "ftc_generic.cu", "ftc_tiled.cu", "ftc_staged.cu", "ftc_staged_inst0.cu", "ftc_staged_inst1.cu", "ftc_staged_inst2.cu", "ftc_staged_inst3.cu", "ftc_expand.cu", "ftc_candidates.cu", "ftc_messages.cu", "ftc_fill.cu", "ftc_probe.cu", "ftc_warp_inst0.cu", "ftc_warp_inst1.cu", "ftc_cand_inst0.cu", "ftc_cand_inst1.cu", "ftc_aheap_inst0.cu", "ftc_aheap_inst1.cu", "ftc_aheap_inst2.cu", "ftc_aheap_inst3.cu"]
HEADERS = ["ftc_device.cuh", "ftc_tile_common.cuh", "ftc_staged_impl.cuh", "ftc_warp_impl.cuh", "ftc_cand_impl.cuh", "ftc_aheap_impl.cuh", "ftc_decode_warp.cuh", "ftc_kernels.h", os.path.join("..", "..", "include", "ftc.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--fmad=false"]


def _newest(paths):
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu into objects and link libftc.so next to this file; returns its path."""
    srcs = [os.path.join(CSRC, s) for s in SOURCES]
    deps = srcs + [os.path.join(CSRC, h) for h in HEADERS]
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest(deps):
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    objs = []
    procs = []
    for src in srcs:
        obj = src[:-3] + ".o"
        objs.append(obj)
        cmd = [nvcc, *NVCC_FLAGS, "-c", src, "-o", obj] + (["-Xptxas", "-v"] if verbose else [])
        procs.append((cmd, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for cmd, pr in procs:
        out, _ = pr.communicate()
        if verbose or pr.returncode:
            sys.stderr.write(out)
        if pr.returncode:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))
    subprocess.check_call([nvcc, "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a"])
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
