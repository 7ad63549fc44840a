"""Builds the CUDA libraries in-tree with nvcc for sm_100a (no JIT cache, no torch extension).

  libpsmc.so           the product: kernels + C-ABI declared in include/psmc.h
  libpsmc_workload.so  synthetic-input generators for tests and benchmarks (not part of the path)
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libpsmc.so")
LIB_WORKLOAD = os.path.join(PKG, "libpsmc_workload.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "--threads", "0", "-std=c++17", "-shared",
              "-Xcompiler", "-fPIC", "--use_fast_math=false"]

PRODUCT_SOURCES = ["context.cu", "logits_pass.cu", "step_fused.cu", "weights_resample.cu", "vocab_shard.cu",
                   "masked_proposal.cu", "reindex_kv.cu", "paged_kv.cu", "select.cu"]
WORKLOAD_SOURCES = ["workload.cu"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _stale(target: str, sources) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    deps = list(sources) + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    deps.append(os.path.join(os.path.dirname(PKG), "include", "psmc.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def _build(target: str, names, verbose: bool, extra=()) -> None:
    sources = [os.path.join(CSRC, n) for n in names]
    tmp = target + ".tmp.%d" % os.getpid()
    cmd = [_nvcc()] + [f for f in NVCC_FLAGS if f != "--use_fast_math=false"] + list(extra) + ["-o", tmp] + sources
    if verbose:
        print(" ".join(cmd), file=sys.stderr)
    subprocess.check_call(cmd)
    os.replace(tmp, target)


def build_all(force: bool = False, verbose: bool = False, ptxas_info: bool = False) -> None:
    extra = ["-Xptxas", "-v"] if ptxas_info else []
    srcs = [os.path.join(CSRC, n) for n in PRODUCT_SOURCES]
    if force or _stale(LIB, srcs):
        _build(LIB, PRODUCT_SOURCES, verbose, extra)
    srcs = [os.path.join(CSRC, n) for n in WORKLOAD_SOURCES]
    if force or _stale(LIB_WORKLOAD, srcs):
        _build(LIB_WORKLOAD, WORKLOAD_SOURCES, verbose, extra)


if __name__ == "__main__":
    build_all(force="--force" in sys.argv, verbose=True, ptxas_info="--ptxas-info" in sys.argv)
