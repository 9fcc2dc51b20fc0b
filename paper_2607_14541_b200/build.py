"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libatrex_agg.so")
SOURCES = ["api.cu", "scatter.cu", "ingest.cu", "finalize.cu", "static_topk.cu", "score.cu", "eq3.cu", "release.cu", "exchange.cu"]
HEADERS = ["atrex_dev.cuh", "kernels.h", os.path.join("..", "..", "include", "atrex_agg.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-fmad=false", "-shared", "-Xcompiler", "-fPIC", "-ldl"]


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libatrex_agg.so if it is missing or older than its sources."""
    srcs = [os.path.join(CSRC, s) for s in SOURCES]
    deps = srcs + [os.path.normpath(os.path.join(CSRC, h)) for h in HEADERS]
    if force or _stale(LIB, deps):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB] + srcs
        subprocess.check_call(cmd)
    return LIB


DEBUG_LIB = os.path.join(_HERE, "libatrex_agg_checked.so")


def build_checked(force: bool = False) -> str:
    """The same library with -DATREX_DEBUG_BOUNDS: every kernel index is range checked (see
    atrex_build_has_bounds_checks in the header).  Select it with ATREX_AGG_LIBRARY=<path>."""
    srcs = [os.path.join(CSRC, s) for s in SOURCES]
    deps = srcs + [os.path.normpath(os.path.join(CSRC, h)) for h in HEADERS]
    if force or _stale(DEBUG_LIB, deps):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.check_call([nvcc] + NVCC_FLAGS + ["-DATREX_DEBUG_BOUNDS", "-o", DEBUG_LIB] + srcs)
    return DEBUG_LIB


# the scatter pass's build-time variant that the test-suite runs the parity cases under
VARIANTS = {"ring4": ["-DATREX_SCATTER_RING=4"]}


def variant_path(name: str) -> str:
    return os.path.join(_HERE, f"libatrex_agg_{name}.so")


def build_variant_if_stale(name: str, flags) -> str:
    srcs = [os.path.join(CSRC, s) for s in SOURCES]
    deps = srcs + [os.path.normpath(os.path.join(CSRC, h)) for h in HEADERS]
    if _stale(variant_path(name), deps):
        build_variant(name, flags)
    return variant_path(name)


def build_all(force: bool = True) -> None:
    """The regular library, the bounds-checked one and the tested variants, compiled side by side."""
    from concurrent.futures import ThreadPoolExecutor
    jobs = [lambda: build(force=force), lambda: build_checked(force=force)]
    jobs += [(lambda n=n, f=f: build_variant(n, f) if force else build_variant_if_stale(n, f)) for n, f in VARIANTS.items()]
    with ThreadPoolExecutor(max_workers=len(jobs)) as pool:
        for fut in [pool.submit(j) for j in jobs]:
            fut.result()


def build_variant(name: str, flags) -> str:
    """The library with extra nvcc flags, as libatrex_agg_<name>.so beside the regular one -- e.g. the
    scatter pass's build-time variant (-DATREX_SCATTER_RING=4).  Select it with
    ATREX_AGG_LIBRARY=<path>."""
    out = os.path.join(_HERE, f"libatrex_agg_{name}.so")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.check_call([nvcc] + NVCC_FLAGS + list(flags) + ["-o", out] + [os.path.join(CSRC, s) for s in SOURCES])
    return out


if __name__ == "__main__":
    import sys
    if len(sys.argv) >= 3 and sys.argv[1] == "--variant":      # build.py --variant NAME [nvcc flags...]
        print(build_variant(sys.argv[2], sys.argv[3:]))
    else:
        print(build(force=True, verbose=True))
