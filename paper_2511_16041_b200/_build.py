"""Builds the C-ABI shared library ``libatb.so`` in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libatb.so")
SOURCES = ["atb_status.cpp", "atb_model.cpp", "atb_quantize.cu", "atb_gemm_sm100.cu", "atb_gemm_pair_sm100.cu",
           "atb_gemm_cfg_sm100.cu"]
HEADERS = ["atb_internal.h", "sm100_ptx.cuh", "atb_gemm_device.cuh", "bfp16_block.cuh"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "atb.h")]
    return any(os.path.getmtime(d) > t for d in deps)


# Diagnostic variants of the library: never the product, each loaded only by the test that needs it.
#   timeout_test: every bounded wait gives up after 2 ms and one dequantiser warp of CTA 0 keeps back its
#                 first arrival, so that the timeout path (abort flag, drain, TMEM release, status) runs.
VARIANTS = {"timeout_test": ["-DATB_TEST_WAIT_NS=2000000ull", "-DATB_TEST_WITHHOLD_DEQ_ARRIVAL"]}


def variant_path(variant: str) -> str:
    return os.path.join(HERE, "libatb_%s.so" % variant)


def build_library(force: bool = False, verbose: bool = False, variant: str | None = None) -> str:
    """Compile every translation unit for sm_100a and link ``libatb.so`` (or, with ``variant``, the
    diagnostic library ``libatb_<variant>.so`` from the same sources plus that variant's flags).
    Returns its path."""
    if variant is not None:
        return _build(variant_path(variant), os.path.join(HERE, "build", variant), VARIANTS[variant], force, verbose)
    return _build(LIB, CSRC, [], force, verbose)


def _build(lib: str, obj_dir: str, extra: list, force: bool, verbose: bool) -> str:
    if not force and not is_stale(lib):
        return lib
    os.makedirs(obj_dir, exist_ok=True)
    objs = []
    common = ["-std=c++17", "-O3", "-lineinfo", "-Xcompiler", "-fPIC",
              "-gencode", "arch=compute_100a,code=sm_100a",
              "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        common += ["-Xptxas", "-v"]
    common += os.environ.get("ATB_NVCC_FLAGS", "").split() + list(extra)
    procs = []
    for src in SOURCES:
        obj = os.path.join(obj_dir, os.path.splitext(src)[0] + ".o")
        objs.append(obj)
        cmd = [_nvcc()] + common + ["-x", "cu", "-c", os.path.join(CSRC, src), "-o", obj]
        procs.append((cmd, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for cmd, p in procs:
        out, _ = p.communicate()
        if verbose and out:
            print(out)
        if p.returncode != 0:
            raise RuntimeError("nvcc failed: %s\n%s" % (" ".join(cmd), out))
    link = [_nvcc(), "-shared", "-o", lib] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"]
    subprocess.run(link, check=True)
    return lib


if __name__ == "__main__":
    import sys
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
    for name in VARIANTS:
        if "--variants" in sys.argv:
            print(build_library(force="--force" in sys.argv, variant=name))
