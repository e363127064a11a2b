"""Build ``libchameleon.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libchameleon.so")
SOURCES = ["cm_cost_shallow_f64.cu", "cm_cost_shallow_i64.cu",
           "cm_kernels.cu", "cm_api.cu", "cm_policy.cu", "cm_noalloc.cu", "cm_cost.cu", "cm_cost_solo.cu", "cm_restore.cu", "cm_cache.cu"]
# cm_cost_deep.cu is compiled once per cost type and range of stage counts (the ranges of
# CM_DEEP_RANGES in cm_internal.h): (object suffix, extra flags)
DEEP_RANGES = [(17, 28), (29, 34), (35, 41), (42, 48), (49, 56), (57, 64)]
DEEP_UNITS = [(f"{tag}_{lo}_{hi}", [f"-DCM_DEEP_T={ctype}", f"-DCM_DEEP_LO={lo}", f"-DCM_DEEP_HI={hi}"])
              for lo, hi in DEEP_RANGES for tag, ctype in (("f64", "double"), ("i64", "long long"))]
HEADERS = ["cm_internal.h", "cm_device.cuh", "cm_plan_eval.cuh", "cm_cost_impl.cuh"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
    "--fmad=false",            # the cost model is written as single IEEE operations
    "-Xcompiler", "-fPIC", "-Xcompiler", "-O2",
]


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(_CSRC, f) for f in SOURCES + HEADERS + ["cm_cost_deep.cu"]] + [os.path.join(_ROOT, "include", "chameleon.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; return its path."""
    if not force and not _stale():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")

    def compile_one(unit) -> str:
        src, suffix, extra = unit
        obj = os.path.join(_CSRC, src.replace(".cu", suffix + ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-I", os.path.join(_ROOT, "include"), "-I", _CSRC,
               "-c", os.path.join(_CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        subprocess.check_call(cmd)
        return obj

    # the translation units are independent: compile them side by side
    from concurrent.futures import ThreadPoolExecutor
    # the heaviest units first, so that they do not end up alone at the tail
    units = [("cm_cost_deep.cu", "_" + tag, flags) for tag, flags in reversed(DEEP_UNITS)] + [(s, "", []) for s in SOURCES]
    with ThreadPoolExecutor(max_workers=max(1, min(len(units), os.cpu_count() or 1))) as pool:
        objs = list(pool.map(compile_one, units))
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
                           "-o", tmp, *objs])
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
