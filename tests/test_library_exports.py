"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol
that include/chameleon.h declares.  No compute call is made here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2508_21613_b200 import build
    return build.build()


def test_every_declared_entry_point_is_exported(lib_path):
    header = open(os.path.join(ROOT, "include", "chameleon.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(cm_[a-z0-9_]+)\s*\(", header))
    assert {"cm_create", "cm_load_profile", "cm_enumerate", "cm_evaluate", "cm_select",
            "cm_search_batch", "cm_decode_plan"} <= declared
    lib = ctypes.CDLL(lib_path)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in chameleon.h but not exported"
    from paper_2508_21613_b200 import binding
    assert set(binding.EXPORTS) == declared


def test_binding_constants_match_the_header():
    from paper_2508_21613_b200 import binding
    header = open(os.path.join(ROOT, "include", "chameleon.h")).read()
    defines = {k: int(v) for k, v in re.findall(r"#define\s+(CM_[A-Z_]+)\s+(\d+)", header)}
    assert binding.NOALLOC_MAX_CANDIDATES == defines["CM_NOALLOC_MAX_CANDIDATES"]
    assert (binding.MAX_PIPES, binding.MAX_STAGES, binding.MAX_LAYERS) == (
        defines["CM_MAX_PIPES"], defines["CM_MAX_STAGES"], defines["CM_MAX_LAYERS"])
    assert (binding.MAX_SHORTLIST, binding.MAX_MATCH) == (defines["CM_MAX_SHORTLIST"], defines["CM_MAX_MATCH"])


def test_transition_time_needs_no_device(lib_path):
    """cm_transition_time is host arithmetic: restart + bytes / bandwidth, floored in integer mode."""
    from paper_2508_21613_b200 import binding, workloads as W
    obj = W.ObjectiveOptions(t_restart_ns=5e9, bw_xfer_Bpns=25)
    t, ti = binding.cm_transition_time(obj, [0, 1000, 1012, -1])
    assert list(t) == [5e9, 5e9 + 40.0, 5e9 + 1012 / 25, -1.0]
    assert list(ti) == [5 * 10**9, 5 * 10**9 + 40, 5 * 10**9 + 40, -1]


def test_struct_layouts_match_the_header():
    from paper_2508_21613_b200 import binding
    assert ctypes.sizeof(binding.cm_plan) == 8 + 8 + 8 + 8 + 8 + 32 + 32 + 128
    assert binding.cm_plan.kappa.offset == 104
    assert ctypes.sizeof(binding.cm_enum_opts) == 40
    assert binding.cm_enum_opts.kappa_cap.offset == 24
    assert binding.cm_enum_opts.cost.offset == 32 and binding.cm_enum_opts.sched.offset == 36
    assert ctypes.sizeof(binding.cm_profile) == 16 + 9 * 8 + 8 + 8 + 16


def test_no_cpu_fallback_without_a_device(lib_path):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2508_21613_b200 import binding
    lib = binding.load_library()
    ctx = ctypes.c_void_p()
    assert lib.cm_create(ctypes.byref(ctx), 0, None) == binding.CM_ECUDA
    with pytest.raises(binding.ChameleonError):
        binding.cm_create(0)


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2508_21613_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.replace("no CPU", "").lower() or f == "workloads.py", f
