"""Thin ctypes binding of ``libchameleon.so`` -- argument marshalling only.

Every step of the search runs in the library's CUDA kernels; this module converts
Python/numpy/torch arguments to the plain pointers and sizes of the C ABI
(``include/chameleon.h``) and turns status codes into exceptions.  The functions carry
the names of the C entry points.  PyTorch is used for device memory and for the
current CUDA stream, nothing else.

There is no CPU fallback: if the library is missing, or no sm_100 device is present,
the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libchameleon.so")

MAX_PIPES, MAX_STAGES, MAX_LAYERS = 16, 64, 128
CM_OK, CM_EINVAL, CM_ENOPROFILE, CM_EOVERFLOW, CM_ENOFEASIBLE, CM_ECUDA, CM_ENOMEM, CM_ETIMEOUT = range(8)
CM_REROUTE, CM_REDUNDANT, CM_DYNPAR = 0, 1, 2
CM_COST_FP64, CM_COST_INT64NS = 0, 1

EXPORTS = ["cm_create", "cm_destroy", "cm_load_profile", "cm_enumerate", "cm_evaluate", "cm_select",
           "cm_decode_plan", "cm_space_free", "cm_search_batch", "cm_batch_prepare", "cm_batch_search",
           "cm_batch_free", "cm_evaluate_argmin_noalloc", "cm_last_stats", "cm_search_objective",
           "cm_objective_stats", "cm_transfer_matching", "cm_cache_build", "cm_cache_lookup", "cm_cache_free",
           "cm_set_sharing", "cm_set_int64_arithmetic", "cm_host_describe", "cm_set_latency_graphs",
           "cm_transition_time", "cm_set_memory_screen", "cm_set_micro_batch_pairs", "cm_set_pipeline_reuse", "cm_int64_runs_in_fp64",
           "cm_strerror", "cm_last_error"]
_STATUS_CALLS = EXPORTS[:28]
NOALLOC_MAX_CANDIDATES = 524288
MAX_SHORTLIST, MAX_MATCH = 16, 256


class ChameleonError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"cm_status {status}: {message}")
        self.status = status


class cm_profile(C.Structure):
    _fields_ = [("L", C.c_int32), ("n_dp", C.c_int32), ("n_pp", C.c_int32), ("n_micro", C.c_int32),
                ("fwd_ns", C.POINTER(C.c_double)), ("bwd_ns", C.POINTER(C.c_double)),
                ("fwd_ns_i", C.POINTER(C.c_int64)), ("bwd_ns_i", C.POINTER(C.c_int64)),
                ("act_bytes", C.POINTER(C.c_int64)), ("param_bytes", C.POINTER(C.c_int64)),
                ("opt_bytes", C.POINTER(C.c_int64)), ("p2p_bytes", C.POINTER(C.c_int64)),
                ("base_cuts", C.POINTER(C.c_int32)),
                ("mem_capacity_bytes", C.c_int64), ("devices_per_node", C.c_int32),
                ("bw_intra_Bpns", C.c_int64), ("bw_inter_Bpns", C.c_int64)]


class cm_enum_opts(C.Structure):
    _fields_ = [("dp_lo", C.c_int32), ("dp_hi", C.c_int32), ("pp_lo", C.c_int32), ("pp_hi", C.c_int32),
                ("lm", C.c_int32), ("bm", C.c_int32), ("kappa_cap", C.c_uint64), ("cost", C.c_int32),
                ("sched", C.c_int32)]


class cm_plan(C.Structure):
    _fields_ = [("policy", C.c_int32), ("feasible", C.c_int32), ("cost", C.c_double),
                ("cost_ns", C.c_int64), ("strategy", C.c_uint32), ("n_pipes", C.c_uint32),
                ("split_rank", C.c_uint64), ("stages", C.c_uint16 * MAX_PIPES),
                ("micro", C.c_uint16 * MAX_PIPES), ("kappa", C.c_uint64 * MAX_PIPES)]


class cm_objective_opts(C.Structure):
    _fields_ = [("topk", C.c_int32), ("sync_rounds", C.c_int32), ("t_gap_ns", C.c_double),
                ("t_restart_ns", C.c_double), ("t_gap_ns_i", C.c_int64), ("t_restart_ns_i", C.c_int64),
                ("bw_xfer_Bpns", C.c_int64)]


class cm_transition(C.Structure):
    _fields_ = [("policy", C.c_int32), ("feasible", C.c_int32), ("rank", C.c_int32), ("n_survivors", C.c_int32),
                ("xfer_bytes", C.c_int64), ("t_trans", C.c_double), ("t_trans_ns", C.c_int64),
                ("objective", C.c_double), ("rounds", C.c_int32), ("domains", C.c_int32),
                ("t_sync", C.c_double), ("t_sync_ns", C.c_int64), ("assign", C.c_uint16 * 256)]


@dataclass
class Plan:
    policy: int
    feasible: bool
    cost: float
    cost_ns: int
    strategy: int
    n_pipes: int
    split_rank: int
    stages: Tuple[int, ...]
    micro: Tuple[int, ...]
    kappa: Tuple[int, ...]

    def key(self):
        """Everything that must match bit for bit between two implementations."""
        return (self.policy, self.feasible, self.strategy, self.n_pipes, self.split_rank,
                self.stages, self.micro, self.kappa)


def _plan_from(c: cm_plan) -> Plan:
    n = c.n_pipes
    return Plan(c.policy, bool(c.feasible), c.cost, c.cost_ns, c.strategy, n, c.split_rank,
                tuple(c.stages[:n]), tuple(c.micro[:n]), tuple(c.kappa[:n]))


def plans_from_array(arr) -> List[Plan]:
    return [_plan_from(arr[i]) for i in range(len(arr))]


_lib = None


def load_library() -> C.CDLL:
    """Load ``libchameleon.so``; raise if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                           "`python -m paper_2508_21613_b200.build` (needs nvcc); there is no CPU path")
    lib = C.CDLL(LIB_PATH)
    vp, u64p = C.c_void_p, C.POINTER(C.c_uint64)
    lib.cm_create.argtypes = [C.POINTER(vp), C.c_int, vp]
    lib.cm_destroy.argtypes = [vp]
    lib.cm_load_profile.argtypes = [vp, C.POINTER(cm_profile)]
    lib.cm_enumerate.argtypes = [vp, C.c_int, C.POINTER(C.c_uint32), C.c_int32, C.POINTER(cm_enum_opts),
                                 C.POINTER(vp), u64p]
    lib.cm_evaluate.argtypes = [vp, vp, C.c_uint64, C.c_uint64, vp, vp, vp, vp]
    lib.cm_select.argtypes = [vp, C.POINTER(vp), C.c_int32, C.POINTER(cm_plan)]
    lib.cm_decode_plan.argtypes = [vp, vp, C.POINTER(cm_plan), C.POINTER(C.c_int32)]
    lib.cm_space_free.argtypes = [vp]
    lib.cm_search_batch.argtypes = [vp, C.POINTER(C.c_uint32), C.POINTER(C.c_int32), C.c_int32,
                                    C.POINTER(cm_enum_opts), C.POINTER(cm_plan), C.POINTER(cm_plan),
                                    C.POINTER(C.c_float)]
    lib.cm_last_stats.argtypes = [vp, u64p]
    lib.cm_strerror.argtypes = [C.c_int]
    lib.cm_strerror.restype = C.c_char_p
    lib.cm_last_error.argtypes = [vp]
    lib.cm_last_error.restype = C.c_char_p
    lib.cm_batch_prepare.argtypes = [vp, C.POINTER(C.c_uint32), C.POINTER(C.c_int32), C.c_int32,
                                     C.POINTER(cm_enum_opts), C.POINTER(vp), u64p]
    lib.cm_batch_search.argtypes = [vp, vp, C.POINTER(cm_plan), C.POINTER(cm_plan)]
    lib.cm_batch_free.argtypes = [vp]
    lib.cm_evaluate_argmin_noalloc.argtypes = [vp, vp, C.c_uint64, C.c_uint64, vp, vp, vp]
    lib.cm_search_objective.argtypes = [vp, C.POINTER(C.c_uint32), C.POINTER(C.c_int32), C.c_int32,
                                        C.POINTER(cm_enum_opts), C.POINTER(cm_objective_opts), C.POINTER(cm_plan),
                                        C.POINTER(cm_transition), C.POINTER(cm_plan), C.POINTER(C.c_int64),
                                        C.POINTER(C.c_int32)]
    lib.cm_objective_stats.argtypes = [vp, u64p]
    lib.cm_transfer_matching.argtypes = [vp, C.c_int32, C.POINTER(C.c_int32), vp, vp, vp, vp,
                                         C.POINTER(C.c_int64), C.POINTER(C.c_uint16)]
    lib.cm_cache_build.argtypes = [vp, C.c_int32, C.POINTER(cm_enum_opts), C.POINTER(vp), u64p]
    lib.cm_cache_lookup.argtypes = [vp, C.POINTER(C.c_uint32), C.c_int32, C.POINTER(cm_plan), C.POINTER(cm_plan)]
    lib.cm_cache_free.argtypes = [vp]
    lib.cm_set_sharing.argtypes = [vp, C.c_int]
    lib.cm_set_latency_graphs.argtypes = [vp, C.c_int]
    lib.cm_set_memory_screen.argtypes = [vp, C.c_int]
    lib.cm_set_micro_batch_pairs.argtypes = [vp, C.c_int]
    lib.cm_set_pipeline_reuse.argtypes = [vp, C.c_int]
    lib.cm_host_describe.argtypes = [C.POINTER(cm_profile), C.POINTER(C.c_uint32), C.c_int32, C.POINTER(cm_enum_opts), u64p]
    lib.cm_set_int64_arithmetic.argtypes = [vp, C.c_int]
    lib.cm_transition_time.argtypes = [C.POINTER(cm_objective_opts), C.c_int32, C.POINTER(C.c_int64),
                                       C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    lib.cm_int64_runs_in_fp64.argtypes = [vp]
    lib.cm_int64_runs_in_fp64.restype = C.c_int
    for name in _STATUS_CALLS:
        getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _check(ctx, status: int, allow: Sequence[int] = ()):
    if status != CM_OK and status not in allow:
        lib = load_library()
        msg = lib.cm_strerror(status).decode()
        if ctx:
            detail = lib.cm_last_error(ctx).decode()
            if detail:
                msg += ": " + detail
        raise ChameleonError(status, msg)
    return status


def _opts(o) -> cm_enum_opts:
    if isinstance(o, cm_enum_opts):
        return o
    return cm_enum_opts(o.dp_lo, o.dp_hi, o.pp_lo, o.pp_hi, o.layer_mode, o.batch_mode, o.kappa_cap, o.cost_mode,
                        int(getattr(o, "schedule", 0)))


# ------------------------------------------------------------------ C-ABI level calls

def cm_create(device: int = 0, stream: Optional[int] = None) -> C.c_void_p:
    """-> context handle.  ``stream`` is a raw cudaStream_t; default: torch's current stream."""
    lib = load_library()
    if stream is None:
        import torch
        if not torch.cuda.is_available():
            raise ChameleonError(CM_ECUDA, "no CUDA device: the plan search has no CPU path")
        stream = torch.cuda.current_stream(device).cuda_stream
    ctx = C.c_void_p()
    _check(None, lib.cm_create(C.byref(ctx), device, C.c_void_p(stream)))
    return ctx


def cm_destroy(ctx) -> None:
    _check(None, load_library().cm_destroy(ctx))


def _profile_struct(profile):
    """cm_profile over host arrays; returns (struct, arrays to keep alive)."""
    f64 = lambda a: np.ascontiguousarray(a, dtype=np.float64)
    i64 = lambda a: np.ascontiguousarray(a, dtype=np.int64)
    keep = [f64(profile.fwd_ns), f64(profile.bwd_ns), i64(profile.fwd_ns_i), i64(profile.bwd_ns_i),
            i64(profile.act_bytes), i64(profile.param_bytes), i64(profile.opt_bytes), i64(profile.p2p_bytes),
            np.ascontiguousarray(profile.base_cuts, dtype=np.int32)]
    dp = lambda a: a.ctypes.data_as(C.POINTER(C.c_double))
    ip = lambda a: a.ctypes.data_as(C.POINTER(C.c_int64))
    cp = cm_profile(profile.L, profile.n_dp, profile.n_pp, profile.n_micro, dp(keep[0]), dp(keep[1]),
                    ip(keep[2]), ip(keep[3]), ip(keep[4]), ip(keep[5]), ip(keep[6]), ip(keep[7]),
                    keep[8].ctypes.data_as(C.POINTER(C.c_int32)), profile.mem_capacity_bytes,
                    profile.devices_per_node, profile.bw_intra_Bpns, profile.bw_inter_Bpns)
    return cp, keep


def cm_load_profile(ctx, profile) -> None:
    """``profile``: an object with the fields of ``workloads.Profile`` (host numpy arrays)."""
    cp, keep = _profile_struct(profile)
    _check(ctx, load_library().cm_load_profile(ctx, C.byref(cp)))


def cm_host_describe(profile, failed: Sequence[int], opts) -> dict:
    """The host-side descriptor builder alone (no GPU needed): counts of the dynamic-parallelism
    space of one failure set."""
    cp, keep = _profile_struct(profile)
    ids = (C.c_uint32 * max(len(failed), 1))(*failed)
    o = _opts(opts)
    out = (C.c_uint64 * 8)()
    _check(None, load_library().cm_host_describe(C.byref(cp), ids, len(failed), C.byref(o), out))
    keys = ["candidates", "strategies", "segments", "splits", "survivors", "launch_classes", "buckets", "node_crossings"]
    return dict(zip(keys, [int(v) for v in out]))


def cm_enumerate(ctx, policy: int, failed: Sequence[int], opts) -> Tuple[C.c_void_p, int]:
    """-> (space handle, number of candidates)."""
    ids = np.ascontiguousarray(failed, dtype=np.uint32)
    space, n = C.c_void_p(), C.c_uint64()
    o = _opts(opts) if opts is not None else None
    _check(ctx, load_library().cm_enumerate(ctx, policy, ids.ctypes.data_as(C.POINTER(C.c_uint32)), len(ids),
                                            C.byref(o) if o is not None else None, C.byref(space), C.byref(n)))
    return space, n.value


def cm_evaluate(ctx, space, first: int, count: int, idx_dev=None, cost_dev=None, cost_ns_dev=None,
                feasible_dev=None) -> None:
    """Device pointers may be torch CUDA tensors (their ``data_ptr`` is passed) or ints."""
    ptr = lambda t: None if t is None else C.c_void_p(t.data_ptr() if hasattr(t, "data_ptr") else int(t))
    _check(ctx, load_library().cm_evaluate(ctx, space, first, count, ptr(idx_dev), ptr(cost_dev),
                                           ptr(cost_ns_dev), ptr(feasible_dev)))


def cm_select(ctx, spaces: Sequence) -> Optional[Plan]:
    """-> best plan over the spaces, or None if nothing is feasible."""
    arr = (C.c_void_p * len(spaces))(*[s.value if isinstance(s, C.c_void_p) else s for s in spaces])
    best = cm_plan()
    st = _check(ctx, load_library().cm_select(ctx, arr, len(spaces), C.byref(best)), allow=(CM_ENOFEASIBLE,))
    return None if st == CM_ENOFEASIBLE else _plan_from(best)


def cm_decode_plan(ctx, space, plan: Plan) -> List[List[int]]:
    c = cm_plan(plan.policy, int(plan.feasible), plan.cost, plan.cost_ns, plan.strategy, plan.n_pipes,
                plan.split_rank)
    for i in range(plan.n_pipes):
        c.stages[i], c.micro[i], c.kappa[i] = plan.stages[i], plan.micro[i], plan.kappa[i]
    out = (C.c_int32 * (MAX_PIPES * (MAX_STAGES + 1)))()
    _check(ctx, load_library().cm_decode_plan(ctx, space, C.byref(c), out))
    res, pos = [], 0
    for i in range(plan.n_pipes):
        S = plan.stages[i]
        res.append(list(out[pos:pos + S + 1]))
        pos += S + 1
    return res


def cm_space_free(space) -> None:
    _check(None, load_library().cm_space_free(space))


def cm_search_batch(ctx, scenarios: Sequence[Sequence[int]], opts, per_policy: bool = False,
                    latency: bool = False):
    """-> (best plan per scenario as a ctypes array of cm_plan, per-policy array or None,
    latency_us numpy array or None).  Inputs and outputs are HOST buffers."""
    B = len(scenarios)
    offsets = np.zeros(B + 1, dtype=np.int32)
    for b, s in enumerate(scenarios):
        offsets[b + 1] = offsets[b] + len(s)
    ids = np.zeros(max(int(offsets[-1]), 1), dtype=np.uint32)
    for b, s in enumerate(scenarios):
        ids[offsets[b]:offsets[b + 1]] = s
    best = (cm_plan * max(B, 1))()
    pol = (cm_plan * (3 * max(B, 1)))() if per_policy else None
    lat = np.zeros(max(B, 1), dtype=np.float32) if latency else None
    o = _opts(opts)
    _check(ctx, load_library().cm_search_batch(
        ctx, ids.ctypes.data_as(C.POINTER(C.c_uint32)), offsets.ctypes.data_as(C.POINTER(C.c_int32)), B,
        C.byref(o), best, pol, lat.ctypes.data_as(C.POINTER(C.c_float)) if latency else None))
    return best, pol, lat


def cm_evaluate_argmin_noalloc(ctx, space, first: int, count: int, best_cost_dev=None, best_cost_ns_dev=None,
                               best_index_dev=None) -> None:
    """Best (cost, index) of a candidate range, for callers that must not allocate: the
    three outputs are caller-owned device buffers (torch tensors or raw pointers) and the
    call itself allocates nothing.  At most NOALLOC_MAX_CANDIDATES candidates per call."""
    ptr = lambda t: None if t is None else C.c_void_p(t.data_ptr() if hasattr(t, "data_ptr") else int(t))
    _check(ctx, load_library().cm_evaluate_argmin_noalloc(ctx, space, first, count, ptr(best_cost_dev),
                                                          ptr(best_cost_ns_dev), ptr(best_index_dev)))


def _objective(obj) -> cm_objective_opts:
    return cm_objective_opts(int(obj.topk), int(getattr(obj, "sync_rounds", 0)), float(obj.t_gap_ns), float(obj.t_restart_ns),
                             int(round(obj.t_gap_ns)), int(round(obj.t_restart_ns)), int(obj.bw_xfer_Bpns))


def cm_search_objective(ctx, scenarios: Sequence[Sequence[int]], opts, objective, shortlist: bool = False):
    """Search plus re-scoring with the transition time.  -> (best plans, transitions,
    shortlisted plans or None, their matched bytes as numpy int64 [B, topk] or None, their
    communication rounds as numpy int32 [B, topk] or None); the first three are ctypes arrays
    (cm_plan / cm_transition), shortlist slots scenario-major."""
    packed = PackedScenarios(scenarios)
    return packed.search_objective(ctx, opts, objective, shortlist)


def cm_transition_time(objective, xfer_bytes) -> Tuple[np.ndarray, np.ndarray]:
    """Transition times of reconstructions that move ``xfer_bytes`` (any shape, int64; -1 = empty
    slot) -> (float64 ns for the fp64 mode, int64 ns for the integer mode), same shape."""
    b = np.ascontiguousarray(xfer_bytes, dtype=np.int64)
    t = np.zeros(b.shape, dtype=np.float64)
    ti = np.zeros(b.shape, dtype=np.int64)
    q = _objective(objective)
    _check(None, load_library().cm_transition_time(C.byref(q), b.size, b.ctypes.data_as(C.POINTER(C.c_int64)),
                                                   t.ctypes.data_as(C.POINTER(C.c_double)),
                                                   ti.ctypes.data_as(C.POINTER(C.c_int64))))
    return t, ti


def cm_objective_stats(ctx) -> dict:
    out = (C.c_uint64 * 8)()
    _check(ctx, load_library().cm_objective_stats(ctx, out))
    keys = ["shortlist_ns", "complete_ns", "matching_ns", "objective_ns", "matchings", "launches", "d2h_bytes",
            "device_ns"]
    return dict(zip(keys, [int(v) for v in out]))


def cm_transfer_matching(ctx, problems: Sequence[Tuple[Sequence[Tuple[int, int]], Sequence[Tuple[int, int]]]]):
    """Weight-transfer matchings over explicit layer ranges.  ``problems`` = [(old ranges,
    new ranges)], ranges as (lo, hi) pairs.  -> (total bytes int64 [n], assignments: list of lists)."""
    n = len(problems)
    sizes = np.zeros(max(n, 1), dtype=np.int32)
    arr = np.zeros((4, max(n, 1), MAX_MATCH), dtype=np.uint8)
    for q, (old, new) in enumerate(problems):
        if len(old) != len(new):
            raise ValueError("a matching needs as many devices as positions")
        sizes[q] = len(old)
        if len(old) <= MAX_MATCH:
            for j, (a, b) in enumerate(old):
                arr[0, q, j], arr[1, q, j] = a, b
            for j, (a, b) in enumerate(new):
                arr[2, q, j], arr[3, q, j] = a, b
    total = np.zeros(max(n, 1), dtype=np.int64)
    assign = np.zeros((max(n, 1), MAX_MATCH), dtype=np.uint16)
    ptr = lambda a: C.c_void_p(a.ctypes.data)
    _check(ctx, load_library().cm_transfer_matching(
        ctx, n, sizes.ctypes.data_as(C.POINTER(C.c_int32)), ptr(arr[0]), ptr(arr[1]), ptr(arr[2]), ptr(arr[3]),
        total.ctypes.data_as(C.POINTER(C.c_int64)), assign.ctypes.data_as(C.POINTER(C.c_uint16))))
    return total[:n], [[int(x) for x in assign[q, :sizes[q]]] for q in range(n)]


def cm_cache_build(ctx, max_failures: int, opts) -> Tuple[C.c_void_p, int]:
    """Plans for every failure set of at most ``max_failures`` devices -> (cache handle, entries)."""
    o = _opts(opts)
    cache, n = C.c_void_p(), C.c_uint64()
    _check(ctx, load_library().cm_cache_build(ctx, max_failures, C.byref(o), C.byref(cache), C.byref(n)))
    return cache, n.value


def cm_cache_lookup(cache, failed: Sequence[int], per_policy: bool = False):
    """-> best Plan (and the three per-policy Plans) of a cached failure set, or None if the set
    is larger than the cache covers."""
    ids = (C.c_uint32 * max(len(failed), 1))(*failed)
    best = cm_plan()
    pol = (cm_plan * 3)() if per_policy else None
    st = load_library().cm_cache_lookup(cache, ids, len(failed), C.byref(best), pol)
    if st == CM_ENOFEASIBLE:
        return (None, None) if per_policy else None
    _check(None, st)
    return (_plan_from(best), plans_from_array(pol)) if per_policy else _plan_from(best)


def cm_set_sharing(ctx, on: bool) -> None:
    """Search scenarios of a batch with identical dynamic-parallelism spaces once (default off)."""
    _check(ctx, load_library().cm_set_sharing(ctx, int(bool(on))))


def cm_set_micro_batch_pairs(ctx, on: bool) -> None:
    """One recurrence for a pipeline's m and m+1 micro-batch variants (on by default)."""
    _check(ctx, load_library().cm_set_micro_batch_pairs(ctx, int(bool(on))))


def cm_set_pipeline_reuse(ctx, on: bool) -> None:
    """Search a pipeline that several strategies of a survivor count have in common once (on by default)."""
    _check(ctx, load_library().cm_set_pipeline_reuse(ctx, int(bool(on))))


def cm_set_memory_screen(ctx, on: bool) -> None:
    """Walk only the listed memory-feasible layer compositions (default on); off: test every
    composition inside the search pass.  Results are identical."""
    _check(ctx, load_library().cm_set_memory_screen(ctx, int(bool(on))))


def cm_set_latency_graphs(ctx, on: bool) -> None:
    """Replay resident one-scenario searches as CUDA graphs (default on)."""
    _check(ctx, load_library().cm_set_latency_graphs(ctx, int(bool(on))))


def cm_set_int64_arithmetic(ctx, native: bool) -> None:
    """Force the 64-bit integer kernels for the integer-nanosecond mode (default: double
    arithmetic on the integer-valued inputs whenever that is exact)."""
    _check(ctx, load_library().cm_set_int64_arithmetic(ctx, int(bool(native))))


def cm_int64_runs_in_fp64(ctx) -> bool:
    return bool(load_library().cm_int64_runs_in_fp64(ctx))


def cm_cache_free(cache) -> None:
    _check(None, load_library().cm_cache_free(cache))


def cm_batch_free(batch) -> None:
    _check(None, load_library().cm_batch_free(batch))


def cm_last_stats(ctx) -> dict:
    out = (C.c_uint64 * 24)()
    _check(ctx, load_library().cm_last_stats(ctx, out))
    keys = ["plans", "cells", "tiebreak_plans", "launches", "device_ns", "segments", "strategies", "splits",
            "cost_kernel_ns", "h2d_bytes", "d2h_bytes", "tiebreak_kernel_ns", "cost_kernel_launches",
            "host_build_ns", "host_enqueue_ns", "host_wait_ns", "plans_simulated", "host_feasible_ns",
            "host_upload_ns", "plans_own"]
    return dict(zip(keys, [int(v) for v in out]))


class PackedScenarios:
    """Failure sets marshalled once (ids + offsets) so that repeated calls pay no Python cost."""

    def __init__(self, scenarios: Sequence[Sequence[int]]):
        self.B = len(scenarios)
        self.offsets = np.zeros(self.B + 1, dtype=np.int32)
        for b, s in enumerate(scenarios):
            self.offsets[b + 1] = self.offsets[b] + len(s)
        self.ids = np.zeros(max(int(self.offsets[-1]), 1), dtype=np.uint32)
        for b, s in enumerate(scenarios):
            self.ids[self.offsets[b]:self.offsets[b + 1]] = s
        self.best = (cm_plan * max(self.B, 1))()
        self.per_policy = (cm_plan * (3 * max(self.B, 1)))()
        self.latency = np.zeros(max(self.B, 1), dtype=np.float32)

    def prepare(self, ctx, opts) -> Tuple[C.c_void_p, int]:
        """cm_batch_prepare: descriptors to the device; -> (batch handle, candidates)."""
        o = _opts(opts)
        batch, n = C.c_void_p(), C.c_uint64()
        _check(ctx, load_library().cm_batch_prepare(
            ctx, self.ids.ctypes.data_as(C.POINTER(C.c_uint32)), self.offsets.ctypes.data_as(C.POINTER(C.c_int32)),
            self.B, C.byref(o), C.byref(batch), C.byref(n)))
        return batch, n.value

    def search_prepared(self, ctx, batch) -> None:
        """cm_batch_search into this object's host plan arrays."""
        _check(ctx, load_library().cm_batch_search(ctx, batch, self.best, self.per_policy))

    def search(self, ctx, opts, latency: bool = False) -> None:
        o = _opts(opts)
        _check(ctx, load_library().cm_search_batch(
            ctx, self.ids.ctypes.data_as(C.POINTER(C.c_uint32)), self.offsets.ctypes.data_as(C.POINTER(C.c_int32)),
            self.B, C.byref(o), self.best, self.per_policy,
            self.latency.ctypes.data_as(C.POINTER(C.c_float)) if latency else None))

    def search_objective(self, ctx, opts, objective, shortlist: bool = False):
        """cm_search_objective into freshly made host arrays (see the module function)."""
        o, q = _opts(opts), _objective(objective)
        B, k = self.B, int(objective.topk)
        best = (cm_plan * max(B, 1))()
        trans = (cm_transition * max(B, 1))()
        sl = (cm_plan * max(B * k, 1))() if shortlist else None
        sb = np.full((max(B, 1), max(k, 1)), -1, dtype=np.int64) if shortlist else None
        sr = np.zeros((max(B, 1), max(k, 1)), dtype=np.int32) if shortlist else None
        _check(ctx, load_library().cm_search_objective(
            ctx, self.ids.ctypes.data_as(C.POINTER(C.c_uint32)), self.offsets.ctypes.data_as(C.POINTER(C.c_int32)),
            B, C.byref(o), C.byref(q), best, trans, sl,
            sb.ctypes.data_as(C.POINTER(C.c_int64)) if shortlist else None,
            sr.ctypes.data_as(C.POINTER(C.c_int32)) if shortlist else None))
        return best, trans, sl, sb, sr
