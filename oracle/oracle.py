"""ctypes front end of the CPU oracle -- TEST INFRASTRUCTURE, not the product.

Only ``tests/``, the smoke check and the bench's CPU-baseline leg may import this
module.  It compiles ``orc_enum.c``, ``orc_restore.c`` and ``orc_model.c`` (the latter twice: double and
integer-nanosecond arithmetic) with gcc into ``liborc.so`` next to the sources and
exposes the entry points.  Nothing here touches CUDA and nothing in the CUDA path
imports this.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liborc.so")
_SOURCES = ["orc_enum.c", "orc_restore.c", "orc_model.c", "orc.h"]

MAX_PIPES = 16
MAX_STAGES = 64

REROUTE, REDUNDANT, DYNPAR = 0, 1, 2
SCHED_1F1B, SCHED_GPIPE = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle if the library is missing or older than its sources."""
    srcs = [os.path.join(_HERE, s) for s in _SOURCES]
    if (not force and os.path.exists(_LIB_PATH)
            and all(os.path.getmtime(_LIB_PATH) >= os.path.getmtime(s) for s in srcs)):
        return _LIB_PATH
    flags = ["-O2", "-fPIC", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-Wall",
             "-Wno-maybe-uninitialized"]
    objs = []
    for name, defs in (("orc_enum", []), ("orc_restore", []), ("orc_model_f64", ["-DORC_INT=0"]),
                       ("orc_model_i64", ["-DORC_INT=1"])):
        src = os.path.join(_HERE, name + ".c" if not defs else "orc_model.c")
        obj = os.path.join(_HERE, name + ".o")
        subprocess.check_call(["gcc", *flags, *defs, "-c", src, "-o", obj])
        objs.append(obj)
    tmp = _LIB_PATH + f".tmp{os.getpid()}"
    subprocess.check_call(["gcc", "-shared", "-o", tmp, *objs, "-lm"])
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


class _Profile(C.Structure):
    _fields_ = [("L", C.c_int32), ("n_dp", C.c_int32), ("n_pp", C.c_int32), ("n_micro", C.c_int32),
                ("fwd_ns", C.POINTER(C.c_double)), ("bwd_ns", C.POINTER(C.c_double)),
                ("fwd_ns_i", C.POINTER(C.c_int64)), ("bwd_ns_i", C.POINTER(C.c_int64)),
                ("act_bytes", C.POINTER(C.c_int64)), ("param_bytes", C.POINTER(C.c_int64)),
                ("opt_bytes", C.POINTER(C.c_int64)), ("p2p_bytes", C.POINTER(C.c_int64)),
                ("base_cuts", C.POINTER(C.c_int32)),
                ("mem_capacity_bytes", C.c_int64), ("devices_per_node", C.c_int32),
                ("bw_intra", C.c_int64), ("bw_inter", C.c_int64)]


class _Opts(C.Structure):
    _fields_ = [("dp_lo", C.c_int32), ("dp_hi", C.c_int32), ("pp_lo", C.c_int32), ("pp_hi", C.c_int32),
                ("layer_mode", C.c_int32), ("batch_mode", C.c_int32), ("kappa_cap", C.c_uint64),
                ("schedule", C.c_int32)]


class _Plan(C.Structure):
    _fields_ = [("policy", C.c_int32), ("feasible", C.c_int32), ("cost", C.c_double),
                ("cost_ns", C.c_int64), ("strategy", C.c_uint32), ("n_pipes", C.c_uint32),
                ("split_rank", C.c_uint64), ("stages", C.c_uint16 * MAX_PIPES),
                ("micro", C.c_uint16 * MAX_PIPES), ("kappa", C.c_uint64 * MAX_PIPES)]


class _Objective(C.Structure):
    _fields_ = [("topk", C.c_int32), ("sync_rounds", C.c_int32), ("t_gap", C.c_double), ("t_restart", C.c_double),
                ("t_gap_ns", C.c_int64), ("t_restart_ns", C.c_int64), ("bw_xfer", C.c_int64)]


class _Transition(C.Structure):
    _fields_ = [("policy", C.c_int32), ("feasible", C.c_int32), ("rank", C.c_int32), ("n_surv", C.c_int32),
                ("xfer_bytes", C.c_int64), ("t_trans", C.c_double), ("t_trans_ns", C.c_int64),
                ("objective", C.c_double), ("rounds", C.c_int32), ("domains", C.c_int32),
                ("t_sync", C.c_double), ("t_sync_ns", C.c_int64)]


@dataclass
class Transition:
    policy: int
    feasible: bool
    rank: int
    n_surv: int
    xfer_bytes: int
    t_trans: float
    t_trans_ns: int
    objective: float
    assign: Tuple[int, ...] = ()
    shortlist: Tuple = ()
    shortlist_bytes: Tuple[int, ...] = ()
    rounds: int = 0
    domains: int = 0
    t_sync: float = 0.0
    t_sync_ns: int = 0
    shortlist_rounds: Tuple[int, ...] = ()


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


def _plan_from(c: _Plan) -> Plan:
    n = c.n_pipes
    return Plan(c.policy, bool(c.feasible), c.cost, c.cost_ns, c.strategy, n, c.split_rank,
                tuple(c.stages[:n]), tuple(c.micro[:n]), tuple(c.kappa[:n]))


def _ptr(a: np.ndarray, ct):
    return a.ctypes.data_as(C.POINTER(ct))


class Oracle:
    """The oracle bound to one profile.  ``cost_mode`` 0 = double, 1 = integer ns."""

    def __init__(self, profile, options=None):
        self._lib = C.CDLL(build())
        self._lib.orc_binom.restype = C.c_uint64
        self._lib.orc_rank_subset.restype = C.c_uint64
        self._lib.orc_split_count.restype = C.c_uint64
        self._lib.orc_layer_count.restype = C.c_uint64
        self._lib.orc_assign.restype = C.c_int64
        self._lib.orc_assign_brute.restype = C.c_int64
        for sfx in ("_f64", "_i64"):
            getattr(self._lib, "orc_pipe_time" + sfx).restype = C.c_double
            getattr(self._lib, "orc_count" + sfx).restype = C.c_uint64
            getattr(self._lib, "orc_plan_transfer" + sfx).restype = C.c_int64
            getattr(self._lib, "orc_plan_async_step" + sfx).restype = C.c_double
        self.profile = profile
        self.options = options
        p = profile
        self._keep = [np.ascontiguousarray(p.fwd_ns, dtype=np.float64),
                      np.ascontiguousarray(p.bwd_ns, dtype=np.float64),
                      np.ascontiguousarray(p.fwd_ns_i, dtype=np.int64),
                      np.ascontiguousarray(p.bwd_ns_i, dtype=np.int64),
                      np.ascontiguousarray(p.act_bytes, dtype=np.int64),
                      np.ascontiguousarray(p.param_bytes, dtype=np.int64),
                      np.ascontiguousarray(p.opt_bytes, dtype=np.int64),
                      np.ascontiguousarray(p.p2p_bytes, dtype=np.int64),
                      np.ascontiguousarray(p.base_cuts, dtype=np.int32)]
        k = self._keep
        self._cp = _Profile(p.L, p.n_dp, p.n_pp, p.n_micro,
                            _ptr(k[0], C.c_double), _ptr(k[1], C.c_double),
                            _ptr(k[2], C.c_int64), _ptr(k[3], C.c_int64),
                            _ptr(k[4], C.c_int64), _ptr(k[5], C.c_int64),
                            _ptr(k[6], C.c_int64), _ptr(k[7], C.c_int64), _ptr(k[8], C.c_int32),
                            p.mem_capacity_bytes, p.devices_per_node, p.bw_intra_Bpns, p.bw_inter_Bpns)

    # -- helpers -------------------------------------------------------------
    def _opts(self, options=None) -> Tuple[_Opts, str]:
        o = options or self.options
        return (_Opts(o.dp_lo, o.dp_hi, o.pp_lo, o.pp_hi, o.layer_mode, o.batch_mode, o.kappa_cap,
                      int(getattr(o, "schedule", 0))),
                "_i64" if o.cost_mode == 1 else "_f64")

    @staticmethod
    def _failed(failed: Sequence[int]):
        a = np.ascontiguousarray(failed, dtype=np.uint32)
        return a, _ptr(a, C.c_uint32), len(a)

    def _fn(self, name, sfx):
        return getattr(self._lib, name + sfx)

    # -- combinatorics -------------------------------------------------------
    def binom(self, n: int, k: int) -> int:
        return self._lib.orc_binom(n, k)

    def unrank_subset(self, rank: int, t: int) -> List[int]:
        out = (C.c_int * max(t, 1))()
        self._lib.orc_unrank_subset(C.c_uint64(rank), t, out)
        return list(out[:t])

    def rank_subset(self, c: Sequence[int]) -> int:
        arr = (C.c_int * max(len(c), 1))(*c)
        return self._lib.orc_rank_subset(len(c), arr)

    def strategies(self, n_surv: int, options=None) -> List[Tuple[int, ...]]:
        o = options or self.options
        n = self._lib.orc_strategies(n_surv, o.dp_lo, o.dp_hi, o.pp_lo, o.pp_hi, self.profile.L, 0, None, None)
        dp = np.zeros(max(n, 1), dtype=np.int32)
        st = np.zeros((max(n, 1), MAX_PIPES), dtype=np.int32)
        self._lib.orc_strategies(n_surv, o.dp_lo, o.dp_hi, o.pp_lo, o.pp_hi, self.profile.L, n,
                                 _ptr(dp, C.c_int32), _ptr(st, C.c_int32))
        return [tuple(int(x) for x in st[i, :dp[i]]) for i in range(n)]

    def split_count(self, batch_mode: int, G: int, n_surv: int, stages: Sequence[int]) -> int:
        st = np.ascontiguousarray(stages, dtype=np.int32)
        return self._lib.orc_split_count(batch_mode, G, n_surv, len(st), _ptr(st, C.c_int32))

    def split_unrank(self, batch_mode: int, G: int, n_surv: int, stages: Sequence[int], beta: int):
        st = np.ascontiguousarray(stages, dtype=np.int32)
        out = np.zeros(len(st), dtype=np.int32)
        ok = self._lib.orc_split_unrank(batch_mode, G, n_surv, len(st), _ptr(st, C.c_int32),
                                        C.c_uint64(beta), _ptr(out, C.c_int32))
        return bool(ok), [int(x) for x in out]

    def layer_count(self, layer_mode: int, S: int) -> int:
        return self._lib.orc_layer_count(layer_mode, self.profile.L, S)

    def layer_unrank(self, layer_mode: int, S: int, kappa: int) -> List[int]:
        out = np.zeros(S + 1, dtype=np.int32)
        self._lib.orc_layer_unrank(layer_mode, self.profile.L, S, C.c_uint64(kappa), _ptr(out, C.c_int32))
        return [int(x) for x in out]

    # -- model -----------------------------------------------------------------
    def pipe_time(self, F, B, xt, m: int, cost_mode: int = 0, schedule: int = 0) -> float:
        S = len(F)
        f = (C.c_double * S)(*F)
        b = (C.c_double * S)(*B)
        x = (C.c_double * S)(*(list(xt) + [0.0] * (S - len(xt))))
        sfx = "_i64" if cost_mode == 1 else "_f64"
        return self._fn("orc_pipe_time", sfx)(S, m, f, b, x, schedule)

    def pipe(self, cuts: Sequence[int], m: int, devs: Sequence[int], n_sync: int, cost_mode: int = 0, schedule: int = 0):
        """-> (feasible, cost as float, cost_ns, peak memory per stage)."""
        S = len(cuts) - 1
        c = np.ascontiguousarray(cuts, dtype=np.int32)
        d = np.ascontiguousarray(devs, dtype=np.int32)
        cost = C.c_double()
        cost_ns = C.c_int64()
        peak = np.zeros(S, dtype=np.int64)
        sfx = "_i64" if cost_mode == 1 else "_f64"
        ok = self._fn("orc_pipe", sfx)(C.byref(self._cp), S, _ptr(c, C.c_int32), m, _ptr(d, C.c_int32),
                                       n_sync, C.byref(cost), C.byref(cost_ns), _ptr(peak, C.c_int64), schedule)
        return bool(ok), cost.value, cost_ns.value, [int(x) for x in peak]

    def minmax(self, S: int, m: int, cost_mode: int = 0, schedule: int = 0):
        cuts = np.zeros(S + 1, dtype=np.int32)
        val = C.c_double()
        sfx = "_i64" if cost_mode == 1 else "_f64"
        ok = self._fn("orc_minmax", sfx)(C.byref(self._cp), S, m, _ptr(cuts, C.c_int32), C.byref(val), schedule)
        return bool(ok), [int(x) for x in cuts], val.value

    # -- search ----------------------------------------------------------------
    def count(self, failed: Sequence[int], options=None):
        o, sfx = self._opts(options)
        _, fp, nf = self._failed(failed)
        ns, ng = C.c_int32(), C.c_int32()
        n = self._fn("orc_count", sfx)(C.byref(self._cp), C.byref(o), fp, nf, C.byref(ns), C.byref(ng))
        return int(n), ns.value, ng.value

    def segment(self, failed: Sequence[int], s: int, options=None):
        o, sfx = self._opts(options)
        _, fp, nf = self._failed(failed)
        desc = (C.c_int32 * 6)()
        K, first = C.c_uint64(), C.c_uint64()
        ok = self._fn("orc_segment", sfx)(C.byref(self._cp), C.byref(o), fp, nf, s, desc, C.byref(K), C.byref(first))
        if not ok:
            return None
        return dict(strategy=desc[0], pipe=desc[1], S=desc[2], m=desc[3], off=desc[4], dp=desc[5],
                    K=K.value, first=first.value)

    def evaluate(self, failed: Sequence[int], first: int = 0, count: Optional[int] = None,
                 idx: Optional[Sequence[int]] = None, options=None):
        """-> (cost float64[n], cost_ns int64[n], feasible uint8[n]) in candidate order."""
        o, sfx = self._opts(options)
        _, fp, nf = self._failed(failed)
        if idx is not None:
            ia = np.ascontiguousarray(idx, dtype=np.uint64)
            n = len(ia)
            ip = _ptr(ia, C.c_uint64)
        else:
            if count is None:
                count = self.count(failed, options)[0] - first
            n, ip = count, None
        cost = np.zeros(n, dtype=np.float64)
        cost_ns = np.zeros(n, dtype=np.int64)
        feas = np.zeros(n, dtype=np.uint8)
        self._fn("orc_eval", sfx)(C.byref(self._cp), C.byref(o), fp, nf, C.c_uint64(first), C.c_uint64(n), ip,
                                  _ptr(cost, C.c_double), _ptr(cost_ns, C.c_int64), _ptr(feas, C.c_uint8))
        return cost, cost_ns, feas

    def search_policy(self, failed: Sequence[int], policy: int, flat: bool = False, options=None):
        o, sfx = self._opts(options)
        _, fp, nf = self._failed(failed)
        pl = _Plan()
        n_flat = C.c_uint64()
        self._fn("orc_search_policy", sfx)(C.byref(self._cp), C.byref(o), fp, nf, policy, int(flat),
                                           C.byref(pl), C.byref(n_flat))
        plan = _plan_from(pl)
        return (plan, n_flat.value) if flat else plan

    def search(self, failed: Sequence[int], options=None):
        """-> (best plan or None, [plan per policy])."""
        o, sfx = self._opts(options)
        _, fp, nf = self._failed(failed)
        best = _Plan()
        per = (_Plan * 3)()
        ok = self._fn("orc_search", sfx)(C.byref(self._cp), C.byref(o), fp, nf, C.byref(best), per)
        return (_plan_from(best) if ok else None), [_plan_from(per[i]) for i in range(3)]

    @staticmethod
    def _cplan(plan: Plan) -> _Plan:
        c = _Plan(plan.policy, int(plan.feasible), plan.cost, plan.cost_ns, plan.strategy, plan.n_pipes,
                  plan.split_rank)
        for i in range(plan.n_pipes):
            c.stages[i], c.micro[i], c.kappa[i] = plan.stages[i], plan.micro[i], plan.kappa[i]
        return c

    # -- weight transfer, full objective ------------------------------------------
    def state_bytes(self) -> np.ndarray:
        """Bytes of model state per layer that a migration moves (parameters + optimizer)."""
        return np.asarray(self.profile.param_bytes, dtype=np.int64) + np.asarray(self.profile.opt_bytes, dtype=np.int64)

    def transfer_cost_matrix(self, old: Sequence[Tuple[int, int]], new: Sequence[Tuple[int, int]],
                             weights: Optional[Sequence[int]] = None) -> np.ndarray:
        """Cost[i][j] of device i (old layer range) serving position j (new layer range)."""
        n = len(old)
        w = np.ascontiguousarray(self.state_bytes() if weights is None else weights, dtype=np.int64)
        olo = np.ascontiguousarray([a for a, _ in old], dtype=np.int32)
        ohi = np.ascontiguousarray([b for _, b in old], dtype=np.int32)
        nlo = np.ascontiguousarray([a for a, _ in new], dtype=np.int32)
        nhi = np.ascontiguousarray([b for _, b in new], dtype=np.int32)
        cost = np.zeros((n, n), dtype=np.int64)
        self._lib.orc_transfer_cost_matrix(len(w), _ptr(w, C.c_int64), n, _ptr(olo, C.c_int32), _ptr(ohi, C.c_int32),
                                           _ptr(nlo, C.c_int32), _ptr(nhi, C.c_int32), _ptr(cost, C.c_int64))
        return cost

    def assign(self, cost: np.ndarray) -> Tuple[int, List[int]]:
        """Minimum-cost perfect matching -> (total, row matched to every column)."""
        c = np.ascontiguousarray(cost, dtype=np.int64)
        n = c.shape[0]
        out = np.zeros(max(n, 1), dtype=np.int32)
        total = self._lib.orc_assign(n, _ptr(c, C.c_int64), _ptr(out, C.c_int32))
        return int(total), [int(x) for x in out[:n]]

    def assign_brute(self, cost: np.ndarray) -> int:
        c = np.ascontiguousarray(cost, dtype=np.int64)
        return int(self._lib.orc_assign_brute(c.shape[0], _ptr(c, C.c_int64)))

    def plan_transfer(self, failed: Sequence[int], plan: Plan, options=None) -> Tuple[int, List[int]]:
        """Bytes moved by the cheapest migration into ``plan`` and its matching."""
        o, sfx = self._opts(options)
        _, fp, nf = self._failed(failed)
        n_surv = self.profile.n_dp * self.profile.n_pp - nf
        out = np.zeros(max(n_surv, 1), dtype=np.int32)
        c = self._cplan(plan)
        b = self._fn("orc_plan_transfer", sfx)(C.byref(self._cp), C.byref(o), fp, nf, C.byref(c), _ptr(out, C.c_int32))
        return int(b), [int(x) for x in out[:n_surv]]

    def comm_rounds(self, stage_of: Sequence[Sequence[int]]) -> Tuple[int, List[int], int]:
        """Greedy communication rounds of a layer placement: stage_of[p][l] = stage of pipeline p
        holding layer l.  -> (rounds, colour per layer, communication domains)."""
        a = np.ascontiguousarray(stage_of, dtype=np.int32)
        dp, L = a.shape
        colour = np.zeros(L, dtype=np.int32)
        r = self._lib.orc_comm_rounds(L, dp, _ptr(a, C.c_int32), _ptr(colour, C.c_int32))
        d = self._lib.orc_comm_domains(L, dp, _ptr(a, C.c_int32))
        return int(r), [int(x) for x in colour], int(d)

    def plan_async_step(self, failed: Sequence[int], plan: Plan, options=None):
        """Step time of a plan under asymmetric synchronisation -> (step, rounds, domains, t_sync);
        times as floats (exact for the integer build below 2^53)."""
        o, sfx = self._opts(options)
        _, fp, nf = self._failed(failed)
        c = self._cplan(plan)
        r, d, ts = C.c_int32(), C.c_int32(), C.c_double()
        t = self._fn("orc_plan_async_step", sfx)(C.byref(self._cp), C.byref(o), fp, nf, C.byref(c),
                                                 C.byref(r), C.byref(d), C.byref(ts))
        return t, r.value, d.value, ts.value

    def search_objective(self, failed: Sequence[int], objective, options=None):
        """Full-objective search -> (best plan or None, Transition).

        ``objective`` carries topk, t_gap_ns, t_restart_ns (floats; rounded for the integer
        build) and bw_xfer_Bpns."""
        o, sfx = self._opts(options)
        _, fp, nf = self._failed(failed)
        k = max(1, int(objective.topk))
        q = _Objective(k, int(getattr(objective, "sync_rounds", 0)), float(objective.t_gap_ns), float(objective.t_restart_ns),
                       int(round(objective.t_gap_ns)), int(round(objective.t_restart_ns)),
                       int(objective.bw_xfer_Bpns))
        n_surv = self.profile.n_dp * self.profile.n_pp - nf
        best, tr = _Plan(), _Transition()
        asg = np.zeros(max(n_surv, 1), dtype=np.int32)
        sp = (_Plan * k)()
        sb = np.zeros(k, dtype=np.int64)
        sr = np.zeros(k, dtype=np.int32)
        ns = C.c_int32()
        ok = self._fn("orc_search_objective", sfx)(C.byref(self._cp), C.byref(o), fp, nf, C.byref(q),
                                                   C.byref(best), C.byref(tr), _ptr(asg, C.c_int32), sp,
                                                   _ptr(sb, C.c_int64), _ptr(sr, C.c_int32), C.byref(ns))
        t = Transition(tr.policy, bool(tr.feasible), tr.rank, tr.n_surv, tr.xfer_bytes, tr.t_trans, tr.t_trans_ns,
                       tr.objective,
                       tuple(int(x) for x in asg[:n_surv]) if (ok and tr.policy == DYNPAR) else (),
                       tuple(_plan_from(sp[i]) for i in range(ns.value)),
                       tuple(int(x) for x in sb[:ns.value]),
                       tr.rounds, tr.domains, tr.t_sync, tr.t_sync_ns, tuple(int(x) for x in sr[:ns.value]))
        return (_plan_from(best) if ok else None), t

    def decode(self, failed: Sequence[int], plan: Plan, options=None) -> List[List[int]]:
        o, sfx = self._opts(options)
        _, fp, nf = self._failed(failed)
        c = self._cplan(plan)
        out = np.zeros(MAX_PIPES * (MAX_STAGES + 1), dtype=np.int32)
        n = self._fn("orc_decode", sfx)(C.byref(self._cp), C.byref(o), fp, nf, C.byref(c), _ptr(out, C.c_int32))
        if n < 0:
            raise ValueError("plan cannot be decoded")
        res, pos = [], 0
        for i in range(plan.n_pipes):
            S = plan.stages[i]
            res.append([int(x) for x in out[pos:pos + S + 1]])
            pos += S + 1
        return res
