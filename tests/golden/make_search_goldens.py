"""Write the stored search results of the full-size workloads.

Calls ONLY the CPU oracle (oracle/) on the seeded workloads; nothing here touches the
CUDA path.  One line per failure scenario and cost mode:

    <policy> <feasible> <cost: double as hex / integer ns> <fingerprint>

where the fingerprint is a 64-bit FNV-1a hash of the selected plan tuple (policy,
feasible, strategy, pipelines, split rank, stages, micro-batches, layer-composition ranks)
and the cost bits -- everything the parity bar requires to be bit-exact.  The GPU tests
recompute the fingerprint from the library's plan and compare.

    python tests/golden/make_search_goldens.py [workload ...] [--procs N] [--objective] [--schedule gpipe]

With --schedule gpipe the time model runs under the all-forward-all-backward order and the
results go to search_<workload>_gpipe_<mode>.txt.

With --objective the full-objective search (default ObjectiveOptions) is stored instead, in
objective_<workload>_<mode>.txt:

    <policy> <rank> <matched bytes> <transition time: double as hex / integer ns> <objective as hex>
    <fingerprint of the chosen plan> <fingerprint of the shortlist: every plan tuple, cost and matched bytes>

The sweep costs about four core-hours per cost mode.
"""
from __future__ import annotations

import argparse
import multiprocessing as mp
import os
import struct
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

HERE = os.path.dirname(os.path.abspath(__file__))
WORKLOADS = ["paper-scale", "70b-like", "175b-like", "sweep"]


def fingerprint(plan, mode: int) -> int:
    """FNV-1a over the plan tuple and the cost bits (works for oracle and library plans)."""
    if plan is None or not plan.feasible:
        words = [0xFFFFFFFFFFFFFFFF]
    else:
        cost_bits = (plan.cost_ns & 0xFFFFFFFFFFFFFFFF) if mode else struct.unpack("<Q", struct.pack("<d", plan.cost))[0]
        words = [plan.policy, 1, plan.strategy, plan.n_pipes, plan.split_rank, cost_bits]
        words += list(plan.stages) + list(plan.micro) + list(plan.kappa)
    h = 0xCBF29CE484222325
    for w in words:
        for byte in struct.pack("<Q", w & 0xFFFFFFFFFFFFFFFF):
            h = ((h ^ byte) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h


def line_of(plan, mode: int) -> str:
    if plan is None or not plan.feasible:
        return f"-1 0 - {fingerprint(plan, mode):016x}"
    cost = str(plan.cost_ns) if mode else float(plan.cost).hex()
    return f"{plan.policy} 1 {cost} {fingerprint(plan, mode):016x}"


_state = {}


def _init(name, mode, schedule=0):
    from oracle.oracle import Oracle
    from paper_2508_21613_b200 import workloads as W
    w = W.ALL_WORKLOADS[name]()
    _state["w"] = w
    _state["o"] = Oracle(w.profile, w.options.with_cost_mode(mode).with_schedule(schedule))
    _state["mode"] = mode


def _one(b):
    best, _ = _state["o"].search(_state["w"].scenarios[b])
    return b, line_of(best, _state["mode"])


def objective_line(best, tr, mode: int) -> str:
    """One stored line of the full-objective search (works for oracle and library results:
    `tr` needs policy, rank, xfer_bytes, t_trans, t_trans_ns, objective, shortlist, shortlist_bytes)."""
    if best is None or not best.feasible:
        return "-1 -1 0 - - ffffffffffffffff ffffffffffffffff"
    h = 0xCBF29CE484222325
    for plan, nbytes in zip(tr.shortlist, tr.shortlist_bytes):
        for w in (fingerprint(plan, mode), nbytes):
            for byte in struct.pack("<Q", int(w) & 0xFFFFFFFFFFFFFFFF):
                h = ((h ^ byte) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    t_trans = str(tr.t_trans_ns) if mode else float(tr.t_trans).hex()
    return (f"{tr.policy} {tr.rank} {tr.xfer_bytes} {t_trans} {float(tr.objective).hex()} "
            f"{fingerprint(best, mode):016x} {h:016x}")


def _one_objective(b):
    from paper_2508_21613_b200 import workloads as W
    best, tr = _state["o"].search_objective(_state["w"].scenarios[b], W.ObjectiveOptions())
    return b, objective_line(best, tr, _state["mode"])


def objective_path(name: str, mode: int) -> str:
    return os.path.join(HERE, f"objective_{name}_{'i64' if mode else 'f64'}.txt")


def golden_path(name: str, mode: int, schedule: int = 0) -> str:
    return os.path.join(HERE, f"search_{name}_{'gpipe_' if schedule else ''}{'i64' if mode else 'f64'}.txt")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("workloads", nargs="*", default=WORKLOADS)
    ap.add_argument("--procs", type=int, default=os.cpu_count())
    ap.add_argument("--modes", type=int, nargs="*", default=[0, 1])
    ap.add_argument("--objective", action="store_true", help="store the full-objective search instead")
    ap.add_argument("--schedule", choices=["1f1b", "gpipe"], default="1f1b")
    args = ap.parse_args()
    schedule = 1 if args.schedule == "gpipe" else 0
    if schedule and args.objective:
        ap.error("the full-objective results are stored for the 1F1B order only")
    from oracle.oracle import build
    build()
    from paper_2508_21613_b200 import workloads as W
    for name in args.workloads:
        n = len(W.ALL_WORKLOADS[name]().scenarios)
        for mode in args.modes:
            t0 = time.time()
            with mp.Pool(args.procs, initializer=_init, initargs=(name, mode, schedule)) as pool:
                lines = [None] * n
                for b, line in pool.imap_unordered(_one_objective if args.objective else _one, range(n), chunksize=1):
                    lines[b] = line
            if args.objective:
                with open(objective_path(name, mode), "w") as f:
                    f.write(f"# {name}, cost mode {'int64 ns' if mode else 'fp64'}: full-objective search per failure scenario "
                            f"from the CPU oracle (tests/golden/make_search_goldens.py --objective)\n"
                            f"# policy rank matched_bytes transition_time objective plan_fingerprint shortlist_fingerprint\n")
                    f.write("\n".join(lines) + "\n")
                print(f"{name} mode {mode} (objective): {n} scenarios in {time.time() - t0:.0f} s", flush=True)
                continue
            with open(golden_path(name, mode, schedule), "w") as f:
                f.write(f"# {name}, cost mode {'int64 ns' if mode else 'fp64'}{', all-forward-all-backward order' if schedule else ''}: best plan per failure scenario from the CPU "
                        f"oracle (tests/golden/make_search_goldens.py)\n# policy feasible cost fingerprint\n")
                f.write("\n".join(lines) + "\n")
            print(f"{name} mode {mode}: {n} scenarios in {time.time() - t0:.0f} s", flush=True)


if __name__ == "__main__":
    main()
