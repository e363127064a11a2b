"""Seeded synthetic inputs for the plan search: profiles, failure sets, search options.

This module only *draws inputs*.  It holds none of the method's arithmetic (no prefix
sums, no cost model, no enumeration), so both the CPU oracle's tests and the CUDA
path's tests can feed the very same arrays to the two independent implementations.

The generator is libm-free so that any language reproduces it bit for bit:
splitmix64 -> 53-bit uniform -> U(a,b) = a + (b-a)u, N(0,1) ~ (sum of 12 uniforms) - 6,
failure sets by a partial Fisher-Yates shuffle with ``z mod n``.

The five workloads take the shapes of the paper's evaluation (Llama-2-7B-like layer
counts and sizes on DP x PP grids, Section "Experimental Setup"), not its dataset or
weights: a profile is per-layer forward/backward time per micro-batch, activation /
parameter / optimizer bytes, the bytes crossing a stage boundary, device memory and
two link tiers.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List

import numpy as np

_MASK = (1 << 64) - 1

# policy / mode ids mirror the C ABI enums (plain integers, no arithmetic)
POLICY_REROUTE, POLICY_REDUNDANT, POLICY_DYNPAR = 0, 1, 2
COST_FP64, COST_INT64NS = 0, 1
LAYERS_FULL, LAYERS_REMAINDER, LAYERS_MINMAX = 0, 1, 2
BATCH_FULL, BATCH_REMAINDER = 0, 1
SCHED_1F1B, SCHED_GPIPE = 0, 1


class SplitMix64:
    """Counter-based generator; every draw consumes exactly one 64-bit output."""

    def __init__(self, seed: int):
        self.state = seed & _MASK

    def next_u64(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & _MASK
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
        return z ^ (z >> 31)

    def uniform01(self) -> float:
        return (self.next_u64() >> 11) * (1.0 / 9007199254740992.0)

    def uniform(self, a: float, b: float) -> float:
        return a + (b - a) * self.uniform01()

    def normal(self) -> float:
        s = 0.0
        for _ in range(12):
            s += self.uniform01()
        return s - 6.0

    def below(self, n: int) -> int:
        return self.next_u64() % n

    def sample_distinct(self, n: int, k: int) -> List[int]:
        """k distinct ids out of range(n): partial Fisher-Yates, returned ascending."""
        ids = list(range(n))
        for i in range(k):
            j = i + self.below(n - i)
            ids[i], ids[j] = ids[j], ids[i]
        return sorted(ids[:k])


@dataclass
class Profile:
    """Per-layer profile plus the fault-free configuration (all host arrays)."""

    L: int
    n_dp: int
    n_pp: int
    n_micro: int
    fwd_ns: np.ndarray       # float64 [L]
    bwd_ns: np.ndarray       # float64 [L]
    fwd_ns_i: np.ndarray     # int64 [L]  (rounded to the nearest ns)
    bwd_ns_i: np.ndarray     # int64 [L]
    act_bytes: np.ndarray    # int64 [L]
    param_bytes: np.ndarray  # int64 [L]
    opt_bytes: np.ndarray    # int64 [L]
    p2p_bytes: np.ndarray    # int64 [L]  bytes crossing a cut placed after layer l
    base_cuts: np.ndarray    # int32 [n_pp+1]
    mem_capacity_bytes: int
    devices_per_node: int
    bw_intra_Bpns: int       # bytes per ns == GB/s
    bw_inter_Bpns: int

    @property
    def n_devices(self) -> int:
        return self.n_dp * self.n_pp


@dataclass
class SearchOptions:
    dp_lo: int
    dp_hi: int
    pp_lo: int
    pp_hi: int
    layer_mode: int
    batch_mode: int
    kappa_cap: int
    cost_mode: int = COST_FP64
    schedule: int = SCHED_1F1B

    def with_cost_mode(self, mode: int) -> "SearchOptions":
        return SearchOptions(self.dp_lo, self.dp_hi, self.pp_lo, self.pp_hi,
                             self.layer_mode, self.batch_mode, self.kappa_cap, mode, self.schedule)

    def with_schedule(self, schedule: int) -> "SearchOptions":
        return SearchOptions(self.dp_lo, self.dp_hi, self.pp_lo, self.pp_hi,
                             self.layer_mode, self.batch_mode, self.kappa_cap, self.cost_mode, schedule)


@dataclass
class ObjectiveOptions:
    """Inputs of the full objective: how many dynamic-parallelism plans are re-scored with
    their transition time, the time between two faults, the restart overhead of a
    reconfiguration and the bandwidth the weight transfer gets (bytes per ns).

    Defaults at the scale of the paper's evaluation: its simulated trace fails each of 32
    devices at 10 % per hour (one fault every 1125 s on average) and its measured recoveries
    take around ten seconds, transfer included."""
    topk: int = 8
    t_gap_ns: float = 1125e9
    t_restart_ns: float = 5e9
    bw_xfer_Bpns: int = 25
    sync_rounds: int = 0     # 1: shortlisted plans are timed with the coloured all-reduce rounds


@dataclass
class Workload:
    name: str
    profile: Profile
    options: SearchOptions
    scenarios: List[List[int]] = field(default_factory=list)  # failed device ids, ascending
    notes: Dict[str, object] = field(default_factory=dict)


def _round_ns(x: np.ndarray) -> np.ndarray:
    # round half away from zero (inputs are positive), as C's llround does
    return np.floor(x + 0.5).astype(np.int64)


def make_profile_ns(L, n_dp, n_pp, n_micro, fwd_ns, bwd_ns, act, param, opt, p2p, base_cuts,
                    cap, dev_per_node, bw_intra, bw_inter) -> Profile:
    """Profile from per-layer times given directly in nanoseconds (scalars broadcast)."""
    fwd_ns = np.asarray(fwd_ns, dtype=np.float64)
    bwd_ns = np.asarray(bwd_ns, dtype=np.float64)

    def arr(v):
        return np.full(L, v, dtype=np.int64) if np.isscalar(v) else np.asarray(v, dtype=np.int64)

    return Profile(L=L, n_dp=n_dp, n_pp=n_pp, n_micro=n_micro,
                   fwd_ns=fwd_ns, bwd_ns=bwd_ns,
                   fwd_ns_i=_round_ns(fwd_ns), bwd_ns_i=_round_ns(bwd_ns),
                   act_bytes=arr(act), param_bytes=arr(param), opt_bytes=arr(opt),
                   p2p_bytes=arr(p2p), base_cuts=np.asarray(base_cuts, dtype=np.int32),
                   mem_capacity_bytes=int(cap), devices_per_node=int(dev_per_node),
                   bw_intra_Bpns=int(bw_intra), bw_inter_Bpns=int(bw_inter))


def _make_profile(L, n_dp, n_pp, n_micro, fwd_ms, bwd_ms, act, param, opt, p2p, base_cuts,
                  cap, dev_per_node, bw_intra, bw_inter) -> Profile:
    """Profile from per-layer times in milliseconds (converted as ns = ms * 1e6)."""
    return make_profile_ns(L, n_dp, n_pp, n_micro,
                           np.asarray(fwd_ms, dtype=np.float64) * 1e6,
                           np.asarray(bwd_ms, dtype=np.float64) * 1e6,
                           act, param, opt, p2p, base_cuts, cap, dev_per_node, bw_intra, bw_inter)


def _gaussian_layer_times(rng: SplitMix64, L: int, mean_ms: float, rel_sigma: float) -> List[float]:
    return [mean_ms * (1.0 + rel_sigma * rng.normal()) for _ in range(L)]


def tiny(mem_bound: bool = False) -> Workload:
    """L=8 on DP2 x PP4, one failed device, every single-device failure.

    ``mem_bound=True`` lowers the device memory to 1.3 GB so that the capacity check
    binds (at most three layers per stage, position dependent)."""
    rng = SplitMix64(1)
    L = 8
    fwd, bwd = [], []
    for _ in range(L):
        f = rng.uniform(1.0, 3.0)
        b = 2.0 * f * rng.uniform(0.9, 1.1)
        fwd.append(f)
        bwd.append(b)
    p = 50_000_000
    prof = _make_profile(L, 2, 4, 8, fwd, bwd, act=8_000_000, param=p, opt=6 * p,
                         p2p=8_000_000, base_cuts=[0, 2, 4, 6, 8],
                         cap=1_300_000_000 if mem_bound else 80_000_000_000,
                         dev_per_node=8, bw_intra=25, bw_inter=25)
    opts = SearchOptions(1, 7, 1, 8, LAYERS_FULL, BATCH_FULL, 1 << 62)
    return Workload("tiny-mem" if mem_bound else "tiny", prof, opts,
                    [[d] for d in range(8)])


def paper_scale(n_triples: int = 1024, n_quads: int = 1024) -> Workload:
    """32 devices DP4 x PP8, L=32 7B-like decoder layers, failure sets of 1-4 devices."""
    rng = SplitMix64(2)
    L = 32
    fwd = _gaussian_layer_times(rng, L, 10.0, 0.05)
    bwd = [2.0 * f for f in fwd]
    act = 2048 * 4096 * 2
    p = 12 * 4096 * 4096 * 2
    prof = _make_profile(L, 4, 8, 32, fwd, bwd, act=act, param=p, opt=6 * p, p2p=act,
                         base_cuts=[4 * i for i in range(9)], cap=80_000_000_000,
                         dev_per_node=8, bw_intra=400, bw_inter=25)
    opts = SearchOptions(3, 5, 4, 12, LAYERS_REMAINDER, BATCH_REMAINDER, 1 << 16)
    scen: List[List[int]] = [[d] for d in range(32)]
    scen += [[a, b] for a in range(32) for b in range(a + 1, 32)]
    frng = SplitMix64(2 ^ 0x5EED)
    scen += [frng.sample_distinct(32, 3) for _ in range(n_triples)]
    scen += [frng.sample_distinct(32, 4) for _ in range(n_quads)]
    return Workload("paper-scale", prof, opts, scen)


def llama70b_like() -> Workload:
    """L=80 on DP2 x PP32, heterogeneous layers (first and last twice the mean),
    80 GB devices with 12 B/param of optimizer state; 1-8 failed devices."""
    rng = SplitMix64(3)
    L = 80
    fwd = _gaussian_layer_times(rng, L, 10.0, 0.05)
    fwd[0] *= 2.0
    fwd[L - 1] *= 2.0
    bwd = [2.0 * f for f in fwd]
    p = 12 * 8192 * 8192 * 2
    cuts = [0]
    for s in range(32):
        cuts.append(cuts[-1] + (3 if s >= 16 else 2))
    prof = _make_profile(L, 2, 32, 64, fwd, bwd, act=34 * 2048 * 8192, param=p, opt=6 * p,
                         p2p=2048 * 8192 * 2, base_cuts=cuts, cap=80_000_000_000,
                         dev_per_node=8, bw_intra=400, bw_inter=25)
    opts = SearchOptions(1, 3, 16, 48, LAYERS_REMAINDER, BATCH_REMAINDER, 1 << 16)
    scen = []
    for size in range(1, 9):
        for s in range(8):
            frng = SplitMix64(3 * 1_000_003 + size * 101 + s)
            scen.append(frng.sample_distinct(64, size))
    return Workload("70b-like", prof, opts, scen)


def _gpt175b_profile() -> Profile:
    rng = SplitMix64(4)
    L = 96
    fwd = _gaussian_layer_times(rng, L, 10.0, 0.05)
    bwd = [2.0 * f for f in fwd]
    act = 2048 * 12288 * 2
    p = 12 * 12288 * 12288 * 2
    return _make_profile(L, 8, 32, 128, fwd, bwd, act=act, param=p, opt=6 * p, p2p=act,
                         base_cuts=[3 * i for i in range(33)], cap=120_000_000_000,
                         dev_per_node=8, bw_intra=400, bw_inter=25)


def _gpt175b_options() -> SearchOptions:
    return SearchOptions(7, 9, 30, 34, LAYERS_REMAINDER, BATCH_REMAINDER, 1 << 13)


def gpt175b_like() -> Workload:
    """L=96 on DP8 x PP32 (256 devices, 8 per node), two link tiers; whole-node and
    single-device failures."""
    prof = _gpt175b_profile()
    scen = [list(range(8 * n, 8 * n + 8)) for n in range(32)]
    frng = SplitMix64(4 ^ 0x5EED)
    scen += [[frng.below(256)] for _ in range(32)]
    return Workload("175b-like", prof, _gpt175b_options(), scen)


def sweep(n_scenarios: int = 1024) -> Workload:
    """Failure-scenario sweep on the 256-device, 96-layer setup: failure sets of size
    U{1..16} with uniformly random members."""
    prof = _gpt175b_profile()
    frng = SplitMix64(5)
    scen = []
    for _ in range(n_scenarios):
        size = 1 + frng.below(16)
        scen.append(frng.sample_distinct(256, size))
    return Workload("sweep", prof, _gpt175b_options(), scen)


def random_small(seed: int, L: int = 10, n_dp: int = 2, n_pp: int = 3, n_micro: int = 5,
                 tight_memory: bool = False) -> Workload:
    """Small randomised profile for brute-force and property tests: non-uniform times,
    non-uniform bytes, two link tiers with 4 devices per node."""
    rng = SplitMix64(0xC0FFEE + seed)
    fwd = [rng.uniform(0.5, 4.0) for _ in range(L)]
    bwd = [f * rng.uniform(1.5, 2.5) for f in fwd]
    act = [int(rng.uniform(1e6, 9e6)) for _ in range(L)]
    par = [int(rng.uniform(2e7, 8e7)) for _ in range(L)]
    opt = [6 * v for v in par]
    p2p = [int(rng.uniform(1e6, 6e7)) for _ in range(L)]
    base = [0]
    q, r = divmod(L, n_pp)
    for s in range(n_pp):
        base.append(base[-1] + q + (1 if s < r else 0))
    cap = int(8 * max(par) * (L / n_pp + 0.6)) if tight_memory else 80_000_000_000
    prof = _make_profile(L, n_dp, n_pp, n_micro, fwd, bwd, act, par, opt, p2p, base,
                         cap=cap, dev_per_node=4, bw_intra=300, bw_inter=20)
    n = n_dp * n_pp
    opts = SearchOptions(1, min(n, 6), 1, min(L, 8), LAYERS_FULL, BATCH_FULL, 1 << 62)
    scen = [[d] for d in range(n)]
    scen += [rng.sample_distinct(n, 2) for _ in range(4)]
    return Workload(f"random-small-{seed}", prof, opts, scen)


ALL_WORKLOADS = {
    "tiny": tiny,
    "tiny-mem": lambda: tiny(mem_bound=True),
    "paper-scale": paper_scale,
    "70b-like": llama70b_like,
    "175b-like": gpt175b_like,
    "sweep": sweep,
}


def deep_pipeline(seed: int = 0) -> Workload:
    """A deliberately deep, narrow job (DP2 x PP40, L=70) whose search window reaches
    pipelines of up to 64 stages: exercises the code paths for pipelines deeper than a
    warp (40 stages fault-free) and deeper than the register-resident kernels cover."""
    rng = SplitMix64(0xDEE9 + seed)
    L, n_dp, n_pp, n_micro = 70, 2, 40, 48
    fwd = [rng.uniform(2.0, 6.0) for _ in range(L)]
    bwd = [f * rng.uniform(1.8, 2.2) for f in fwd]
    act = [int(rng.uniform(2e6, 6e6)) for _ in range(L)]
    par = [int(rng.uniform(4e7, 9e7)) for _ in range(L)]
    p2p = [int(rng.uniform(1e6, 4e7)) for _ in range(L)]
    base = [0]
    for s in range(n_pp):
        base.append(base[-1] + (2 if s < L - n_pp else 1))
    prof = _make_profile(L, n_dp, n_pp, n_micro, fwd, bwd, act, par, [6 * v for v in par], p2p, base,
                         cap=4_000_000_000, dev_per_node=8, bw_intra=300, bw_inter=20)
    opts = SearchOptions(1, 3, 18, 64, LAYERS_REMAINDER, BATCH_REMAINDER, 40)
    n = n_dp * n_pp
    scen = [[7], [0], [41, 42], rng.sample_distinct(n, 3), rng.sample_distinct(n, 6), [39, 79]]
    return Workload(f"deep-pipeline-{seed}", prof, opts, scen)
