"""The allocation-free entry point against the existing one and against the CPU oracle.

cm_evaluate_argmin_noalloc serves callers that cannot allocate device memory when a
failure strikes (the training framework's allocator owns the GPU, or the handler must not
trigger the device-wide synchronisation an allocation implies).  It must return exactly
what a caller would get by running cm_evaluate over the same range and taking the
cheapest candidate (lowest index on ties) -- and that, in turn, is what the oracle's
per-candidate costs give.  Called twice in a row on purpose: both calls share one fixed
scratch array inside the library, and the second must not see leftovers of the first.
This file sorts last so that a run stopping at the first failure has already executed
every other test."""
import numpy as np
import pytest

from paper_2508_21613_b200 import workloads as W

pytestmark = pytest.mark.gpu

REL_TOL = 1e-12
NO_INDEX = 2**64 - 1
INT64_MAX = 2**63 - 1


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2508_21613_b200 import binding, build
    build.build()
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device; there is no CPU path")
    return binding


def _argmin(vals, ok, first):
    """Least value among the feasible entries, lowest index on ties."""
    ok = ok.astype(bool)
    if not ok.any():
        return None, None
    best = vals[ok].min()
    return best, first + int(np.flatnonzero(ok & (vals == best))[0])


def _reference(gpu, ctx, space, first, count, mode):
    """Cheapest candidate of the range from the existing entry point's per-candidate output."""
    import torch
    cost = torch.zeros(count, dtype=torch.float64, device="cuda")
    cost_ns = torch.zeros(count, dtype=torch.int64, device="cuda")
    feas = torch.zeros(count, dtype=torch.uint8, device="cuda")
    gpu.cm_evaluate(ctx, space, first, count, None, cost, cost_ns, feas)
    torch.cuda.synchronize()
    return _argmin((cost_ns if mode else cost).cpu().numpy(), feas.cpu().numpy(), first)


def _oracle_reference(orc, failed, first, count, mode):
    cost, cost_ns, feas = orc.evaluate(failed, first, count)
    return _argmin(cost_ns if mode else cost, feas, first)


def _buffers():
    import torch
    # the caller's own output buffers, allocated once, ahead of time
    return (torch.zeros(1, dtype=torch.float64, device="cuda"),
            torch.zeros(1, dtype=torch.int64, device="cuda"),
            torch.zeros(1, dtype=torch.int64, device="cuda"))


def _no_alloc(gpu, ctx, space, first, count, mode, out):
    import torch
    cost, cost_ns, index = out
    gpu.cm_evaluate_argmin_noalloc(ctx, space, first, count, cost, cost_ns, index)
    torch.cuda.synchronize()
    idx = int(index.cpu().numpy().view(np.uint64)[0])
    if idx == NO_INDEX:
        return None, None
    return (int(cost_ns.item()) if mode else float(cost.item())), idx


def _same(got, want, mode):
    (got_cost, got_idx), (want_cost, want_idx) = got, want
    assert got_idx == want_idx
    if want_idx is not None:
        if mode:
            assert got_cost == want_cost
        else:
            assert abs(got_cost - want_cost) <= REL_TOL * abs(want_cost)


@pytest.mark.parametrize("mode,native", [(0, False), (1, False), (1, True)])
def test_two_calls_in_a_row_match_cm_evaluate_and_the_oracle(gpu, oracle_factory, mode, native):
    for w, failed in ((W.tiny(mem_bound=True), [2]), (W.paper_scale(0, 0), [5, 17])):
        ctx = gpu.cm_create(0)
        try:
            gpu.cm_load_profile(ctx, w.profile)
            if native:
                gpu.cm_set_int64_arithmetic(ctx, True)      # the 64-bit integer kernels instead of exact doubles
            opts = w.options.with_cost_mode(mode)
            orc = oracle_factory(w.profile, opts)
            space, n = gpu.cm_enumerate(ctx, W.POLICY_DYNPAR, failed, opts)
            assert n > 1000
            out = _buffers()
            half = n // 2
            for first, count in ((0, min(n, gpu.NOALLOC_MAX_CANDIDATES)), (half, n - half), (3, 1)):
                got = _no_alloc(gpu, ctx, space, first, count, mode, out)
                _same(got, _reference(gpu, ctx, space, first, count, mode), mode)
                _same(got, _oracle_reference(orc, failed, first, count, mode), mode)
            gpu.cm_space_free(space)
        finally:
            gpu.cm_destroy(ctx)


@pytest.mark.parametrize("mode", [0, 1])
def test_the_largest_allowed_range_fills_the_whole_scratch_array(gpu, oracle_factory, mode):
    """Exactly NOALLOC_MAX_CANDIDATES candidates: every block partial of the fixed array is in
    use.  Twice in a row over different windows of the 70b-like space (memory decides most of
    its candidates), each checked against cm_evaluate and, on the first window, the oracle."""
    w = W.llama70b_like()
    failed = w.scenarios[0]
    opts = w.options.with_cost_mode(mode)
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        space, n = gpu.cm_enumerate(ctx, W.POLICY_DYNPAR, failed, opts)
        count = gpu.NOALLOC_MAX_CANDIDATES
        assert n >= 2 * count
        out = _buffers()
        for k, first in enumerate((0, n - count)):
            got = _no_alloc(gpu, ctx, space, first, count, mode, out)
            _same(got, _reference(gpu, ctx, space, first, count, mode), mode)
            if k == 0:
                orc = oracle_factory(w.profile, opts)
                # the oracle walks the window in slices that each finish in seconds
                best = (None, None)
                for lo in range(0, count, 65536):
                    c, i = _oracle_reference(orc, failed, first + lo, min(65536, count - lo), mode)
                    if i is not None and (best[1] is None or c < best[0]):
                        best = (c, i)
                _same(got, best, mode)
        gpu.cm_space_free(space)
    finally:
        gpu.cm_destroy(ctx)


@pytest.mark.parametrize("mode,native", [(0, False), (1, False), (1, True)])
def test_a_range_without_a_feasible_candidate_returns_the_sentinels(gpu, mode, native):
    import torch
    w = W.tiny()
    w.profile.mem_capacity_bytes = 1000          # nothing fits: every candidate fails the memory check
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        if native:
            gpu.cm_set_int64_arithmetic(ctx, True)
        space, n = gpu.cm_enumerate(ctx, W.POLICY_DYNPAR, [1], w.options.with_cost_mode(mode))
        cost, cost_ns, index = _buffers()
        for _ in range(2):
            cost.fill_(-1.0); cost_ns.fill_(-1); index.fill_(7)
            gpu.cm_evaluate_argmin_noalloc(ctx, space, 0, min(n, gpu.NOALLOC_MAX_CANDIDATES), cost, cost_ns, index)
            torch.cuda.synchronize()
            assert int(index.cpu().numpy().view(np.uint64)[0]) == NO_INDEX
            if mode:
                assert int(cost_ns.item()) == INT64_MAX and float(cost.item()) == -1.0   # the other buffer is untouched
            else:
                assert float(cost.item()) == float("inf") and int(cost_ns.item()) == -1
        gpu.cm_space_free(space)
    finally:
        gpu.cm_destroy(ctx)


def test_index_alone_may_be_asked_for(gpu):
    import torch
    w = W.tiny(mem_bound=True)
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        space, n = gpu.cm_enumerate(ctx, W.POLICY_DYNPAR, [2], w.options)
        index = torch.zeros(1, dtype=torch.int64, device="cuda")
        for _ in range(2):
            gpu.cm_evaluate_argmin_noalloc(ctx, space, 0, n, None, None, index)
            torch.cuda.synchronize()
            assert int(index.item()) == _reference(gpu, ctx, space, 0, n, 0)[1]
        gpu.cm_space_free(space)
    finally:
        gpu.cm_destroy(ctx)


def test_ranges_beyond_the_fixed_scratch_are_refused(gpu):
    w = W.llama70b_like()
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        space, n = gpu.cm_enumerate(ctx, W.POLICY_DYNPAR, w.scenarios[0], w.options)
        assert n > gpu.NOALLOC_MAX_CANDIDATES
        for count in (gpu.NOALLOC_MAX_CANDIDATES + 1, 0):
            with pytest.raises(gpu.ChameleonError) as e:
                gpu.cm_evaluate_argmin_noalloc(ctx, space, 0, count)
            assert e.value.status == gpu.CM_EINVAL
        with pytest.raises(gpu.ChameleonError):
            gpu.cm_evaluate_argmin_noalloc(ctx, space, n - 5, 10)
        gpu.cm_space_free(space)
    finally:
        gpu.cm_destroy(ctx)
