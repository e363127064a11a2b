"""The allocation-free entry point against the existing one.

cm_evaluate_argmin_noalloc serves callers that cannot allocate device memory when a
failure strikes (the training framework's allocator owns the GPU, or the handler must not
trigger the device-wide synchronisation an allocation implies).  It must return exactly
what a caller would get by running cm_evaluate over the same range and taking the
cheapest candidate (lowest index on ties).  Called twice in a row on purpose: both calls
share one fixed scratch array inside the library, and the second must not see leftovers
of the first.  This file sorts last so that a run stopping at the first failure has
already executed every other test."""
import numpy as np
import pytest

from paper_2508_21613_b200 import workloads as W

pytestmark = pytest.mark.gpu

REL_TOL = 1e-12


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2508_21613_b200 import binding, build
    build.build()
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device; there is no CPU path")
    return binding


def _reference(gpu, ctx, space, first, count, mode):
    """Cheapest candidate of the range from the existing entry point's per-candidate output."""
    import torch
    cost = torch.zeros(count, dtype=torch.float64, device="cuda")
    cost_ns = torch.zeros(count, dtype=torch.int64, device="cuda")
    feas = torch.zeros(count, dtype=torch.uint8, device="cuda")
    gpu.cm_evaluate(ctx, space, first, count, None, cost, cost_ns, feas)
    torch.cuda.synchronize()
    vals = (cost_ns if mode else cost).cpu().numpy()
    ok = feas.cpu().numpy().astype(bool)
    if not ok.any():
        return None, None
    best = vals[ok].min()
    return best, first + int(np.flatnonzero(ok & (vals == best))[0])


def _no_alloc(gpu, ctx, space, first, count, mode, out):
    import torch
    cost, cost_ns, index = out
    gpu.cm_evaluate_argmin_noalloc(ctx, space, first, count, cost, cost_ns, index)
    torch.cuda.synchronize()
    idx = int(index.cpu().numpy().view(np.uint64)[0])
    if idx == 2**64 - 1:
        return None, None
    return (int(cost_ns.item()) if mode else float(cost.item())), idx


@pytest.mark.parametrize("mode", [0, 1])
def test_two_calls_in_a_row_match_cm_evaluate(gpu, mode):
    import torch
    for w, failed in ((W.tiny(mem_bound=True), [2]), (W.paper_scale(0, 0), [5, 17])):
        ctx = gpu.cm_create(0)
        try:
            gpu.cm_load_profile(ctx, w.profile)
            opts = w.options.with_cost_mode(mode)
            space, n = gpu.cm_enumerate(ctx, W.POLICY_DYNPAR, failed, opts)
            assert n > 1000
            # the caller's own output buffers, allocated once, ahead of time
            out = (torch.zeros(1, dtype=torch.float64, device="cuda"),
                   torch.zeros(1, dtype=torch.int64, device="cuda"),
                   torch.zeros(1, dtype=torch.int64, device="cuda"))
            half = n // 2
            for first, count in ((0, min(n, gpu.NOALLOC_MAX_CANDIDATES)), (half, n - half), (3, 1)):
                want_cost, want_idx = _reference(gpu, ctx, space, first, count, mode)
                got_cost, got_idx = _no_alloc(gpu, ctx, space, first, count, mode, out)
                assert got_idx == want_idx
                if want_idx is not None:
                    if mode:
                        assert got_cost == want_cost
                    else:
                        assert abs(got_cost - want_cost) <= REL_TOL * abs(want_cost)
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
