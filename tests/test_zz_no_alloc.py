"""The allocation-free top-k entry point gives exactly what the context-based one gives.

Some callers cannot call cudaMalloc (a loop that must not block on the allocator, a process
whose device memory all belongs to a pool, a plug-in whose host forbids it); for them the library has
`distsim_topk_static`, whose scratch is a fixed array inside the library.  This file is named so
that pytest collects it last: if it fails, a run that stops at the first failure has already
run every other test.
"""
import numpy as np
import pytest

from paper_2306_08423_b200 import workloads as W

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def test_static_topk_matches_context_topk_twice_in_a_row():
    from paper_2306_08423_b200 import engine as E
    ctx = E.Context(0)
    try:
        w = W.config3()
        E.distsim_load_event_table(ctx, w.table)
        n = E.distsim_set_space(ctx, w.space)
        batch = torch.empty(n, dtype=torch.int64, device="cuda")
        E.distsim_eval_strategies(ctx, 0, n, batch)
        # second input: another order and plenty of ties, so that state left over from the
        # first call (histogram, thresholds, output cursor) would show
        second = torch.flip(batch, dims=[0]) // 1000
        for arr, first, k in ((batch, 0, 1000), (second, 17, E.TOPK_STATIC_MAX_K)):
            want_i = torch.empty(k, dtype=torch.int64, device="cuda")
            want_t = torch.empty(k, dtype=torch.int64, device="cuda")
            E.distsim_topk(ctx, arr, first, n, k, want_i, want_t)
            got_i = torch.full((k,), -1, dtype=torch.int64, device="cuda")
            got_t = torch.full((k,), -1, dtype=torch.int64, device="cuda")
            torch.cuda.synchronize()
            free_before, _ = torch.cuda.mem_get_info()
            E.distsim_topk_static(arr, first, n, k, got_i, got_t)
            torch.cuda.synchronize()
            free_after, _ = torch.cuda.mem_get_info()
            if arr is second:
                # the call allocates nothing: by its second use (the first one may load the
                # kernels' code) the device's free memory is the same before and after
                assert free_after == free_before
            assert torch.equal(got_i, want_i) and torch.equal(got_t, want_t)    # integers: bit-exact
            st, si = torch.sort(arr, stable=True)
            assert torch.equal(got_t, st[:k]) and torch.equal(got_i, si[:k] + first)
        # a k beyond the fixed scratch is refused and nothing is written
        k = E.TOPK_STATIC_MAX_K + 1
        out = torch.full((k,), -1, dtype=torch.int64, device="cuda")
        with pytest.raises(E.DistsimError) as ei:
            E.distsim_topk_static(batch, 0, n, k, out)
        assert ei.value.code == E.E_CAPACITY
        torch.cuda.synchronize()
        assert (out == -1).all()
    finally:
        ctx.close()
