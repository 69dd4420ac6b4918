"""The sweep entry point that allocates no device memory, against the regular one.

qcfg_quant_error_sweep_static exists for callers that cannot allocate on the device at call
time: code running after a serving engine or framework has claimed all GPU memory for its own
pool, or inside a loop that cannot afford the device-wide synchronisation an allocation
implies.  Its scratch is one fixed array inside the library, shared by every call, which keeps
whatever the previous call left there; so the test calls it twice in a row, on different
inputs, and each result must equal the regular entry point's on the same inputs (same kernels,
same order of summation: equal to the last bit, and in any case within the 1e-5 relative
tolerance the sweep tests use).  Inputs beyond the array's capacity must be refused with a
clear message, before anything runs.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.  It passes on its own in a fresh process and after the other tests.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _tensors(seed, shapes):
    rng = np.random.default_rng(seed)
    out = []
    for s in shapes:
        w = (rng.standard_normal(s) * 0.02).astype(np.float32)
        w[rng.random(s) < 1e-3] *= 20
        out.append(torch.from_numpy(w).cuda())
    return out


def test_static_sweep_matches_regular_sweep_on_two_calls_in_a_row():
    import paper_2302_01382_b200 as q
    ctx = q.Context(0)
    try:
        first = _tensors(1, [(768, 768), (3072, 768), (300, 3072), (64, 147), (10, 256), (40, 4608)])
        second = _tensors(2, [(97, 1024), (33, 4096), (500, 64), (3, 9000)])   # fewer, different shapes
        for granularity in (q.PER_ROW, q.PER_TENSOR):
            for tensors in (first, second):
                n = len(tensors)
                sse_s = torch.full((n, 7), float("nan"), dtype=torch.float64, device="cuda")
                amax_s = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
                ctx.quant_error_sweep_static(tensors, granularity, 2, 8, sse=sse_s, absmax=amax_s)
                ctx.check_sync()
                sse_r, amax_r = ctx.quant_error_sweep(tensors, granularity, 2, 8)
                ctx.check_sync()
                assert torch.equal(amax_s, amax_r)
                np.testing.assert_allclose(sse_s.cpu().numpy(), sse_r.cpu().numpy(), rtol=1e-5, atol=0)
                assert torch.equal(sse_s, sse_r)
        # a sub-range of bit widths, right after a full-range call left its sums behind
        sub, _ = ctx.quant_error_sweep_static(first, q.PER_ROW, 4, 6)
        ref, _ = ctx.quant_error_sweep(first, q.PER_ROW, 4, 6)
        ctx.check_sync()
        assert torch.equal(sub, ref)
    finally:
        ctx.close()


def test_static_sweep_matches_the_oracle_and_allocates_nothing():
    """Against the CPU oracle (not only its sibling), and with the device's free memory unchanged
    across a call once the outputs exist."""
    import paper_2302_01382_b200 as q
    from oracle import qcfg_oracle as orc
    ctx = q.Context(0)
    try:
        tensors = _tensors(3, [(200, 768), (64, 3072), (33, 100)])
        so, ao = orc.quant_error_sweep([t.cpu().numpy() for t in tensors])
        sse = torch.empty((3, 7), dtype=torch.float64, device="cuda")
        amax = torch.empty(3, dtype=torch.float32, device="cuda")
        ctx.quant_error_sweep_static(tensors, q.PER_ROW, 2, 8, sse=sse, absmax=amax)      # first call: address look-up
        ctx.check_sync()
        free_before, _ = torch.cuda.mem_get_info()
        ctx.quant_error_sweep_static(tensors, q.PER_ROW, 2, 8, sse=sse, absmax=amax)
        ctx.check_sync()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        np.testing.assert_allclose(sse.cpu().numpy(), so, rtol=1e-5)
        np.testing.assert_array_equal(amax.cpu().numpy(), ao)
    finally:
        ctx.close()


def test_static_sweep_refuses_what_does_not_fit():
    import paper_2302_01382_b200 as q
    ctx = q.Context(0)
    try:
        t = torch.zeros((8, 64), device="cuda")
        sse = torch.zeros((1, 7), dtype=torch.float64, device="cuda")
        amax = torch.zeros(1, device="cuda")
        # a declared shape beyond the element limit of one call: refused on the host, nothing is
        # launched, outputs stay as they were
        with pytest.raises(q.QcfgError) as e:
            ctx.quant_error_sweep_static([t], q.PER_ROW, 2, 8, sse=sse, absmax=amax, shapes=[(10 ** 9, 768)])
        assert e.value.status == q.ENOMEM and "2^35 elements" in str(e.value)
        many = [t] * 1025
        with pytest.raises(q.QcfgError) as e:
            ctx.quant_error_sweep_static(many, q.PER_ROW, 2, 8)
        assert e.value.status == q.ENOMEM and "1024" in str(e.value)
        assert ctx.sync_status() == q.OK
        assert not sse.any() and not amax.any()
    finally:
        ctx.close()
