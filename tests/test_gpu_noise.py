"""E_N (Eqs. 3-5) through the C-ABI against the noise oracle."""
import numpy as np
import pytest
import torch

import qcfg_workloads as wl
from oracle import noise_oracle as nz

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2302_01382_b200 as q
    c = q.Context(0)
    yield c
    c.close()


def _run(ctx, w, nus, lam):
    import paper_2302_01382_b200 as q
    weights = [torch.from_numpy(a).cuda() for a in w.weights]
    model = q.Model(ctx, w.layers, weights)
    x = torch.from_numpy(np.ascontiguousarray(w.x)).cuda()
    noises = [None if a is None else torch.from_numpy(a).cuda() for a in nus]
    e = model.noise_sensitivity(x, w.m, noises, lam)
    ctx.check_sync()
    model.close()
    return np.array(e)


@pytest.mark.parametrize("make", [lambda: wl.tiny_mlp(), lambda: wl.bert_stack(41, 333, 128, 512, 2),
                                  lambda: wl.resnet50(seed=3, batch=2, in_hw=32, width=16, n_classes=10, blocks=(1, 1, 1, 1))])
def test_noise_sensitivity_matches_oracle(ctx, make):
    w = make()
    nus = wl.standard_normal_like(w.weights, 99)
    nus[1] = None                                         # a skipped layer reports 0
    lam = 0.05
    got = _run(ctx, w, nus, lam)
    want = np.array(nz.noise_sensitivity(w.layers, w.weights, w.x, nus, lam))
    assert got[1] == 0.0 and want[1] == 0.0
    # both sides round operands to bf16; the GPU accumulates in fp32, the oracle wider, so a few
    # intermediate activations round to the other bf16 neighbour: agreement to about 1e-3 of E_N,
    # 1e-2 required, with a floor for layers whose effect is below the rounding noise
    np.testing.assert_allclose(got, want, rtol=1e-2, atol=2e-4)
    # layers nothing downstream reads: exactly zero on both sides
    assert np.array_equal(got == 0.0, want == 0.0)
    # and the ordering of clearly separated layers (the use the paper makes of the metric) agrees
    order = np.argsort(want)
    for a, b in zip(order[:-1], order[1:]):
        if want[b] > 1.05 * want[a] + 4e-4:
            assert got[b] > got[a]


def test_noise_sensitivity_zero_lambda_and_errors(ctx):
    import paper_2302_01382_b200 as q
    w = wl.tiny_mlp()
    nus = wl.standard_normal_like(w.weights, 3)
    assert np.all(_run(ctx, w, nus, 0.0) == 0.0)
    weights = [torch.from_numpy(a).cuda() for a in w.weights]
    model = q.Model(ctx, w.layers, weights)
    x = torch.from_numpy(w.x).cuda()
    with pytest.raises(q.QcfgError) as e:
        model.noise_sensitivity(x, w.m, [None] * 3, -1.0)
    assert e.value.status == q.EINVAL
    model.close()
