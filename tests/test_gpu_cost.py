"""Latency table and configuration cost through the C-ABI against the cost oracle."""
import numpy as np
import pytest
import torch

import qcfg_workloads as wl
from oracle import cost_oracle as cost

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def setup():
    import paper_2302_01382_b200 as q
    ctx = q.Context(0)
    w = wl.bert_stack(31, 2048, 256, 1024, 2)
    weights = [torch.from_numpy(a).cuda() for a in w.weights]
    model = q.Model(ctx, w.layers, weights)
    x = torch.from_numpy(w.x).cuda()
    model.calibrate_model(x, w.m)
    yield q, ctx, model, w, x
    model.close()
    ctx.close()


def test_latency_table_and_cost_match_oracle(setup):
    q, ctx, model, w, x = setup
    bs = [16, 8, 4]
    table = model.latency_table(x, w.m, bs, reps=3)
    ctx.check_sync()
    t = np.array(table)
    assert t.shape == (len(w.layers), 3)
    assert np.all(np.isfinite(t)) and np.all(t > 0)
    rng = np.random.default_rng(5)
    for _ in range(4):
        bits = [int(b) for b in rng.choice(bs, len(w.layers))]
        lat, size = model.config_cost(bits, bs, table)
        assert size == cost.size_bytes(w.layers, bits)                      # exact: small integers over 8
        assert lat == pytest.approx(cost.latency_ms(table, bs, bits), rel=1e-12)
    # all integer widths share the int8 tensor path here: their columns agree up to timing noise
    assert t[:, 2].sum() == pytest.approx(t[:, 1].sum(), rel=0.35)
    # size alone needs no table
    lat, size = model.config_cost([8] * len(w.layers))
    assert lat is None and size == cost.size_bytes(w.layers, [8] * len(w.layers))


def test_cost_argument_errors(setup):
    q, ctx, model, w, x = setup
    n = len(w.layers)
    table = [[1.0, 2.0]] * n
    with pytest.raises(q.QcfgError) as e:
        model.config_cost([4] * n, [16, 8], table)            # 4 bit is not a column of the table
    assert e.value.status == q.EBITS
    with pytest.raises(q.QcfgError) as e:
        model.config_cost([9] * n)
    assert e.value.status == q.EBITS
    with pytest.raises(q.QcfgError) as e:
        model.latency_table(x, w.m, [8, 1], reps=1)
    assert e.value.status == q.EBITS
