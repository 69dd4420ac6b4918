"""The host search drivers (Algorithms 1 and 2 over qcfg_eval_config) against the search oracle.

Both sides evaluate configurations of the same small model; the oracle side uses the CPU oracle's
forward and an fp64 fidelity.  Fidelities agree to float tolerance, so for targets that no visited
configuration comes close to, the two searches must take identical decisions: identical
configurations visited, in the same order, and the same final configuration."""
import numpy as np
import pytest
import torch

import qcfg_workloads as wl
from oracle import qcfg_oracle as orc
from oracle import search_oracle as so

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def setup():
    import paper_2302_01382_b200 as q
    ctx = q.Context(0)
    w = wl.bert_stack(31, 300, 128, 512, 2, bit_choices=None)
    weights = [torch.from_numpy(a).cuda() for a in w.weights]
    x = torch.from_numpy(w.x).cuda()
    model = q.Model(ctx, w.layers, weights)
    model.calibrate_model(x, w.m)
    act = [np.float32(a) for a in model.act_absmax()]
    wmax = [orc.absmax(a, orc.PER_ROW) for a in w.weights]
    sse, amax = ctx.quant_error_sweep(weights)
    ctx.check_sync()
    sizes = np.array([a.size for a in w.weights], np.float64)
    eqe = np.sqrt(sse.cpu().numpy()[:, 2] / sizes) / amax.cpu().numpy()
    order = [int(i) for i in np.argsort(eqe, kind="stable")]
    so_sse, so_amax = orc.quant_error_sweep(w.weights)
    assert order == [int(i) for i in orc.ranking(orc.e_qe_table(so_sse, sizes, so_amax)[:, 2])]
    ref = orc.eval_config(w.layers, w.weights, [16] * len(w.layers), w.x, act, wmax)[-1].astype(np.float64)
    cache = {}

    def evaluate(cfg):
        key = tuple(cfg)
        if key not in cache:
            y = orc.eval_config(w.layers, w.weights, cfg, w.x, act, wmax)[-1].astype(np.float64)
            cache[key] = 1.0 - np.linalg.norm(y - ref) / np.linalg.norm(ref)
        return cache[key]

    yield q, ctx, model, w, x, order, evaluate
    model.close()
    ctx.close()


@pytest.mark.parametrize("algorithm", [0, 1])
def test_search_matches_oracle_search(setup, algorithm):
    q, ctx, model, w, x, order, evaluate = setup
    n = len(w.layers)
    bs = [16, 8, 4]
    oracle_search = so.bisection_search if algorithm == 0 else so.greedy_search
    checked = 0
    for target in (0.995, 0.99, 0.98, 0.95, 0.9, 0.8, 0.5):
        w_o, vis_o = oracle_search(n, order, bs, target, evaluate)
        margin = min(abs(evaluate(c) - target) for c in vis_o)
        if margin < 2e-3:                      # a decision too close to call at float tolerance
            continue
        bits, vis, acc, n_evals = model.search(algorithm, order, bs, target, x, w.m)
        assert n_evals == len(vis_o)
        assert vis == [list(c) for c in vis_o]
        assert bits == list(w_o)
        np.testing.assert_allclose(acc, [evaluate(c) for c in vis_o], atol=5e-4)
        if algorithm == 0:
            assert n_evals <= 2 * (int(np.ceil(np.log2(n + 1))) + 2)
        else:
            assert n <= n_evals <= 2 * n
        checked += 1
    assert checked >= 3


def test_search_argument_errors(setup):
    q, ctx, model, w, x, order, evaluate = setup
    with pytest.raises(q.QcfgError) as e:
        model.search(0, [0] * len(order), [16, 8], 0.9, x, w.m)
    assert e.value.status == q.EINVAL
    with pytest.raises(q.QcfgError) as e:
        model.search(1, order, [16, 9], 0.9, x, w.m)
    assert e.value.status == q.EBITS
    bits, vis, acc, n_evals = model.search(1, order, [16], 0.9, x, w.m)     # nothing to lower
    assert bits == [16] * len(order) and n_evals == 0
