"""Pins of the scale-adjustment oracle (Section 3.1, second step; learning rate of Section 4).

The oracle's gradient code is checked against things other than itself: central finite
differences of a rounding-free surrogate forward (where the straight-through gradient is the exact
one), a closed form on a one-layer model, and structural facts (16-bit layers have no scale
gradients, clipped elements do not move the pre-rounding scale, weights are never written, the
forward with calibrated scales is the evaluation oracle's forward bit for bit, a small step lowers
the surrogate loss by lr * |gradient|^2 to first order)."""
import copy

import numpy as np
import pytest

import qcfg_workloads as wl
from oracle import adjust_oracle as adj
from oracle import qcfg_oracle as orc

F64 = np.float64


def _setup(seed=5, m=24, bits=None, residual=False, gelu=True):
    rng = np.random.default_rng(seed)
    L = wl.Layer
    layers = [L("a", 20, 16, src=-1, act=orc.ACT_RELU),
              L("b", 20, 20, src=0, act=orc.ACT_GELU_TANH if gelu else orc.ACT_NONE),
              L("c", 12, 8, src=1, src_col0=4, act=orc.ACT_NONE),           # reads a column slice
              L("d", 20, 12, src=2, act=orc.ACT_RELU, residual_from=1 if residual else -1),
              L("e", 6, 20, src=3, act=orc.ACT_NONE)]
    x = rng.standard_normal((m, 16)).astype(np.float32)
    weights = [(rng.standard_normal((l.n_out, l.k_in)) / np.sqrt(l.k_in)).astype(np.float32) for l in layers]
    bits = bits or [8, 6, 16, 4, 8]
    act, wmax = orc.calibrate_model(layers, weights, x)
    return layers, weights, bits, x, act, wmax


def _soft_loss(layers, weights, bits, x, scales, y_ref):
    return adj.loss(adj.forward(layers, weights, bits, x, scales, soft=True)[-1]["y"], y_ref)


@pytest.mark.parametrize("residual", [False, True])
def test_gradients_match_finite_differences_of_the_rounding_free_surrogate(residual):
    layers, weights, bits, x, act, wmax = _setup(residual=residual)
    n = len(layers)
    y_ref = adj.forward(layers, weights, [16] * n, x, [None] * n, soft=True)[-1]["y"]
    scales = adj.calibrated_scales(layers, weights, bits, act, wmax)
    # move the scales off their calibrated values so that some elements clip
    rng = np.random.default_rng(1)
    for sc in scales:
        if sc is None:
            continue
        sc["ix"] = np.float32(sc["ix"] * 1.3)
        sc["sx"] = np.float32(sc["sx"] * 0.9)
        sc["iw"] = (sc["iw"] * rng.uniform(0.9, 1.4, sc["iw"].shape)).astype(np.float32)
        sc["sw"] = (sc["sw"] * rng.uniform(0.8, 1.1, sc["sw"].shape)).astype(np.float32)
    taps = adj.forward(layers, weights, bits, x, scales, soft=True)
    assert any(np.any(np.abs(t["tx"]) > orc.qmax(t["bits"])) for t in taps if t["bits"] != 16)   # the clip is live
    g = adj.gradients(layers, weights, bits, scales, taps, y_ref)
    checked = 0
    for l, sc in enumerate(scales):
        if sc is None:
            assert g[l] is None
            continue
        for key in ("sx", "ix", "sw", "iw"):
            idxs = [None] if key in ("sx", "ix") else [0, sc[key].size // 2, sc[key].size - 1]
            for i in idxs:
                base = float(sc[key]) if i is None else float(sc[key][i])
                h = 1e-4 * abs(base)
                vals = []
                for sign in (+1, -1):
                    s2 = copy.deepcopy(scales)
                    s2 = [None if t is None else {k: (np.array(v, F64) if np.ndim(v) else F64(v)) for k, v in t.items()} for t in s2]
                    if i is None:
                        s2[l][key] = F64(base + sign * h)
                    else:
                        s2[l][key][i] = base + sign * h
                    vals.append(_soft_loss(layers, weights, bits, x, s2, y_ref))
                fd = (vals[0] - vals[1]) / (2 * h)
                an = g[l][key] if i is None else g[l][key][i]
                assert abs(fd - an) <= 2e-5 * max(abs(fd), abs(an)) + 1e-12, (l, key, i, fd, an)
                checked += 1
    assert checked >= 30


def test_closed_form_for_one_layer_post_rounding_scales():
    # one linear layer, no activation: y = acc * sx * sw[n]; L = sum (y - r)^2 / sum r^2
    rng = np.random.default_rng(3)
    lay = [wl.Layer("a", 5, 7, src=-1)]
    x = rng.standard_normal((9, 7)).astype(np.float32)
    w = [rng.standard_normal((5, 7)).astype(np.float32)]
    act, wmax = orc.calibrate_model(lay, w, x)
    scs = adj.calibrated_scales(lay, w, [4], act, wmax)
    sc = scs[0]
    taps = adj.forward(lay, w, [4], x, scs)
    y_ref = rng.standard_normal((9, 5)).astype(np.float32)
    g = adj.gradients(lay, w, [4], scs, taps, y_ref)[0]
    acc = orc.int_gemm(taps[0]["qx"].astype(np.int8), taps[0]["qw"].astype(np.int8)).astype(F64)
    y = taps[0]["y"].astype(F64)
    r2 = np.sum(y_ref.astype(F64) ** 2)
    d = 2 * (y - y_ref) / r2
    np.testing.assert_allclose(g["sx"], np.sum(d * acc * sc["sw"].astype(F64)[None, :]), rtol=1e-12)
    np.testing.assert_allclose(g["sw"], np.sum(d * acc, axis=0) * float(sc["sx"]), rtol=1e-12)
    # hand-sized case: x = [[1, -2]], w = [[3, 1]] at 8 bit on exact grids
    lay = [wl.Layer("a", 1, 2, src=-1)]
    x1 = np.array([[1.0, -2.0]], np.float32); w1 = [np.array([[3.0, 1.0]], np.float32)]
    s1 = [{"sx": np.float32(2 / 127), "ix": np.float32(127 / 2), "sw": np.array([3 / 127], np.float32), "iw": np.array([127 / 3], np.float32)}]
    t1 = adj.forward(lay, w1, [8], x1, s1)
    acc1 = float(orc.int_gemm(t1[0]["qx"].astype(np.int8), t1[0]["qw"].astype(np.int8))[0, 0])
    assert acc1 == 64 * 127 + (-127) * 42              # codes (64, -127) and (127, 42)
    yr = np.array([[2.0]], np.float32)
    g1 = adj.gradients(lay, w1, [8], s1, t1, yr)[0]
    y1 = float(t1[0]["y"][0, 0])
    assert g1["sx"] == pytest.approx(2 * (y1 - 2.0) / 4.0 * acc1 * float(s1[0]["sw"][0]), rel=1e-12)


def test_structure_sixteen_bit_layers_clipped_elements_untouched_weights():
    layers, weights, bits, x, act, wmax = _setup(gelu=False)
    n = len(layers)
    before = [w.copy() for w in weights]
    scales, losses = adj.adjust(layers, weights, bits, x, act, wmax, steps=2, lr=1e-5)
    assert len(losses) == 3 and all(np.isfinite(losses))
    for a, b in zip(before, weights):
        np.testing.assert_array_equal(a, b)                         # the model's parameters are frozen
    assert scales[2] is None                                        # the 16-bit layer has no scales
    # forward with calibrated scales is the evaluation oracle's forward
    sc0 = adj.calibrated_scales(layers, weights, bits, act, wmax)
    taps = adj.forward(layers, weights, bits, x, sc0)
    ref = orc.eval_config(layers, weights, bits, x, act, wmax)
    for l in range(n):
        np.testing.assert_array_equal(taps[l]["y"].view(np.uint32), ref[l].view(np.uint32))
    # an element beyond the clip range contributes nothing to d/d(inv_scale): blow one input up
    y_ref = adj.forward(layers, weights, [16] * n, x, [None] * n)[-1]["y"]
    g0 = adj.gradients(layers, weights, bits, sc0, taps, y_ref)
    x2 = x.copy(); x2[3, 5] = 1e4                                    # far outside the calibrated range
    taps2 = adj.forward(layers, weights, bits, x2, sc0)
    assert abs(taps2[0]["tx"][3, 5]) > 127
    g2 = adj.gradients(layers, weights, bits, sc0, taps2, y_ref)
    # recompute layer 0's d/d(ix) by hand without the clipped element
    t = taps2[0]; sc = sc0[0]
    n_all = len(layers)
    # the gradient reaching layer 0's codes is whatever it is; zeroing the clipped element's input
    # value must not change d_ix (its term is masked), while an unclipped one does
    x3 = x2.copy(); x3[3, 5] = 2e4
    g3 = adj.gradients(layers, weights, bits, sc0, adj.forward(layers, weights, bits, x3, sc0), y_ref)
    assert g2[0]["ix"] == g3[0]["ix"]                                # still clipped to the same code
    assert g0[0]["ix"] != g2[0]["ix"]
    # layers whose output never reaches the loss get exactly zero
    L = wl.Layer
    lay2 = [L("a", 8, 16, src=-1), L("tap", 8, 16, src=-1), L("b", 4, 8, src=0)]
    w2 = [np.random.default_rng(9).standard_normal((l.n_out, l.k_in)).astype(np.float32) for l in lay2]
    a2, m2 = orc.calibrate_model(lay2, w2, x)
    s2 = adj.calibrated_scales(lay2, w2, [8, 8, 8], a2, m2)
    t2 = adj.forward(lay2, w2, [8, 8, 8], x, s2)
    yr = adj.forward(lay2, w2, [16] * 3, x, [None] * 3)[-1]["y"]
    gg = adj.gradients(lay2, w2, [8, 8, 8], s2, t2, yr)
    assert gg[1]["sx"] == 0.0 and gg[1]["ix"] == 0.0 and not gg[1]["sw"].any() and not gg[1]["iw"].any()
    assert gg[0]["sx"] != 0.0


def test_small_step_lowers_the_surrogate_loss_to_first_order():
    layers, weights, bits, x, act, wmax = _setup(seed=8)
    n = len(layers)
    y_ref = adj.forward(layers, weights, [16] * n, x, [None] * n, soft=True)[-1]["y"]
    scales = adj.calibrated_scales(layers, weights, bits, act, wmax)
    taps = adj.forward(layers, weights, bits, x, scales, soft=True)
    g = adj.gradients(layers, weights, bits, scales, taps, y_ref)
    norm2 = sum(gl["sx"] ** 2 + gl["ix"] ** 2 + np.sum(gl["sw"] ** 2) + np.sum(gl["iw"] ** 2) for gl in g if gl)
    l0 = adj.loss(taps[-1]["y"], y_ref)
    lr = 1e-3 * l0 / norm2
    s64 = [None if t is None else {k: np.array(v, F64) for k, v in t.items()} for t in scales]
    s1 = [None if t is None else {k: t[k] - lr * (g[i][k] if np.ndim(g[i][k]) else F64(g[i][k])) for k in t} for i, t in enumerate(s64)]
    l1 = _soft_loss(layers, weights, bits, x, s1, y_ref)
    assert l1 < l0
    assert (l0 - l1) == pytest.approx(lr * norm2, rel=2e-2)
    # and the update rule itself: fp32(scale - lr * gradient)
    new = adj.sgd_step(scales, g, 1e-5)
    assert new[0]["sx"] == np.float32(np.float64(scales[0]["sx"]) - 1e-5 * g[0]["sx"])
    assert new[0]["iw"].dtype == np.float32 and new[2] is None
