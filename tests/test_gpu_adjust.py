"""Scale adjustment on the GPU (Section 3.1, second step) against the adjustment oracle.

Forward quantities are exact (the loss agrees to fp64-sum accuracy); the backward pass runs its two
GEMMs per layer with bf16 operands on the tensor cores, so gradients agree with the oracle's fp64
ones to bf16 accuracy (2e-2 of each gradient vector's norm); the update rule is exact given the
gradient; the model's weights are never written; an evaluation after the adjustment uses the
adapted scales (checked bit for bit against the oracle's forward at those scales)."""
import numpy as np
import pytest
import torch

import qcfg_workloads as wl
from oracle import adjust_oracle as adj
from oracle import qcfg_oracle as orc

pytestmark = pytest.mark.gpu


def _close(a, b, tol=2e-2, floor=1e-12):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return np.linalg.norm(a - b) <= tol * max(np.linalg.norm(b), floor) + floor


def _gpu_scales(model, layers, bits):
    out = []
    for l, b in enumerate(bits):
        if int(b) == 16:
            out.append(None)
            continue
        sx, ix, sw, iw = model.scales(l, int(b))
        out.append({"sx": np.float32(sx), "ix": np.float32(ix), "sw": np.array(sw, np.float32), "iw": np.array(iw, np.float32)})
    return out


@pytest.mark.parametrize("kind", ["tiny_mlp", "bert_block", "residual"])
def test_gradients_update_and_evaluation_match_the_oracle(kind):
    import paper_2302_01382_b200 as q
    if kind == "tiny_mlp":
        w = wl.tiny_mlp()
        bits = [8, 4, 8]
    elif kind == "bert_block":
        w = wl.bert_stack(41, 320, 128, 512, 1, bit_choices=None)
        bits = [8, 4, 6, 16, 8, 4]
    else:
        L = wl.Layer
        layers = [L("a", 96, 64, src=-1, act=orc.ACT_RELU), L("b", 96, 96, src=0, act=orc.ACT_RELU),
                  L("c", 96, 40, src=1, src_col0=8, act=orc.ACT_RELU, residual_from=0), L("d", 24, 96, src=2)]
        rng = np.random.default_rng(42)
        x = rng.standard_normal((200, 64)).astype(np.float32)
        ws = [(rng.standard_normal((l.n_out, l.k_in)) / np.sqrt(l.k_in)).astype(np.float32) for l in layers]
        w = wl.Workload("residual", 42, layers, 200, x, ws)
        bits = [8, 5, 4, 8]
    n = len(w.layers)
    ctx = q.Context(0)
    try:
        weights = [torch.from_numpy(a).cuda() for a in w.weights]
        before = [t.clone() for t in weights]
        x = torch.from_numpy(w.x).cuda()
        model = q.Model(ctx, w.layers, weights)
        model.calibrate_model(x, w.m)
        act = [np.float32(a) for a in model.act_absmax()]
        wmax = [orc.absmax(a, orc.PER_ROW) for a in w.weights]
        # oracle at the calibrated scales, fed with the GPU's calibration table
        sc0 = adj.calibrated_scales(w.layers, w.weights, bits, act, wmax)
        y_ref = adj.forward(w.layers, w.weights, [16] * n, w.x, [None] * n)[-1]["y"]
        taps = adj.forward(w.layers, w.weights, bits, w.x, sc0)
        g_o = adj.gradients(w.layers, w.weights, bits, sc0, taps, y_ref)
        loss_o = adj.loss(taps[-1]["y"], y_ref)
        loss_g, dsx, dix, dsw, diw = model.scale_gradients(bits, x, w.m)
        # the 16-bit reference forward differs in its last bits between the two sides (fp32 against fp64
        # accumulation of bf16 products), which moves the loss by about 1e-3 of itself
        assert loss_g == pytest.approx(loss_o, rel=5e-3)
        for l in range(n):
            if int(bits[l]) == 16:
                assert dsx[l] == 0.0 and dix[l] == 0.0 and not any(dsw[l]) and not any(diw[l])
                continue
        live = [l for l in range(n) if int(bits[l]) != 16]
        assert _close([dsx[l] for l in live], [g_o[l]["sx"] for l in live])
        assert _close([dix[l] for l in live], [g_o[l]["ix"] for l in live])
        for l in live:
            assert _close(dsw[l], g_o[l]["sw"], floor=1e-9 * abs(g_o[l]["sx"])), (kind, l, "scale_w")
            assert _close(diw[l], g_o[l]["iw"], floor=1e-9 * abs(g_o[l]["ix"])), (kind, l, "inv_scale_w")
        # layers the loss never sees (the q and k projections of the block) get exactly zero
        if kind == "bert_block":
            for l in (0, 1):
                assert dsx[l] == 0.0 and dix[l] == 0.0 and not any(dsw[l]) and not any(diw[l])
                assert g_o[l]["sx"] == 0.0
        # two steps at the paper's learning rate: update rule, frozen weights, losses
        lr = 1e-5
        losses = model.adjust_scales(bits, x, w.m, steps=2, lr=lr)
        assert len(losses) == 3 and losses[0] == pytest.approx(loss_g, rel=1e-12)
        for a, b in zip(before, weights):
            assert torch.equal(a, b)
        sc_o, losses_o = adj.adjust(w.layers, w.weights, bits, w.x, act, wmax, steps=2, lr=lr)
        sc_g = _gpu_scales(model, w.layers, bits)
        for l in live:
            for key in ("sx", "ix", "sw", "iw"):
                moved = np.abs(np.asarray(sc_o[l][key], np.float64) - np.asarray(sc0[l][key], np.float64))
                diff = np.abs(np.asarray(sc_g[l][key], np.float64) - np.asarray(sc_o[l][key], np.float64))
                ulp = np.abs(np.asarray(sc_o[l][key], np.float64)) * 2.0 ** -23
                assert np.all(diff <= 0.1 * moved.max() + 2 * ulp), (kind, l, key)
        # first step alone: exact update rule on the GPU's own gradients
        model.reset_scales()
        loss1, dsx1, dix1, dsw1, diw1 = model.scale_gradients(bits, x, w.m)
        model.adjust_scales(bits, x, w.m, steps=1, lr=lr)
        sc1 = _gpu_scales(model, w.layers, bits)
        for l in live:
            assert sc1[l]["sx"] == np.float32(np.float64(sc0[l]["sx"]) - lr * dsx1[l])
            assert sc1[l]["ix"] == np.float32(np.float64(sc0[l]["ix"]) - lr * dix1[l])
            np.testing.assert_array_equal(sc1[l]["sw"], (sc0[l]["sw"].astype(np.float64) - lr * np.array(dsw1[l])).astype(np.float32))
            np.testing.assert_array_equal(sc1[l]["iw"], (sc0[l]["iw"].astype(np.float64) - lr * np.array(diw1[l])).astype(np.float32))
        # an evaluation now runs at the adapted scales: bit-identical to the oracle's forward at them
        ys = [torch.empty((w.m, lay.n_out), device="cuda") for lay in w.layers]
        model.eval_config(bits, x, w.m, ys)
        ctx.check_sync()
        taps1 = adj.forward(w.layers, w.weights, bits, w.x, sc1)
        for l in range(n):
            got, ref = ys[l].cpu().numpy(), taps1[l]["y"]
            if int(bits[l]) == 16 or any(int(bits[j]) == 16 for j in range(l + 1)) or w.layers[l].act == orc.ACT_GELU_TANH \
                    or any(w.layers[j].act == orc.ACT_GELU_TANH for j in range(l)):
                assert np.linalg.norm(got - ref) <= 1e-2 * np.linalg.norm(ref)
            else:
                np.testing.assert_array_equal(got.view(np.uint32), ref.view(np.uint32), err_msg=f"{kind} layer {l}")
        # back to max calibration
        model.reset_scales()
        sc_back = _gpu_scales(model, w.layers, bits)
        for l in live:
            assert sc_back[l]["sx"] == sc0[l]["sx"] and np.array_equal(sc_back[l]["iw"], sc0[l]["iw"])
        model.close()
    finally:
        ctx.close()


def test_adjust_argument_errors():
    import paper_2302_01382_b200 as q
    ctx = q.Context(0)
    try:
        w = wl.resnet50(seed=23, batch=1, in_hw=32, width=8, n_classes=8, blocks=(1, 1, 1, 1))
        weights = [torch.from_numpy(a).cuda() for a in w.weights]
        x = torch.from_numpy(w.x).cuda()
        model = q.Model(ctx, w.layers, weights)
        model.calibrate_model(x, w.m)
        with pytest.raises(q.QcfgError) as e:
            model.adjust_scales([8] * len(w.layers), x, w.m, steps=1)
        assert e.value.status == q.ESHAPE
        model.close()
    finally:
        ctx.close()
