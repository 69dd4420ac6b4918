"""Prefix reuse between consecutive configurations (the searches change one layer, or a slice of
the ordering, per evaluation): with reuse on, every evaluation of a search sequence must give
bit-identical outputs to a full recompute, while launching fewer kernels."""
import numpy as np
import pytest
import torch

import qcfg_workloads as wl

pytestmark = pytest.mark.gpu


def _sequences(n, rng):
    order = [int(i) for i in rng.permutation(n)]
    accept = rng.random(n) < 0.5
    greedy = wl.greedy_sequence(order, accept)
    bisect = wl.bisection_sequence(order, rng.random(8) < 0.5, max(2, (3 * n) // 4), 8)
    wild = [rng.choice(np.array([4, 8, 16], np.uint8), size=n) for _ in range(6)]
    return greedy[:24] + bisect + wild + [wild[-1], wild[-1]]      # the last two: nothing changes


@pytest.mark.parametrize("kind", ["bert", "bert_wide_qkv", "resnet"])
def test_reuse_is_bit_identical_on_search_sequences(kind):
    import paper_2302_01382_b200 as q
    rng = np.random.default_rng(11)
    if kind == "bert":
        w = wl.bert_stack(21, 640, 256, 1024, 3, bit_choices=None)
    elif kind == "bert_wide_qkv":
        w = wl.bert_stack_wide_qkv(22, 384, 256, 1024, 2)
    else:
        w = wl.resnet50(seed=23, batch=2, in_hw=64, width=16, n_classes=24, blocks=(2, 1, 1, 1))
    n = len(w.layers)
    ctx = q.Context(0)
    try:
        weights = [torch.from_numpy(a).cuda() for a in w.weights]
        x = torch.from_numpy(w.x).cuda()
        model = q.Model(ctx, w.layers, weights)
        model.calibrate_model(x, w.m)
        rows_out = wl.layer_rows(w.layers, n - 1, w.m)
        out_a = torch.empty((rows_out, w.layers[-1].n_out), device="cuda")
        out_b = torch.empty_like(out_a)
        tap = n // 2
        tap_a = torch.empty((wl.layer_rows(w.layers, tap, w.m), w.layers[tap].n_out), device="cuda")
        tap_b = torch.empty_like(tap_a)
        seq = _sequences(n, rng)
        # reference: full recompute of every configuration
        ref, launches_full = [], 0
        for i, bits in enumerate(seq):
            ys = [None] * n
            ys[-1] = out_a
            if i % 5 == 3:
                ys[tap] = tap_a
            l0 = ctx.launch_count()
            model.eval_config(bits, x, w.m, ys)
            launches_full += ctx.launch_count() - l0
            ctx.check_sync()
            ref.append((out_a.clone(), tap_a.clone() if i % 5 == 3 else None))
        ctx.set_prefix_reuse(True)
        launches_reuse = 0
        for i, bits in enumerate(seq):
            ys = [None] * n
            ys[-1] = out_b
            if i % 5 == 3:
                ys[tap] = tap_b
            l0 = ctx.launch_count()
            model.eval_config(bits, x, w.m, ys)
            launches_reuse += ctx.launch_count() - l0
            ctx.check_sync()
            assert torch.equal(out_b, ref[i][0]), f"{kind}: configuration {i} differs under reuse"
            if ref[i][1] is not None:
                assert torch.equal(tap_b, ref[i][1]), f"{kind}: tapped layer differs at configuration {i}"
        assert launches_reuse < launches_full
        # a switch in between invalidates what is kept: the next evaluation is a full one and still right
        ctx.set_fusion(False)
        ys = [None] * n
        ys[-1] = out_b
        model.eval_config(seq[3], x, w.m, ys)
        ctx.check_sync()
        assert torch.equal(out_b, ref[3][0])
        model.close()
    finally:
        ctx.close()
