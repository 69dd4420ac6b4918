"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot run a whole 72- or 144-layer evaluation at full token count in seconds, so
these tests check a seeded sample of rows under teacher forcing (rows of a linear layer are
independent): for every layer the GPU's own fp32 input rows go to the oracle, which must
reproduce the input codes, weight codes, int32 accumulators (bit-exact) and the outputs
(bit-exact, 1e-6 for GELU, 1e-2 normwise for 16-bit layers).  The sweep is checked in full on a
sample of tensors and by its invariants on all of them.
"""
import numpy as np
import pytest
import torch

import qcfg_workloads as wl
from oracle import qcfg_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2302_01382_b200 as q
    c = q.Context(0)
    yield c
    c.close()


def sampled_teacher_forced(ctx, model, w, x, bits, n_rows=256, layers=None):
    rows = np.sort(np.random.default_rng(7).choice(w.m, n_rows, replace=False))
    rows[0], rows[-1] = 0, w.m - 1                       # first and last row of the ragged edges
    rows_d = torch.from_numpy(rows).cuda()
    ys = [torch.full((w.m, lay.n_out), float("nan"), device="cuda") for lay in w.layers]
    model.eval_config(bits, x, w.m, ys)
    ctx.check_sync()
    outs = [y.index_select(0, rows_d).cpu().numpy() for y in ys]
    xs = w.x[rows]
    act_g = np.array(model.act_absmax(), np.float32)
    for l, lay in enumerate(w.layers):
        assert np.all(np.isfinite(outs[l])), f"layer {l}: unwritten output"
        if layers is not None and l not in layers:
            continue
        b = int(bits[l])
        src = xs if lay.src < 0 else outs[lay.src]
        xin = src[:, lay.src_col0:lay.src_col0 + lay.k_in]
        w_amax = orc.absmax(w.weights[l], orc.PER_ROW)
        y_ref, taps = orc.eval_layer_teacher_forced(lay, w.weights[l], xin, b, act_g[l], w_amax)
        if b == 16:
            assert np.linalg.norm(outs[l] - y_ref) <= 1e-2 * np.linalg.norm(y_ref), l
            assert np.abs(outs[l] - y_ref).max() <= 1e-2 * np.abs(y_ref).max(), l
            continue
        qx = torch.empty((w.m, lay.k_in), dtype=torch.int8, device="cuda")
        qw = torch.empty((lay.n_out, lay.k_in), dtype=torch.int8, device="cuda")
        acc = torch.empty((w.m, lay.n_out), dtype=torch.int32, device="cuda")
        model.debug_dump(l, qx, qw, acc)
        ctx.check_sync()
        np.testing.assert_array_equal(qx.index_select(0, rows_d).cpu().numpy(), taps["qx"], err_msg=f"layer {l} input codes")
        np.testing.assert_array_equal(qw.cpu().numpy(), taps["qw"], err_msg=f"layer {l} weight codes")
        np.testing.assert_array_equal(acc.index_select(0, rows_d).cpu().numpy(), taps["acc"], err_msg=f"layer {l} accumulators")
        if lay.act == orc.ACT_GELU_TANH:
            np.testing.assert_allclose(outs[l], y_ref, rtol=1e-6, atol=1e-6 * np.abs(y_ref).max(), err_msg=f"layer {l}")
        else:
            np.testing.assert_array_equal(outs[l].view(np.uint32), y_ref.view(np.uint32), err_msg=f"layer {l}")
    return ys


def build(ctx, w):
    import paper_2302_01382_b200 as q
    weights = [torch.from_numpy(a).cuda() for a in w.weights]
    x = torch.from_numpy(w.x).cuda()
    model = q.Model(ctx, w.layers, weights)
    model.calibrate_model(x, w.m)
    return model, x, weights


def check_sweep(ctx, w, weights, full_on):
    sse, amax = ctx.quant_error_sweep(weights)
    ctx.check_sync()
    sse, amax = sse.cpu().numpy(), amax.cpu().numpy()
    assert np.all(np.diff(sse, axis=1) < 0)                         # error shrinks with every added bit
    for t in range(len(weights)):
        assert amax[t] == np.max(np.abs(w.weights[t]))
    for t in full_on:
        so, ao = orc.quant_error_sweep([w.weights[t]])
        np.testing.assert_allclose(sse[t], so[0], rtol=1e-5)
    for j, b in enumerate(range(2, 9)):                              # bound SSE <= sum_rows n * s^2 / 4
        for t in full_on:
            s, _ = orc.scales_from_absmax(orc.absmax(w.weights[t], orc.PER_ROW), b)
            assert sse[t, j] <= float(np.sum(w.weights[t].shape[1] * s.astype(np.float64) ** 2 / 4)) * (1 + 1e-6)
    sizes = np.array([a.size for a in w.weights], np.float64)
    return np.argsort(np.sqrt(sse[:, 2] / sizes) / amax, kind="stable"), sse, amax


def test_bert_base_block_full(ctx):
    w = wl.bert_base_block()
    assert set(np.unique(w.bits)) <= {4, 8, 16}
    model, x, weights = build(ctx, w)
    sampled_teacher_forced(ctx, model, w, x, w.bits, n_rows=512)
    rank, sse, amax = check_sweep(ctx, w, weights, full_on=range(6))
    so, ao = orc.quant_error_sweep(w.weights)
    eo = orc.e_qe_table(so, [a.size for a in w.weights], ao)
    np.testing.assert_array_equal(rank, orc.ranking(eo[:, 2]))
    model.close()


def test_bert_base_x12_greedy_step(ctx):
    w = wl.bert_base_x12()
    model, x, weights = build(ctx, w)
    rank, sse, amax = check_sweep(ctx, w, weights, full_on=[0, 4, 5, 37, 70, 71])
    seq = wl.greedy_sequence(rank, w.accept)
    assert len(seq) == 72
    # the first and a late configuration of the pass; every layer checked on 256 sampled rows
    sampled_teacher_forced(ctx, model, w, x, seq[0])
    sampled_teacher_forced(ctx, model, w, x, seq[40], layers=set(range(0, 72, 5)))
    model.close()


def test_bert_large_x24_bisection_step(ctx):
    w = wl.bert_large_x24()
    model, x, weights = build(ctx, w)
    rank, sse, amax = check_sweep(ctx, w, weights, full_on=[0, 5, 143])
    seq = wl.bisection_sequence(rank, w.accept, 108, 8)
    assert sorted(set(np.unique(seq[0]))) == [4, 8, 16]
    sampled_teacher_forced(ctx, model, w, x, seq[0], layers=set(range(0, 144, 3)))
    sampled_teacher_forced(ctx, model, w, x, seq[3], layers={0, 1, 2, 3, 4, 5, 70, 71, 142, 143})
    model.close()


def test_resnet50_batch128_sampled_images(ctx):
    """ResNet-50 v1.5 table at batch 128: every layer checked under teacher forcing on two whole
    images (rows of different images are independent), from the GPU's own inputs to that layer."""
    import paper_2302_01382_b200 as q
    w = wl.resnet50()
    assert len(w.layers) == 54 and w.bits[0] == 16 and w.bits[-1] == 16
    weights = [torch.from_numpy(a).cuda() for a in w.weights]
    x = torch.from_numpy(w.x).cuda()
    model = q.Model(ctx, w.layers, weights)
    model.calibrate_model(x, w.m)
    act_g = np.array(model.act_absmax(), np.float32)
    rows_of = [wl.layer_rows(w.layers, l, w.m) for l in range(54)]
    ys = [torch.full((rows_of[l], lay.n_out), float("nan"), device="cuda") for l, lay in enumerate(w.layers)]
    model.eval_config(w.bits, x, w.m, ys)
    ctx.check_sync()
    for img in (0, 127):
        per = [r // w.m for r in rows_of]
        outs = [ys[l][img * per[l]:(img + 1) * per[l]].cpu().numpy() for l in range(54)]
        x_img = w.x[img:img + 1]
        for l, lay in enumerate(w.layers):
            assert np.all(np.isfinite(outs[l])), f"layer {l}: unwritten output"
            b = int(w.bits[l])
            xin = orc.layer_input(w.layers, l, x_img, outs)
            res = outs[lay.residual_from] if lay.residual_from >= 0 else None
            w_amax = orc.absmax(w.weights[l], orc.PER_ROW)
            y_ref, taps = orc.eval_layer_teacher_forced(lay, w.weights[l], xin, b, act_g[l], w_amax, residual=res)
            if b == 16:
                assert np.linalg.norm(outs[l] - y_ref) <= 1e-2 * np.linalg.norm(y_ref), l
                assert np.abs(outs[l] - y_ref).max() <= 1e-2 * np.abs(y_ref).max(), l
                continue
            if img == 0:      # codes and accumulators once per layer (the dumps are whole-batch buffers)
                qx = torch.empty((rows_of[l], lay.k_in), dtype=torch.int8, device="cuda")
                acc = torch.empty((rows_of[l], lay.n_out), dtype=torch.int32, device="cuda")
                model.debug_dump(l, qx, None, acc)
                ctx.check_sync()
                np.testing.assert_array_equal(qx[:per[l]].cpu().numpy(), taps["qx"], err_msg=f"layer {l} input codes")
                np.testing.assert_array_equal(acc[:per[l]].cpu().numpy(), taps["acc"], err_msg=f"layer {l} accumulators")
                del qx, acc
            np.testing.assert_array_equal(outs[l].view(np.uint32), y_ref.view(np.uint32), err_msg=f"layer {l} image {img}")
    model.close()


def test_bench_launch_configuration_gives_the_checked_outputs(ctx):
    """bench.py asks for the last layer's output only, so most layers write nothing but their
    consumers' codes (fast epilogue bodies) and the GEMMs go out as chains.  The teacher-forced
    checks above ask for every layer's output.  Here the two meet: for configurations of the greedy
    pass and one with 16-bit layers, the last layer's output of the benchmark's configuration (chains
    on and off) equals, bit for bit, the one of the every-output evaluation."""
    w = wl.bert_base_x12()
    model, x, weights = build(ctx, w)
    n = len(w.layers)
    rank = np.arange(n)
    seq = wl.greedy_sequence(rank, w.accept)
    mixed = np.array([16 if i % 7 == 3 else (4 if i % 3 == 0 else 8) for i in range(n)], dtype=np.uint8)
    last = torch.empty((w.m, w.layers[-1].n_out), device="cuda")
    try:
        for bits in (seq[0], seq[40], seq[71], mixed):
            ys = [torch.full((w.m, lay.n_out), float("nan"), device="cuda") for lay in w.layers]
            model.eval_config(bits, x, w.m, ys)
            ctx.check_sync()
            ref = ys[-1].cpu().numpy()
            del ys
            assert np.all(np.isfinite(ref))
            for chained in (True, False):
                ctx.set_gemm_chains(chained)
                last.fill_(float("nan"))
                n0 = ctx.launch_count()
                model.eval_config(bits, x, w.m, [None] * (n - 1) + [last])
                ctx.check_sync()
                launches = ctx.launch_count() - n0
                np.testing.assert_array_equal(last.cpu().numpy().view(np.uint32), ref.view(np.uint32),
                                              err_msg=f"chains {chained}")
                if chained and not np.any(np.asarray(bits) == 16):
                    assert launches <= 5, launches          # one input quantization and three chains
    finally:
        ctx.set_gemm_chains(True)
        model.close()
