"""Parity of whole configuration evaluations with the CPU oracle, through the C-ABI.

Primary gate: layer-wise teacher forcing.  For every layer the test downloads the fp32
input the GPU actually fed to it, lets the oracle recompute scale, codes, int32 accumulators
and output from that input, and requires codes, scale bit patterns and accumulators to be
bit-exact, outputs to be bit-exact (no activation / ReLU), within 1e-6 relative with a floor
of 1e-6 * max|y| (GELU), or within 1e-2 normwise (16-bit layers).  End-to-end chained outputs
are compared with float tolerances; the ReLU-only integer model must be bit-exact end to end.
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


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.detach().cpu().numpy()


def build(ctx, w):
    import paper_2302_01382_b200 as q
    weights = [dev(a) for a in w.weights]
    model = q.Model(ctx, w.layers, weights)
    x = dev(w.x.reshape(w.x.shape[0], -1) if w.x.ndim == 2 else w.x)
    model.calibrate_model(x, w.m)
    return model, x


def run_eval(ctx, model, w, x, bits):
    ys = [torch.full((wl.layer_rows(w.layers, l, w.m), lay.n_out), float("nan"), device="cuda")
          for l, lay in enumerate(w.layers)]
    model.eval_config(bits, x, w.m, ys)
    ctx.check_sync()
    return ys


def check_calibration(model, w):
    act_o, w_o = orc.calibrate_model(w.layers, w.weights, w.x)
    act_g = np.array(model.act_absmax(), np.float32)
    # the 16-bit forward accumulates in fp32 on the GPU and fp64 in the oracle: maxima agree to
    # bf16-product accumulation accuracy, not bit for bit (except for external inputs)
    for l, lay in enumerate(w.layers):
        if lay.src < 0 and lay.pool_before == 0:
            assert act_g[l] == act_o[l]
        else:
            assert act_g[l] == pytest.approx(float(act_o[l]), rel=2e-3)
        np.testing.assert_array_equal(np.array(model.weight_absmax(l), np.float32), w_o[l])
    return act_g, w_o


def teacher_forced_check(ctx, model, w, x, bits, ys, act_g, w_amax, sample_rows=None):
    outs = [host(y) for y in ys]
    for o in outs:
        assert np.all(np.isfinite(o)), "an output element was never written"
    for l, lay in enumerate(w.layers):
        b = int(bits[l])
        xin = orc.layer_input(w.layers, l, w.x, outs)          # built from the GPU's own outputs
        res = outs[lay.residual_from] if lay.residual_from >= 0 else None
        rows = None
        if sample_rows is not None and outs[l].shape[0] > sample_rows:
            rows = np.sort(np.random.default_rng(l).choice(outs[l].shape[0], sample_rows, replace=False))
        y_ref, taps = orc.eval_layer_teacher_forced(lay, w.weights[l], xin, b, act_g[l], w_amax[l], residual=res, rows=rows)
        y_gpu = outs[l] if rows is None else outs[l][rows]
        if b == 16:
            assert np.linalg.norm(y_gpu - y_ref) <= 1e-2 * max(np.linalg.norm(y_ref), 1e-30), l
            assert np.abs(y_gpu - y_ref).max() <= 1e-2 * max(np.abs(y_ref).max(), 1e-30), l
            continue
        m_rows, k = outs[l].shape[0], lay.k_in
        qx = torch.empty((m_rows, k), dtype=torch.int8, device="cuda")
        qw = torch.empty((lay.n_out, k), dtype=torch.int8, device="cuda")
        acc = torch.empty((m_rows, lay.n_out), dtype=torch.int32, device="cuda")
        model.debug_dump(l, qx, qw, acc)
        ctx.check_sync()
        qx, acc = host(qx), host(acc)
        if rows is not None:
            qx, acc = qx[rows], acc[rows]
        np.testing.assert_array_equal(qx, taps["qx"], err_msg=f"layer {l} input codes")
        np.testing.assert_array_equal(host(qw), taps["qw"], err_msg=f"layer {l} weight codes")
        np.testing.assert_array_equal(acc, taps["acc"], err_msg=f"layer {l} accumulators")
        if lay.act == orc.ACT_GELU_TANH:
            np.testing.assert_allclose(y_gpu, y_ref, rtol=1e-6, atol=1e-6 * np.abs(y_ref).max(), err_msg=f"layer {l}")
        else:
            np.testing.assert_array_equal(y_gpu.view(np.uint32), y_ref.view(np.uint32), err_msg=f"layer {l}")


def test_tiny_mlp_bit_exact_end_to_end(ctx):
    w = wl.tiny_mlp()
    model, x = build(ctx, w)
    act_g, w_amax = check_calibration(model, w)
    ys = run_eval(ctx, model, w, x, w.bits)
    teacher_forced_check(ctx, model, w, x, w.bits, ys, act_g, w_amax)
    # chained oracle with the GPU's calibration table: integers and ReLU only -> bit-exact
    outs = orc.eval_config(w.layers, w.weights, w.bits, w.x, list(act_g), w_amax)
    for l in range(3):
        np.testing.assert_array_equal(host(ys[l]), outs[l])
    model.close()


@pytest.mark.parametrize("fuse", [True, False])
@pytest.mark.parametrize("seed,m,hidden,ffn,blocks", [(11, 300, 192, 768, 2), (12, 1100, 256, 1024, 1)])
def test_bert_stack_teacher_forced(ctx, fuse, seed, m, hidden, ffn, blocks):
    ctx.set_fusion(fuse)
    try:
        w = wl.bert_stack(seed, m, hidden, ffn, blocks)
        model, x = build(ctx, w)
        act_g, w_amax = check_calibration(model, w)
        for bits in (w.bits, [8] * len(w.layers), [4, 8, 16, 3, 16, 2] * blocks):
            ys = run_eval(ctx, model, w, x, bits)
            teacher_forced_check(ctx, model, w, x, bits, ys, act_g, w_amax)
            # end to end against the chained oracle: float tolerance only (GELU, bf16 layers)
            outs = orc.eval_config(w.layers, w.weights, bits, w.x, list(act_g), w_amax)
            last = host(ys[-1])
            assert np.linalg.norm(last - outs[-1]) <= 2e-2 * np.linalg.norm(outs[-1])
        model.close()
    finally:
        ctx.set_fusion(True)


@pytest.mark.parametrize("fuse", [True, False])
def test_column_slice_consumers_teacher_forced(ctx, fuse):
    """One wide projection layer (3h output channels) whose column thirds are read by three
    consumers through src_col0 = 0, h, 2h: calibration maxima, input codes, accumulators and
    outputs of every slice reader against the oracle, and the wide layer's thirds against three
    separate projections with the same weight rows."""
    ctx.set_fusion(fuse)
    try:
        h, ffn, m = 192, 768, 333
        w = wl.bert_stack_wide_qkv(33, m, h, ffn, 2)
        model, x = build(ctx, w)
        act_g, w_amax = check_calibration(model, w)
        for bits in (w.bits, [8] * len(w.layers), [4, 8, 16, 3, 16, 2] * 2, [16, 8, 4, 8, 8, 8] * 2):
            ys = run_eval(ctx, model, w, x, bits)
            teacher_forced_check(ctx, model, w, x, bits, ys, act_g, w_amax)
        ys8 = run_eval(ctx, model, w, x, [8] * len(w.layers))
        model.close()
        # all-8: the wide layer's thirds equal three separate projections
        sep = wl.Workload("sep", 33, wl.bert_layers(h, ffn, 2), m, w.x, [], bits=np.full(12, 8, np.uint8))
        for blk in range(2):
            wide = w.weights[6 * blk]
            sep.weights += [wide[:h], wide[h:2 * h], wide[2 * h:]] + w.weights[6 * blk + 3:6 * blk + 6]
        model_s, xs = build(ctx, sep)
        ys_s = run_eval(ctx, model_s, sep, xs, sep.bits)
        for blk in range(2):
            for j in range(3):
                assert torch.equal(ys8[6 * blk][:, j * h:(j + 1) * h], ys_s[6 * blk + j])
            for j in (3, 4, 5):
                assert torch.equal(ys8[6 * blk + j], ys_s[6 * blk + j])
        model_s.close()
    finally:
        ctx.set_fusion(True)


def test_fused_and_unfused_agree_bitwise_and_taps_are_optional(ctx):
    w = wl.bert_stack(21, 515, 128, 512, 2, bit_choices=(4, 8))
    model, x = build(ctx, w)
    ys_f = run_eval(ctx, model, w, x, w.bits)
    ctx.set_fusion(False)
    ys_u = run_eval(ctx, model, w, x, w.bits)
    ctx.set_fusion(True)
    for a, b in zip(ys_f, ys_u):
        assert torch.equal(a, b)
    # only the last layer requested: same values
    ys = [None] * (len(w.layers) - 1) + [torch.empty_like(ys_f[-1])]
    model.eval_config(w.bits, x, w.m, ys)
    ctx.check_sync()
    assert torch.equal(ys[-1], ys_f[-1])
    model.eval_config(w.bits, x, w.m, None)
    ctx.check_sync()
    model.close()


@pytest.mark.parametrize("bits_kind", ["uniform8", "mixed_int", "with16"])
def test_grouped_and_single_launches_agree_bitwise(ctx, bits_kind):
    """The three projections of a block read one input: when their GEMMs have the same shape and
    operand type they run as one grouped launch (also with different bit widths, i.e. different
    input codes and scales per group); a 16-bit layer among them splits the group."""
    w = wl.bert_stack(23, 700, 256, 1024, 2, bit_choices=(4, 8))
    n = len(w.layers)
    bits = {"uniform8": [8] * n, "mixed_int": [4, 8, 6, 8, 3, 8] * 2, "with16": [8, 16, 8, 4, 16, 8] * 2}[bits_kind]
    model, x = build(ctx, w)
    res = []
    for grouping in (True, False):
        ctx.set_grouping(grouping)
        try:
            ys = run_eval(ctx, model, w, x, bits)
        finally:
            ctx.set_grouping(True)
        res.append(ys)
    for a, b in zip(*res):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    act_g = np.array(model.act_absmax(), np.float32)
    w_amax = [np.array(model.weight_absmax(l), np.float32) for l in range(n)]
    teacher_forced_check(ctx, model, w, x, bits, res[0], act_g, w_amax)
    model.close()


def test_model_argument_errors(ctx):
    import paper_2302_01382_b200 as q
    w = wl.tiny_mlp()
    weights = [dev(a) for a in w.weights]
    model = q.Model(ctx, w.layers, weights)
    x = dev(w.x)
    with pytest.raises(q.QcfgError) as e:
        model.eval_config(w.bits, x, w.m)
    assert e.value.status == q.ESTATE
    model.calibrate_model(x, w.m)
    with pytest.raises(q.QcfgError) as e:
        model.eval_config([8, 9, 8], x, w.m)
    assert e.value.status == q.EBITS
    bad = [wl.Layer("a", 8, 16), wl.Layer("b", 8, 16, src=0)]      # reads 16 columns of an 8-wide output
    with pytest.raises(q.QcfgError) as e:
        q.Model(ctx, bad, [torch.zeros((8, 16), device="cuda")] * 2)
    assert e.value.status == q.ESHAPE
    xn = x.clone()
    xn[3, 3] = float("nan")
    with pytest.raises(q.QcfgError) as e:
        model.calibrate_model(xn, w.m)
    assert e.value.status == q.ENONFINITE
    model.close()


@pytest.mark.parametrize("fuse", [True, False])
def test_resnet_small_teacher_forced(ctx, fuse):
    """Convolutional table at reduced size: im2col operands (3-channel 7x7/2 stem, 3x3 with stride 1
    and 2, 1x1 with stride 1 and 2), max-pool, shortcuts, global average pool, 16-bit stem and fc."""
    ctx.set_fusion(fuse)
    try:
        w = wl.resnet50(seed=3, batch=3, in_hw=64, width=16, n_classes=10, blocks=(2, 1, 2, 1))
        model, x = build(ctx, w)
        act_g, w_amax = check_calibration(model, w)
        for bits in (w.bits, [8] * len(w.layers)):
            ys = run_eval(ctx, model, w, x, bits)
            teacher_forced_check(ctx, model, w, x, bits, ys, act_g, w_amax)
        outs = orc.eval_config(w.layers, w.weights, w.bits, w.x, list(act_g), w_amax)
        last = host(ys[-1])
        ref_all8 = orc.eval_config(w.layers, w.weights, [8] * len(w.layers), w.x, list(act_g), w_amax)
        assert np.linalg.norm(last - ref_all8[-1]) <= 2e-2 * np.linalg.norm(ref_all8[-1])
        model.close()
    finally:
        ctx.set_fusion(True)


@pytest.mark.parametrize("fuse", [True, False])
def test_implicit_and_materialised_convolutions_agree_bitwise(ctx, fuse):
    """The GEMM that gathers its patches from the input's NHWC codes gives, layer by layer, the same
    bits as the GEMM on a materialised patch matrix: 3x3 with stride 1 and 2, strided 1x1, channel
    counts of one to several 16-byte chunks, int8 and 16-bit layers, ragged last row tiles."""
    for width, batch, hw in ((16, 3, 64), (48, 2, 40)):
        w = wl.resnet50(seed=5, batch=batch, in_hw=hw, width=width, n_classes=10, blocks=(2, 1, 1, 1))
        model, x = build(ctx, w)
        model.calibrate_model(x, w.m)
        n = len(w.layers)
        with16 = np.array(w.bits).copy()
        with16[3::4] = 16
        for bits in (w.bits, [8] * n, with16):
            outs = {}
            for implicit in (True, False):
                ctx.set_implicit_conv(implicit)
                ctx.set_fusion(fuse)
                ys = run_eval(ctx, model, w, x, bits)
                outs[implicit] = [host(y) for y in ys]
            for l in range(n):
                np.testing.assert_array_equal(outs[True][l].view(np.uint32), outs[False][l].view(np.uint32),
                                              err_msg=f"width {width} layer {l} ({w.layers[l].name})")
        ctx.set_implicit_conv(True)
        ctx.set_fusion(True)
        model.close()


@pytest.mark.parametrize("m", [19200, 19000])
def test_chained_and_separate_launches_agree_bitwise(ctx, m):
    """A forward pass whose GEMMs go to the device as chains (one cooperative launch for up to sixteen
    consecutive GEMMs, tiles started by per-row-tile counters; a GEMM joins a chain only if it has at
    least one tile per CTA pair, hence the row counts) gives the same bits as one launch
    per GEMM: all-int8, a mix with 4-bit and 16-bit layers (both operand types chain), every
    output requested (general epilogue) and only the last one (fast epilogue bodies), whole and
    ragged last row tiles.  The launch counter shows that the chains were in fact used."""
    w = wl.bert_stack(11, m, 256, 1024, 3, bit_choices=None)
    model, x = build(ctx, w)
    n = len(w.layers)
    mixed = [16 if i % 5 == 4 else (4 if i % 3 == 0 else 8) for i in range(n)]
    last = torch.empty((m, w.layers[-1].n_out), device="cuda")
    try:
        for bits in ([8] * n, mixed, [16] * n):
            outs, lasts, launches = {}, {}, {}
            for chained in (True, False):
                ctx.set_gemm_chains(chained)
                ys = run_eval(ctx, model, w, x, bits)
                outs[chained] = [host(y) for y in ys]
                last.fill_(float("nan"))
                n0 = ctx.launch_count()
                model.eval_config(bits, x, m, [None] * (n - 1) + [last])
                ctx.check_sync()
                launches[chained] = ctx.launch_count() - n0
                lasts[chained] = host(last).copy()
            for l in range(n):
                np.testing.assert_array_equal(outs[True][l].view(np.uint32), outs[False][l].view(np.uint32),
                                              err_msg=f"layer {l} ({w.layers[l].name}) bits {bits[l]}")
            np.testing.assert_array_equal(lasts[True].view(np.uint32), lasts[False].view(np.uint32))
            assert np.all(np.isfinite(lasts[True]))
            assert launches[True] < launches[False], launches
    finally:
        ctx.set_gemm_chains(True)
        model.close()


def test_calibration_maxima_do_not_depend_on_fusion_or_chaining(ctx):
    """The calibration forward may take an activation's range in the epilogue of the GEMM that
    produces it (fusion on: the 16-bit operand codes come from there too, and the GEMMs chain) or in
    the kernel that builds the 16-bit operand (fusion off).  Both read the same fp32 values and fold
    bit patterns with an integer maximum, so the tables agree bit for bit."""
    w = wl.bert_stack(5, 19200, 256, 1024, 2, bit_choices=None)
    model, x = build(ctx, w)
    try:
        tables = {}
        for fuse in (True, False):
            for chained in (True, False):
                ctx.set_fusion(fuse)
                ctx.set_gemm_chains(chained)
                model.calibrate_model(x, w.m)
                tables[(fuse, chained)] = np.array(model.act_absmax(), np.float32)
        ref = tables[(False, False)]
        assert np.all(ref > 0)
        for key, t in tables.items():
            np.testing.assert_array_equal(t.view(np.uint32), ref.view(np.uint32), err_msg=str(key))
    finally:
        ctx.set_fusion(True)
        ctx.set_gemm_chains(True)
        model.close()
