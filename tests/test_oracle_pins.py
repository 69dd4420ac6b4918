"""Pins for the CPU oracle: closed forms, invariants, library routines and brute force.

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong
sign or index, a transposed operand, a wrong rounding rule) makes it fail.  None of them
needs a GPU and none calls the CUDA path.
"""
import math
import os

import numpy as np
import pytest
import torch

import qcfg_workloads as wl
from oracle import qcfg_oracle as orc
from oracle import cost_oracle as cost

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
BITS = list(range(2, 9))


def _golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append(line.split())
    return rows


# ----------------------------------------------------------------------- absmax and scales

@pytest.mark.parametrize("b", BITS)
def test_absmax_element_maps_to_qmax(b):
    rng = np.random.default_rng(b)
    for _ in range(200):
        x = (rng.standard_normal(257) * 10.0 ** rng.uniform(-6, 6)).astype(np.float32)
        A = orc.absmax(x)
        s, inv = orc.scales_from_absmax(A, b)
        q = orc.quantize(x, inv, b)
        i = int(np.argmax(np.abs(x)))
        assert abs(int(q[i])) == orc.qmax(b)
        assert int(np.sign(q[i])) == int(np.sign(x[i]))
        assert abs(float(s) * float(inv) - 1.0) < 3 * 2.0 ** -23


def test_absmax_is_absolute_and_per_row():
    x = np.array([[1.0, -7.0, 3.0], [-0.5, 0.25, 0.125]], dtype=np.float32)
    assert orc.absmax(x) == np.float32(7.0)            # a signed max would give 3
    np.testing.assert_array_equal(orc.absmax(x, orc.PER_ROW), np.array([7.0, 0.5], np.float32))


def test_zero_tensor_is_defined():
    x = np.zeros((3, 4), np.float32)
    s, inv = orc.scales_from_absmax(orc.absmax(x), 4)
    assert s == 1 and inv == 1
    assert not orc.quantize(x, inv, 4).any()
    sse, amax = orc.quant_error_sweep([x])
    assert not sse.any() and amax[0] == 0
    assert orc.e_qe(0.0, 12, 0.0) == 0.0


# ----------------------------------------------------------------------- quantizer (Eq. 1)

@pytest.mark.parametrize("b", BITS)
def test_levels_monotone_odd(b):
    rng = np.random.default_rng(100 + b)
    x = np.sort(rng.standard_normal(20000).astype(np.float32) * 3)
    _, inv = orc.scales_from_absmax(orc.absmax(x), b)
    q = orc.quantize(x, inv, b).astype(np.int32)
    assert len(np.unique(q)) <= 2 ** b - 1
    assert q.min() >= -orc.qmax(b) and q.max() <= orc.qmax(b)
    assert np.all(np.diff(q) >= 0)
    np.testing.assert_array_equal(orc.quantize(-x, inv, b).astype(np.int32), -q)


@pytest.mark.parametrize("b", BITS)
def test_idempotent_all_codes(b):
    rng = np.random.default_rng(7)
    codes = np.arange(-orc.qmax(b), orc.qmax(b) + 1, dtype=np.int8)
    for _ in range(300):
        A = np.float32(10.0 ** rng.uniform(-8, 8))
        s, inv = orc.scales_from_absmax(A, b)
        np.testing.assert_array_equal(orc.quantize(orc.dequantize(codes, s), inv, b), codes)


@pytest.mark.parametrize("b", [3, 4, 8])
def test_ties_round_to_even_and_clip(b):
    qm = orc.qmax(b)
    A = np.float32(qm * 0.25)                 # scale = 0.25 and inv_scale = 4 exactly
    s, inv = orc.scales_from_absmax(A, b)
    assert s == np.float32(0.25) and inv == np.float32(4.0)
    k = np.arange(-qm, qm, dtype=np.float32)
    x = (k + np.float32(0.5)) * np.float32(0.25)      # exact ties
    q = orc.quantize(x, inv, b).astype(np.int32)
    assert np.all(q % 2 == 0)
    assert np.all(np.abs(q - (k + 0.5)) == 0.5)
    big = np.array([10 * A, -10 * A], np.float32)     # beyond the calibrated range
    np.testing.assert_array_equal(orc.quantize(big, inv, b), np.array([qm, -qm], np.int8))


@pytest.mark.parametrize("b", BITS)
def test_fake_quant_matches_library_on_exact_scales(b):
    """With a power-of-two scale both the oracle and torch's fake-quantize are exact."""
    rng = np.random.default_rng(b)
    qm = orc.qmax(b)
    rows = np.array([qm * 2.0 ** -3, qm * 2.0 ** -5, qm * 2.0 ** 1], np.float32)
    x = rng.uniform(-1, 1, size=(3, 500)).astype(np.float32) * rows[:, None]
    x[:, 0] = rows                                      # the row maxima
    got = orc.fake_quant(x, b, orc.PER_ROW)
    scale = torch.tensor(rows / qm)
    want = torch.fake_quantize_per_channel_affine(torch.from_numpy(x), scale,
                                                  torch.zeros(3, dtype=torch.int32), 0, -qm, qm)
    np.testing.assert_array_equal(got, want.numpy())


def test_bf16_round_matches_library_everywhere():
    hi = np.arange(2 ** 16, dtype=np.uint32) << 16
    lows = np.array([0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF], np.uint32)
    u = (hi[:, None] | lows[None, :]).reshape(-1)
    x = u.view(np.float32)
    finite = np.isfinite(x)
    got = orc.bf16_round(x[finite])
    want = torch.from_numpy(x[finite].copy()).to(torch.bfloat16).to(torch.float32).numpy()
    ok = np.isfinite(want)                              # rounding up to inf is out of scope
    np.testing.assert_array_equal(got[ok].view(np.uint32), want[ok].view(np.uint32))


# ----------------------------------------------------------------------- E_QE (Eq. 2)

def test_uniform_closed_form():
    n = 1 << 20
    A = 3.0
    x = (np.linspace(-A, A, n, dtype=np.float64)).astype(np.float32)[None, :]
    sse, amax = orc.quant_error_sweep([x], orc.PER_TENSOR)
    for b, want in _golden("uniform_eqe.txt"):
        got = orc.e_qe(sse[0, int(b) - 2], n, amax[0])
        assert got == pytest.approx(float(want), rel=2e-3), b


def test_sse_bound_decreasing_and_zero_on_grid():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((37, 301)).astype(np.float32) * rng.uniform(0.1, 10, (37, 1)).astype(np.float32)
    sse, amax = orc.quant_error_sweep([x], orc.PER_ROW)
    assert np.all(np.diff(sse[0]) < 0)
    for j, b in enumerate(BITS):
        s, _ = orc.scales_from_absmax(orc.absmax(x, orc.PER_ROW), b)
        bound = float(np.sum(x.shape[1] * s.astype(np.float64) ** 2 / 4))
        assert sse[0, j] <= bound * (1 + 1e-6)
        xg = orc.fake_quant(x, b, orc.PER_ROW)            # already on the b-bit grid
        assert orc.quant_error_sse(xg, b, orc.PER_ROW) <= 1e-12 * float(np.sum(xg.astype(np.float64) ** 2))


def test_sse_brute_force_small():
    rng = np.random.default_rng(11)
    x = rng.standard_normal((3, 5)).astype(np.float32)
    sse, amax = orc.quant_error_sweep([x], orc.PER_ROW)
    for j, b in enumerate(BITS):
        qm = 2 ** (b - 1) - 1
        tot = 0.0
        for r in range(3):
            A = max(abs(float(v)) for v in x[r])
            for v in x[r]:
                v = float(v)
                code = max(-qm, min(qm, round(v * qm / A)))      # python round: half-even
                tot += (v - code * A / qm) ** 2
        assert sse[0, j] == pytest.approx(tot, rel=1e-5)
    assert float(amax[0]) == max(abs(float(v)) for v in x.reshape(-1))


def test_per_row_reduces_to_per_tensor_and_eqe_normalisation():
    rng = np.random.default_rng(5)
    x = rng.uniform(-1, 1, (8, 64)).astype(np.float32)
    x[:, 3] = np.float32(2.0) * np.where(np.arange(8) % 2, 1, -1)   # every row has absmax 2
    for b in (2, 5, 8):
        assert orc.quant_error_sse(x, b, orc.PER_ROW) == orc.quant_error_sse(x, b, orc.PER_TENSOR)
    sse = orc.quant_error_sse(x, 4, orc.PER_TENSOR)
    e = orc.e_qe(sse, x.size, 2.0)
    assert e == pytest.approx(math.sqrt(sse / x.size) / 2.0, rel=1e-12)
    # scale invariance of Eq. 2 under power-of-two rescaling of the tensor (exact in fp32)
    sse4 = orc.quant_error_sse(x * np.float32(4), 4, orc.PER_TENSOR)
    assert orc.e_qe(sse4, x.size, 8.0) == pytest.approx(e, rel=1e-12)


def test_ranking_stable_ascending():
    r = orc.ranking([0.3, 0.1, 0.3, 0.05, 0.1])
    np.testing.assert_array_equal(r, [3, 1, 4, 0, 2])


# ----------------------------------------------------------------------- integer GEMM

def test_int_gemm_brute_force_and_library():
    rng = np.random.default_rng(2)
    qx = rng.integers(-127, 128, (5, 19), dtype=np.int8)
    qw = rng.integers(-127, 128, (7, 19), dtype=np.int8)
    acc = orc.int_gemm(qx, qw)
    assert acc.dtype == np.int32 and acc.shape == (5, 7)
    for m in range(5):
        for n in range(7):
            assert int(acc[m, n]) == sum(int(qx[m, k]) * int(qw[n, k]) for k in range(19))
    qx = rng.integers(-127, 128, (33, 300), dtype=np.int8)
    qw = rng.integers(-127, 128, (21, 300), dtype=np.int8)
    np.testing.assert_array_equal(orc.int_gemm(qx, qw), qx.astype(np.int64) @ qw.astype(np.int64).T)


def test_int_gemm_worst_case_magnitude():
    K = 4608
    qx = np.full((2, K), 127, np.int8)
    qw = np.stack([np.full(K, 127, np.int8), np.full(K, -127, np.int8)])
    acc = orc.int_gemm(qx, qw)
    assert acc[0, 0] == K * 127 * 127 and acc[1, 1] == -K * 127 * 127


# ----------------------------------------------------------------------- epilogue

def test_gelu_identity_limits_and_library():
    y = np.concatenate([np.linspace(-12, 12, 4001), [0.0, 50.0, -50.0, 1e4, -1e4]]).astype(np.float32)
    g = orc.gelu_tanh(y)
    assert np.all(np.isfinite(g))
    y64 = y.astype(np.float64)
    ref = 0.5 * y64 * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (y64 + 0.044715 * y64 ** 3)))
    np.testing.assert_allclose(g, ref, rtol=1e-6, atol=1e-12)
    lib = torch.nn.functional.gelu(torch.from_numpy(y64), approximate="tanh").numpy()
    np.testing.assert_allclose(g, lib, rtol=1e-6, atol=1e-12)
    assert orc.gelu_tanh(np.float32(0)) == 0
    assert orc.gelu_tanh(np.float32(50)) == np.float32(50)
    assert orc.gelu_tanh(np.float32(-50)) == 0


def test_dequant_and_relu_exact():
    acc = np.array([[3, -5], [2 ** 24 + 1, -7]], np.int32)
    sw = np.array([0.5, 0.25], np.float32)
    y = orc.dequant_output(acc, np.float32(2.0), sw)
    np.testing.assert_array_equal(y, np.array([[3.0, -2.5], [float(np.float32(2 ** 24 + 1)), -3.5]], np.float32))
    np.testing.assert_array_equal(orc.activation(y, orc.ACT_RELU)[:, 1], [0, 0])


# ----------------------------------------------------------------------- layers and chains

def test_bf16_layer_matches_library_matmul():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((40, 96)).astype(np.float32)
    w = rng.standard_normal((24, 96)).astype(np.float32)
    got = orc.bf16_gemm(x, w)
    xb = torch.from_numpy(x).to(torch.bfloat16).double()
    wb = torch.from_numpy(w).to(torch.bfloat16).double()
    np.testing.assert_allclose(got, (xb @ wb.T).numpy(), rtol=1e-6, atol=1e-6)
    full = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.linalg.norm(got - full) / np.linalg.norm(full) < 1e-2


@pytest.mark.parametrize("k,stride,pad", [(1, 1, 0), (1, 2, 0), (3, 1, 1), (3, 2, 1), (7, 2, 3)])
def test_conv_as_im2col_matches_library(k, stride, pad):
    rng = np.random.default_rng(k * 10 + stride)
    B, H, W, C, N = 2, 13, 11, 5, 6
    x = orc.bf16_round(rng.standard_normal((B, H, W, C)).astype(np.float32))
    w = orc.bf16_round(rng.standard_normal((N, k, k, C)).astype(np.float32))     # OHWI
    lay = wl.Layer("c", N, k * k * C, kh=k, kw=k, stride=stride, pad=pad, in_h=H, in_w=W, in_c=C)
    y = orc.bf16_gemm(orc.gemm_rows(lay, x), w.reshape(N, -1))
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double().permute(0, 3, 1, 2),
                                     torch.from_numpy(w).double().permute(0, 3, 1, 2),
                                     stride=stride, padding=pad)
    ref = ref.permute(0, 2, 3, 1).reshape(-1, N).numpy()
    assert y.shape == (B * lay.out_h * lay.out_w, N)
    np.testing.assert_allclose(y, ref, rtol=1e-5, atol=1e-5)


def test_pools_match_library():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 9, 12, 3)).astype(np.float32)
    t = torch.from_numpy(x).permute(0, 3, 1, 2)
    mp = torch.nn.functional.max_pool2d(t, 3, 2, 1).permute(0, 2, 3, 1).numpy()
    np.testing.assert_array_equal(orc.maxpool3s2(x), mp)
    ap = t.double().mean(dim=(2, 3)).float().numpy()
    np.testing.assert_allclose(orc.global_avgpool(x), ap, rtol=1e-6)


def test_quantized_layer_tracks_float_layer():
    """A quantized layer approximates the float product with an error that shrinks with b;
    a transposed operand, a missing scale or a wrong dequantization would break this."""
    rng = np.random.default_rng(4)
    x = rng.standard_normal((64, 128)).astype(np.float32)
    w = (rng.standard_normal((48, 128)) * 0.05).astype(np.float32)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    lay = wl.Layer("l", 48, 128)
    errs = []
    for b in (4, 6, 8):
        y = orc.layer_forward(lay, w, x, b, orc.absmax(x), orc.absmax(w, orc.PER_ROW))
        errs.append(np.linalg.norm(y - ref) / np.linalg.norm(ref))
    assert errs[0] > errs[1] > errs[2]
    assert errs[2] < 0.02 and errs[0] < 0.35


def test_chain_all16_equals_calibration_forward_and_taps_consistent():
    w = wl.bert_stack(seed=5, m=24, hidden=32, ffn=64, n_blocks=2)
    act_amax, w_amax = orc.calibrate_model(w.layers, w.weights, w.x)
    outs16 = orc.eval_config(w.layers, w.weights, [16] * 12, w.x, act_amax, w_amax)
    # the calibrated activation maxima are the maxima of the 16-bit forward's layer inputs
    for l, lay in enumerate(w.layers):
        src = w.x if lay.src < 0 else outs16[lay.src]
        assert act_amax[l] == np.max(np.abs(src))
    outs, taps = orc.eval_config(w.layers, w.weights, w.bits, w.x, act_amax, w_amax, want_taps=True)
    for l, lay in enumerate(w.layers):
        if w.bits[l] == 16:
            continue
        t = taps[l]
        src = w.x if lay.src < 0 else outs[lay.src]
        np.testing.assert_array_equal(t["a"], src)
        y, t2 = orc.eval_layer_teacher_forced(lay, w.weights[l], src, int(w.bits[l]), act_amax[l], w_amax[l])
        np.testing.assert_array_equal(y, outs[l])
        np.testing.assert_array_equal(t2["acc"], t["acc"])
    # dependence structure of the stand-in graph: V feeds O, Q/K feed nobody
    assert w.layers[3].src == 2 and w.layers[4].src == 3 and w.layers[6].src == 5
    assert all(l.src not in (0, 1) for l in w.layers)


def test_resnet_chain_small_runs_and_residual_is_used():
    w = wl.resnet50(seed=3, batch=1, in_hw=32, width=8, n_classes=10, blocks=(1, 1, 1, 1))
    act_amax, w_amax = orc.calibrate_model(w.layers, w.weights, w.x)
    outs = orc.eval_config(w.layers, w.weights, w.bits, w.x, act_amax, w_amax)
    assert outs[-1].shape == (1, 10)
    assert all(np.all(np.isfinite(o)) for o in outs)
    c = next(i for i, l in enumerate(w.layers) if l.residual_from >= 0)
    lay = w.layers[c]
    xin = orc.layer_input(w.layers, c, w.x, outs)
    no_res = orc.layer_forward(lay, w.weights[c], xin, int(w.bits[c]), act_amax[c], w_amax[c])
    assert not np.array_equal(no_res, outs[c])
    assert np.all(outs[c] >= 0)


def test_e_qe_table_is_e_qe_elementwise():
    sse = np.array([[4.0, 1.0, 0.25], [9.0, 0.0, 16.0], [1.0, 1.0, 1.0]])
    sizes = [4, 9, 100]
    amax = np.array([2.0, 0.5, 0.0], np.float32)           # the last tensor is all zero
    tab = orc.e_qe_table(sse, sizes, amax)
    # Eq. 2 by hand: sqrt(sse/n)/A
    want = np.array([[0.5, 0.25, 0.125], [2.0, 0.0, 8.0 / 3.0], [0.0, 0.0, 0.0]])
    np.testing.assert_allclose(tab, want, rtol=1e-15)
    for t in range(3):
        for j in range(3):
            assert tab[t, j] == orc.e_qe(sse[t, j], sizes[t], float(amax[t]))


@pytest.mark.parametrize("b", [3, 4, 8])
def test_layer_forward_exact_on_grid_with_unequal_row_scales(b):
    """Inputs and weights that already lie on their b-bit grids with power-of-two scales: every
    step of the quantized layer is then exact, so its output must equal the real product bit for
    bit.  The weight rows have maxima 2^8 apart, so a per-row scale taken from the wrong row, a
    per-tensor weight scale, a transposed operand or a dropped activation scale all fail."""
    rng = np.random.default_rng(40 + b)
    qm = orc.qmax(b)
    M, K, N = 9, 24, 5
    cx = rng.integers(-qm, qm + 1, (M, K)).astype(np.float64)
    cx[2, 7] = -qm                                         # the activation maximum
    cw = rng.integers(-qm, qm + 1, (N, K)).astype(np.float64)
    cw[np.arange(N), (3 * np.arange(N) + 1) % K] = qm * np.array([1, -1, 1, -1, 1])   # every row reaches +-qmax
    e_x = -4
    e_w = np.array([-3, 1, -7, 0, -5])
    x = (cx * 2.0 ** e_x).astype(np.float32)
    w = (cw * 2.0 ** e_w[:, None]).astype(np.float32)
    lay = wl.Layer("l", N, K)
    taps = {}
    y = orc.layer_forward(lay, w, x, b, orc.absmax(x), orc.absmax(w, orc.PER_ROW), taps=taps)
    np.testing.assert_array_equal(taps["qx"], cx.astype(np.int8))
    np.testing.assert_array_equal(taps["qw"], cw.astype(np.int8))
    np.testing.assert_array_equal(taps["scale_w"], (2.0 ** e_w).astype(np.float32))
    assert taps["scale_x"] == np.float32(2.0 ** e_x)
    want = x.astype(np.float64) @ w.astype(np.float64).T   # exact: integers times powers of two
    np.testing.assert_array_equal(y.astype(np.float64), want)


def test_layer_forward_shortcut_relu_and_clip_by_hand():
    """2 x 2 x 2 case written out: the shortcut is added before the ReLU, and an input beyond the
    CALIBRATED maximum is clipped (the activation scale is the calibrated one, not the input's)."""
    lay = wl.Layer("l", 2, 2, act=orc.ACT_RELU)
    b = 4                                                  # qmax 7
    x = np.array([[1.0, -0.5], [3.5, 0.25]], np.float32)   # calibrated max 1.75 -> scale 0.25; 3.5 clips to 7
    w = np.array([[7.0, -7.0], [0.5, 3.5]], np.float32)    # row maxima 7 and 3.5 -> scales 1 and 0.5
    res = np.array([[-30.0, 0.125], [1.0, -100.0]], np.float32)
    # codes: x -> [[4, -2], [7, 1]];  w -> [[7, -7], [1, 7]]
    # acc  = [[4*7 + 2*7, 4*1 - 2*7], [7*7 - 1*7, 7*1 + 1*7]] = [[42, -10], [42, 14]]
    # y    = acc * 0.25 * [1, 0.5]   = [[10.5, -1.25], [10.5, 1.75]]
    # + res                          = [[-19.5, -1.125], [11.5, -98.25]];  ReLU -> [[0, 0], [11.5, 0]]
    taps = {}
    y = orc.layer_forward(lay, w, x, b, np.float32(1.75), orc.absmax(w, orc.PER_ROW), residual=res, taps=taps)
    np.testing.assert_array_equal(taps["qx"], np.array([[4, -2], [7, 1]], np.int8))
    np.testing.assert_array_equal(taps["acc"], np.array([[42, -10], [42, 14]], np.int32))
    np.testing.assert_array_equal(y, np.array([[0.0, 0.0], [11.5, 0.0]], np.float32))
    lay_none = wl.Layer("l", 2, 2)
    y2 = orc.layer_forward(lay_none, w, x, b, np.float32(1.75), orc.absmax(w, orc.PER_ROW), residual=res)
    np.testing.assert_array_equal(y2, np.array([[-19.5, -1.125], [11.5, -98.25]], np.float32))


def test_conv_pool_reshape_chain_matches_library():
    """layer_input's convolution / pooling / reshape branch, value by value: a 7x7/2 stem, a 3x3/2
    max-pool, a 1x1 convolution, a 3x3/2 convolution and a global-average-pooled linear layer on a
    NON-square image, every layer at 16 bit.  Inputs and weights are small integers, so every
    product, sum and bf16 rounding is exact and the library's convolutions must agree bit for bit.
    A swapped height/width in the reshape, a wrong pooling window or a wrong patch order fails."""
    F = torch.nn.functional
    rng = np.random.default_rng(77)
    B, H, W = 2, 20, 14
    L = [
        wl.Layer("stem", 6, 7 * 7 * 3, src=-1, act=wl.ACT_RELU, kh=7, kw=7, stride=2, pad=3, in_h=H, in_w=W, in_c=3,
                 src_h=H, src_w=W),                                                        # -> 10 x 7
        wl.Layer("p1", 4, 6, src=0, act=wl.ACT_RELU, kh=1, kw=1, stride=1, pad=0, in_h=5, in_w=4, in_c=6,
                 pool_before=wl.POOL_MAX3S2, src_h=10, src_w=7),                            # pool -> 5 x 4
        wl.Layer("c3", 5, 3 * 3 * 4, src=1, act=wl.ACT_NONE, kh=3, kw=3, stride=2, pad=1, in_h=5, in_w=4, in_c=4,
                 src_h=5, src_w=4),                                                        # -> 3 x 2
        wl.Layer("fc", 3, 5, src=2, pool_before=wl.POOL_GLOBAL_AVG, src_h=3, src_w=2),
    ]
    x = rng.integers(-3, 4, (B, H, W, 3)).astype(np.float32)
    ws = [rng.integers(-2, 3, (l.n_out, l.k_in)).astype(np.float32) for l in L]
    outs = orc.eval_config(L, ws, [16] * 4, x, [None] * 4, [None] * 4)

    def bf(t):
        return t.float().to(torch.bfloat16).double()

    def conv(t, w, lay):
        w4 = torch.from_numpy(w).double().reshape(lay.n_out, lay.kh, lay.kw, lay.in_c).permute(0, 3, 1, 2)
        return F.conv2d(bf(t), bf(w4), stride=lay.stride, padding=lay.pad).float()

    t = torch.from_numpy(x).permute(0, 3, 1, 2)                       # NCHW
    y0 = torch.relu(conv(t, ws[0], L[0]))
    assert y0.shape[2:] == (10, 7)
    y1 = torch.relu(conv(F.max_pool2d(y0, 3, 2, 1), ws[1], L[1]))
    assert y1.shape[2:] == (5, 4)
    y2 = conv(y1, ws[2], L[2])
    assert y2.shape[2:] == (3, 2)
    y3 = (bf(y2.double().mean(dim=(2, 3)).float()) @ bf(torch.from_numpy(ws[3])).T).float()
    for got, want in zip(outs[:3], (y0, y1, y2)):
        np.testing.assert_array_equal(got, want.permute(0, 2, 3, 1).reshape(-1, want.shape[1]).numpy())
    np.testing.assert_array_equal(outs[3], y3.numpy())
    assert float(np.abs(outs[2]).max()) > 100                        # the chain is not trivially zero


def test_column_slice_consumers_equal_separate_projections():
    """src_col0: a layer of 3h output channels whose thirds are read by three consumers must give
    what three separate h-channel layers with the same weight rows give (rows of a product are
    independent, per-row weight scales do not mix rows).  Ignoring src_col0, or slicing rows
    instead of columns, makes the consumer of the last third read the wrong tensor."""
    h, ffn, m = 16, 48, 21
    ww = wl.bert_stack_wide_qkv(31, m, h, ffn, 2, bit_choices=(4, 8))
    sep = wl.bert_layers(h, ffn, 2)
    w_sep, bits_sep = [], []
    for blk in range(2):
        wide = ww.weights[6 * blk]
        w_sep += [wide[:h], wide[h:2 * h], wide[2 * h:], ww.weights[6 * blk + 3], ww.weights[6 * blk + 4], ww.weights[6 * blk + 5]]
        bq = int(ww.bits[6 * blk])
        bits_sep += [bq, bq, bq] + [int(v) for v in ww.bits[6 * blk + 3:6 * blk + 6]]
    act_w, wam_w = orc.calibrate_model(ww.layers, ww.weights, ww.x)
    act_s, wam_s = orc.calibrate_model(sep, w_sep, ww.x)
    outs_w = orc.eval_config(ww.layers, ww.weights, ww.bits, ww.x, act_w, wam_w)
    outs_s = orc.eval_config(sep, w_sep, bits_sep, ww.x, act_s, wam_s)
    for blk in range(2):
        base = 6 * blk
        wide = outs_w[base]
        for j in range(3):
            np.testing.assert_array_equal(wide[:, j * h:(j + 1) * h], outs_s[base + j])
        for j in (3, 4, 5):
            np.testing.assert_array_equal(outs_w[base + j], outs_s[base + j])
            assert act_w[base + j] == act_s[base + j]
        # what each slice reader was fed, by manual slicing
        for j, lay_idx in enumerate((base + 1, base + 2, base + 3)):
            xin = orc.layer_input(ww.layers, lay_idx, ww.x, outs_w)
            np.testing.assert_array_equal(xin, wide[:, j * h:(j + 1) * h])
            assert act_w[lay_idx] == np.max(np.abs(orc.eval_config(ww.layers, ww.weights, [16] * 12, ww.x, act_w, wam_w)[base][:, j * h:(j + 1) * h]))
    assert not np.array_equal(outs_w[0][:, :h], outs_w[0][:, 2 * h:])


# ----------------------------------------------------------------------- tables and sequences

def test_layer_tables_match_table1_sizes():
    res = wl.resnet50_layers()
    bert = wl.bert_layers(1024, 4096, 24)
    assert len(res) == 54 and wl.param_count(res) == 25_502_912
    assert len(bert) == 144 and wl.param_count(bert) == 301_989_888
    assert wl.param_count(wl.bert_layers(768, 3072, 12)) == 84_934_656
    tables = {"resnet50": res, "bert": bert}
    for model, b, mb in _golden("table1_sizes.txt"):
        L = tables[model]
        assert wl.size_mb(L, [int(b)] * len(L)) == pytest.approx(float(mb), abs=0.0075)
        assert cost.size_bytes(L, [int(b)] * len(L)) / 1e6 == pytest.approx(float(mb), abs=0.0075)


def test_cost_oracle_latency_is_the_selected_entries_sum_and_size_is_linear_in_bits():
    L = wl.mlp_layers([256, 256, 256, 10])
    table = [[1.0, 2.0, 4.0], [8.0, 16.0, 32.0], [64.0, 128.0, 256.0]]      # distinct powers of two: the sum names its terms
    assert cost.latency_ms(table, [4, 8, 16], [4, 8, 16]) == 1.0 + 16.0 + 256.0
    assert cost.latency_ms(table, [4, 8, 16], [16, 4, 8]) == 4.0 + 8.0 + 128.0
    assert cost.latency_ms(table, [16, 8, 4], [4, 4, 4]) == 4.0 + 32.0 + 256.0    # columns follow bs, not the width
    with pytest.raises(KeyError):
        cost.latency_ms(table, [4, 8, 16], [4, 2, 16])
    # hand count: 256*256 + 256*256 + 10*256 parameters
    assert cost.size_bytes(L, [8, 8, 8]) == 256 * 256 * 2 + 2560
    assert cost.size_bytes(L, [4, 8, 16]) == 256 * 256 * 0.5 + 256 * 256 + 2560 * 2
    assert cost.size_bytes(L, [2, 2, 2]) * 8 == cost.size_bytes(L, [16, 16, 16])


def test_search_sequences_follow_the_algorithms():
    n = 72
    rank = np.random.default_rng(0).permutation(n)
    acc = np.random.default_rng(1).random(n) < 0.5
    seq = wl.greedy_sequence(rank, acc)
    assert len(seq) == n                                   # one evaluation per layer per bit width
    for i, cfg in enumerate(seq):
        assert cfg[rank[i]] == 4
        kept = [rank[j] for j in range(i) if acc[j]]
        dropped = [rank[j] for j in range(i) if not acc[j]]
        assert np.all(cfg[kept] == 4) and np.all(cfg[dropped] == 8)
    rank = np.arange(144)
    seq = wl.bisection_sequence(rank, [True, False, True, True, False, False, True, True], 108, 8)
    counts = [int(np.sum(c == 4)) for c in seq]
    assert counts[:4] == [54, 81, 68, 74]                  # +27, -(27//2), +(13//2): floor halving
    assert all(int(np.sum(c == 16)) == 36 for c in seq)
    assert len(seq) <= 3 * math.ceil(math.log2(144)) + 3
