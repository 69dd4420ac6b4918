"""CPU oracle of the scale-adjustment step (test infrastructure: only tests, the smoke check and
the benchmark's CPU baseline may import this package).

Section 3.1, second step of the scale estimation ("adjustment"): after max calibration the
quantization scales are adapted by backpropagation to lower the model loss on the calibration
data, the model's own parameters staying untouched; Section 4 gives the learning rate 1e-5.

What is written here, step by step:
  * the forward of a model under a bit configuration with EXPLICIT scales (the two scales of
    Eq. 1 kept apart: inv_scale before the rounding, scale after it), using the quantizer,
    integer GEMM and rescale of `qcfg_oracle` unchanged;
  * the loss  L = sum (y - y_ref)^2 / sum y_ref^2  on the last layer's output, y_ref being the
    output of the 16-bit model;
  * its gradient with respect to every scale, in fp64, with the straight-through estimator for
    the rounding (d round(t)/dt := 1) and the exact derivative of the clip (0 where clipped);
  * one plain gradient-descent step on the scales.

Readings where the paper is silent:
  * optimizer: plain gradient descent (no momentum), one step per call, full batch;
  * which scales: all four kinds -- activation scale and inv_scale per layer, weight scale and
    inv_scale per output channel -- of the layers that run at an integer width; 16-bit layers have
    no scales and get none;
  * rounding: straight-through; the 16-bit rounding of operands is passed through as the identity;
  * graphs: linear layers with optional shortcut adds and column-slice consumers (the convolutional
    table is not covered).

Parity unpinned: the loss.  The paper minimises the model's task loss, which needs labels; the
output-distance used here is this build's convention (the arithmetic around it is pinned by finite
differences on a rounding-free surrogate, closed forms and structural checks).
"""
from __future__ import annotations

import numpy as np

from . import qcfg_oracle as orc

F32 = np.float32
F64 = np.float64


def calibrated_scales(layers, weights, bits, act_amax, w_amax):
    """The starting point: the max-calibrated scales of every integer layer (None for 16 bit)."""
    out = []
    for l, lay in enumerate(layers):
        b = int(bits[l])
        if b == 16:
            out.append(None)
            continue
        sx, ix = orc.scales_from_absmax(act_amax[l], b)
        sw, iw = orc.scales_from_absmax(w_amax[l], b)
        out.append({"sx": F32(sx), "ix": F32(ix), "sw": sw.astype(F32).copy(), "iw": iw.astype(F32).copy()})
    return out


def _codes(t: np.ndarray, b: int, soft: bool) -> np.ndarray:
    """Codes of Eq. 1 from the pre-scaled values t = x * inv_scale (fp32).  soft=True leaves out the
    rounding (a smooth surrogate used only to check the gradient code by finite differences)."""
    qm = float(orc.qmax(b))
    if soft:
        return np.clip(t.astype(F64), -qm, qm)
    return np.clip(np.rint(t), -qm, qm).astype(F64)


def _activation64(y: np.ndarray, act: int) -> np.ndarray:
    """The activations in fp64 (surrogate forward only)."""
    if act == orc.ACT_NONE:
        return y
    if act == orc.ACT_RELU:
        return np.maximum(y, 0.0)
    u = 0.7978845608028654 * (y + 0.044715 * y ** 3)
    return y / (1.0 + np.exp(-2.0 * u))


def forward(layers, weights, bits, x_ext, scales, soft: bool = False):
    """Forward with explicit scales.  Returns per layer a dict of what the backward pass needs:
    xin (fp32 input), t (pre-scaled input), qx, qw (codes as fp64), y_lin (rescaled accumulators),
    y_pre (after the shortcut add), y (after the activation).  With soft=False and calibrated
    scales the outputs equal qcfg_oracle.eval_config's bit for bit."""
    taps, outputs = [], []
    for l, lay in enumerate(layers):
        if lay.is_conv or lay.pool_before != orc.POOL_NONE:
            raise ValueError("adjust oracle: linear layers only")
        b = int(bits[l])
        w = weights[l]
        if soft:          # everything in fp64, no rounding anywhere: a smooth function of the scales
            xin = orc.layer_input(layers, l, np.asarray(x_ext, F64), outputs)
            if b == 16:
                y_lin = xin @ w.astype(F64).T
                tap = {"xin": xin, "wq": w.astype(F64), "bits": 16}
            else:
                sc = scales[l]
                tx, tw = xin * F64(sc["ix"]), w.astype(F64) * sc["iw"].astype(F64)[:, None]
                qx, qw = _codes(tx, b, True), _codes(tw, b, True)
                y_lin = (qx @ qw.T) * (F64(sc["sx"]) * sc["sw"].astype(F64))[None, :]
                tap = {"xin": xin, "tx": tx, "tw": tw, "qx": qx, "qw": qw, "bits": b}
            y_pre = y_lin + outputs[lay.residual_from] if lay.residual_from >= 0 else y_lin
            y = _activation64(y_pre, lay.act)
            tap.update(y_lin=y_lin, y_pre=y_pre, y=y)
            taps.append(tap)
            outputs.append(y)
            continue
        xin = orc.layer_input(layers, l, x_ext, outputs).astype(F32)
        if b == 16:
            xb, wb = orc.bf16_round(xin).astype(F64), orc.bf16_round(w).astype(F64)
            y_lin = (xb @ wb.T).astype(F32)
            tap = {"xin": xin, "wq": wb, "bits": 16}
        else:
            sc = scales[l]
            tx = (xin * F32(sc["ix"])).astype(F32)
            tw = (w.astype(F32) * sc["iw"][:, None].astype(F32)).astype(F32)
            qx, qw = _codes(tx, b, False), _codes(tw, b, False)
            acc = orc.int_gemm(qx.astype(np.int8), qw.astype(np.int8))
            y_lin = orc.dequant_output(acc, sc["sx"], sc["sw"])
            tap = {"xin": xin, "tx": tx, "tw": tw, "qx": qx, "qw": qw, "bits": b}
        y_pre = y_lin
        if lay.residual_from >= 0:
            y_pre = (y_lin + outputs[lay.residual_from]).astype(F32)
        y = orc.activation(y_pre, lay.act)
        tap.update(y_lin=y_lin, y_pre=y_pre, y=y)
        taps.append(tap)
        outputs.append(y)
    return taps


def loss(y: np.ndarray, y_ref: np.ndarray) -> float:
    """L = sum (y - y_ref)^2 / sum y_ref^2 in fp64."""
    d = y.astype(F64) - y_ref.astype(F64)
    return float(np.sum(d * d) / np.sum(y_ref.astype(F64) ** 2))


def _act_grad(y_pre: np.ndarray, act: int) -> np.ndarray:
    """d act(y)/dy at the fp32 pre-activation values, in fp64."""
    y = y_pre.astype(F64)
    if act == orc.ACT_NONE:
        return np.ones_like(y)
    if act == orc.ACT_RELU:
        return (y > 0).astype(F64)
    if act == orc.ACT_GELU_TANH:
        c, a = 0.7978845608028654, 0.044715
        u = c * (y + a * y ** 3)
        with np.errstate(over="ignore"):
            sig = 1.0 / (1.0 + np.exp(-2.0 * u))
        return sig + y * sig * (1.0 - sig) * 2.0 * c * (1.0 + 3.0 * a * y * y)
    raise ValueError("unknown activation")


def gradients(layers, weights, bits, scales, taps, y_ref):
    """dL/d(scale) for every scale, by backpropagation through the taps of `forward`.

    Returns a list (per layer) of None (16-bit layer) or {"sx", "ix", "sw"[n], "iw"[n]} in fp64.
    Straight-through rounding: d q/d t = 1 inside the clip range, 0 outside."""
    n = len(layers)
    y_last = taps[-1]["y"].astype(F64)
    norm2 = float(np.sum(y_ref.astype(F64) ** 2))
    g_out = [None] * n                                   # dL/d(output of layer l), accumulated over its readers
    g_out[n - 1] = 2.0 * (y_last - y_ref.astype(F64)) / norm2
    grads = [None] * n
    for l in range(n - 1, -1, -1):
        lay, tap = layers[l], taps[l]
        if g_out[l] is None:                             # nothing downstream reaches the loss
            if tap["bits"] != 16:
                k = weights[l].shape[0]
                grads[l] = {"sx": 0.0, "ix": 0.0, "sw": np.zeros(k), "iw": np.zeros(k)}
            continue
        g_pre = g_out[l] * _act_grad(tap["y_pre"], lay.act)          # through the activation
        if lay.residual_from >= 0:                                    # the shortcut passes it on unchanged
            r = lay.residual_from
            g_out[r] = g_pre.copy() if g_out[r] is None else g_out[r] + g_pre
        if tap["bits"] == 16:
            g_x = g_pre @ tap["wq"]                                   # rounding to bf16 passed through
        else:
            sc = scales[l]
            sx, ix = float(sc["sx"]), float(sc["ix"])
            sw, iw = sc["sw"].astype(F64), sc["iw"].astype(F64)
            qm = float(orc.qmax(tap["bits"]))
            qx, qw = tap["qx"], tap["qw"]
            acc = qx @ qw.T
            # y_lin[m, n] = acc[m, n] * sx * sw[n]
            d_sx = float(np.sum(g_pre * acc * sw[None, :]))
            d_sw = np.sum(g_pre * acc, axis=0) * sx
            # codes: y_lin = sum_k (sx qx[m,k]) (sw[n] qw[n,k])
            g_qx = (g_pre * sw[None, :]) @ qw * sx                    # dL/d qx
            g_qw = (g_pre * sw[None, :]).T @ qx * sx                  # dL/d qw
            in_x = (np.abs(tap["tx"].astype(F64)) <= qm).astype(F64)  # derivative of the clip
            in_w = (np.abs(tap["tw"].astype(F64)) <= qm).astype(F64)
            xin, w = tap["xin"].astype(F64), weights[l].astype(F64)
            d_ix = float(np.sum(g_qx * in_x * xin))                   # qx ~ clip(x * ix)
            d_iw = np.sum(g_qw * in_w * w, axis=1)
            g_x = g_qx * in_x * ix
            grads[l] = {"sx": d_sx, "ix": d_ix, "sw": d_sw, "iw": d_iw}
        if lay.src >= 0:
            p = lay.src
            if g_out[p] is None:
                g_out[p] = np.zeros(taps[p]["y"].shape, F64)
            g_out[p][:, lay.src_col0:lay.src_col0 + lay.k_in] += g_x
    return grads


def sgd_step(scales, grads, lr: float):
    """scale <- fp32(scale - lr * gradient), every scale of every integer layer; returns new scales."""
    out = []
    for sc, g in zip(scales, grads):
        if sc is None:
            out.append(None)
            continue
        out.append({"sx": F32(F64(sc["sx"]) - lr * g["sx"]), "ix": F32(F64(sc["ix"]) - lr * g["ix"]),
                    "sw": (sc["sw"].astype(F64) - lr * g["sw"]).astype(F32),
                    "iw": (sc["iw"].astype(F64) - lr * g["iw"]).astype(F32)})
    return out


def adjust(layers, weights, bits, x_ext, act_amax, w_amax, steps: int, lr: float = 1e-5):
    """The adjustment step: `steps` gradient-descent steps on the scales from their calibrated
    values.  Returns (scales, losses) with losses[i] the loss before step i and losses[steps] the
    final one.  The model's weights are read, never written."""
    n = len(layers)
    ref_taps = forward(layers, weights, [16] * n, x_ext, [None] * n)
    y_ref = ref_taps[-1]["y"]
    scales = calibrated_scales(layers, weights, bits, act_amax, w_amax)
    losses = []
    for _ in range(steps):
        taps = forward(layers, weights, bits, x_ext, scales)
        losses.append(loss(taps[-1]["y"], y_ref))
        scales = sgd_step(scales, gradients(layers, weights, bits, scales, taps, y_ref), lr)
    losses.append(loss(forward(layers, weights, bits, x_ext, scales)[-1]["y"], y_ref))
    return scales, losses
