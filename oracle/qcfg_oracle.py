"""CPU oracle for the bit-configuration evaluator.  TEST INFRASTRUCTURE, not product code.

A plain, slow, readable numpy statement of what the hot path computes, written from the
paper (Schaefer et al., "Mixed Precision Post Training Quantization of Neural Networks
with Sensitivity Guided Search"): the quantizer of Eq. 1 with max calibration
(Section 3.1), the quantization-error sensitivity of Eq. 2 (Section 3.2), and the
evaluation of a model under one bit configuration (the "Evaluate f(x, w)" step of
Algorithms 1 and 2).  It shares no code with the CUDA path and imports nothing from it.
Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.

Readings of the paper taken here (where it is silent or inconsistent):
  * Eq. 1 clips to [-1, 1] and multiplies by 2^(b-1), which would give 2^b + 1 levels;
    a b-bit signed code holds at most 2^b - 1 symmetric levels, so the grid used is
    +-qmax with qmax = 2^(b-1) - 1.
  * Section 3.1 writes alpha = 1/max(x); Eq. 2 normalises by max|x|.  The absolute
    maximum is used for both.
  * "round" is round-half-to-even.
  * The two scales of Eq. 1 are kept apart: inv_scale = qmax/A multiplies before the
    rounding (alpha * 2^(b-1) in the paper's notation) and scale = A/qmax multiplies
    after it (2^-(b-1) * gamma).  Each comes from ONE IEEE fp32 division.
  * Weights are calibrated per output channel (row), activations per tensor.  With
    per-row scales E_QE sums the squared error over all rows, takes the mean over all
    n elements and normalises by the tensor-wide max|x|; this is Eq. 2 when all rows
    share one scale.
  * "16 bit floating point" layers use bfloat16 operands with wide accumulation.

Parity unpinned (conventions of this build that the paper does not fix, so no value in
the paper can confirm them): the stand-in model graphs (which layer reads which), the
bit width at which E_QE ranks the layers, the scripted accept/reject streams.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
PER_TENSOR = 0
PER_ROW = 1
ACT_NONE, ACT_RELU, ACT_GELU_TANH = 0, 1, 2
POOL_NONE, POOL_MAX3S2, POOL_GLOBAL_AVG = 0, 1, 2


# --------------------------------------------------------------------------- Eq. 1 pieces

def qmax(b: int) -> int:
    """Largest code magnitude of a b-bit symmetric signed grid (reading of Eq. 1)."""
    if not 2 <= b <= 8:
        raise ValueError("integer bit widths are 2..8")
    return 2 ** (b - 1) - 1


def absmax(x: np.ndarray, granularity: int = PER_TENSOR) -> np.ndarray:
    """Max calibration (Section 3.1): A = max|x| over the tensor, or per row."""
    x = np.asarray(x, dtype=F32)
    if granularity == PER_TENSOR:
        return F32(np.max(np.abs(x))) if x.size else F32(0)
    return np.max(np.abs(x.reshape(x.shape[0], -1)), axis=1).astype(F32)


def scales_from_absmax(A, b: int):
    """scale = A/qmax (post-rounding scale), inv_scale = qmax/A (pre-rounding scale).

    One fp32 division each.  A == 0 gives scale = inv_scale = 1 (all codes 0).
    """
    A = np.asarray(A, dtype=F32)
    q = F32(qmax(b))
    zero = A == 0
    safe = np.where(zero, F32(1), A).astype(F32)
    scale = np.where(zero, F32(1), safe / q).astype(F32)
    inv_scale = np.where(zero, F32(1), q / safe).astype(F32)
    return scale, inv_scale


def quantize(x: np.ndarray, inv_scale, b: int) -> np.ndarray:
    """Codes of Eq. 1: round-half-even of x*inv_scale (one fp32 multiply), clipped to +-qmax.

    inv_scale is a scalar (per tensor) or a column vector broadcast over rows (per row).
    """
    t = (np.asarray(x, dtype=F32) * np.asarray(inv_scale, dtype=F32)).astype(F32)
    r = np.rint(t)                      # round-half-to-even in fp32
    qm = F32(qmax(b))
    return np.clip(r, -qm, qm).astype(np.int8)


def dequantize(q: np.ndarray, scale) -> np.ndarray:
    """x_hat = float(q) * scale, one fp32 multiply."""
    return (q.astype(F32) * np.asarray(scale, dtype=F32)).astype(F32)


def fake_quant(x: np.ndarray, b: int, granularity: int) -> np.ndarray:
    """Q(x) of Eq. 1 with max-calibrated scales of x itself."""
    A = absmax(x, granularity)
    scale, inv = scales_from_absmax(A, b)
    if granularity == PER_ROW:
        scale, inv = scale[:, None], inv[:, None]
    return dequantize(quantize(x, inv, b), scale)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (round-to-nearest-even on the bit pattern), returned as fp32."""
    u = np.ascontiguousarray(x, dtype=F32).view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) & 0xFFFF0000).astype(np.uint32)
    return r.view(F32).reshape(np.shape(x))


# --------------------------------------------------------------------------- Eq. 2

def quant_error_sse(x: np.ndarray, b: int, granularity: int = PER_ROW) -> float:
    """Sum over the tensor of (x - Q(x))^2 in fp64 (the expectation of Eq. 2 times n)."""
    x = np.asarray(x, dtype=F32)
    x2 = x.reshape(x.shape[0], -1)
    xh = fake_quant(x2, b, granularity)
    d = x2.astype(np.float64) - xh.astype(np.float64)
    return float(np.sum(d * d))


def e_qe(sse: float, n: int, A_tensor: float) -> float:
    """Eq. 2: sqrt(E[(Q(x)-x)^2]) / max|x|.  Defined as 0 for an all-zero tensor."""
    if A_tensor == 0 or n == 0:
        return 0.0
    return float(np.sqrt(sse / n) / float(A_tensor))


def quant_error_sweep(tensors, granularity: int = PER_ROW, b_lo: int = 2, b_hi: int = 8):
    """All (tensor, b) quantization errors.  Returns (sse[T][nb] fp64, absmax[T] fp32)."""
    nb = b_hi - b_lo + 1
    sse = np.zeros((len(tensors), nb), dtype=np.float64)
    amax = np.zeros(len(tensors), dtype=F32)
    for t, x in enumerate(tensors):
        amax[t] = absmax(x, PER_TENSOR)
        for j in range(nb):
            sse[t, j] = quant_error_sse(x, b_lo + j, granularity)
    return sse, amax


def e_qe_table(sse: np.ndarray, sizes, amax: np.ndarray) -> np.ndarray:
    out = np.zeros_like(sse)
    for t in range(sse.shape[0]):
        for j in range(sse.shape[1]):
            out[t, j] = e_qe(sse[t, j], int(sizes[t]), float(amax[t]))
    return out


def ranking(scores) -> np.ndarray:
    """Layer list sorted ascending by sensitivity (Algorithms 1 and 2), ties by index."""
    return np.argsort(np.asarray(scores, dtype=np.float64), kind="stable")


# --------------------------------------------------------------------------- quantized layer

def int_gemm(qx: np.ndarray, qw: np.ndarray) -> np.ndarray:
    """acc[m][n] = sum_k qx[m][k] * qw[n][k], exact, returned as int32.

    The products are formed in fp64 by the BLAS matmul; every partial sum is an integer
    of magnitude at most K*127^2 < 2^53, so the fp64 result is the exact integer.
    """
    acc = qx.astype(np.float64) @ qw.astype(np.float64).T
    if acc.size and np.max(np.abs(acc)) >= 2.0 ** 31:
        raise OverflowError("int32 accumulator overflow")
    return acc.astype(np.int64).astype(np.int32)


def gelu_tanh(y: np.ndarray) -> np.ndarray:
    """tanh-GELU of the fp32 value y, evaluated in fp64 as y / (1 + exp(-2u)),
    u = sqrt(2/pi) * (y + 0.044715 y^3), which equals 0.5*y*(1 + tanh u); rounded to fp32."""
    y64 = np.asarray(y, dtype=F32).astype(np.float64)
    u = 0.7978845608028654 * (y64 + 0.044715 * y64 * y64 * y64)
    with np.errstate(over="ignore"):
        g = y64 / (1.0 + np.exp(-2.0 * u))
    return g.astype(F32)


def activation(y: np.ndarray, act: int) -> np.ndarray:
    if act == ACT_NONE:
        return y
    if act == ACT_RELU:
        return np.maximum(y, F32(0))
    if act == ACT_GELU_TANH:
        return gelu_tanh(y)
    raise ValueError("unknown activation")


def dequant_output(acc: np.ndarray, scale_x, scale_w: np.ndarray) -> np.ndarray:
    """y = float(acc) * (scale_x * scale_w[n]); two fp32 multiplies, int->float is RNE."""
    c = (F32(scale_x) * np.asarray(scale_w, dtype=F32)).astype(F32)
    return (acc.astype(F32) * c[None, :]).astype(F32)


def bf16_gemm(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """16-bit layer: operands rounded to bfloat16, products and sums in fp64, result fp32."""
    xb = bf16_round(x).astype(np.float64)
    wb = bf16_round(w).astype(np.float64)
    return (xb @ wb.T).astype(F32)


# --------------------------------------------------------------------------- glue (fp32)

def maxpool3s2(x_nhwc: np.ndarray) -> np.ndarray:
    """3x3 max-pool, stride 2, pad 1 (padding never wins the max)."""
    B, H, W, C = x_nhwc.shape
    oh, ow = (H + 2 - 3) // 2 + 1, (W + 2 - 3) // 2 + 1
    xp = np.full((B, H + 2, W + 2, C), -np.inf, dtype=F32)
    xp[:, 1:H + 1, 1:W + 1, :] = x_nhwc
    out = np.full((B, oh, ow, C), -np.inf, dtype=F32)
    for dy in range(3):
        for dx in range(3):
            out = np.maximum(out, xp[:, dy:dy + 2 * oh:2, dx:dx + 2 * ow:2, :])
    return out


def global_avgpool(x_nhwc: np.ndarray) -> np.ndarray:
    """Mean over H*W, summed in fp64 and rounded to fp32."""
    B, H, W, C = x_nhwc.shape
    return (x_nhwc.astype(np.float64).sum(axis=(1, 2)) / float(H * W)).astype(F32)


def im2col(x_nhwc: np.ndarray, kh: int, kw: int, stride: int, pad: int) -> np.ndarray:
    """Patches in (kh, kw, cin) order, zero padded: [B*OH*OW, kh*kw*C]."""
    B, H, W, C = x_nhwc.shape
    oh, ow = (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1
    xp = np.zeros((B, H + 2 * pad, W + 2 * pad, C), dtype=x_nhwc.dtype)
    xp[:, pad:pad + H, pad:pad + W, :] = x_nhwc
    cols = np.empty((B, oh, ow, kh, kw, C), dtype=x_nhwc.dtype)
    for dy in range(kh):
        for dx in range(kw):
            cols[:, :, :, dy, dx, :] = xp[:, dy:dy + stride * oh:stride, dx:dx + stride * ow:stride, :]
    return cols.reshape(B * oh * ow, kh * kw * C)


# --------------------------------------------------------------------------- model evaluation

def layer_input(layers, l: int, x_ext: np.ndarray, outputs) -> np.ndarray:
    """The fp32 tensor layer l reads: a column slice of its producer's output (after the
    producer's activation), pooled if the layer says so.  Linear: [M, K].  Conv: NHWC."""
    lay = layers[l]
    src = x_ext if lay.src < 0 else outputs[lay.src]
    if lay.is_conv or lay.pool_before != POOL_NONE:
        if src.ndim == 2:   # a GEMM output [B*H*W, C] is an NHWC tensor
            B = src.shape[0] // (lay.src_h * lay.src_w)
            src = src.reshape(B, lay.src_h, lay.src_w, src.shape[1])
        if lay.pool_before == POOL_MAX3S2:
            src = maxpool3s2(src)
        elif lay.pool_before == POOL_GLOBAL_AVG:
            src = global_avgpool(src)
        return src
    return src[:, lay.src_col0:lay.src_col0 + lay.k_in]


def gemm_rows(lay, xin: np.ndarray) -> np.ndarray:
    """The [M, K] operand of the layer's GEMM (im2col for a convolution)."""
    if lay.is_conv:
        return im2col(xin, lay.kh, lay.kw, lay.stride, lay.pad)
    return xin


def layer_forward(lay, w: np.ndarray, xin: np.ndarray, b: int, act_absmax, w_absmax,
                  residual=None, taps=None) -> np.ndarray:
    """One layer under bit width b.

    b in 2..8: the input is quantized with the layer's CALIBRATED activation scale (the
    clip of Eq. 1 is live: evaluation values may exceed the calibrated maximum), the
    weight with its per-row scale, the product is an exact integer GEMM, the output is
    rescaled (the 2^-(b-1)*gamma factor of Eq. 1 for both operands), the shortcut is added
    in fp32 and the non-linearity applied.  b = 16: bfloat16 operands, wide accumulation.
    """
    a = gemm_rows(lay, xin)
    if b == 16:
        y = bf16_gemm(a, w)
        if taps is not None:
            taps.update(a=a)
    else:
        sx, ix = scales_from_absmax(act_absmax, b)
        sw, iw = scales_from_absmax(w_absmax, b)
        qx = quantize(a, ix, b)
        qw = quantize(w, iw[:, None], b)
        acc = int_gemm(qx, qw)
        y = dequant_output(acc, sx, sw)
        if taps is not None:
            taps.update(a=a, qx=qx, qw=qw, acc=acc, scale_x=sx, inv_scale_x=ix, scale_w=sw)
    if residual is not None:
        y = (y + residual).astype(F32)
    return activation(y, lay.act)


def calibrate_model(layers, weights, x_ext: np.ndarray):
    """Max calibration of every tensor (Section 3.1) from a forward of the float model:
    every layer at 16 bit.  Returns (act_absmax[l] of each layer's input, w_absmax[l] per row)."""
    outputs, act_amax, w_amax = [], [], []
    for l, lay in enumerate(layers):
        xin = layer_input(layers, l, x_ext, outputs)
        act_amax.append(absmax(xin, PER_TENSOR))
        w_amax.append(absmax(weights[l], PER_ROW))
        res = outputs[lay.residual_from] if lay.residual_from >= 0 else None
        outputs.append(layer_forward(lay, weights[l], xin, 16, None, None, residual=res))
    return act_amax, w_amax


def eval_config(layers, weights, bits, x_ext: np.ndarray, act_amax, w_amax, want_taps=False):
    """Evaluate f(x, w): forward under the bit configuration `bits` (Algorithms 1, 2).
    Returns the list of fp32 layer outputs (and per-layer taps when asked)."""
    outputs, taps = [], []
    for l, lay in enumerate(layers):
        xin = layer_input(layers, l, x_ext, outputs)
        res = outputs[lay.residual_from] if lay.residual_from >= 0 else None
        t = {} if want_taps else None
        outputs.append(layer_forward(lay, weights[l], xin, int(bits[l]), act_amax[l], w_amax[l],
                                     residual=res, taps=t))
        taps.append(t)
    return (outputs, taps) if want_taps else outputs


def eval_layer_teacher_forced(lay, w, xin_gpu: np.ndarray, b: int, act_amax_l, w_amax_l,
                              residual=None, rows=None):
    """One layer recomputed from an input produced elsewhere (teacher forcing).  `rows`
    optionally restricts the GEMM to a sample of rows (rows of a GEMM are independent)."""
    taps = {}
    a = gemm_rows(lay, xin_gpu)
    if rows is not None:
        a = a[rows]
        if residual is not None:
            residual = residual[rows]
    lin = type("L", (), dict(is_conv=False, act=lay.act))()
    y = layer_forward(lin, w, a, b, act_amax_l, w_amax_l, residual=residual, taps=taps)
    return y, taps
