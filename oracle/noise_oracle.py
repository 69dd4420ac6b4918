"""CPU oracle of the noise-injection sensitivity E_N (test infrastructure: only tests, the smoke
check and the benchmark's CPU baseline may import this package).

Section 3.1, Eqs. 3-5: E_N(i) = L(x, W*) - L(x, W), where W* is W with nu ~ N(0, lambda max|w_i|)
added to tensor w_i alone.  Readings: the second argument of N is the standard deviation; max|w_i|
is the whole tensor's maximum; the loss (the paper's needs labels) is the relative L2 distance of
the last layer's output from the noise-free output, so L(x, W) = 0; the model is the 16-bit
floating-point baseline.  The standard-normal draws are inputs.

Parity unpinned: the loss.  The paper's L needs labels; the output-distance proxy used here is this
build's convention, so no value in the paper can pin it (the arithmetic around it is pinned).
"""
import numpy as np

from . import qcfg_oracle as orc

F32 = np.float32


def perturbed_weight(w: np.ndarray, nu: np.ndarray, lam: float) -> np.ndarray:
    """w_i + nu (Eq. 4, 5): deviation lambda * max|w_i| and the sum in fp32, one rounding per operation."""
    sigma = F32(lam) * F32(np.max(np.abs(w))) if w.size else F32(0)
    return (w.astype(F32) + (F32(sigma) * nu.astype(F32)).astype(F32)).astype(F32)


def noise_sensitivity(layers, weights, x_ext: np.ndarray, noises, lam: float):
    """E_N of every layer (0 where noises[i] is None)."""
    n = len(layers)
    bits = [16] * n
    none = [None] * n
    y0 = orc.eval_config(layers, weights, bits, x_ext, none, none)[-1].astype(np.float64)
    ref = np.sqrt(np.sum(y0 * y0))
    out = []
    for i in range(n):
        if noises[i] is None:
            out.append(0.0)
            continue
        ws = list(weights)
        ws[i] = perturbed_weight(weights[i], noises[i], lam)        # Eq. 4: only w_i is replaced
        y = orc.eval_config(layers, ws, bits, x_ext, none, none)[-1].astype(np.float64)
        d = np.sqrt(np.sum((y - y0) ** 2))
        out.append(float(d / ref) if ref > 0 else (0.0 if d == 0 else float("inf")))   # Eq. 3 with L(x, W) = 0
    return out
