"""Pins of the E_N oracle (Eqs. 3-5) against closed forms and structural facts."""
import math

import numpy as np
import pytest

import qcfg_workloads as wl
from oracle import noise_oracle as nz


def _identity_model(k, n):
    # y = x w^T with x the k x k identity: the output IS w^T, so E_N has a closed form
    layers = wl.mlp_layers([k, n])
    return layers, np.eye(k, dtype=np.float32)


def test_single_layer_closed_form_uses_tensor_max_and_standard_deviation():
    """x = I, w and nu small integers, lambda * max|w| a power of two: every value is exact in
    bf16, y* - y = sigma nu^T, so E_N = sigma ||nu||_F / ||w||_F with sigma = lambda * max|w|
    taken over the WHOLE tensor (rows of different magnitude would give another number per row)."""
    layers, x = _identity_model(8, 4)
    rng = np.random.default_rng(0)
    w = rng.integers(-3, 4, (4, 8)).astype(np.float32)
    w[2, 5] = 16.0                                   # the tensor maximum sits in one row only
    nu = rng.integers(-2, 3, (4, 8)).astype(np.float32)
    lam = 0.125                                      # sigma = 2: w + 2 nu are small integers
    e = nz.noise_sensitivity(layers, [w], x, [nu], lam)
    assert e[0] == pytest.approx(2.0 * math.sqrt(float((nu ** 2).sum())) / math.sqrt(float((w ** 2).sum())), rel=1e-12)
    # the sign of the noise does not matter for one linear layer, its scale does, linearly
    assert nz.noise_sensitivity(layers, [w], x, [-nu], lam)[0] == pytest.approx(e[0], rel=1e-12)
    assert nz.noise_sensitivity(layers, [w], x, [nu], 2 * lam)[0] == pytest.approx(2 * e[0], rel=1e-12)


def test_zero_lambda_and_missing_noise_give_zero():
    w = wl.tiny_mlp()
    nus = wl.standard_normal_like(w.weights, 7)
    assert nz.noise_sensitivity(w.layers, w.weights, w.x, nus, 0.0) == [0.0, 0.0, 0.0]
    e = nz.noise_sensitivity(w.layers, w.weights, w.x, [None, nus[1], None], 0.05)
    assert e[0] == 0.0 and e[2] == 0.0 and e[1] > 0.0


def test_only_the_named_tensor_is_perturbed():
    """Eq. 4: a layer whose output nothing downstream reads cannot change the model's output
    (q and k of the synthetic BERT stack), while every layer on the path to the output does."""
    w = wl.bert_stack(5, 48, 32, 64, 1)
    nus = wl.standard_normal_like(w.weights, 8)
    e = nz.noise_sensitivity(w.layers, w.weights, w.x, nus, 0.1)
    names = [l.name for l in w.layers]
    dead = [i for i, l in enumerate(w.layers) if not any(c.src == i or c.residual_from == i for c in w.layers) and i != len(w.layers) - 1]
    assert dead, names
    for i in range(len(w.layers)):
        if i in dead:
            assert e[i] == 0.0, names[i]
        else:
            assert e[i] > 0.0, names[i]


def test_perturbed_weight_rounding_order():
    w = np.array([[1.0, -4.0], [0.5, 2.0]], np.float32)
    nu = np.array([[1.0, 1.0], [-1.0, 3.0]], np.float32)
    lam = np.float32(0.1)
    sigma = np.float32(lam * np.float32(4.0))
    want = np.array([[np.float32(1.0) + sigma, np.float32(-4.0) + sigma], [np.float32(0.5) - sigma, np.float32(2.0) + np.float32(sigma * np.float32(3.0))]], np.float32)
    np.testing.assert_array_equal(nz.perturbed_weight(w, nu, 0.1), want)
    # monotone in lambda for a fixed draw: larger noise, larger first-order output change
    layers, x = _identity_model(2, 2)
    es = [nz.noise_sensitivity(layers, [w], x, [nu], l)[0] for l in (0.01, 0.05, 0.25)]
    assert es[0] < es[1] < es[2]
