"""Pins for the oracle's scaled layer norm: a library implementation with autograd, brute-force loops,
finite differences, invariants of the normalisation and the table's scale factors."""
import math

import numpy as np
import torch

from oracle import ops as O
from oracle import scales as S


def _case(seed, b=6, n=40, shift=0.7, spread=2.5):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((b, n)) * spread + shift
    w = 1 + 0.3 * rng.standard_normal(n)
    c = 0.2 * rng.standard_normal(n)
    G = rng.standard_normal((b, n))
    return X, w, c, G


def test_forward_and_backward_match_library_layer_norm():
    """torch's CPU layer_norm in float64 and its autograd gradients (another implementation of the
    same definition); the oracle's weight and bias gradients carry beta = b^-1/2 on top."""
    for eps in (0.0, 1e-5):
        X, w, c, G = _case(0)
        Xt, wt, ct = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (X, w, c))
        Y = torch.nn.functional.layer_norm(Xt, (X.shape[1],), wt, ct, eps)
        Y.backward(torch.tensor(G))
        assert np.allclose(O.layer_norm_fwd(X, w, c, eps), Y.detach().numpy(), rtol=1e-12, atol=1e-12)
        dX, dw, dc = O.layer_norm_bwd(X, w, G, eps)
        beta = float(np.float32(X.shape[0] ** -0.5))
        assert np.allclose(dX, Xt.grad.numpy(), rtol=1e-10, atol=1e-12)
        assert np.allclose(dw, beta * wt.grad.numpy(), rtol=1e-10, atol=1e-12)
        assert np.allclose(dc, beta * ct.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_forward_brute_force_from_the_table_formula():
    X, w, c, _ = _case(1, b=3, n=7)
    Y = O.layer_norm_fwd(X, w, c)
    for i in range(3):
        mu = sum(X[i]) / 7
        sigma = math.sqrt(sum(x * x for x in X[i]) / 7 - mu * mu)
        for j in range(7):
            assert abs(Y[i, j] - (c[j] + w[j] * (X[i, j] - mu) / sigma)) < 1e-12


def test_normalised_rows_have_zero_mean_unit_variance_and_ignore_shift_and_scale():
    X, w, c, _ = _case(2, b=9, n=128)
    ones, zeros = np.ones(128), np.zeros(128)
    Y = O.layer_norm_fwd(X, ones, zeros)
    assert np.abs(Y.mean(axis=1)).max() < 1e-13 and np.abs((Y * Y).mean(axis=1) - 1).max() < 1e-12
    assert np.allclose(O.layer_norm_fwd(3.5 * X + 11.0, ones, zeros), Y, atol=1e-10)      # alpha = 1: output scale is fixed
    assert np.allclose(O.layer_norm_fwd(X, w, c), c + w * Y, atol=1e-13)


def test_backward_is_the_scaled_gradient_by_finite_differences():
    X, w, c, G = _case(3, b=4, n=6)
    beta_x, beta_wc = 1.75, 0.3
    dX, dw, dc = O.layer_norm_bwd(X, w, G, 0.0, beta_x, beta_wc)
    f = lambda X_, w_, c_: float(np.sum(G * O.layer_norm_fwd(X_, w_, c_)))
    h = 1e-6
    for i in range(4):
        for j in range(6):
            E = np.zeros_like(X); E[i, j] = h
            fd = (f(X + E, w, c) - f(X - E, w, c)) / (2 * h)
            assert abs(dX[i, j] - beta_x * fd) < 1e-7
    for j in range(6):
        e = np.zeros(6); e[j] = h
        assert abs(dw[j] - beta_wc * (f(X, w + e, c) - f(X, w - e, c)) / (2 * h)) < 1e-7
        assert abs(dc[j] - beta_wc * (f(X, w, c + e) - f(X, w, c - e)) / (2 * h)) < 1e-7


def test_input_gradient_is_orthogonal_to_ones_and_to_the_normalised_row():
    """The normalisation removes the row mean and the row scale, so the input gradient has no component
    along either direction."""
    X, w, c, G = _case(4, b=5, n=64)
    dX, _, _ = O.layer_norm_bwd(X, w, G)
    xhat = O.layer_norm_fwd(X, np.ones(64), np.zeros(64))
    assert np.abs(dX.sum(axis=1)).max() < 1e-12
    assert np.abs((dX * xhat).sum(axis=1)).max() < 1e-12


def test_scale_factors_of_the_table_and_unit_scale_of_the_weight_gradient():
    assert S.layer_norm_scales(8192) == (1.0, 1.0, 8192 ** -0.5, 8192 ** -0.5)
    # with unit-variance G and unit-variance normalised input, sum over b rows has variance b: b^-1/2 restores 1
    rng = np.random.default_rng(5)
    b, n = 4096, 64
    X, G = rng.standard_normal((b, n)), rng.standard_normal((b, n))
    _, dw, dc = O.layer_norm_bwd(X, np.ones(n), G)
    assert abs(dw.std() - 1) < 0.25 and abs(dc.std() - 1) < 0.25
