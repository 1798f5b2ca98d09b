"""Pins for the oracle's softmax cross-entropy: library log-softmax, finite differences, and the table's
beta = s / sqrt(s - 1) giving a unit-scale gradient at initialisation."""
import numpy as np
from scipy import special

from oracle import ops as O
from oracle import scales as S


def test_forward_is_the_library_log_softmax_at_the_target():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((9, 37)) * 4
    X[0] += 900.0                                                   # no overflow
    t = rng.integers(0, 37, 9)
    ref = special.log_softmax(X, axis=-1)[np.arange(9), t]
    assert np.allclose(O.softmax_xent_fwd(X, t), ref, rtol=1e-12, atol=1e-12)
    assert (O.softmax_xent_fwd(X, t) <= 0).all()
    # brute force on one row
    x = X[3]
    assert abs(O.softmax_xent_fwd(X, t)[3] - np.log(np.exp(x[t[3]]) / np.exp(x).sum())) < 1e-12


def test_backward_is_beta_times_the_gradient_and_sums_to_zero():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((4, 7))
    t = rng.integers(0, 7, 4)
    g = rng.standard_normal(4)
    beta = 2.5
    dX = O.softmax_xent_bwd(X, t, g, beta)
    h = 1e-6
    for i in range(4):
        for j in range(7):
            E = np.zeros_like(X); E[i, j] = h
            fd = (np.sum(g * O.softmax_xent_fwd(X + E, t)) - np.sum(g * O.softmax_xent_fwd(X - E, t))) / (2 * h)
            assert abs(dX[i, j] - beta * fd) < 1e-8
    assert np.abs(dX.sum(axis=1)).max() < 1e-14                     # onehot - softmax sums to zero


def test_table_beta_gives_unit_scale_at_initialisation():
    """Near-uniform predictions: (onehot - p) has mean square (s - 1) / s^2 per element, so beta = s / sqrt(s - 1)."""
    s = 1000
    assert S.softmax_xent_scales(s) == (1.0, s / np.sqrt(s - 1))
    rng = np.random.default_rng(2)
    X = rng.standard_normal((256, s)) * 0.01
    t = rng.integers(0, s, 256)
    dX = O.softmax_xent_bwd(X, t, np.ones(256), S.softmax_xent_scales(s)[1])
    assert abs(np.sqrt(np.mean(dX ** 2)) - 1) < 0.01
