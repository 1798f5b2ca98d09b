"""Pins for the oracle's scaled softmax: library softmax, invariants, finite differences."""
import numpy as np
from scipy import special

from oracle import ops as O


def test_softmax_matches_library_and_sums_to_alpha():
    rng = np.random.default_rng(0)
    S = rng.standard_normal((7, 33)) * 3
    P = O.softmax_fwd(S, 33.0)
    assert np.allclose(P, 33.0 * special.softmax(S, axis=-1), rtol=1e-13)
    assert np.allclose(P.sum(axis=-1), 33.0, rtol=1e-13)
    assert np.allclose(O.softmax_fwd(S + 100.0, 33.0), P, rtol=1e-12)          # shift invariance
    big = O.softmax_fwd(np.array([[1000.0, 1000.0, -1000.0]]), 1.0)            # no overflow
    assert np.allclose(big, [[0.5, 0.5, 0.0]])


def test_scaled_softmax_is_about_one_for_small_scores():
    """Appendix "Softmax (followed by matmul)": with alpha = s the output is approximately a vector of ones."""
    rng = np.random.default_rng(1)
    S = rng.standard_normal((64, 512)) * 0.1
    P = O.softmax_fwd(S, 512.0)
    assert abs(P.mean() - 1) < 1e-12 and np.abs(P - 1).max() < 0.6 and P.std() < 0.11


def test_softmax_backward_is_the_gradient_times_beta():
    rng = np.random.default_rng(2)
    S, G = rng.standard_normal((3, 9)), rng.standard_normal((3, 9))
    alpha, beta = 9.0, 2.5
    P = O.softmax_fwd(S, alpha)
    dS = O.softmax_bwd(P, G, alpha, beta)
    h = 1e-6
    fd = np.zeros_like(S)
    for i in range(S.shape[0]):
        for j in range(S.shape[1]):
            E = np.zeros_like(S); E[i, j] = h
            # unscaled op f = softmax; f*_grad = beta * g^T df/dx
            fd[i, j] = np.sum(G * (special.softmax(S + E, axis=-1) - special.softmax(S - E, axis=-1))) / (2 * h)
    assert np.allclose(dS, beta * fd, atol=1e-8)
    assert np.allclose(dS.sum(axis=-1), 0.0, atol=1e-12)                       # gradients of a simplex map sum to zero


def test_softmax_backward_scale_with_s():
    """With alpha = beta = s and near-uniform probabilities the gradient is about (g - mean g): unit scale."""
    rng = np.random.default_rng(3)
    s = 512
    S, G = rng.standard_normal((256, s)) * 0.1, rng.standard_normal((256, s))
    dS = O.softmax_bwd(O.softmax_fwd(S, s), G, s, s)
    assert abs(dS.std() - 1) < 0.05
