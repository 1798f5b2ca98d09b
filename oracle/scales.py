"""Unit-scaling factors (test infrastructure, fp64).

Follows the section "A scaling strategy for unit variance" (alpha = 1/sigma_Y,
beta_i = 1/sigma_{x'_i} under unit-normal inputs; constrained groups take the
geometric mean) and the appendix table "Table of unit scaling factors".
"""
from __future__ import annotations

import math

import numpy as np
from scipy import integrate, special


def linear_scales(b: int, m: int, n: int, constrained: bool = False):
    """(alpha, beta_X, beta_W) of matmul(X[b x m], W[m x n]).

    Unconstrained (table row "matmul"): alpha = m^-1/2, beta_X = n^-1/2,
    beta_W = b^-1/2.  Constrained (section "Example": the edge carrying X is not
    a cut-edge): alpha = beta_X = (m n)^-1/4, beta_W unchanged.
    """
    alpha = m ** -0.5
    beta_x = n ** -0.5
    beta_w = b ** -0.5
    if constrained:
        alpha = beta_x = geometric_mean([alpha, beta_x])
    return alpha, beta_x, beta_w


def geometric_mean(factors) -> float:
    """(f_0 * f_1 * ... * f_l)^(1/(l+1)) for a constrained group of l+1 factors."""
    factors = [float(f) for f in factors]
    return math.exp(sum(math.log(f) for f in factors) / len(factors))


def _normal_pdf(z):
    return np.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)


def _normal_cdf(z):
    return 0.5 * special.erfc(-z / math.sqrt(2.0))      # = (1 + erf(z / sqrt 2)) / 2, accurate in the lower tail


def gaussian_expectation(f, breakpoints=(0.0,)) -> float:
    """E[f(Z)] for Z ~ N(0,1) by adaptive quadrature over [-40, 40]."""
    val, _ = integrate.quad(
        lambda z: f(z) * _normal_pdf(z), -40.0, 40.0,
        points=list(breakpoints), epsabs=1e-14, epsrel=1e-13, limit=800,
    )
    return val


def activation_scales(f, df):
    """(alpha, beta) of an elementwise activation under a unit-normal input.

    alpha = 1 / std(f(Z)) (the output's standard deviation about its mean) and
    beta = 1 / sqrt(E[f'(Z)^2]): the incoming gradient is zero-mean, unit-variance
    and independent of Z, so the variance of f'(Z) * G is E[f'(Z)^2].
    """
    mean = gaussian_expectation(f)
    second = gaussian_expectation(lambda z: f(z) ** 2)
    grad_second = gaussian_expectation(lambda z: df(z) ** 2)
    return 1.0 / math.sqrt(second - mean * mean), 1.0 / math.sqrt(grad_second)


def gelu(z):
    """gelu(x) = x * Phi(x), Phi the standard normal CDF (table row "gelu")."""
    return z * _normal_cdf(z)


def gelu_grad(z):
    """d/dx [x Phi(x)] = Phi(x) + x phi(x)."""
    return _normal_cdf(z) + z * _normal_pdf(z)


def gelu_scales(constrained: bool = False):
    """(alpha_g, beta_g) for gelu; the geometric mean of the two when constrained."""
    a, b = activation_scales(gelu, gelu_grad)
    if constrained:
        a = b = geometric_mean([a, b])
    return a, b


def relu_scales():
    return activation_scales(lambda z: np.maximum(z, 0.0), lambda z: (z > 0) * 1.0)


def tanh_scales():
    return activation_scales(np.tanh, lambda z: 1.0 - np.tanh(z) ** 2)


def sigmoid_scales():
    sg = lambda z: 1.0 / (1.0 + np.exp(-z))
    return activation_scales(sg, lambda z: sg(z) * (1.0 - sg(z)))


def residual_coefficients(tau: float):
    """(sqrt(1 - tau), sqrt(tau)) of the fixed(tau) residual scheme."""
    return math.sqrt(1.0 - tau), math.sqrt(tau)


def rescale_flop_ratio(b: int, m: int, n: int) -> float:
    """FLOP_rescaling / FLOP_matmul = (1/6)(1/b + 1/m + 1/n) (appendix "Computational overhead")."""
    return (b * n + n * m + b * m) / (6.0 * b * n * m)


def layer_norm_scales(b: int):
    """(alpha, beta_x, beta_w, beta_c) of layer_norm on a b x n input (table row "layer_norm"):
    alpha = 1, beta_x = 1, beta_w = beta_c = b^-1/2."""
    return 1.0, 1.0, b ** -0.5, b ** -0.5


def softmax_xent_scales(s: int):
    """(alpha, beta) of softmax_xent over s classes (table row "softmax_xent"): alpha = 1, beta = s / sqrt(s - 1)."""
    return 1.0, s / math.sqrt(s - 1)
