"""Pins for the oracle's scaled relu / tanh / sigmoid (and gelu through the same entry): library
functions, finite differences, and unit scale of output and gradient with the table's constants."""
import numpy as np
import pytest
from scipy import special

from oracle import ops as O
from oracle import scales as S

def _sigmoid(z):
    """The table's (1 + e^-x)^-1, written so that neither tail overflows: e^x / (1 + e^x) for x < 0."""
    z = np.asarray(z, np.float64)
    e = np.exp(-np.abs(z))
    return np.where(z >= 0, 1.0 / (1.0 + e), e / (1.0 + e))


LIB = {"relu": lambda z: np.where(z > 0, z, 0.0), "tanh": lambda z: np.expm1(2 * np.clip(z, -300, 300)) / (np.expm1(2 * np.clip(z, -300, 300)) + 2),
       "sigmoid": _sigmoid, "gelu": lambda z: z * special.ndtr(z)}
SCALES = {"relu": S.relu_scales, "tanh": S.tanh_scales, "sigmoid": S.sigmoid_scales, "gelu": S.gelu_scales}


@pytest.mark.parametrize("fn", ["relu", "tanh", "sigmoid", "gelu"])
def test_forward_is_the_library_function_and_backward_its_derivative(fn):
    rng = np.random.default_rng(0)
    H = np.concatenate([rng.standard_normal(200) * 3, [-800.0, -40.0, 0.0, 40.0, 800.0]])
    s_in, alpha, beta = 1.25, 1.7, 0.6
    A = O.activation_fwd(fn, H, s_in, alpha)
    assert np.allclose(A, np.float64(np.float32(alpha)) * LIB[fn](s_in * H), rtol=1e-12, atol=1e-300), fn
    assert np.isfinite(A).all()
    G = rng.standard_normal(H.shape)
    dH = O.activation_bwd(fn, H, G, s_in, beta)
    h = 1e-6
    Hs = H[:200][np.abs(H[:200]) > 1e-3] if fn == "relu" else H[:200]      # relu: away from the kink
    Gs = G[:200][np.abs(H[:200]) > 1e-3] if fn == "relu" else G[:200]
    fd = (LIB[fn](s_in * (Hs + h)) - LIB[fn](s_in * (Hs - h))) / (2 * h)
    ref = np.float64(np.float32(beta)) * fd * Gs
    got = O.activation_bwd(fn, Hs, Gs, s_in, beta)
    assert np.allclose(got, ref, atol=1e-8)
    assert dH.shape == H.shape and np.isfinite(dH).all()


def test_relu_derivative_at_zero_is_zero_and_gelu_entry_equals_gelu_ops():
    assert O.activation_bwd("relu", np.zeros(3), np.ones(3), 1.0, 1.0).tolist() == [0.0, 0.0, 0.0]
    z = np.linspace(-5, 5, 101)
    assert np.allclose(O.activation_fwd("gelu", z, 0.7, 1.701), O.gelu_fwd(z, 0.7, 1.701), rtol=1e-14, atol=0)
    assert np.allclose(O.activation_bwd("gelu", z, 2 * z, 0.7, 1.481), O.gelu_bwd(z, 2 * z, 0.7, 1.481), rtol=1e-14, atol=0)


@pytest.mark.parametrize("fn", ["relu", "tanh", "sigmoid"])
def test_unit_scale_of_output_and_gradient_with_the_table_constants(fn):
    """Section "Unit Scaling": with alpha and beta of the table row, output and input gradient of the op
    have unit standard deviation for unit-normal inputs and gradients."""
    alpha, beta = SCALES[fn]()
    rng = np.random.default_rng(1)
    z, g = rng.standard_normal(400000), rng.standard_normal(400000)
    assert abs(O.activation_fwd(fn, z, 1.0, alpha).std() - 1) < 0.01
    assert abs(np.sqrt(np.mean(O.activation_bwd(fn, z, g, 1.0, beta) ** 2)) - 1) < 0.01
