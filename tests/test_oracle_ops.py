"""Pins for the oracle's ops: brute force on tiny shapes, finite differences, unit variance, the theorem."""
import math

import numpy as np
import pytest

from oracle import formats as F
from oracle import ops as O
from oracle import scales as S


def loops_matmul(A, B):
    """Textbook triple loop in Python floats: C[i][j] = sum_k A[i][k] B[k][j]."""
    n, k, m = len(A), len(B), len(B[0])
    return [[sum(A[i][t] * B[t][j] for t in range(k)) for j in range(m)] for i in range(n)]


def test_linear_ops_by_triple_loop():
    rng = np.random.default_rng(0)
    b, m, n = 3, 4, 5
    X, W, G = rng.standard_normal((b, m)), rng.standard_normal((m, n)), rng.standard_normal((b, n))
    a = 0.37
    a32 = float(np.float32(a))
    Y = np.array(loops_matmul(X.tolist(), W.tolist())) * a32
    dX = np.array(loops_matmul(G.tolist(), W.T.tolist())) * a32
    dW = np.array(loops_matmul(X.T.tolist(), G.tolist())) * a32
    assert O.linear_fwd(X, W, a).shape == (b, n) and np.allclose(O.linear_fwd(X, W, a), Y, rtol=1e-14)
    assert O.linear_bwd_x(G, W, a).shape == (b, m) and np.allclose(O.linear_bwd_x(G, W, a), dX, rtol=1e-14)
    assert O.linear_bwd_w(X, G, a).shape == (m, n) and np.allclose(O.linear_bwd_w(X, G, a), dW, rtol=1e-14)


def test_linear_identity_and_one_hot():
    X = np.arange(12.0).reshape(3, 4)
    assert np.array_equal(O.linear_fwd(X, np.eye(4), 1.0), X)
    W = np.arange(20.0).reshape(4, 5)
    e = np.zeros((1, 4)); e[0, 2] = 1
    assert np.array_equal(O.linear_fwd(e, W, 0.5), 0.5 * W[2:3])
    g = np.zeros((1, 5)); g[0, 3] = 1
    assert np.array_equal(O.linear_bwd_x(g, W, 2.0), 2.0 * W[:, 3][None, :])
    assert np.array_equal(O.linear_bwd_w(e, g, 1.0), np.outer(e[0], g[0]))


def test_linear_gradients_are_true_gradients_up_to_the_scale():
    """d<G, X W>/dX = G W^T and d/dW = X^T G: the scaled grads are beta times these."""
    rng = np.random.default_rng(1)
    b, m, n = 4, 5, 3
    X, W, G = rng.standard_normal((b, m)), rng.standard_normal((m, n)), rng.standard_normal((b, n))
    L = lambda X_, W_: float(np.sum(G * (X_ @ W_)))
    h = 1e-6
    fdX = np.zeros_like(X); fdW = np.zeros_like(W)
    for i in range(b):
        for j in range(m):
            E = np.zeros_like(X); E[i, j] = h
            fdX[i, j] = (L(X + E, W) - L(X - E, W)) / (2 * h)
    for i in range(m):
        for j in range(n):
            E = np.zeros_like(W); E[i, j] = h
            fdW[i, j] = (L(X, W + E) - L(X, W - E)) / (2 * h)
    assert np.allclose(O.linear_bwd_x(G, W, 0.25) / 0.25, fdX, atol=1e-7)
    assert np.allclose(O.linear_bwd_w(X, G, 0.125) / 0.125, fdW, atol=1e-7)


def test_unit_variance_of_the_three_matmuls():
    b, m, n = 1024, 1536, 1280
    rng = np.random.default_rng(2)
    X, W, G = rng.standard_normal((b, m)), rng.standard_normal((m, n)), rng.standard_normal((b, n))
    a, bx, bw = S.linear_scales(b, m, n)
    for out in (O.linear_fwd(X, W, a), O.linear_bwd_x(G, W, bx), O.linear_bwd_w(X, G, bw)):
        assert abs(np.std(out) - 1) < 0.05 and abs(np.mean(out)) < 0.01


def test_unit_variance_survives_fp8_operands():
    b, m, n = 512, 1024, 768
    rng = np.random.default_rng(3)
    X = F.quantise(rng.standard_normal((b, m)), F.E4M3)
    W = F.quantise(rng.standard_normal((m, n)), F.E4M3)
    G = F.quantise(rng.standard_normal((b, n)), F.E5M2)
    a, bx, bw = S.linear_scales(b, m, n)
    for out in (O.linear_fwd(X, W, a), O.linear_bwd_x(G, W, bx), O.linear_bwd_w(X, G, bw)):
        assert abs(np.std(out) - 1) < 0.05


def test_gelu_ops_match_scalar_math():
    H = np.linspace(-6, 6, 97)
    s_in, ag, bg = 0.75, 1.7, 1.48
    s32, a32, b32 = (float(np.float32(v)) for v in (s_in, ag, bg))
    want = [a32 * (s32 * h) * 0.5 * math.erfc(-(s32 * h) / math.sqrt(2)) for h in H]
    assert np.allclose(O.gelu_fwd(H, s_in, ag), want, rtol=1e-14, atol=1e-16)
    import mpmath
    mpmath.mp.dps = 40
    for h in (-5.5, -1.25, 0.0, 0.4375, 3.0):
        z = mpmath.mpf(s32) * mpmath.mpf(h)
        ref = mpmath.mpf(a32) * z * mpmath.ncdf(z)
        assert abs(float(O.gelu_fwd(np.float64(h), s_in, ag)) - float(ref)) <= 4e-16 * max(abs(float(ref)), 1e-300)
        dref = mpmath.mpf(b32) * mpmath.mpf(s32) * (mpmath.ncdf(z) + z * mpmath.npdf(z)) * mpmath.mpf(0.5)
        assert abs(float(O.gelu_bwd(np.float64(h), np.float64(0.5), s_in, bg)) - float(dref)) <= 1e-15 * abs(float(dref))
    dA = np.cos(H)
    fd = (O.gelu_fwd(H + 1e-6, s_in, 1.0) - O.gelu_fwd(H - 1e-6, s_in, 1.0)) / 2e-6
    assert np.allclose(O.gelu_bwd(H, dA, s_in, bg), b32 * fd * dA, atol=1e-8)


def test_residual_add():
    rng = np.random.default_rng(4)
    a, b = rng.standard_normal(100000), rng.standard_normal(100000)
    assert np.allclose(O.residual_add(a, b, 0.5), (a + b) * float(np.float32(math.sqrt(0.5))), rtol=1e-15)
    for tau in (0.2, 0.5, 0.8):
        assert abs(np.std(O.residual_add(a, b, tau)) - 1) < 0.02
    assert np.allclose(O.residual_add(a, b, 0.0), a) and np.allclose(O.residual_add(a, b, 1.0), b)


def test_epilogue_rounds_once_and_stores_preactivation():
    val = np.array([[0.3, -1.2, 2.5, 300.0]])
    out, codes, aux = O.apply_epilogue(val, O.Epilogue(act="gelu", act_out_scale=1.7), "e4m3")
    assert np.array_equal(aux, F.quantise(val, F.BF16))
    assert np.array_equal(out, F.quantise(O.gelu_fwd(val, 1.0, 1.7), F.E4M3))   # from unrounded val
    assert out[0, 3] == 448.0 and codes[0, 3] == 126
    skip = np.ones_like(val)
    out, _, _ = O.apply_epilogue(val, O.Epilogue(skip=skip, skip_coef=0.5, out_coef=2.0), "f32")
    assert np.allclose(out, 0.5 + 2.0 * val, rtol=1e-7)


def _ffn_loss_fd(X, W1, W2, G, sc, wrt, idx, h=1e-6):
    def R(X_, W1_, W2_):
        return O.ffn_block(X_, W1_, W2_, G, sc, operand="f64", h_dtype="f64", io_dtype="f64").R
    args = [X.copy(), W1.copy(), W2.copy()]
    args[wrt][idx] += h
    up = float(np.sum(G * R(*args)))
    args[wrt][idx] -= 2 * h
    dn = float(np.sum(G * R(*args)))
    return (up - dn) / (2 * h)


@pytest.fixture(scope="module")
def tiny_ffn():
    rng = np.random.default_rng(5)
    T, d, f = 6, 5, 7
    return (rng.standard_normal((T, d)), rng.standard_normal((d, f)),
            rng.standard_normal((f, d)), rng.standard_normal((T, d)), (T, d, f))


def test_ffn_constrained_graph_gives_true_input_gradient(tiny_ffn):
    """Theorem (constraint-scaled graphs are scaled ops): with alpha = beta on every op that
    consumes the non-cut residual-branch edge, dX is the true gradient of <G, R>."""
    X, W1, W2, G, (T, d, f) = tiny_ffn
    sc = O.FFNScales.constrained(T, d, f, tau=0.3)
    r = O.ffn_block(X, W1, W2, G, sc, operand="f64", h_dtype="f64", io_dtype="f64")
    for idx in [(0, 0), (2, 3), (5, 4), (3, 1)]:
        fd = _ffn_loss_fd(X, W1, W2, G, sc, 0, idx)
        assert abs(r.dX[idx] - fd) < 2e-6 * max(1, abs(fd))


def test_ffn_weight_gradients_are_true_gradients_times_a_constant(tiny_ffn):
    X, W1, W2, G, (T, d, f) = tiny_ffn
    sc = O.FFNScales.unconstrained(T, d, f, tau=0.5)
    r = O.ffn_block(X, W1, W2, G, sc, operand="f64", h_dtype="f64", io_dtype="f64")
    f32 = lambda v: float(np.float32(v))
    st = f32(math.sqrt(sc.tau))
    k2 = f32(sc.beta_w) / (st * f32(sc.alpha2))
    k1 = f32(sc.beta_w) * f32(sc.beta_g) * f32(sc.beta_x2) / (f32(sc.alpha1) * f32(sc.alpha_g) * st * f32(sc.alpha2))
    for idx in [(0, 0), (3, 2), (6, 4)]:
        fd = _ffn_loss_fd(X, W1, W2, G, sc, 2, idx)
        assert abs(r.dW2[idx] - k2 * fd) < 2e-6 * max(1, abs(k2 * fd))
    for idx in [(0, 0), (4, 6), (2, 3)]:
        fd = _ffn_loss_fd(X, W1, W2, G, sc, 1, idx)
        assert abs(r.dW1[idx] - k1 * fd) < 2e-6 * max(1, abs(k1 * fd))


def test_ffn_unconstrained_input_gradient_is_not_the_true_gradient(tiny_ffn):
    """Counter-example in the text (x + f*(x) with alpha != beta is not a scaled op)."""
    X, W1, W2, G, (T, d, f) = tiny_ffn
    sc = O.FFNScales.unconstrained(T, d, f, tau=0.5)
    r = O.ffn_block(X, W1, W2, G, sc, operand="f64", h_dtype="f64", io_dtype="f64")
    fd = np.array([_ffn_loss_fd(X, W1, W2, G, sc, 0, (i, 0)) for i in range(T)])
    ratio = r.dX[:, 0] / fd
    assert np.std(ratio) > 1e-3


def test_ffn_chain_statistics_at_initialisation():
    """H is unit-variance; the second matmul sees gelu outputs whose second moment is
    alpha_g^2 E[gelu(z)^2], so std(Y) = alpha_g * rms(gelu(z)) ~ 1.109 (non-zero-mean
    activation, cf. the remark on ReLU in the scaling-analysis appendix)."""
    from paper_2303_11257_b200 import synth
    shape = synth.FFNShape("t", 1024, 512, 2048)
    X, W1, W2, G = synth.ffn_tensors(shape, seed=7)
    sc = O.FFNScales.unconstrained(shape.tokens, shape.d_model, shape.d_ff)
    r = O.ffn_block(X, W1, W2, G, sc, operand="fp8")
    assert abs(np.std(r.H) - 1) < 0.03
    assert abs(np.std(r.Aq) - 1) < 0.03                      # alpha_g * gelu has unit std
    rms_gelu = math.sqrt(S.gaussian_expectation(lambda z: S.gelu(z) ** 2))
    expect = S.gelu_scales()[0] * rms_gelu
    assert abs(expect - 1.1092) < 1e-3
    Y = (r.R - np.float32(math.sqrt(0.5)) * X.astype(np.float64)) / np.float32(math.sqrt(0.5))
    assert abs(np.std(Y) - expect) < 0.04
    for t in (r.dW1, r.dW2, r.dHq):
        assert 0.8 < np.std(t) < 1.25
    # every stored FP8 tensor holds representable values only
    assert np.array_equal(F.quantise(r.Aq, F.E4M3), r.Aq) and np.array_equal(F.quantise(r.dHq, F.E5M2), r.dHq)
    assert np.array_equal(F.quantise(r.H, F.BF16), r.H)


def test_ffn_flops():
    assert O.ffn_flops(8192, 1024, 4096) == 6 * 2 * 8192 * 1024 * 4096


def test_weighted_add_n_keeps_unit_variance_and_reduces_to_the_residual_add():
    rng = np.random.default_rng(11)
    xs = [rng.standard_normal((64, 512)) for _ in range(3)]
    out = O.weighted_add_n(xs, [1.0, 0.5, 2.0])
    assert abs(out.std() - 1) < 0.02                                   # alpha = (sum gamma^2)^-1/2
    direct = (1.0 * xs[0] + 0.5 * xs[1] + 2.0 * xs[2]) / np.sqrt(1 + 0.25 + 4)
    assert np.allclose(out, direct, rtol=1e-6, atol=1e-6)
    tau = 0.3                                                          # n = 2 with gamma = (sqrt(1-tau), sqrt(tau)): alpha = 1
    two = O.weighted_add_n(xs[:2], [np.sqrt(1 - tau), np.sqrt(tau)], alpha=1.0)
    assert np.allclose(two, O.residual_add(xs[0], xs[1], tau), rtol=1e-12, atol=1e-12)
    l = 5                                                              # running-mean residual: tau = 1 / (l + 1)
    assert np.allclose(O.residual_add(xs[0], xs[1], 1 / (l + 1)), np.sqrt(l / (l + 1)) * xs[0] + np.sqrt(1 / (l + 1)) * xs[1], rtol=1e-6, atol=1e-6)
