"""Pins for the oracle's scaled dot-product attention with unrounded scores (ops.attention_fwd):
closed forms, a brute-force loop on tiny inputs, the library softmax, and the unit-scale property the
appendix "Unit scaling and attention" states for the chosen scale factors."""
import math

import numpy as np
from scipy import special

from oracle import formats as F
from oracle import ops as O
from oracle import encoder as E


def test_equal_keys_give_uniform_weights_and_the_scaled_mean_of_values():
    """All keys equal -> softmax is uniform, s * softmax = 1 exactly, C = alpha_c * column sums of V."""
    rng = np.random.default_rng(0)
    s, d = 48, 8
    Q = rng.standard_normal((5, d))
    K = np.tile(rng.standard_normal((1, d)), (s, 1))
    V = F.quantise(rng.standard_normal((s, d)), F.FORMATS["bf16"])
    P, C = O.attention_fwd(Q, K, V, d ** -0.5, float(s), s ** -0.5, "bf16")
    assert np.array_equal(P, np.ones((5, s)))
    assert np.allclose(C, np.float64(np.float32(s ** -0.5)) * V.sum(axis=0, keepdims=True).repeat(5, 0), rtol=1e-14)


def test_one_dominant_key_selects_its_value_row():
    """A key whose score exceeds the others by 120 takes all the weight: P = s at that key (rounded to the
    operand format, which saturates E4M3 at 448 for s = 512), C = alpha_c * P * that row of V."""
    s, d = 512, 4
    Q = np.zeros((3, d)); Q[:, 0] = 1.0
    K = np.zeros((s, d)); K[7, 0] = 120.0
    V = np.arange(s * d, dtype=np.float64).reshape(s, d) / 64.0
    P, C = O.attention_fwd(Q, K, V, 1.0, float(s), 1.0, "bf16")
    assert P[0, 7] == 512.0 and np.count_nonzero(P) == 3
    assert np.allclose(C[1], 512.0 * V[7])
    P8, _ = O.attention_fwd(Q, K, V, 1.0, float(s), 1.0, "e4m3")
    assert P8[0, 7] == 448.0


def test_brute_force_on_a_tiny_problem():
    rng = np.random.default_rng(1)
    sq, sk, d = 3, 5, 4
    Q, K, V = rng.standard_normal((sq, d)), rng.standard_normal((sk, d)), rng.standard_normal((sk, d))
    a_s, sm, a_c = 0.5, 5.0, 0.25            # exactly representable in float32
    P, C = O.attention_fwd(Q, K, V, a_s, sm, a_c, "f64")
    for i in range(sq):
        scores = [a_s * sum(Q[i][t] * K[j][t] for t in range(d)) for j in range(sk)]
        den = sum(math.exp(x) for x in scores)
        w = [sm * math.exp(x) / den for x in scores]
        for j in range(sk):
            assert abs(P[i, j] - w[j]) < 1e-13
        for t in range(d):
            assert abs(C[i, t] - a_c * sum(w[j] * V[j][t] for j in range(sk))) < 1e-13


def test_matches_library_softmax_and_rounds_only_the_weights():
    rng = np.random.default_rng(2)
    Q, K, V = rng.standard_normal((2, 3, 16, 8)), rng.standard_normal((2, 3, 24, 8)), rng.standard_normal((2, 3, 24, 8))
    a_s = float(np.float32(8 ** -0.5)); a_c = float(np.float32(24 ** -0.5))
    P, C = O.attention_fwd(Q, K, V, 8 ** -0.5, 24.0, 24 ** -0.5, "e4m3")
    ref = 24.0 * special.softmax(a_s * np.einsum("bhqd,bhkd->bhqk", Q, K), axis=-1)
    assert np.array_equal(P, F.quantise(ref, F.FORMATS["e4m3"]))
    assert np.allclose(C, a_c * np.einsum("bhqk,bhkd->bhqd", P, V), rtol=1e-13)
    # the scores themselves are not rounded: rounding them to BF16 first changes some weights
    S16 = F.quantise(a_s * np.einsum("bhqd,bhkd->bhqk", Q, K), F.FORMATS["bf16"])
    assert not np.array_equal(F.quantise(24.0 * special.softmax(S16, axis=-1), F.FORMATS["e4m3"]), P)


def test_unit_scale_of_scores_weights_and_context():
    """Unit-variance Q, K, V: scores have variance ~1 with alpha = d^-1/2; s * softmax has mean exactly 1;
    the context alpha_c * P V with alpha_c = s^-1/2 has variance close to E[p^2] (independent of s up to that
    factor), i.e. of order one."""
    rng = np.random.default_rng(3)
    s, d = 256, 64
    Q, K, V = rng.standard_normal((s, d)), rng.standard_normal((s, d)), rng.standard_normal((s, d))
    P, C = O.attention_fwd(Q, K, V, d ** -0.5, float(s), s ** -0.5, "f64")
    S = np.float64(np.float32(d ** -0.5)) * Q @ K.T
    assert abs(S.std() - 1) < 0.02
    assert np.allclose(P.mean(axis=1), 1.0, rtol=1e-12)
    assert abs(C.var() / (P ** 2).mean() - 1) < 0.1


def test_encoder_layer_with_unrounded_scores_differs_only_from_the_scores_on():
    rng = np.random.default_rng(4)
    nseq, slen, d, nhead, f = 2, 16, 32, 2, 64
    X, G = rng.standard_normal((nseq * slen, d)), rng.standard_normal((nseq * slen, d))
    Wqkv, Wo = rng.standard_normal((d, 3 * d)), rng.standard_normal((d, d))
    W1, W2 = rng.standard_normal((d, f)), rng.standard_normal((f, d))
    a = E.encoder_layer(X, Wqkv, Wo, W1, W2, G, nseq, slen, nhead, att="bf16")
    b = E.encoder_layer(X, Wqkv, Wo, W1, W2, G, nseq, slen, nhead, att="bf16", fused_scores=True)
    assert np.array_equal(a.QKV, b.QKV)
    assert np.array_equal(F.quantise(b.S, F.FORMATS["bf16"]), a.S)         # same scores before rounding
    hd = d // nhead
    Q, K, V = (E._heads(b.QKV, nseq, slen, nhead, hd, i, d) for i in range(3))
    P, C = O.attention_fwd(Q, K, V, hd ** -0.5, float(slen), slen ** -0.5, "bf16")
    assert np.array_equal(b.P, P.reshape(-1, slen))
    assert np.array_equal(b.Cq, F.quantise(E._unheads(C, nseq, slen, nhead, hd), F.FORMATS["e4m3"]))
    assert np.abs(a.P - b.P).max() < 0.05 * np.abs(a.P).max()             # close, not identical


def test_backward_to_the_scores_by_finite_differences():
    """dS and dQ of attention_bwd_scores are beta-scaled gradients of L = sum(G * (P V)) with P = alpha softmax(S):
    central differences in S for dS (through the unscaled softmax, table row "softmax") and the plain products for dQ."""
    rng = np.random.default_rng(5)
    sq, sk, d = 3, 6, 4
    Q, K, V = rng.standard_normal((sq, d)), rng.standard_normal((sk, d)), rng.standard_normal((sk, d))
    G = rng.standard_normal((sq, d))
    alpha, beta, b_p, b_q = 6.0, 6.0, 0.5, 0.25
    S = 0.5 * Q @ K.T
    P = O.softmax_fwd(S, alpha)
    dS, dQ = O.attention_bwd_scores(G, P, K, V, b_p, alpha, beta, b_q, "f64")
    fd = np.zeros_like(S)
    h = 1e-6
    for i in range(sq):
        for j in range(sk):
            E = np.zeros_like(S); E[i, j] = h
            f = lambda s_: np.sum(G * (special.softmax(s_, axis=-1) @ V))       # unscaled ops
            fd[i, j] = (f(S + E) - f(S - E)) / (2 * h)
    assert np.allclose(dS, beta * b_p * fd, atol=1e-8)
    assert np.allclose(dQ, b_q * dS @ K, rtol=1e-14)


def test_backward_rows_sum_to_zero_and_uniform_gradient_vanishes():
    rng = np.random.default_rng(6)
    s, d = 40, 8
    P = O.softmax_fwd(rng.standard_normal((5, s)), float(s))
    K, V = rng.standard_normal((s, d)), rng.standard_normal((s, d))
    dS, _ = O.attention_bwd_scores(rng.standard_normal((5, d)), P, K, V, d ** -0.5, float(s), float(s), d ** -0.5, "f64")
    assert np.abs(dS.sum(axis=1)).max() < 1e-12                      # softmax gradients are orthogonal to 1
    # every value row equal: dP is constant along a row, so dS = 0
    Vc = np.tile(rng.standard_normal((1, d)), (s, 1))
    dS0, dQ0 = O.attention_bwd_scores(rng.standard_normal((5, d)), P, K, Vc, 1.0, float(s), float(s), 1.0, "bf16")
    assert np.abs(dS0).max() < 1e-12 and np.abs(dQ0).max() < 1e-10
