"""Pins for the oracle's encoder layer: per-head attention against a direct loop, unit scale at
initialisation, and agreement of its pieces with the single-op functions."""
import numpy as np

from oracle import encoder as E
from oracle import ops as O
from paper_2303_11257_b200 import synth


def _tensors(nseq, slen, d, f, seed=0):
    T = nseq * slen
    return (synth.normal(seed, 0, (T, d)), synth.normal(seed, 1, (d, 3 * d)), synth.normal(seed, 2, (d, d)),
            synth.normal(seed, 3, (d, f)), synth.normal(seed, 4, (f, d)), synth.normal(seed, 5, (T, d)))


import pytest


@pytest.mark.parametrize("att", ["bf16", "fp8"])
def test_attention_pieces_match_a_direct_per_head_loop(att):
    nseq, slen, d, nhead, f = 2, 16, 32, 4, 64
    hd = d // nhead
    X, Wqkv, Wo, W1, W2, G = _tensors(nseq, slen, d, f)
    r = E.encoder_layer(X, Wqkv, Wo, W1, W2, G, nseq, slen, nhead, att=att)
    act, grad, wide = ("e4m3", "e5m2", "bf16") if att == "fp8" else ("bf16",) * 3
    from oracle import formats as F
    for t, fmt in ((r.QKV, act), (r.P, act), (r.dC, grad), (r.dS, grad), (r.dQKV, grad), (r.S, wide), (r.dP, wide)):
        assert np.array_equal(F.quantise(t, F.FORMATS[fmt]), t)          # every stored tensor is on its format's grid
    for i in range(nseq):
        for j in range(nhead):
            rows = slice(i * slen, (i + 1) * slen)
            q, k, v = (r.QKV[rows, o + j * hd:o + (j + 1) * hd] for o in (0, d, 2 * d))
            pr = slice((i * nhead + j) * slen, (i * nhead + j + 1) * slen)
            s_ref = O.store(O.linear_bwd_x(q, k, hd ** -0.5), wide)[0]            # alpha Q K^T
            assert np.array_equal(r.S[pr], s_ref)
            p_ref = O.store(O.softmax_fwd(s_ref, slen), act)[0]
            assert np.array_equal(r.P[pr], p_ref)
            c_ref = O.store(O.linear_fwd(p_ref, v, slen ** -0.5), "e4m3")[0]
            assert np.array_equal(r.Cq[rows, j * hd:(j + 1) * hd], c_ref)
            dc = r.dC[rows, j * hd:(j + 1) * hd]
            assert np.array_equal(r.dP[pr], O.store(O.linear_bwd_x(dc, v, hd ** -0.5), wide)[0])
            dv = O.linear_bwd_w(p_ref, dc, slen ** -0.5)
            assert np.array_equal(r.dQKV[rows, 2 * d + j * hd:2 * d + (j + 1) * hd], O.store(dv, grad)[0])
            ds = r.dS[pr]
            assert np.array_equal(r.dQKV[rows, j * hd:(j + 1) * hd], O.store(O.linear_fwd(ds, k, hd ** -0.5), grad)[0])
            assert np.array_equal(r.dQKV[rows, d + j * hd:d + (j + 1) * hd], O.store(O.linear_bwd_w(ds, q, hd ** -0.5), grad)[0])


@pytest.mark.parametrize("att", ["bf16", "fp8"])
def test_unit_scale_at_initialisation(att):
    nseq, slen, d, nhead, f = 2, 128, 256, 4, 512
    X, Wqkv, Wo, W1, W2, G = _tensors(nseq, slen, d, f, seed=1)
    r = E.encoder_layer(X, Wqkv, Wo, W1, W2, G, nseq, slen, nhead, att=att)
    assert abs(r.QKV.std() - 1) < 0.05
    assert abs(r.S.std() - 1) < 0.1                       # scores scaled by 1 / sqrt(d_head)
    assert abs(r.P.mean() - 1) < 0.01                     # scaled softmax output is about one
    # unit-normal scores make the softmax output far from uniform (std 1.26 instead of 0), so the
    # tensors downstream of it come out at 1.4 - 2.3 rather than exactly one
    assert 0.5 < r.R1.std() < 2.5 and 0.5 < r.dX.std() < 2.5
    for t in (r.dWqkv, r.dWo, r.dQKV, r.dC):
        assert 0.3 < t.std() < 3.0


def test_fp8_attention_stays_close_to_16_bit_attention():
    """FP8 operands change every attention tensor by quantisation noise only (E5M2 gradients carry two
    mantissa bits, so a few percent per rounding): no tensor of the layer moves by more than a fraction
    of its scale on average, and the two runs stay almost perfectly correlated (a wiring or format mix-up
    in either mode would break both)."""
    nseq, slen, d, nhead, f = 2, 128, 256, 4, 512
    t = _tensors(nseq, slen, d, f, seed=2)
    a = E.encoder_layer(*t, nseq, slen, nhead, att="bf16")
    b = E.encoder_layer(*t, nseq, slen, nhead, att="fp8")
    for name in ("S", "P", "R1", "dC", "dP", "dS", "dQKV", "dX", "dWqkv", "dWo"):
        x, y = getattr(a, name), getattr(b, name)
        assert np.abs(x - y).mean() < 0.25 * max(1.0, np.abs(x).std()), name
        assert np.corrcoef(x.ravel(), y.ravel())[0, 1] > 0.985, name


def test_post_norm_layer_chains_the_single_op_functions_and_normalises_its_outputs():
    nseq, slen, d, nhead, f = 2, 32, 64, 4, 128
    t = _tensors(nseq, slen, d, f, seed=3)
    rng = np.random.default_rng(3)
    ln = (1 + 0.2 * rng.standard_normal(d), 0.1 * rng.standard_normal(d), 1 + 0.2 * rng.standard_normal(d), 0.1 * rng.standard_normal(d))
    r = E.encoder_layer(*t, nseq, slen, nhead, norm="post", ln=ln)
    plain = E.encoder_layer(*t, nseq, slen, nhead)
    assert np.array_equal(r.U1, plain.R1)                                   # same attention block in front of the norm
    eps = float(np.float32(1e-5))
    assert np.array_equal(r.R1, O.store(O.layer_norm_fwd(r.U1, ln[0], ln[1], eps), "bf16")[0])
    assert np.array_equal(r.R2, O.store(O.layer_norm_fwd(r.ffn.R, ln[2], ln[3], eps), "bf16")[0])
    G = t[5]
    dU2, dw2, dc2 = O.layer_norm_bwd(r.ffn.R, ln[2], G, eps)
    assert np.array_equal(r.dU2, O.store(dU2, "bf16")[0]) and np.allclose(r.dln2[0], dw2, rtol=1e-6) and np.allclose(r.dln2[1], dc2, rtol=1e-6, atol=1e-7)
    dU1, dw1, _ = O.layer_norm_bwd(r.U1, ln[0], r.ffn.dX, eps)
    assert np.array_equal(r.dU1, O.store(dU1, "bf16")[0]) and np.allclose(r.dln1[0], dw1, rtol=1e-6)
    # with unit weight and zero bias every token of the layer output has zero mean and unit variance
    ones, zeros = np.ones(d), np.zeros(d)
    u = E.encoder_layer(*t, nseq, slen, nhead, norm="post", ln=(ones, zeros, ones, zeros))
    assert np.abs(u.R2.mean(axis=1)).max() < 0.02 and np.abs(u.R2.std(axis=1) - 1).max() < 0.02
    # the norm gradients carry beta = T^-1/2: unit-ish scale
    assert 0.3 < r.dln2[0].std() < 3 and 0.3 < r.dln1[0].std() < 3
