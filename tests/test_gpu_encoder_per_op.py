"""Encoder layer, op by op, strictly: every launch of the layer is checked against the oracle's
single-op function evaluated on the inputs the device actually stored for that launch.

Feeding each op the device's own stored operands removes the propagation of legitimate one-code
differences through the chain, so the per-op tolerances of the stand-alone tests apply unchanged:
GEMM outputs within 2e-3 of the fp64 result at unit scale, 16-bit outputs additionally within one
ulp, FP8 outputs within one code, casts of identical values bit-exact, softmax within 3e-6 of the row
scale.  A transposed head, a wrong scale factor on any of the attention GEMMs or swapped dQ / dK fail
here.  Small layers are checked in full, the BERT-large-shaped layer on sampled (sequence, head)
problems and sampled rows."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import ops as O
from oracle import scales as S
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _run(nseq, slen, d, nhead, f, seed, attention, fused=False):
    from paper_2303_11257_b200 import encoder, synth
    T = nseq * slen
    host = (synth.normal(seed, 0, (T, d)), synth.normal(seed, 1, (d, 3 * d)), synth.normal(seed, 2, (d, d)),
            synth.normal(seed, 3, (d, f)), synth.normal(seed, 4, (f, d)), synth.normal(seed, 5, (T, d)))
    layer = encoder.UnitScaledEncoderLayer(nseq, slen, d, nhead, f, attention=attention, fused_attention=fused)
    layer.ffn.keep_h = True                                  # the per-op comparison below reads the FFN's pre-activation
    layer.step(*[torch.from_numpy(t).cuda() for t in host])
    layer.check()
    return layer, host


def _fmt_of(t):
    return {torch.float32: "f32", torch.bfloat16: "bf16", torch.float16: "fp16",
            torch.float8_e4m3fn: "e4m3", torch.float8_e5m2: "e5m2"}[t.dtype]


def _check(got_rows, ref, fmt, tol, what):
    """got_rows: float64 values the device stored; ref: fp64 oracle values before the storage rounding."""
    if fmt in ("e4m3", "e5m2"):
        fm = F.FORMATS[fmt]
        d = U.code_distance(F.quantise_codes(got_rows, fm), F.quantise_codes(ref, fm), fmt)
        ok = (d <= 1) | (np.abs(got_rows - F.quantise(ref, fm)) <= tol)
        assert ok.all(), f"{what}: FP8 code distance {d.max()} at {(~ok).sum()} places"
    else:
        lim = tol + (U.ulp_of(ref, fmt) if fmt != "f32" else 0.0)
        err = np.abs(got_rows - ref)
        assert (err <= lim).all(), f"{what}: {(err > lim).sum()} elements out, worst {err.max():.3e}"


def _per_op(layer, host, problems, rows, wrows):
    """problems: list of (sequence, head); rows: token rows checked in the projections; wrows: rows of
    the weight gradients checked (the contraction always runs over all tokens)."""
    X, Wqkv, Wo, W1, W2, G = host
    nseq, slen, d, nhead, hd = layer.nseq, layer.slen, layer.d, layer.nhead, layer.hd
    T = nseq * slen
    sc = {k: float(np.float32(v)) for k, v in layer.sc.items()}
    cs, cb = S.residual_coefficients(layer.tau)
    H = U.host_values
    # ---- casts that open the step: bit-exact
    assert np.array_equal(U.codes_of(layer.Xq), F.quantise_codes(X, F.E4M3))
    assert np.array_equal(U.codes_of(layer.Wqkv_q), F.quantise_codes(Wqkv, F.E4M3))
    assert np.array_equal(U.codes_of(layer.Wo_q), F.quantise_codes(Wo, F.E4M3))
    Xq, Wqkv_q, Wo_q = H(layer.Xq), H(layer.Wqkv_q), H(layer.Wo_q)
    QKV, Cq = H(layer.QKV), H(layer.Cq)
    f_act, f_grad = _fmt_of(layer.QKV), _fmt_of(layer.dS)
    f_qkv_grad = _fmt_of(layer.dQKV)          # E5M2 where the producers write the projection GEMMs' operand format directly
    f_wide = _fmt_of(layer.dP) if layer.dP is not None else None
    fused = layer.S is None          # fused attention forward: the scores are never stored
    # ---- QKV projection
    _check(QKV[rows], O.linear_fwd(Xq[rows], Wqkv_q, sc["alpha_qkv"]), f_act, TOL, "QKV")
    dC, dQKV = H(layer.dC), H(layer.dQKV)
    for (i, j) in problems:
        r = slice(i * slen, (i + 1) * slen)
        pr = slice((i * nhead + j) * slen, (i * nhead + j + 1) * slen)
        q, k, v = (QKV[r, o + j * hd:o + (j + 1) * hd] for o in (0, d, 2 * d))
        c = slice(j * hd, (j + 1) * hd)
        tag = f"problem ({i}, {j})"
        Pp, dSp = H(layer.P[pr]), H(layer.dS[pr])   # score-sized tensors: this problem only
        # forward: scores, scaled softmax, context
        if fused:
            p_ref, _ = O.attention_fwd(q, k, v, sc["alpha_s"], sc["sm"], sc["alpha_c"], "f64")     # from unrounded scores
            _check(Pp, p_ref, f_act, 3e-6 * sc["sm"], "P (fused) " + tag)
        else:
            Sp = H(layer.S[pr])
            _check(Sp, O.linear_bwd_x(q, k, sc["alpha_s"]), f_wide, TOL, "S " + tag)
            _check(Pp, O.softmax_fwd(Sp, sc["sm"]), f_act, 3e-6 * sc["sm"], "P " + tag)
        ref_c = O.linear_fwd(Pp, v, sc["alpha_c"])
        _check(Cq[r, c], ref_c, "e4m3", TOL * max(1.0, np.abs(ref_c).max()), "C " + tag)
        # backward: dP = beta dC V^T, dV = beta P^T dC, dS, dQ = beta dS K, dK = beta dS^T Q
        dc = dC[r, c]
        ref = O.linear_bwd_x(dc, v, sc["beta_P"])
        if fused:
            dPp = ref                                  # never stored: the softmax gradient sees it unrounded
        else:
            dPp = H(layer.dP[pr])
            _check(dPp, ref, f_wide, TOL * max(1.0, np.abs(ref).max()), "dP " + tag)
        ref = O.linear_bwd_w(Pp, dc, sc["beta_V"])
        _check(dQKV[r, 2 * d + j * hd:2 * d + (j + 1) * hd], ref, f_qkv_grad, TOL * max(1.0, np.abs(ref).max()), "dV " + tag)
        ref = O.softmax_bwd(Pp, dPp, sc["sm"], sc["sm"])
        scale = np.abs(ref).max() + np.abs(dPp).max()
        _check(dSp, ref, f_grad, 3e-6 * scale * max(1.0, slen / 512), "dS " + tag)
        ref = O.linear_fwd(dSp, k, sc["beta_Q"])
        _check(dQKV[r, j * hd:(j + 1) * hd], ref, f_qkv_grad, TOL * max(1.0, np.abs(ref).max()), "dQ " + tag)
        ref = O.linear_bwd_w(dSp, q, sc["beta_K"])
        _check(dQKV[r, d + j * hd:d + (j + 1) * hd], ref, f_qkv_grad, TOL * max(1.0, np.abs(ref).max()), "dK " + tag)
    # ---- output projection with the residual epilogue
    ref = O.weighted_add(X[rows].astype(np.float64), O.linear_fwd(Cq[rows], Wo_q, sc["alpha_o"]), cs, cb)
    _check(H(layer.R1)[rows], ref, "bf16", TOL, "R1")
    # ---- FFN block on R1 (the block's own stored tensors)
    f = layer.ffn
    fs = f.sc
    R1 = H(layer.R1)
    assert np.array_equal(U.codes_of(f.Xq), F.quantise_codes(R1, F.E4M3))
    assert np.array_equal(U.codes_of(f.W1q), F.quantise_codes(W1, F.E4M3))
    assert np.array_equal(U.codes_of(f.W2q), F.quantise_codes(W2, F.E4M3))
    assert np.array_equal(U.codes_of(f.Gq), F.quantise_codes(G, F.E5M2))
    fXq, W1q, W2q, Gq, Hh, Aq, dHq = H(f.Xq), H(f.W1q), H(f.W2q), H(f.Gq), H(f.H), H(f.Aq), H(f.dHq)
    h_ref = O.linear_fwd(fXq[rows], W1q, np.float32(fs.alpha1))
    _check(Hh[rows], h_ref, "bf16", TOL, "H")
    _check(Aq[rows], O.gelu_fwd(h_ref, fs.s_in, np.float32(fs.alpha_g)), "e4m3", TOL, "A")
    ref = O.weighted_add(R1[rows], O.linear_fwd(Aq[rows], W2q, np.float32(fs.alpha2)), cs, cb)
    _check(H(f.R)[rows], ref, "bf16", TOL, "R2")
    ref = O.gelu_bwd(Hh[rows], O.linear_bwd_x(Gq[rows], W2q, np.float32(fs.beta_x2)), fs.s_in, np.float32(fs.beta_g))
    _check(dHq[rows], ref, "e5m2", TOL, "dH")
    g1 = H(f.dX)
    ref = O.weighted_add(G[rows].astype(np.float64), O.linear_bwd_x(dHq[rows], W1q, np.float32(fs.beta_x1)), cs, cb)
    _check(g1[rows], ref, "bf16", TOL, "g1 (FFN input gradient)")
    fw = wrows[wrows < min(W1.shape[0], W2.shape[0])]
    _check(H(f.dW1)[fw], O.linear_bwd_w(fXq[:, fw], dHq, np.float32(fs.beta_w)), "f32", TOL, "dW1")
    _check(H(f.dW2)[fw], O.linear_bwd_w(Aq[:, fw], Gq, np.float32(fs.beta_w)), "f32", TOL, "dW2")
    # ---- attention block backward: projections
    assert np.array_equal(U.codes_of(layer.g1q), F.quantise_codes(g1, F.E5M2))
    g1q = H(layer.g1q)
    _check(dC[rows], O.linear_bwd_x(g1q[rows], Wo_q, sc["beta_o"]), f_grad, TOL, "dC")
    dw = wrows[wrows < d]
    _check(H(layer.dWo)[dw], O.linear_bwd_w(Cq[:, dw], g1q, sc["beta_w"]), "f32", TOL, "dWo")
    if layer.dQKV is not layer.dQKVq:
        assert np.array_equal(U.codes_of(layer.dQKVq), F.quantise_codes(dQKV, F.E5M2))
    dQKVq = H(layer.dQKVq)
    ref = O.weighted_add(g1[rows], O.linear_bwd_x(dQKVq[rows], Wqkv_q, sc["beta_qkv"]), cs, cb)
    _check(H(layer.dX)[rows], ref, "bf16", TOL, "dX")
    _check(H(layer.dWqkv)[dw], O.linear_bwd_w(Xq[:, dw], dQKVq, sc["beta_w"]), "f32", TOL, "dWqkv")


@pytest.mark.parametrize("attention", ["bf16", "fp16", "fp8"])
@pytest.mark.parametrize("cfg", [(2, 128, 256, 4, 512), (3, 80, 192, 3, 400)])
def test_encoder_layer_every_op_small(cfg, attention):
    nseq, slen, d, nhead, f = cfg
    layer, host = _run(nseq, slen, d, nhead, f, seed=51, attention=attention)
    problems = [(i, j) for i in range(nseq) for j in range(nhead)]
    _per_op(layer, host, problems, np.arange(nseq * slen), np.arange(max(d, f)))


@pytest.mark.parametrize("attention", ["bf16", "fp16", "fp8"])
@pytest.mark.parametrize("cfg", [(2, 128, 256, 4, 512), (3, 80, 192, 3, 400)])
def test_encoder_layer_every_op_small_fused_attention(cfg, attention):
    nseq, slen, d, nhead, f = cfg
    layer, host = _run(nseq, slen, d, nhead, f, seed=53, attention=attention, fused=True)
    problems = [(i, j) for i in range(nseq) for j in range(nhead)]
    _per_op(layer, host, problems, np.arange(nseq * slen), np.arange(max(d, f)))


@pytest.mark.parametrize("attention,fused", [("bf16", False), ("fp8", False), ("bf16", True), ("fp8", True)])
def test_encoder_layer_every_op_bert_large_shape(attention, fused):
    """Config 5 at its stated size (16 sequences x 512 tokens, d = 1024, 16 heads x 64, d_ff = 4096)."""
    nseq, slen, d, nhead, f = 16, 512, 1024, 16, 4096
    layer, host = _run(nseq, slen, d, nhead, f, seed=52, attention=attention, fused=fused)
    rng = np.random.default_rng(7)
    problems = [(0, 0), (0, nhead - 1), (nseq - 1, 0), (nseq - 1, nhead - 1)] + \
               [(int(rng.integers(nseq)), int(rng.integers(nhead))) for _ in range(4)]
    T = nseq * slen
    rows = np.unique(np.concatenate([[0, 127, 128, 511, 512, T - 1], rng.integers(0, T, 18)]))
    wrows = np.unique(np.concatenate([[0, 255, 256, d - 1, f - 1], rng.integers(0, f, 11)]))
    _per_op(layer, host, problems, rows, wrows)
