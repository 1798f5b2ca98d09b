"""Fused scaled dot-product attention forward (us_attention_fwd) against the oracle, element by element.

The weights P are compared with ops.attention_fwd evaluated on the operands the device holds (16-bit
output: within one ulp plus 3e-6 of the row scale, the allowance of the stand-alone softmax tests); the
context C is compared with alpha_context * P V evaluated on the device's OWN stored weights, so that a
legitimate one-ulp difference in a weight does not leak into the second check (2e-3 at unit scale, one ulp /
one FP8 code of the output format on top).  Problems are strided head slices of a [tokens x 3 d] matrix as in
the encoder layer, with ragged lengths, one and two halves of keys, and every output format of C."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import ops as O
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _run(nseq, nhead, s, fmt, c_fmt, seed, store_p=True, scale=1.0):
    from paper_2303_11257_b200 import lib as L, synth
    hd, d, T = 64, nhead * 64, nseq * s
    qkv = scale * synth.normal(seed, 0, (T, 3 * d))
    QKV = U.to_device(qkv, fmt)
    qkv_v = U.values_of(qkv, fmt)
    Cx = U.empty(T, d, c_fmt)
    P = U.empty(nseq * nhead * s, s, fmt) if store_p else None
    ws = L.new_workspace()
    a_s, sm, a_c = hd ** -0.5, float(s), s ** -0.5
    st = (s * 3 * d, hd)
    bt = L.attention_batch((nseq, nhead), st, st, st, (s * d, hd), (nhead * s * s, s * s))
    L.us_attention_fwd(QKV[:s, 0:hd], QKV[:s, d:d + hd], QKV[:s, 2 * d:2 * d + hd], a_s, sm, a_c,
                       Cx[:s, :hd], P[:s] if store_p else None, bt, ws)
    assert L.us_workspace_status(ws) == 0
    return qkv_v, Cx, P, (a_s, sm, a_c)


def _heads(M, nseq, s, nhead, which):
    d = nhead * 64
    return M[:, which * d:(which + 1) * d].reshape(nseq, s, nhead, 64).transpose(0, 2, 1, 3)


def _check_c(Cx, c_ref, c_fmt, nseq, s, nhead):
    ref = c_ref.transpose(0, 2, 1, 3).reshape(nseq * s, nhead * 64)
    got = U.host_values(Cx)
    tol = TOL * max(1.0, np.abs(ref).max())
    if c_fmt in ("e4m3", "e5m2"):
        fm = F.FORMATS[c_fmt]
        dist = U.code_distance(F.quantise_codes(got, fm), F.quantise_codes(ref, fm), c_fmt)
        ok = (dist <= 1) | (np.abs(got - F.quantise(ref, fm)) <= tol)
        assert ok.all(), f"C: code distance {dist.max()} at {(~ok).sum()} places"
    else:
        lim = tol + (U.ulp_of(ref, c_fmt) if c_fmt != "f32" else 0.0)
        err = np.abs(got - ref)
        assert (err <= lim).all(), f"C: {(err > lim).sum()} elements out, worst {err.max():.3e}"


@pytest.mark.parametrize("fmt", ["bf16", "fp16"])
@pytest.mark.parametrize("nseq,nhead,s", [(2, 3, 128), (1, 2, 200), (2, 2, 512), (1, 1, 72), (1, 2, 264), (3, 1, 8)])
def test_weights_and_context_against_the_oracle(fmt, nseq, nhead, s):
    c_fmt = "e4m3"
    qkv_v, Cx, P, (a_s, sm, a_c) = _run(nseq, nhead, s, fmt, c_fmt, seed=61)
    Q, K, V = (_heads(qkv_v, nseq, s, nhead, i) for i in range(3))
    p_ref, _ = O.attention_fwd(Q, K, V, a_s, sm, a_c, "f64")            # unrounded weights
    p_dev = U.host_values(P).reshape(nseq, nhead, s, s)
    lim = U.ulp_of(p_ref, fmt) + 3e-6 * sm
    err = np.abs(p_dev - p_ref)
    assert (err <= lim).all(), f"P: {(err > lim).sum()} elements beyond one ulp, worst {err.max():.3e}"
    assert np.allclose(p_dev.sum(axis=-1), sm, rtol=4e-3)                # rows of s * softmax sum to s
    _check_c(Cx, np.float64(np.float32(a_c)) * (p_dev @ V), c_fmt, nseq, s, nhead)


@pytest.mark.parametrize("c_fmt", ["f32", "bf16", "fp16", "e4m3", "e5m2"])
def test_every_context_format_and_weights_not_stored(c_fmt):
    nseq, nhead, s = 2, 2, 192
    qkv_v, Cx, P, (a_s, sm, a_c) = _run(nseq, nhead, s, "bf16", c_fmt, seed=62, store_p=False)
    Q, K, V = (_heads(qkv_v, nseq, s, nhead, i) for i in range(3))
    p_ref, c_ref = O.attention_fwd(Q, K, V, a_s, sm, a_c, "bf16")
    # without the device's weights at hand, allow for one-ulp differences in them: sum_j ulp(p_j) |v_j| * alpha_c
    slack = np.float64(np.float32(a_c)) * (U.ulp_of(p_ref, "bf16") @ np.abs(V))
    ref = c_ref.transpose(0, 2, 1, 3).reshape(nseq * s, nhead * 64)
    got = U.host_values(Cx)
    lim = TOL + 0.05 * slack.transpose(0, 2, 1, 3).reshape(ref.shape) + \
        (U.ulp_of(ref, c_fmt) if c_fmt != "f32" else 0.0)
    err = np.abs(got - ref)
    assert (err <= lim).all(), f"C ({c_fmt}): {(err > lim).sum()} out, worst {err.max():.3e}"


def test_peaked_rows_large_scores():
    """Scores of standard deviation ~8: rows dominated by one key, weights from 0 to several hundred."""
    nseq, nhead, s = 1, 2, 320
    qkv_v, Cx, P, (a_s, sm, a_c) = _run(nseq, nhead, s, "bf16", "bf16", seed=63, scale=2.8)
    Q, K, V = (_heads(qkv_v, nseq, s, nhead, i) for i in range(3))
    p_ref, _ = O.attention_fwd(Q, K, V, a_s, sm, a_c, "f64")
    p_dev = U.host_values(P).reshape(nseq, nhead, s, s)
    assert p_ref.max() > 100
    # exp of a float32 argument of magnitude up to ~60: relative error up to 60 * 2^-23
    lim = U.ulp_of(p_ref, "bf16") + 3e-6 * sm + 1.5e-5 * p_ref
    assert (np.abs(p_dev - p_ref) <= lim).all()
    _check_c(Cx, np.float64(np.float32(a_c)) * (p_dev @ V), "bf16", nseq, s, nhead)


def test_bert_large_attention_shape_sampled_problems():
    """16 sequences x 16 heads x 512 tokens: first / last and sampled (sequence, head) problems in full."""
    nseq, nhead, s = 16, 16, 512
    qkv_v, Cx, P, (a_s, sm, a_c) = _run(nseq, nhead, s, "bf16", "e4m3", seed=64)
    rng = np.random.default_rng(5)
    probs = [(0, 0), (0, 15), (15, 0), (15, 15)] + [(int(rng.integers(16)), int(rng.integers(16))) for _ in range(6)]
    Cv = U.host_values(Cx)
    for (i, j) in probs:
        r = slice(i * s, (i + 1) * s)
        q, k, v = (qkv_v[r, o * 1024 + j * 64:o * 1024 + (j + 1) * 64] for o in range(3))
        p_ref, _ = O.attention_fwd(q, k, v, a_s, sm, a_c, "f64")
        p_dev = U.host_values(P[(i * nhead + j) * s:(i * nhead + j + 1) * s])
        assert (np.abs(p_dev - p_ref) <= U.ulp_of(p_ref, "bf16") + 3e-6 * sm).all(), (i, j)
        ref = np.float64(np.float32(a_c)) * (p_dev @ v)
        fm = F.FORMATS["e4m3"]
        got = Cv[r, j * 64:(j + 1) * 64]
        dist = U.code_distance(F.quantise_codes(got, fm), F.quantise_codes(ref, fm), "e4m3")
        ok = (dist <= 1) | (np.abs(got - F.quantise(ref, fm)) <= TOL * max(1.0, np.abs(ref).max()))
        assert ok.all(), (i, j, dist.max())


def test_argument_checks():
    from paper_2303_11257_b200 import lib as L
    ws = L.new_workspace()
    q = U.empty(128, 64, "bf16"); k = U.empty(128, 64, "bf16"); c = U.empty(128, 64, "bf16")
    bt = L.attention_batch((1, 1), (0, 0), (0, 0), (0, 0), (0, 0))
    wide = U.empty(128, 128, "bf16")
    with pytest.raises(L.UnitScaleError) as e:
        L.us_attention_fwd(wide, wide, wide, 0.125, 128.0, 0.1, wide, None, bt, ws)
    assert e.value.status == L.US_ERR_UNSUPPORTED                    # head width 128
    k_long = U.empty(640, 64, "bf16")
    with pytest.raises(L.UnitScaleError) as e:
        L.us_attention_fwd(q, k_long, k_long, 0.125, 640.0, 0.1, c, None, bt, ws)
    assert e.value.status == L.US_ERR_UNSUPPORTED                    # more than 512 keys
    q8 = U.empty(128, 64, "e5m2")
    with pytest.raises(L.UnitScaleError) as e:
        L.us_attention_fwd(q8, q8, q8, 0.125, 128.0, 0.1, c, None, bt, ws)
    assert e.value.status == L.US_ERR_UNSUPPORTED                    # E5M2 (gradient format) operands in the forward pass
    with pytest.raises(L.UnitScaleError) as e:
        L.us_attention_fwd(q, k, U.empty(64, 64, "bf16"), 0.125, 128.0, 0.1, c, None, bt, ws)
    assert e.value.status == L.US_ERR_INVALID_ARG                    # V rows != K rows
    L.us_attention_fwd(q[:0], k, k, 0.125, 128.0, 0.1, c[:0], None, bt, ws)   # no queries: nothing to do


@pytest.mark.parametrize("nseq,nhead,s", [(2, 3, 128), (1, 2, 208), (2, 2, 512), (1, 1, 80), (1, 2, 272), (3, 1, 16)])
def test_fp8_operands_weights_and_context(nseq, nhead, s):
    """Q, K, V and the stored weights as E4M3 (all matmul inputs quantised): P within one code of the oracle's
    (weights up to s = 512 saturate at 448), the context against alpha_c * P V on the device's own stored P."""
    qkv_v, Cx, P, (a_s, sm, a_c) = _run(nseq, nhead, s, "e4m3", "e4m3", seed=65)
    Q, K, V = (_heads(qkv_v, nseq, s, nhead, i) for i in range(3))
    p_ref, _ = O.attention_fwd(Q, K, V, a_s, sm, a_c, "f64")
    fm = F.FORMATS["e4m3"]
    p_dev = U.host_values(P).reshape(nseq, nhead, s, s)
    dist = U.code_distance(U.codes_of(P).reshape(p_ref.shape), F.quantise_codes(p_ref, fm), "e4m3")
    ok = (dist <= 1) | (np.abs(p_dev - F.quantise(p_ref, fm)) <= 3e-6 * sm)
    assert ok.all(), f"P: code distance {dist.max()} at {(~ok).sum()} places"
    assert (dist > 0).mean() < 2e-3
    _check_c(Cx, np.float64(np.float32(a_c)) * (p_dev @ V), "e4m3", nseq, s, nhead)


def test_fp8_operands_bert_large_attention_shape_sampled_problems():
    nseq, nhead, s = 16, 16, 512
    qkv_v, Cx, P, (a_s, sm, a_c) = _run(nseq, nhead, s, "e4m3", "e4m3", seed=66)
    rng = np.random.default_rng(9)
    probs = [(0, 0), (0, 15), (15, 0), (15, 15)] + [(int(rng.integers(16)), int(rng.integers(16))) for _ in range(4)]
    Cv = U.host_values(Cx)
    fm = F.FORMATS["e4m3"]
    for (i, j) in probs:
        r = slice(i * s, (i + 1) * s)
        q, k, v = (qkv_v[r, o * 1024 + j * 64:o * 1024 + (j + 1) * 64] for o in range(3))
        p_ref, _ = O.attention_fwd(q, k, v, a_s, sm, a_c, "f64")
        Pt = P[(i * nhead + j) * s:(i * nhead + j + 1) * s]
        p_dev = U.host_values(Pt)
        dist = U.code_distance(U.codes_of(Pt), F.quantise_codes(p_ref, fm), "e4m3")
        assert ((dist <= 1) | (np.abs(p_dev - F.quantise(p_ref, fm)) <= 3e-6 * sm)).all(), (i, j)
        ref = np.float64(np.float32(a_c)) * (p_dev @ v)
        got = Cv[r, j * 64:(j + 1) * 64]
        dc = U.code_distance(F.quantise_codes(got, fm), F.quantise_codes(ref, fm), "e4m3")
        assert ((dc <= 1) | (np.abs(got - F.quantise(ref, fm)) <= TOL * max(1.0, np.abs(ref).max()))).all(), (i, j)


# ------------------------------------------------------------------------------------------------ backward

def _run_bwd(nseq, nhead, s, fmt, dq_fmt, seed, scale=1.0, gfmt=None):
    """Weights P as the oracle's forward pass rounds them (uploaded bit patterns), random dC; returns host values of the
    operands and the device outputs.  gfmt: format of the gradients dC and dS when it differs from fmt (FP8: E5M2)."""
    from paper_2303_11257_b200 import lib as L, synth
    gfmt = gfmt or fmt
    hd, d, T = 64, nhead * 64, nseq * s
    qkv = scale * synth.normal(seed, 0, (T, 3 * d))
    dc = synth.normal(seed, 1, (T, d))
    QKV, dCt = U.to_device(qkv, fmt), U.to_device(dc, gfmt)
    qkv_v, dc_v = U.values_of(qkv, fmt), U.values_of(dc, gfmt)
    Q, K, V = (_heads(qkv_v, nseq, s, nhead, i) for i in range(3))
    a_s, sm, a_c = hd ** -0.5, float(s), s ** -0.5
    p_host, _ = O.attention_fwd(Q, K, V, a_s, sm, a_c, fmt)                    # as stored by a forward pass
    P = U.to_device(p_host.reshape(-1, s), fmt)
    dS = U.empty(nseq * nhead * s, s, gfmt)
    dQ = U.empty(T, d, dq_fmt)
    ws = L.new_workspace()
    b_p, b_q = hd ** -0.5, hd ** -0.5
    st, td, sq = (s * 3 * d, hd), (s * d, hd), (nhead * s * s, s * s)
    bt = L.attention_bwd_batch((nseq, nhead), td, sq, st, st, sq, td)
    L.us_attention_bwd(dCt[:s, :hd], P[:s], QKV[:s, d:d + hd], QKV[:s, 2 * d:2 * d + hd], b_p, sm, sm, b_q, dS[:s], dQ[:s, :hd], bt, ws)
    assert L.us_workspace_status(ws) == 0
    dC4 = dc_v.reshape(nseq, s, nhead, 64).transpose(0, 2, 1, 3)
    return dC4, p_host, K, V, dS, dQ, (b_p, sm, b_q)


@pytest.mark.parametrize("fmt", ["bf16", "fp16"])
@pytest.mark.parametrize("nseq,nhead,s", [(2, 3, 128), (1, 2, 200), (2, 2, 512), (1, 1, 72), (1, 2, 264), (3, 1, 8)])
def test_backward_scores_and_queries_against_the_oracle(fmt, nseq, nhead, s):
    dC4, p_host, K, V, dS, dQ, (b_p, sm, b_q) = _run_bwd(nseq, nhead, s, fmt, fmt, seed=71)
    dp = np.float64(np.float32(b_p)) * (dC4 @ V.transpose(0, 1, 3, 2))          # unrounded, as in the kernel
    ref = O.softmax_bwd(p_host, dp, sm, sm)
    got = U.host_values(dS).reshape(ref.shape)
    scale = np.abs(ref).max() + np.abs(dp).max()
    lim = U.ulp_of(ref, fmt) + 3e-6 * scale * max(1.0, s / 512)
    err = np.abs(got - ref)
    assert (err <= lim).all(), f"dS: {(err > lim).sum()} elements out, worst {err.max():.3e}"
    ref_q = (np.float64(np.float32(b_q)) * (got @ K)).transpose(0, 2, 1, 3).reshape(nseq * s, nhead * 64)   # from the device's own dS
    gq = U.host_values(dQ)
    lim_q = TOL * max(1.0, np.abs(ref_q).max()) + U.ulp_of(ref_q, fmt)
    assert (np.abs(gq - ref_q) <= lim_q).all(), f"dQ: worst {np.abs(gq - ref_q).max():.3e}"
    # and the whole chain against the oracle's single function, loosely (a one-ulp flip in dS moves dQ by ulp * |K|)
    ds_o, dq_o = O.attention_bwd_scores(dC4, p_host, K, V, b_p, sm, sm, b_q, fmt)
    assert np.abs(gq - dq_o.transpose(0, 2, 1, 3).reshape(gq.shape)).max() < 0.02 * max(1.0, np.abs(dq_o).max())


@pytest.mark.parametrize("dq_fmt", ["f32", "e5m2"])
def test_backward_query_gradient_formats(dq_fmt):
    nseq, nhead, s = 2, 2, 192
    dC4, p_host, K, V, dS, dQ, (b_p, sm, b_q) = _run_bwd(nseq, nhead, s, "bf16", dq_fmt, seed=72)
    got = U.host_values(dS).reshape(nseq, nhead, s, s)
    ref_q = (np.float64(np.float32(b_q)) * (got @ K)).transpose(0, 2, 1, 3).reshape(nseq * s, nhead * 64)
    gq = U.host_values(dQ)
    if dq_fmt == "f32":
        assert np.abs(gq - ref_q).max() <= TOL * max(1.0, np.abs(ref_q).max())
    else:
        fm = F.FORMATS[dq_fmt]
        dist = U.code_distance(F.quantise_codes(gq, fm), F.quantise_codes(ref_q, fm), dq_fmt)
        assert ((dist <= 1) | (np.abs(gq - F.quantise(ref_q, fm)) <= TOL * max(1.0, np.abs(ref_q).max()))).all()


def test_backward_bert_large_attention_shape_sampled_problems():
    nseq, nhead, s = 16, 16, 512
    dC4, p_host, K, V, dS, dQ, (b_p, sm, b_q) = _run_bwd(nseq, nhead, s, "bf16", "bf16", seed=73)
    rng = np.random.default_rng(8)
    probs = [(0, 0), (0, 15), (15, 0), (15, 15)] + [(int(rng.integers(16)), int(rng.integers(16))) for _ in range(4)]
    gq = U.host_values(dQ)
    for (i, j) in probs:
        dp = np.float64(np.float32(b_p)) * (dC4[i, j] @ V[i, j].T)
        ref = O.softmax_bwd(p_host[i, j], dp, sm, sm)
        got = U.host_values(dS[(i * nhead + j) * s:(i * nhead + j + 1) * s])
        lim = U.ulp_of(ref, "bf16") + 3e-6 * (np.abs(ref).max() + np.abs(dp).max())
        assert (np.abs(got - ref) <= lim).all(), (i, j)
        ref_q = np.float64(np.float32(b_q)) * (got @ K[i, j])
        g = gq[i * s:(i + 1) * s, j * 64:(j + 1) * 64]
        assert (np.abs(g - ref_q) <= TOL * max(1.0, np.abs(ref_q).max()) + U.ulp_of(ref_q, "bf16")).all(), (i, j)


@pytest.mark.parametrize("nseq,nhead,s", [(2, 3, 128), (1, 2, 208), (2, 2, 512), (1, 1, 80), (3, 1, 16)])
def test_backward_fp8_operands(nseq, nhead, s):
    """dC and dS as E5M2, P, K, V as E4M3: dS within one code of the oracle's softmax gradient on the unrounded dP,
    dQ against beta * dS K on the device's own stored dS."""
    dC4, p_host, K, V, dS, dQ, (b_p, sm, b_q) = _run_bwd(nseq, nhead, s, "e4m3", "e5m2", seed=74, gfmt="e5m2")
    dp = np.float64(np.float32(b_p)) * (dC4 @ V.transpose(0, 1, 3, 2))
    ref = O.softmax_bwd(p_host, dp, sm, sm)
    fm = F.FORMATS["e5m2"]
    got = U.host_values(dS).reshape(ref.shape)
    dist = U.code_distance(U.codes_of(dS).reshape(ref.shape), F.quantise_codes(ref, fm), "e5m2")
    scale = np.abs(ref).max() + np.abs(dp).max()
    ok = (dist <= 1) | (np.abs(got - F.quantise(ref, fm)) <= 3e-6 * scale)
    assert ok.all(), f"dS: code distance {dist.max()} at {(~ok).sum()} places"
    assert (dist > 0).mean() < 2e-3
    ref_q = (np.float64(np.float32(b_q)) * (got @ K)).transpose(0, 2, 1, 3).reshape(nseq * s, nhead * 64)
    gq = U.host_values(dQ)
    dq = U.code_distance(F.quantise_codes(gq, fm), F.quantise_codes(ref_q, fm), "e5m2")
    assert ((dq <= 1) | (np.abs(gq - F.quantise(ref_q, fm)) <= TOL * max(1.0, np.abs(ref_q).max()))).all()


def test_separate_contiguous_operands_and_repeatability():
    """Q, K, V as three contiguous [problems * s x 64] tensors (strides of a different shape than the packed QKV matrix),
    different query and key counts, and bit-identical outputs from two launches (no atomics anywhere)."""
    from paper_2303_11257_b200 import lib as L, synth
    nb0, nb1, s_q, s_k = 2, 3, 200, 328
    n = nb0 * nb1
    q, k, v = (synth.normal(81, i, (n * r, 64)) for i, r in ((0, s_q), (1, s_k), (2, s_k)))
    Q, K, V = U.to_device(q, "bf16"), U.to_device(k, "bf16"), U.to_device(v, "bf16")
    ws = L.new_workspace()
    a_s, sm, a_c = 0.125, float(s_k), s_k ** -0.5
    bt = L.attention_batch((nb0, nb1), (nb1 * s_q * 64, s_q * 64), (nb1 * s_k * 64, s_k * 64), (nb1 * s_k * 64, s_k * 64),
                           (nb1 * s_q * 64, s_q * 64), (nb1 * s_q * s_k, s_q * s_k))
    outs = []
    for _ in range(2):
        Cx, P = U.empty(n * s_q, 64, "bf16"), U.empty(n * s_q, s_k, "bf16")
        L.us_attention_fwd(Q[:s_q], K[:s_k], V[:s_k], a_s, sm, a_c, Cx[:s_q], P[:s_q], bt, ws)
        assert L.us_workspace_status(ws) == 0
        outs.append((U.codes_of(Cx), U.codes_of(P)))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    qv, kv, vv = (U.values_of(t, "bf16") for t in (q, k, v))
    p_ref, _ = O.attention_fwd(qv.reshape(n, s_q, 64), kv.reshape(n, s_k, 64), vv.reshape(n, s_k, 64), a_s, sm, a_c, "f64")
    p_dev = U.host_values(P).reshape(n, s_q, s_k)
    assert (np.abs(p_dev - p_ref) <= U.ulp_of(p_ref, "bf16") + 3e-6 * sm).all()
    c_ref = np.float64(np.float32(a_c)) * (p_dev @ vv.reshape(n, s_k, 64))
    got = U.host_values(Cx).reshape(n, s_q, 64)
    assert (np.abs(got - c_ref) <= TOL * max(1.0, np.abs(c_ref).max()) + U.ulp_of(c_ref, "bf16")).all()


@pytest.mark.parametrize("s_q,s_k", [(100, 100), (37, 413), (130, 33)])
def test_lengths_that_are_not_multiples_of_eight(s_q, s_k):
    """Key counts that end inside a 32-column chunk and inside a 16-byte piece (masking of the zero-filled key rows);
    P goes to a padded buffer so that its row pitch stays a multiple of 16 bytes."""
    from paper_2303_11257_b200 import lib as L, synth
    q, k, v = synth.normal(82, 0, (s_q, 64)), synth.normal(82, 1, (s_k, 64)), synth.normal(82, 2, (s_k, 64))
    Q, K, V = U.to_device(q, "fp16"), U.to_device(k, "fp16"), U.to_device(v, "fp16")
    ld = (s_k + 7) // 8 * 8
    P = U.empty(s_q, s_k, "fp16", ld=ld)
    Cx = U.empty(s_q, 64, "f32")
    ws = L.new_workspace()
    a_s, sm, a_c = 0.125, float(s_k), s_k ** -0.5
    bt = L.attention_batch((1, 1), (0, 0), (0, 0), (0, 0), (0, 0))
    L.us_attention_fwd(Q, K, V, a_s, sm, a_c, Cx, P, bt, ws)
    assert L.us_workspace_status(ws) == 0
    qv, kv, vv = (U.values_of(t, "fp16") for t in (q, k, v))
    p_ref, _ = O.attention_fwd(qv, kv, vv, a_s, sm, a_c, "f64")
    p_dev = U.host_values(P)
    assert (np.abs(p_dev - p_ref) <= U.ulp_of(p_ref, "fp16") + 3e-6 * sm).all()
    c_ref = np.float64(np.float32(a_c)) * (p_dev @ vv)
    assert np.abs(U.host_values(Cx) - c_ref).max() <= TOL * max(1.0, np.abs(c_ref).max())
    # backward on the same problem
    dc = synth.normal(82, 3, (s_q, 64))
    dCt, dS, dQ = U.to_device(dc, "fp16"), U.empty(s_q, s_k, "fp16", ld=ld), U.empty(s_q, 64, "f32")
    btb = L.attention_bwd_batch((1, 1), *[(0, 0)] * 6)
    L.us_attention_bwd(dCt, P, K, V, 0.125, sm, sm, 0.125, dS, dQ, btb, ws)
    assert L.us_workspace_status(ws) == 0
    dp = 0.125 * (U.values_of(dc, "fp16") @ vv.T)
    ref = O.softmax_bwd(p_dev, dp, sm, sm)
    got = U.host_values(dS)
    assert (np.abs(got - ref) <= U.ulp_of(ref, "fp16") + 3e-6 * (np.abs(ref).max() + np.abs(dp).max())).all()
    ref_q = 0.125 * (got @ kv)
    assert np.abs(U.host_values(dQ) - ref_q).max() <= TOL * max(1.0, np.abs(ref_q).max())
