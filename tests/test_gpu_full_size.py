"""Parity at the stated sizes of the configurations, in the launch shapes the benchmark uses.

* the BERT-large FFN block (8192 x 1024 x 4096) with BF16 and FP16 operands: sampled token rows of the
  forward pass and the input gradient, every element of both weight gradients;
* each 16-bit linear op at a shape whose contraction is 8192 long;
* the row-wise kernels (scaled softmax, scaled layer norm) with more rows than the device holds
  resident warps, so that the persistent warps take several rows each: every element compared;
* the batched attention GEMMs at 16 x 16 problems of 512 x 64: sampled problems including the first
  and last of each batch index."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import ops as O
from oracle import scales as S
from tests import util as U
from tests.test_gpu_ffn import _compare_chain, _run

pytestmark = pytest.mark.gpu
TOL = 2e-3


@pytest.mark.parametrize("operand", ["bf16", "fp16"])
def test_ffn_bert_large_16bit_operands(operand):
    from paper_2303_11257_b200 import synth
    shape = synth.FFN_BERT_LARGE
    blk, (X, W1, W2, G) = _run(shape, operand, seed=2)
    T, d, f = shape.tokens, shape.d_model, shape.d_ff
    sc = O.FFNScales.unconstrained(T, d, f)
    fm = F.FORMATS[operand]
    assert np.array_equal(U.codes_of(blk.Xq), F.quantise_codes(X, fm))
    assert np.array_equal(U.codes_of(blk.W2q), F.quantise_codes(W2, fm))
    rng = np.random.default_rng(3)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, T - 1], rng.integers(0, T, 26)]))
    # the forward pass and the input gradient are row-wise independent given the weights
    r = O.ffn_block(X[rows], W1, W2, G[rows], sc, operand=operand)
    _compare_chain(blk, r, None, operand, rows=rows, weights=False)
    # weight gradients: the device's own stored operands through the oracle's single op, every element
    Hv = U.host_values
    sc_w = np.float32(blk.sc.beta_w)
    U.assert_close_stored(blk.dW2, O.linear_bwd_w(Hv(blk.Aq), Hv(blk.Gq), sc_w), "f32", TOL, "dW2")
    U.assert_close_stored(blk.dW1, O.linear_bwd_w(Hv(blk.Xq), Hv(blk.dHq), sc_w), "f32", TOL, "dW1")
    assert abs(blk.H.float().std().item() - 1) < 0.02


@pytest.mark.parametrize("fmt", ["bf16", "fp16"])
@pytest.mark.parametrize("op,b,m,n", [("fwd", 520, 8192, 400), ("bwd_x", 400, 520, 8192), ("bwd_w", 8192, 272, 528)])
def test_16bit_linear_with_a_long_contraction(fmt, op, b, m, n):
    from paper_2303_11257_b200 import lib as L, synth
    X, W, G = synth.linear_tensors(b, m, n, 61)
    a, bx, bw = S.linear_scales(b, m, n)
    A, B, scale, ref_fn, oshape = {"fwd": (X, W, a, O.linear_fwd, (b, n)), "bwd_x": (G, W, bx, O.linear_bwd_x, (b, m)),
                                   "bwd_w": (X, G, bw, O.linear_bwd_w, (m, n))}[op]
    ws = L.new_workspace()
    ref = ref_fn(U.values_of(A, fmt), U.values_of(B, fmt), scale)
    for out_fmt in ("f32", fmt):
        out = U.empty(oshape[0], oshape[1], out_fmt)
        getattr(L, "us_linear_" + op)(U.to_device(A, fmt), U.to_device(B, fmt), float(scale), out, ws)
        U.assert_close_stored(out, ref, out_fmt, TOL, f"{op} {fmt} -> {out_fmt}")
    assert L.us_workspace_status(ws) == 0


@pytest.mark.parametrize("rows,cols", [(8192, 512), (9000, 1024), (8200, 200)])
def test_softmax_more_rows_than_resident_warps(rows, cols):
    from paper_2303_11257_b200 import lib as L, synth
    alpha = beta = float(cols)
    s = synth.normal(62, 0, (rows, cols), 2.0)
    St = U.to_device(s, "bf16")
    P = U.empty(rows, cols, "bf16")
    L.us_softmax_fwd(St, alpha, P)
    sv = U.values_of(s, "bf16")
    U.assert_close_stored(P, O.softmax_fwd(sv, alpha), "bf16", 3e-6 * alpha, "softmax fwd")
    g = synth.normal(62, 1, (rows, cols))
    gv = U.values_of(g, "bf16")
    Gt = U.to_device(g, "bf16")
    # backward from the stored BF16 output, and from an output stored as E4M3 for an FP8 matmul
    for p_fmt, out_fmt in (("bf16", "bf16"), ("e4m3", "e5m2"), ("e4m3", "bf16")):
        p_host = O.softmax_fwd(sv, alpha).astype(np.float32)
        Pt = U.to_device(p_host, p_fmt)
        pv = U.values_of(p_host, p_fmt)
        dS = U.empty(rows, cols, out_fmt)
        L.us_softmax_bwd(Pt, Gt, alpha, beta, dS)
        ref = O.softmax_bwd(pv, gv, alpha, beta)
        scale = np.abs(ref).max() + np.abs(gv).max()
        U.assert_close_stored(dS, ref, out_fmt, 3e-6 * scale * max(1.0, cols / 512), f"softmax bwd P {p_fmt} -> {out_fmt}")


@pytest.mark.parametrize("rows,cols,g_fmt", [(8192, 1024, "bf16"), (8192, 1024, "f32"), (9001, 768, "bf16"), (8200, 2048, "bf16")])
def test_layer_norm_more_rows_than_resident_warps(rows, cols, g_fmt):
    from paper_2303_11257_b200 import lib as L, synth
    X = F.quantise(synth.normal(63, 0, (rows, cols), 1.5) + np.float32(0.5), F.BF16).astype(np.float32)
    G = synth.normal(63, 1, (rows, cols))
    if g_fmt != "f32":
        G = F.quantise(G, F.FORMATS[g_fmt]).astype(np.float32)
    w = (1 + 0.25 * synth.normal(63, 2, (1, cols))).astype(np.float32)
    c = (0.1 * synth.normal(63, 3, (1, cols))).astype(np.float32)
    eps = 1e-5
    wt, ct = torch.from_numpy(w[0]).cuda(), torch.from_numpy(c[0]).cuda()
    Xt = U.to_device(X, "bf16")
    Y = U.empty(rows, cols, "bf16")
    L.us_layer_norm_fwd(Xt, wt, ct, eps, Y)
    U.assert_close_stored(Y, O.layer_norm_fwd(X, w, c, np.float32(eps)), "bf16", 2e-5, "layer norm fwd")
    beta_wc = float(np.float32(rows ** -0.5))
    dX, dw, dc = U.empty(rows, cols, "bf16"), torch.empty(cols, device="cuda"), torch.empty(cols, device="cuda")
    ws = torch.empty(L.us_layer_norm_bwd_workspace_bytes(rows, cols), dtype=torch.uint8, device="cuda")
    L.us_layer_norm_bwd(Xt, wt, U.to_device(G, g_fmt), eps, 1.0, beta_wc, dX, dw, dc, ws)
    rdX, rdw, rdc = O.layer_norm_bwd(X, w, G, np.float32(eps), 1.0, beta_wc)
    scale = 1.0 / np.sqrt(X.var(axis=1).min() + eps)
    U.assert_close_stored(dX, rdX, "bf16", 3e-5 * max(1.0, scale), "layer norm dX")
    tol = 8 * (2e-6 * np.sqrt(rows) + 1e-6)
    assert np.abs(dw.cpu().numpy() - rdw.reshape(-1)).max() <= tol
    assert np.abs(dc.cpu().numpy() - rdc.reshape(-1)).max() <= tol


@pytest.mark.parametrize("fmt", ["bf16", "e4m3"])
def test_batched_gemms_at_the_attention_problem_count(fmt):
    """16 sequences x 16 heads, 512 tokens x 64 per head: 256 problems per launch, all three forms."""
    from paper_2303_11257_b200 import lib as L, synth
    nseq, nhead, slen, hd = 16, 16, 512, 64
    d, T = nhead * hd, nseq * slen
    qkv = synth.normal(64, 0, (T, 3 * d))
    do = synth.normal(64, 2, (T, d))
    QKV, dO = U.to_device(qkv, fmt), U.to_device(do, fmt)
    qkv_v, do_v = U.values_of(qkv, fmt), U.values_of(do, fmt)
    ws = L.new_workspace()
    alpha_s, alpha_c, beta_w = hd ** -0.5, slen ** -0.5, slen ** -0.5
    Q, K, V = QKV[:slen, 0:hd], QKV[:slen, d:d + hd], QKV[:slen, 2 * d:2 * d + hd]
    qkv_stride = (slen * 3 * d, hd)
    sq_stride = (nhead * slen * slen, slen * slen)
    S_out = U.empty(nseq * nhead * slen, slen, "bf16")
    L.us_linear_bwd_x_batched(Q, K, alpha_s, S_out[:slen], L.batch((nseq, nhead), qkv_stride, qkv_stride, sq_stride), ws)
    # P: a positive tensor of the softmax output's scale, stored in the operand format (made on the device from S)
    P = torch.empty(nseq * nhead * slen, slen, device="cuda", dtype=U.TORCH_OF[fmt])
    L.us_softmax_fwd(S_out, float(slen), P)
    Oc = U.empty(T, d, "f32")
    L.us_linear_fwd_batched(P[:slen], V, alpha_c, Oc[:slen, :hd], L.batch((nseq, nhead), sq_stride, qkv_stride, (slen * d, hd)), ws)
    dV = U.empty(T, d, "bf16")
    L.us_linear_bwd_w_batched(P[:slen], dO[:slen, :hd], beta_w, dV[:slen, :hd],
                              L.batch((nseq, nhead), sq_stride, (slen * d, hd), (slen * d, hd)), ws)
    assert L.us_workspace_status(ws) == 0
    rng = np.random.default_rng(5)
    problems = {(0, 0), (0, nhead - 1), (nseq - 1, 0), (nseq - 1, nhead - 1)}
    problems |= {(i, int(rng.integers(nhead))) for i in range(nseq)} | {(int(rng.integers(nseq)), j) for j in range(nhead)}
    assert len(problems) >= 32
    O_h, dV_h = U.host_values(Oc), U.host_values(dV)
    for (i, j) in sorted(problems):
        r = slice(i * slen, (i + 1) * slen)
        q, k, v = (qkv_v[r, o + j * hd:o + (j + 1) * hd] for o in (0, d, 2 * d))
        pr = slice((i * nhead + j) * slen, (i * nhead + j + 1) * slen)
        ref_s = O.linear_bwd_x(q, k, alpha_s)
        assert np.all(np.abs(U.host_values(S_out[pr]) - ref_s) <= TOL + U.ulp_of(ref_s, "bf16")), (i, j)
        p_v = U.host_values(P[pr])
        c = slice(j * hd, (j + 1) * hd)
        ref_o = O.linear_fwd(p_v, v, alpha_c)
        assert np.abs(O_h[r, c] - ref_o).max() <= TOL * max(1.0, np.abs(ref_o).max()), (i, j)
        ref_dv = O.linear_bwd_w(p_v, do_v[r, c], beta_w)
        assert np.all(np.abs(dV_h[r, c] - ref_dv) <= TOL * max(1.0, np.abs(ref_dv).max()) + U.ulp_of(ref_dv, "bf16")), (i, j)
