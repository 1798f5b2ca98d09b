"""Batched linear ops on the (sequence, head) problems of scaled dot-product attention: scores
Q K^T (backward-input form), context P V (forward form) and P^T dO (backward-weight form), with the
heads taken as strided column slices of a [tokens x 3 d] QKV matrix."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _mods():
    from paper_2303_11257_b200 import lib, synth
    return lib, synth


@pytest.mark.parametrize("fmt", ["bf16", "fp16", "e4m3"])
@pytest.mark.parametrize("nseq,nhead,slen,hd", [(2, 3, 160, 64), (1, 2, 512, 64), (3, 1, 272, 128)])
def test_attention_shaped_batches(fmt, nseq, nhead, slen, hd):
    L, synth = _mods()
    d = nhead * hd
    T = nseq * slen
    qkv = synth.normal(31, 0, (T, 3 * d))
    p_all = np.abs(synth.normal(31, 1, (nseq * nhead * slen, slen)))         # stand-in for scaled softmax outputs
    do = synth.normal(31, 2, (T, d))
    QKV, P, dO = U.to_device(qkv, fmt), U.to_device(p_all, fmt), U.to_device(do, fmt)
    qkv_v, p_v, do_v = U.values_of(qkv, fmt), U.values_of(p_all, fmt), U.values_of(do, fmt)
    ws = L.new_workspace()
    alpha_s, alpha_c, beta_w = hd ** -0.5, slen ** -0.5, slen ** -0.5
    Q, K, V = QKV[:slen, 0:hd], QKV[:slen, d:d + hd], QKV[:slen, 2 * d:2 * d + hd]
    qkv_stride = (slen * 3 * d, hd)
    sq_stride = (nhead * slen * slen, slen * slen)
    # scores S = alpha Q K^T
    S = U.empty(nseq * nhead * slen, slen, "f32")
    bt = L.batch((nseq, nhead), qkv_stride, qkv_stride, sq_stride)
    L.us_linear_bwd_x_batched(Q, K, alpha_s, S[:slen], bt, ws)
    # context O = alpha P V, written head by head into a [T x d] matrix
    Oc = U.empty(T, d, "f32")
    bt = L.batch((nseq, nhead), sq_stride, qkv_stride, (slen * d, hd))
    L.us_linear_fwd_batched(P[:slen], V, alpha_c, Oc[:slen, :hd], bt, ws)
    # dV = beta P^T dO
    dV = U.empty(T, d, "bf16")
    bt = L.batch((nseq, nhead), sq_stride, (slen * d, hd), (slen * d, hd))
    L.us_linear_bwd_w_batched(P[:slen], dO[:slen, :hd], beta_w, dV[:slen, :hd], bt, ws)
    assert L.us_workspace_status(ws) == 0
    S_h, O_h, dV_h = U.host_values(S), U.host_values(Oc), U.host_values(dV)
    for i in range(nseq):
        for j in range(nhead):
            r = slice(i * slen, (i + 1) * slen)
            q, k, v = (qkv_v[r, o + j * hd:o + (j + 1) * hd] for o in (0, d, 2 * d))
            pr = slice((i * nhead + j) * slen, (i * nhead + j + 1) * slen)
            assert np.abs(S_h[pr] - O.linear_bwd_x(q, k, alpha_s)).max() <= TOL
            c = slice(j * hd, (j + 1) * hd)
            ref_o = O.linear_fwd(p_v[pr], v, alpha_c)
            assert np.abs(O_h[r, c] - ref_o).max() <= TOL * max(1.0, np.abs(ref_o).max())
            ref_dv = O.linear_bwd_w(p_v[pr], do_v[r, c], beta_w)
            assert np.all(np.abs(dV_h[r, c] - ref_dv) <= TOL + U.ulp_of(ref_dv, "bf16"))


def test_batched_argument_errors():
    L, _ = _mods()
    ws = L.new_workspace()
    A, B, out = U.empty(64, 64, "bf16"), U.empty(64, 64, "bf16"), U.empty(64, 64, "f32")
    bt = L.batch((2, 1), (64 * 64, 0), (64 * 64, 0), (64 * 64 + 1, 0))
    with pytest.raises(L.UnitScaleError) as e:
        L.us_linear_fwd_batched(A, B, 1.0, out, bt, ws)
    assert e.value.status == 3                      # output stride not a multiple of 16 bytes
    bt = L.batch((0, 1), (0, 0), (0, 0), (0, 0))
    with pytest.raises(L.UnitScaleError) as e:
        L.us_linear_fwd_batched(A, B, 1.0, out, bt, ws)
    assert e.value.status == 1
