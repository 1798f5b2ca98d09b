"""us_softmax_fwd / us_softmax_bwd against the oracle.  The kernels compute exp through ex2.approx
in float32 (relative error about 2e-7), so values agree to 2e-6 relative to the row scale alpha
(beta * max|dP| for the gradient) plus the rounding of the output format."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from tests import util as U

pytestmark = pytest.mark.gpu


def _mods():
    from paper_2303_11257_b200 import lib, synth
    return lib, synth


@pytest.mark.parametrize("shape,ld", [((1, 8), None), ((5, 7), None), ((33, 512), None), ((130, 200), 208), ((9, 2048), None),
                                      ((4, 2056), None), ((3, 5000), None), ((64, 1024), 1040)])
@pytest.mark.parametrize("in_fmt,out_fmt", [("f32", "f32"), ("bf16", "bf16"), ("fp16", "f32"), ("f32", "e4m3")])
def test_softmax_fwd_bwd(shape, ld, in_fmt, out_fmt):
    L, synth = _mods()
    rows, cols = shape
    alpha = beta = float(cols)
    s = synth.normal(21, 0, shape, 2.0)
    St = U.to_device(s, in_fmt, ld)
    P = U.empty(rows, cols, out_fmt, ld)
    L.us_softmax_fwd(St, alpha, P)
    ref = O.softmax_fwd(U.values_of(s, in_fmt), alpha)
    U.assert_close_stored(P, ref, out_fmt, 3e-6 * alpha, "softmax fwd")
    if out_fmt == "f32":
        assert np.allclose(U.host_values(P).sum(axis=-1), alpha, rtol=1e-5)
    # backward from a stored scaled output (16-bit or float32) and an upstream gradient
    p_fmt = in_fmt
    p_host = O.softmax_fwd(s.astype(np.float64), alpha).astype(np.float32)
    g = synth.normal(21, 1, shape)
    Pt, Gt = U.to_device(p_host, p_fmt, ld), U.to_device(g, in_fmt, ld)
    dS = U.empty(rows, cols, out_fmt if out_fmt != "e4m3" else "e5m2", ld)
    L.us_softmax_bwd(Pt, Gt, alpha, beta, dS)
    gv = U.values_of(g, in_fmt)
    refb = O.softmax_bwd(U.values_of(p_host, p_fmt), gv, alpha, beta)
    fmt_b = out_fmt if out_fmt != "e4m3" else "e5m2"
    scale = np.abs(refb).max() + np.abs(gv).max()
    U.assert_close_stored(dS, refb, fmt_b, 3e-6 * scale * max(1.0, cols / 512), "softmax bwd")


@pytest.mark.parametrize("shape,ld", [((5, 8), None), ((33, 512), None), ((130, 200), 208), ((7, 100), 112), ((4, 2056), None)])
def test_softmax_bwd_from_an_fp8_stored_output(shape, ld):
    """P as the E4M3 tensor an FP8 matmul consumes, dP in BF16, dS written as E5M2."""
    L, synth = _mods()
    rows, cols = shape
    alpha = beta = float(cols)
    p_host = O.softmax_fwd(synth.normal(23, 0, shape, 1.0).astype(np.float64), alpha).astype(np.float32)
    g = synth.normal(23, 1, shape)
    Pt, Gt = U.to_device(p_host, "e4m3", ld), U.to_device(g, "bf16", ld)
    gv, pv = U.values_of(g, "bf16"), U.values_of(p_host, "e4m3")
    refb = O.softmax_bwd(pv, gv, alpha, beta)
    scale = np.abs(refb).max() + np.abs(gv).max()
    for out_fmt in ("f32", "e5m2"):
        dS = U.empty(rows, cols, out_fmt, ld)
        L.us_softmax_bwd(Pt, Gt, alpha, beta, dS)
        U.assert_close_stored(dS, refb, out_fmt, 3e-6 * scale * max(1.0, cols / 512), "softmax bwd from FP8 P")


def test_attention_shape_statistics():
    """16 x 16 x 512 rows of 512 scores would be 67 M elements; a 1/16 sample keeps the test quick."""
    L, synth = _mods()
    rows, s = 8192, 512
    S = torch.from_numpy(synth.normal(22, 0, (rows, s), 0.125)).cuda().to(torch.bfloat16)
    P = torch.empty_like(S)
    L.us_softmax_fwd(S, float(s), P)
    assert abs(P.float().mean().item() - 1) < 1e-3 and P.float().std().item() < 0.2
    G = torch.from_numpy(synth.normal(22, 1, (rows, s))).cuda().to(torch.bfloat16)
    dS = torch.empty_like(S)
    L.us_softmax_bwd(P, G, float(s), float(s), dS)
    assert abs(dS.float().std().item() - 1) < 0.05


def test_softmax_argument_errors():
    L, _ = _mods()
    a = torch.zeros((4, 8), device="cuda")
    with pytest.raises(L.UnitScaleError) as e:
        L.us_softmax_fwd(a, 8.0, torch.zeros((4, 9), device="cuda"))
    assert e.value.status == 1
    with pytest.raises(L.UnitScaleError) as e:
        L.us_softmax_bwd(a, a, 0.0, 1.0, a)
    assert e.value.status == 1
    with pytest.raises(L.UnitScaleError) as e:
        L.us_softmax_fwd(U.empty(4, 16, "e4m3"), 8.0, a)
    assert e.value.status == 2
    L.us_softmax_fwd(torch.zeros((0, 8), device="cuda"), 8.0, torch.zeros((0, 8), device="cuda"))
