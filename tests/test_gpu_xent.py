"""us_softmax_xent_fwd / us_softmax_xent_bwd against the oracle.  exp and log go through ex2.approx /
lg2.approx in float32: 2e-6 relative to the row's score range for the log-likelihood, 3e-6 * beta * |g|
for the gradient, plus the rounding of the output format."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import scales as S
from tests import util as U

pytestmark = pytest.mark.gpu


def _mods():
    from paper_2303_11257_b200 import lib, synth
    return lib, synth


@pytest.mark.parametrize("shape,ld", [((1, 8), None), ((5, 7), None), ((33, 512), None), ((130, 200), 208), ((9, 2048), None),
                                      ((4, 2056), None), ((3, 30522), None)])
@pytest.mark.parametrize("in_fmt,out_fmt", [("f32", "f32"), ("bf16", "bf16"), ("fp16", "e5m2")])
def test_softmax_xent_fwd_bwd(shape, ld, in_fmt, out_fmt):
    L, synth = _mods()
    rows, s = shape
    x = synth.normal(31, 0, shape, 2.0)
    rng = np.random.default_rng(31)
    t = rng.integers(0, s, rows).astype(np.int32)
    g = synth.normal(31, 1, (1, rows))[0]
    beta = S.softmax_xent_scales(s)[1] if s > 1 else 1.0
    Xt = U.to_device(x, in_fmt, ld)
    xv = U.values_of(x, in_fmt)
    tt, gt = torch.from_numpy(t).cuda(), torch.from_numpy(g).cuda()
    out = torch.empty(rows, device="cuda")
    L.us_softmax_xent_fwd(Xt, tt, out)
    ref = O.softmax_xent_fwd(xv, t)
    assert np.abs(out.cpu().numpy() - ref).max() <= 4e-6 * (1 + np.abs(ref).max())
    dX = U.empty(rows, s, out_fmt, ld)
    L.us_softmax_xent_bwd(Xt, tt, gt, beta, dX)
    refb = O.softmax_xent_bwd(xv, t, g.astype(np.float64), beta)
    U.assert_close_stored(dX, refb, out_fmt, 3e-6 * beta * np.abs(g).max(), "xent bwd")
    # g = NULL means ones
    L.us_softmax_xent_bwd(Xt, tt, None, beta, dX)
    U.assert_close_stored(dX, O.softmax_xent_bwd(xv, t, np.ones(rows), beta), out_fmt, 3e-6 * beta, "xent bwd, unit g")


def test_softmax_xent_unit_scale_and_bad_targets():
    L, synth = _mods()
    rows, s = 512, 4096
    X = torch.from_numpy(synth.normal(32, 0, (rows, s), 0.01)).cuda()
    t = torch.from_numpy(np.random.default_rng(32).integers(0, s, rows).astype(np.int32)).cuda()
    dX = torch.empty_like(X)
    L.us_softmax_xent_bwd(X, t, None, S.softmax_xent_scales(s)[1], dX)
    assert abs(dX.pow(2).mean().sqrt().item() - 1) < 0.01            # table row: beta = s / sqrt(s - 1)
    assert dX.sum(dim=1).abs().max().item() < 1e-3
    bad = t.clone(); bad[3] = s; bad[5] = -1
    out = torch.empty(rows, device="cuda")
    L.us_softmax_xent_fwd(X, bad, out)
    assert torch.isnan(out[[3, 5]]).all() and torch.isfinite(out[[0, 1, 2, 4]]).all()
    L.us_softmax_xent_bwd(X, bad, None, 1.0, dX)
    assert (dX[3] < 0).all() and (dX[5] < 0).all()                    # no one-hot term: -softmax only
    with pytest.raises(L.UnitScaleError) as e:
        L.us_softmax_xent_bwd(X, t, None, 1.0, torch.empty((rows, s + 8), device="cuda"))
    assert e.value.status == 1
