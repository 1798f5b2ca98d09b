"""us_linear_fwd_static_ws: the entry point for callers that cannot allocate device memory.

Such callers (a plug-in given only its inputs and outputs, a serving loop that forbids
allocation while running, a process whose framework owns all device memory) cannot create the
workspace that us_linear_fwd asks for, so the library carries a small built-in scratch array
for them.  The test drives the new entry point through the C ABI twice in a row -- the second
call finds the array as the first one left it -- and checks each result against the ordinary
us_linear_fwd on the same operands, at the tolerance the linear-op tests use.  It must pass on
its own in a fresh process as well as after every other test, hence a file that sorts last.
"""
import numpy as np
import pytest
import torch

from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3


def test_static_workspace_entry_point_matches_us_linear_fwd_twice():
    from paper_2303_11257_b200 import lib as L
    from paper_2303_11257_b200 import synth
    for call, (b, m, n, seed) in enumerate(((264, 400, 304, 21), (256, 128, 512, 22))):
        X, W, _ = synth.linear_tensors(b, m, n, seed)
        Xt, Wt = U.to_device(X, "e4m3"), U.to_device(W, "e4m3")
        alpha, _, _ = L.us_scales_linear(b, m, n)
        want = U.empty(b, n, "f32")
        ws = L.new_workspace()
        L.us_linear_fwd(Xt, Wt, alpha, want, ws)
        assert L.us_workspace_status(ws) == 0
        got = U.empty(b, n, "f32")
        ws_ptr = L.us_linear_fwd_static_ws(Xt, Wt, alpha, got)
        assert ws_ptr and L.us_workspace_status_ptr(ws_ptr) == 0
        diff = (got - want).abs().max().item()
        assert diff <= TOL, f"call {call}: |static_ws - us_linear_fwd| = {diff}"
        assert abs(got.std().item() - 1) < 0.1                      # and it is a real result, not zeros
    # fused epilogue through the same entry point, third use of the shared array
    H = U.empty(b, n, "bf16")
    A1, A2 = U.empty(b, n, "e4m3"), U.empty(b, n, "e4m3")
    ep = L.epilogue(act=L.US_ACT_GELU, act_out_scale=1.7, aux=H)
    L.us_linear_fwd(Xt, Wt, alpha, A1, ws, ep)
    L.us_linear_fwd_static_ws(Xt, Wt, alpha, A2, ep)
    torch.cuda.synchronize()
    assert U.code_distance(U.codes_of(A2), U.codes_of(A1), "e4m3").max() <= 1


def test_static_workspace_entry_point_validates_like_us_linear_fwd():
    from paper_2303_11257_b200 import lib as L
    with pytest.raises(L.UnitScaleError) as e:
        L.us_linear_fwd_static_ws(U.empty(32, 64, "e4m3"), U.empty(65, 48, "e4m3"), 1.0, U.empty(32, 48, "f32"))
    assert e.value.status == 1
