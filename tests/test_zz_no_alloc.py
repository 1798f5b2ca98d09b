"""us_linear_fwd_static_ws: the entry point for callers that cannot allocate device memory.

Such callers (a plug-in given only its inputs and outputs, a serving loop that forbids
allocation while running, a process whose framework owns all device memory) cannot create the
workspace that us_linear_fwd asks for, so the library carries a small built-in scratch array
for them.  The test drives the new entry point through the C ABI twice in a row -- the second
call finds the array as the first one left it -- and checks each result against the ordinary
us_linear_fwd on the same operands and against the oracle, at the tolerance the linear-op tests
use.  It must pass on its own in a fresh process as well as after every other test, hence a file
that sorts last.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import ops as O
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3
US_ERR_TIMEOUT = 6


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
        ref = O.linear_fwd(U.values_of(X, "e4m3"), U.values_of(W, "e4m3"), np.float32(alpha))
        U.assert_close_stored(got, ref, "f32", TOL, f"call {call} against the oracle")
    # fused epilogue through the same entry point, third use of the shared array
    H = U.empty(b, n, "bf16")
    A1, A2 = U.empty(b, n, "e4m3"), U.empty(b, n, "e4m3")
    ep = L.epilogue(act=L.US_ACT_GELU, act_out_scale=1.7, aux=H)
    L.us_linear_fwd(Xt, Wt, alpha, A1, ws, ep)
    L.us_linear_fwd_static_ws(Xt, Wt, alpha, A2, ep)
    torch.cuda.synchronize()
    assert U.code_distance(U.codes_of(A2), U.codes_of(A1), "e4m3").max() <= 1
    U.assert_close_stored(A2, O.gelu_fwd(ref, 1.0, 1.7), "e4m3", TOL, "fused GELU through the built-in scratch")


def test_static_workspace_starts_each_call_from_a_clear_status_word():
    """The built-in array keeps what the previous call left.  Leave a raised status word in it (a
    launch whose waits run out, made on that very array) and check that the next call through the
    entry point clears it and is correct, while a call that fails its host checks leaves it alone."""
    from paper_2303_11257_b200 import lib as L
    from paper_2303_11257_b200 import synth
    b, m, n = 200, 144, 336
    X, W, _ = synth.linear_tensors(b, m, n, 23)
    Xt, Wt = U.to_device(X, "e4m3"), U.to_device(W, "e4m3")
    alpha, _, _ = L.us_scales_linear(b, m, n)
    out = U.empty(b, n, "f32")
    ws_ptr = L.us_linear_fwd_static_ws(Xt, Wt, alpha, out)
    assert L.us_workspace_status_ptr(ws_ptr) == 0
    # raise the word in the built-in array itself
    raw = L.raw()
    st = raw.us_test_linear_fwd_starved(C.byref(L.mat(Xt)), C.byref(L.mat(Wt)), alpha, C.byref(L.mat(out)),
                                        ws_ptr, L.us_workspace_bytes(), 2000, None)
    assert st == 0
    assert L.us_workspace_status_ptr(ws_ptr) == US_ERR_TIMEOUT
    # a call that fails validation enqueues nothing: the word stays raised
    with pytest.raises(L.UnitScaleError):
        L.us_linear_fwd_static_ws(Xt, U.empty(m + 1, n, "e4m3"), alpha, out)
    assert L.us_workspace_status_ptr(ws_ptr) == US_ERR_TIMEOUT
    # a valid call starts from a clear word and computes the right thing
    out.zero_()
    assert L.us_linear_fwd_static_ws(Xt, Wt, alpha, out) == ws_ptr
    assert L.us_workspace_status_ptr(ws_ptr) == 0
    ref = O.linear_fwd(U.values_of(X, "e4m3"), U.values_of(W, "e4m3"), np.float32(alpha))
    U.assert_close_stored(out, ref, "f32", TOL, "call after a raised status word")


def test_static_workspace_entry_point_validates_like_us_linear_fwd():
    from paper_2303_11257_b200 import lib as L
    with pytest.raises(L.UnitScaleError) as e:
        L.us_linear_fwd_static_ws(U.empty(32, 64, "e4m3"), U.empty(65, 48, "e4m3"), 1.0, U.empty(32, 48, "f32"))
    assert e.value.status == 1
