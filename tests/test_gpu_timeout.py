"""The bounded-wait failure path of the linear kernels, driven without faulting the GPU.

us_test_linear_fwd_starved launches the forward kernel with its operand loads withheld and a short
wait limit: nothing is in flight, every role's wait runs out, the kernel raises the status word, frees its
tensor memory and returns.  The context must stay usable: after clearing the word, an ordinary call
on the same workspace has to match the oracle."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import scales as S
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3
US_ERR_TIMEOUT = 6


@pytest.mark.parametrize("shape", [(96, 64, 80), (520, 272, 1040)])      # one 128-row tile; CTA-pair tiles (256 x 256)
def test_starved_launch_times_out_and_the_next_call_is_correct(shape):
    from paper_2303_11257_b200 import lib as L, synth
    b, m, n = shape
    X, W, _ = synth.linear_tensors(b, m, n, 31)
    Xt, Wt = U.to_device(X, "e4m3"), U.to_device(W, "e4m3")
    alpha, _, _ = S.linear_scales(b, m, n)
    ws = L.new_workspace()
    junk = U.empty(b, n, "f32")
    L.us_test_linear_fwd_starved(Xt, Wt, float(alpha), junk, ws, wait_limit=2000)
    assert L.us_workspace_status(ws) == US_ERR_TIMEOUT            # synchronises: the kernel has returned by itself
    # the word is sticky until the caller clears it
    out = U.empty(b, n, "f32")
    L.us_linear_fwd(Xt, Wt, float(alpha), out, ws)
    assert L.us_workspace_status(ws) == US_ERR_TIMEOUT
    ref = O.linear_fwd(U.values_of(X, "e4m3"), U.values_of(W, "e4m3"), alpha)
    U.assert_close_stored(out, ref, "f32", TOL, "call after a timed-out launch")   # the kernel itself ran normally
    ws.zero_()
    out2 = U.empty(b, n, "bf16")
    L.us_linear_fwd(Xt, Wt, float(alpha), out2, ws)
    assert L.us_workspace_status(ws) == 0
    U.assert_close_stored(out2, ref, "bf16", TOL, "call after clearing the word")
    # tensor memory was released: a kernel that needs all of it (two 256-column accumulators per SM) still runs
    big = U.empty(512, 512, "f32")
    Xb, Wb, _ = synth.linear_tensors(512, 256, 512, 32)
    L.us_linear_fwd(U.to_device(Xb, "e4m3"), U.to_device(Wb, "e4m3"), 1.0 / 16, big, ws)
    assert L.us_workspace_status(ws) == 0
    refb = O.linear_fwd(U.values_of(Xb, "e4m3"), U.values_of(Wb, "e4m3"), 1.0 / 16)
    U.assert_close_stored(big, refb, "f32", TOL, "full-width kernel after the timed-out launch")


def test_starved_launch_argument_checks():
    from paper_2303_11257_b200 import lib as L
    ws = L.new_workspace()
    X, W, Y = U.empty(32, 64, "e4m3"), U.empty(64, 48, "e4m3"), U.empty(32, 48, "f32")
    for bad in (0, 1 << 17):
        with pytest.raises(L.UnitScaleError) as e:
            L.us_test_linear_fwd_starved(X, W, 1.0, Y, ws, wait_limit=bad)
        assert e.value.status == 1
    assert L.us_workspace_status(ws) == 0
