"""us_layer_norm_fwd / us_layer_norm_bwd against the oracle."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import ops as O
from tests import util as U

pytestmark = pytest.mark.gpu


def _lib():
    from paper_2303_11257_b200 import lib
    return lib


def _inputs(seed, rows, cols, x_fmt, shift=0.5, spread=1.5):
    from paper_2303_11257_b200 import synth
    X = synth.normal(seed, 0, (rows, cols), spread) + np.float32(shift)
    G = synth.normal(seed, 1, (rows, cols), 1.0)
    w = (1 + 0.25 * synth.normal(seed, 2, (1, cols), 1.0)).astype(np.float32)
    c = (0.1 * synth.normal(seed, 3, (1, cols), 1.0)).astype(np.float32)
    if x_fmt != "f32":
        X = F.quantise(X, F.FORMATS[x_fmt]).astype(np.float32)
        G = F.quantise(G, F.FORMATS[x_fmt]).astype(np.float32)
    return X, G, w, c


CASES = [(1, 8, "f32", None), (5, 24, "f32", None), (33, 100, "f32", None), (64, 256, "bf16", None), (130, 768, "bf16", 800),
         (257, 1024, "bf16", None), (19, 1000, "fp16", 1008), (40, 2048, "bf16", None), (9, 4096, "f32", None), (6, 2056, "bf16", None)]


@pytest.mark.parametrize("rows,cols,x_fmt,ld", CASES)
@pytest.mark.parametrize("out_fmt", ["f32", "bf16", "e4m3"])
def test_layer_norm_forward(rows, cols, x_fmt, ld, out_fmt):
    L = _lib()
    X, _, w, c = _inputs(3, rows, cols, x_fmt)
    eps = 1e-5
    Y = U.empty(rows, cols, out_fmt, ld)
    L.us_layer_norm_fwd(U.to_device(X, x_fmt, ld), torch.from_numpy(w[0]).cuda(), torch.from_numpy(c[0]).cuda(), eps, Y)
    ref = O.layer_norm_fwd(X, w, c, np.float32(eps))
    # float32 arithmetic on O(1) values with sums over up to 4096 elements: 2e-5 absolute before the output rounding
    U.assert_close_stored(Y, ref, out_fmt, 2e-5)


@pytest.mark.parametrize("rows,cols,x_fmt,ld", CASES)
def test_layer_norm_backward(rows, cols, x_fmt, ld):
    L = _lib()
    X, G, w, _ = _inputs(4, rows, cols, x_fmt)
    eps, beta_x, beta_wc = 1e-5, 1.0, float(np.float32(rows ** -0.5))
    dX = U.empty(rows, cols, "f32", ld)
    dw = torch.empty(cols, device="cuda")
    dc = torch.empty(cols, device="cuda")
    ws = torch.empty(max(L.us_layer_norm_bwd_workspace_bytes(rows, cols), 16), dtype=torch.uint8, device="cuda")
    args = (U.to_device(X, x_fmt, ld), torch.from_numpy(w[0]).cuda(), U.to_device(G, x_fmt, ld), eps, beta_x, beta_wc)
    L.us_layer_norm_bwd(*args, dX, dw, dc, ws)
    rdX, rdw, rdc = O.layer_norm_bwd(X, w, G, np.float32(eps), beta_x, beta_wc)
    scale = 1.0 / np.sqrt(X.var(axis=1).min() + eps)          # dX grows with 1 / sigma
    assert np.abs(U.host_values(dX) - rdX).max() <= 3e-5 * max(1.0, scale)
    # column sums of `rows` products of O(1) values in float32, scaled by rows^-1/2
    tol = 2e-6 * np.sqrt(rows) + 1e-6
    assert np.abs(dw.cpu().numpy() - rdw.reshape(-1)).max() <= tol * 8
    assert np.abs(dc.cpu().numpy() - rdc.reshape(-1)).max() <= tol * 8
    # a second call gives bit-identical results (fixed summation order)
    dX2, dw2, dc2 = U.empty(rows, cols, "f32", ld), torch.empty_like(dw), torch.empty_like(dc)
    L.us_layer_norm_bwd(*args, dX2, dw2, dc2, ws)
    assert torch.equal(dw, dw2) and torch.equal(dc, dc2) and torch.equal(dX.contiguous(), dX2.contiguous())


def test_layer_norm_large_offset_rows_keep_their_variance():
    """Rows with a mean far above their spread: the variance about the mean survives float32
    (mean(x^2) - mu^2 in float32 would not)."""
    L = _lib()
    X, _, w, c = _inputs(5, 16, 1024, "f32", shift=300.0, spread=0.5)
    Y = U.empty(16, 1024, "f32")
    L.us_layer_norm_fwd(torch.from_numpy(X).cuda(), torch.from_numpy(w[0]).cuda(), torch.from_numpy(c[0]).cuda(), 0.0, Y)
    assert np.abs(U.host_values(Y) - O.layer_norm_fwd(X, w, c, 0.0)).max() < 5e-4      # input ulp 3e-5 / sigma 0.5


def test_layer_norm_errors_and_empty():
    L = _lib()
    x = torch.zeros((4, 16), device="cuda")
    v = torch.ones(16, device="cuda")
    with pytest.raises(L.UnitScaleError) as e:
        L.us_layer_norm_fwd(x, torch.ones(8, device="cuda"), v, 0.0, torch.empty_like(x))
    assert e.value.status == 1
    with pytest.raises(L.UnitScaleError) as e:
        L.us_layer_norm_fwd(x, v, v, -1.0, torch.empty_like(x))
    assert e.value.status == 1
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(L.UnitScaleError) as e:                       # workspace too small
        L.us_layer_norm_bwd(x, v, x, 0.0, 1.0, 0.5, torch.empty_like(x), torch.empty_like(v), torch.empty_like(v), ws)
    assert e.value.status == 4
    big = torch.zeros((2, 4104), device="cuda")
    vb = torch.ones(4104, device="cuda")
    wsb = torch.empty(L.us_layer_norm_bwd_workspace_bytes(2, 4104), dtype=torch.uint8, device="cuda")
    with pytest.raises(L.UnitScaleError) as e:                       # rows longer than the backward supports
        L.us_layer_norm_bwd(big, vb, big, 0.0, 1.0, 0.5, torch.empty_like(big), torch.empty_like(vb), torch.empty_like(vb), wsb)
    assert e.value.status == 2
    L.us_layer_norm_fwd(torch.zeros((0, 16), device="cuda"), v, v, 0.0, torch.zeros((0, 16), device="cuda"))


@pytest.mark.parametrize("rows,cols,ld", [(64, 256, None), (130, 768, 800), (257, 1024, None), (40, 512, None)])
def test_layer_norm_backward_with_a_float32_gradient(rows, cols, ld):
    """16-bit X with a float32 incoming gradient (the gradient of a layer's output)."""
    L = _lib()
    X, G, w, _ = _inputs(6, rows, cols, "bf16")
    from paper_2303_11257_b200 import synth
    G = synth.normal(6, 4, (rows, cols), 1.0)                      # not on the BF16 grid
    eps, beta_wc = 1e-5, float(np.float32(rows ** -0.5))
    dX, dw, dc = U.empty(rows, cols, "bf16", ld), torch.empty(cols, device="cuda"), torch.empty(cols, device="cuda")
    ws = torch.empty(L.us_layer_norm_bwd_workspace_bytes(rows, cols), dtype=torch.uint8, device="cuda")
    L.us_layer_norm_bwd(U.to_device(X, "bf16", ld), torch.from_numpy(w[0]).cuda(), U.to_device(G, "f32", ld), eps, 1.0, beta_wc,
                        dX, dw, dc, ws)
    rdX, rdw, rdc = O.layer_norm_bwd(X, w, G, np.float32(eps), 1.0, beta_wc)
    scale = 1.0 / np.sqrt(X.var(axis=1).min() + eps)
    U.assert_close_stored(dX, rdX, "bf16", 3e-5 * max(1.0, scale), "dX")
    tol = 8 * (2e-6 * np.sqrt(rows) + 1e-6)
    assert np.abs(dw.cpu().numpy() - rdw.reshape(-1)).max() <= tol and np.abs(dc.cpu().numpy() - rdc.reshape(-1)).max() <= tol
