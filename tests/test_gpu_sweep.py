"""Linear GEMM sweep (each of Y, dX, dW separately): squares 1024 ... 16384 and the skinny
M = 512, N = K = 8192 case, E4M3 x E4M3 and E5M2 x E4M3 operands, float32 and FP8-cast outputs.

Up to 4096 the whole output is compared with the oracle; beyond that the oracle evaluates sampled
rows x columns (full-K fp64 dot products on operands it quantised itself from the same float32
inputs; the device operands come from us_cast_fp8, which is bit-exact against the oracle's cast)."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import ops as O
from oracle import scales as S
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3

PAIRS = {"fwd": [("e4m3", "e4m3")], "bwd_x": [("e5m2", "e4m3"), ("e4m3", "e4m3")], "bwd_w": [("e4m3", "e5m2"), ("e4m3", "e4m3")]}


def _mods():
    from paper_2303_11257_b200 import lib, synth
    return lib, synth


def _device_operand(L, host_f32, fmt):
    src = torch.from_numpy(host_f32).cuda()
    dst = U.empty(host_f32.shape[0], host_f32.shape[1], fmt)
    L.us_cast_fp8(src, 1.0, dst)
    return dst


def _run(L, op, At, Bt, scale, out_fmt, oshape):
    out = U.empty(oshape[0], oshape[1], out_fmt)
    ws = L.new_workspace()
    getattr(L, "us_linear_" + op)(At, Bt, float(scale), out, ws)
    assert L.us_workspace_status(ws) == 0
    return out


def _setup(op, b, m, n, synth, seed):
    X, W, G = synth.linear_tensors(b, m, n, seed)
    a, bx, bw = S.linear_scales(b, m, n)
    if op == "fwd":
        return X, W, a, (b, n)
    if op == "bwd_x":
        return G, W, bx, (b, m)
    return X, G, bw, (m, n)


@pytest.mark.parametrize("size", [1024, 2048, 4096])
@pytest.mark.parametrize("op", ["fwd", "bwd_x", "bwd_w"])
def test_square_full_compare(op, size):
    L, synth = _mods()
    A, B, scale, oshape = _setup(op, size, size, size, synth, seed=size)
    ref_fn = {"fwd": O.linear_fwd, "bwd_x": O.linear_bwd_x, "bwd_w": O.linear_bwd_w}[op]
    for fa, fb in PAIRS[op]:
        At, Bt = _device_operand(L, A, fa), _device_operand(L, B, fb)
        ref = ref_fn(U.values_of(A, fa), U.values_of(B, fb), scale)
        for out_fmt in ("f32", "e4m3"):
            out = _run(L, op, At, Bt, scale, out_fmt, oshape)
            U.assert_close_stored(out, ref, out_fmt, TOL, f"{op} {size}^3 {fa}x{fb}->{out_fmt}")
        assert abs(ref.std() - 1) < 0.05


def _sampled(op, Aq_rows_or_cols, Bq_rows_or_cols, scale):
    """Reference block for sampled output rows R x columns C, from the operand slices that feed them."""
    a, b = Aq_rows_or_cols, Bq_rows_or_cols
    s = float(np.float32(scale))
    if op == "fwd":       # a = Xq[R, :], b = Wq[:, C]
        return s * (a @ b)
    if op == "bwd_x":     # a = Gq[R, :], b = Wq[C, :]
        return s * (a @ b.T)
    return s * (a.T @ b)  # a = Xq[:, R], b = Gq[:, C]


@pytest.mark.parametrize("shape", [(8192, 8192, 8192), (16384, 16384, 16384), (512, 8192, 8192)])
@pytest.mark.parametrize("op", ["fwd", "bwd_x", "bwd_w"])
def test_large_sampled(op, shape):
    L, synth = _mods()
    b, m, n = shape
    A, B, scale, oshape = _setup(op, b, m, n, synth, seed=b + n)
    rng = np.random.default_rng(b)
    R = np.unique(np.concatenate([[0, 127, 128, 255, 256, oshape[0] - 1], rng.integers(0, oshape[0], 10)]))
    Cc = np.unique(np.concatenate([[0, 127, 128, 255, 256, oshape[1] - 1], rng.integers(0, oshape[1], 10)]))
    for fa, fb in PAIRS[op]:
        At, Bt = _device_operand(L, A, fa), _device_operand(L, B, fb)
        if op == "fwd":
            a_s, b_s = U.values_of(A[R], fa), U.values_of(B[:, Cc], fb)
        elif op == "bwd_x":
            a_s, b_s = U.values_of(A[R], fa), U.values_of(B[Cc], fb)
        else:
            a_s, b_s = U.values_of(A[:, R], fa), U.values_of(B[:, Cc], fb)
        ref = _sampled(op, a_s, b_s, scale)
        for out_fmt in ("f32", "e4m3"):
            out = _run(L, op, At, Bt, scale, out_fmt, oshape)
            block = out[torch.from_numpy(R).cuda()][:, torch.from_numpy(Cc).cuda()]
            U.assert_close_stored(block, ref, out_fmt, TOL, f"{op} {shape} {fa}x{fb}->{out_fmt}")
            if out_fmt == "f32":
                assert abs(out[:2048].std().item() - 1) < 0.03          # unit variance at initialisation
        del At, Bt
    torch.cuda.empty_cache()
