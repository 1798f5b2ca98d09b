"""us_linear_fwd / bwd_x / bwd_w against the oracle on identically quantised operands.

Tolerances: float32 outputs within 2e-3 absolute of the fp64 result (outputs are unit scale);
16-bit outputs additionally within one ulp; FP8-cast outputs within one code step."""
import math

import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import scales as S
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _lib():
    from paper_2303_11257_b200 import lib, synth
    return lib, synth


def _operands(op, b, m, n, seed, synth):
    X, W, G = synth.linear_tensors(b, m, n, seed)
    a, bx, bw = S.linear_scales(b, m, n)
    if op == "fwd":
        return X, W, a, O.linear_fwd, (b, n)
    if op == "bwd_x":
        return G, W, bx, O.linear_bwd_x, (b, m)
    return X, G, bw, O.linear_bwd_w, (m, n)


def _fp8_pair(op):
    return {"fwd": ("e4m3", "e4m3"), "bwd_x": ("e5m2", "e4m3"), "bwd_w": ("e4m3", "e5m2")}[op]


SHAPES = [(1, 16, 16), (7, 16, 48), (128, 32, 128), (200, 144, 336), (256, 128, 512), (256, 512, 128),
          (384, 1040, 272), (520, 272, 1040), (129, 2064, 257 + 15)]


@pytest.mark.parametrize("op", ["fwd", "bwd_x", "bwd_w"])
@pytest.mark.parametrize("operand", ["fp8", "fp8_e4e4", "bf16", "fp16"])
@pytest.mark.parametrize("shape", SHAPES)
def test_linear_f32_out(op, operand, shape):
    L, synth = _lib()
    b, m, n = shape
    A, B, scale, ref_fn, oshape = _operands(op, b, m, n, 1, synth)
    fa, fb = _fp8_pair(op) if operand == "fp8" else ("e4m3", "e4m3") if operand == "fp8_e4e4" else (operand, operand)
    out = U.empty(oshape[0], oshape[1], "f32")
    ws = L.new_workspace()
    getattr(L, "us_linear_" + op)(U.to_device(A, fa), U.to_device(B, fb), float(scale), out, ws)
    assert L.us_workspace_status(ws) == 0
    ref = ref_fn(U.values_of(A, fa), U.values_of(B, fb), scale)
    U.assert_close_stored(out, ref, "f32", TOL, f"{op} {shape} {fa}x{fb}")


@pytest.mark.parametrize("op", ["fwd", "bwd_x", "bwd_w"])
@pytest.mark.parametrize("out_fmt", ["bf16", "fp16", "e4m3", "e5m2"])
def test_linear_cast_outputs_and_padded_rows(op, out_fmt):
    L, synth = _lib()
    b, m, n = 264, 400, 304
    A, B, scale, ref_fn, oshape = _operands(op, b, m, n, 2, synth)
    fa, fb = _fp8_pair(op)
    At = U.to_device(A, fa, ld=A.shape[1] + 16)
    Bt = U.to_device(B, fb, ld=B.shape[1] + 32)
    out = U.empty(oshape[0], oshape[1], out_fmt, ld=oshape[1] + 16)
    ws = L.new_workspace()
    getattr(L, "us_linear_" + op)(At, Bt, float(scale), out, ws)
    assert L.us_workspace_status(ws) == 0
    ref = ref_fn(U.values_of(A, fa), U.values_of(B, fb), scale)
    U.assert_close_stored(out, ref, out_fmt, TOL, f"{op} -> {out_fmt}")
    pad = out.as_strided((oshape[0], 16), (oshape[1] + 16, 1), oshape[1])
    assert not pad.view(torch.uint8).any().item() if out.element_size() == 1 else not pad.any().item()


@pytest.mark.parametrize("shape", [(256, 128, 512), (200, 144, 336)])
@pytest.mark.parametrize("aux_fmt", ["bf16", "fp16"])
def test_gelu_epilogue(shape, aux_fmt):
    """GEMM-1 of the FFN: H stored in 16 bit, A = q_E4(alpha_g gelu(s_in H)) from the unrounded H."""
    L, synth = _lib()
    b, m, n = shape
    X, W, _ = synth.linear_tensors(b, m, n, 3)
    a, _, _ = S.linear_scales(b, m, n)
    ag, _ = S.gelu_scales()
    H = U.empty(b, n, aux_fmt)
    Aq = U.empty(b, n, "e4m3")
    ws = L.new_workspace()
    ep = L.epilogue(act=L.US_ACT_GELU, act_in_scale=0.9, act_out_scale=float(ag), aux=H)
    L.us_linear_fwd(U.to_device(X, "e4m3"), U.to_device(W, "e4m3"), float(a), Aq, ws, ep)
    assert L.us_workspace_status(ws) == 0
    val = O.linear_fwd(U.values_of(X, "e4m3"), U.values_of(W, "e4m3"), a)
    oep = O.Epilogue(act="gelu", act_in_scale=0.9, act_out_scale=ag, aux_dtype=aux_fmt)
    ref_out = O.gelu_fwd(val, 0.9, ag)
    U.assert_close_stored(H, val, aux_fmt, TOL, "stored pre-activation")
    U.assert_close_stored(Aq, ref_out, "e4m3", TOL, "gelu output")
    _, codes, _ = O.apply_epilogue(val, oep, "e4m3")
    assert (U.codes_of(Aq) != codes).mean() < 2e-3          # flips only at near-ties


@pytest.mark.parametrize("shape", [(256, 128, 512), (200, 144, 336)])
def test_gelu_grad_and_residual_epilogues(shape):
    L, synth = _lib()
    b, m, n = shape
    _, W, G = synth.linear_tensors(b, m, n, 4)
    _, bx, _ = S.linear_scales(b, m, n)
    _, bg = S.gelu_scales()
    Hh = synth.normal(4, 7, (b, m))
    ws = L.new_workspace()
    # dH = q_E5(beta_g gelu'(H) * beta_x G W^T)
    Ht = U.to_device(Hh, "bf16")
    dH = U.empty(b, m, "e5m2")
    ep = L.epilogue(act=L.US_ACT_GELU_GRAD, act_in_scale=1.0, act_out_scale=float(bg), aux=Ht)
    L.us_linear_bwd_x(U.to_device(G, "e5m2"), U.to_device(W, "e4m3"), float(bx), dH, ws, ep)
    val = O.linear_bwd_x(U.values_of(G, "e5m2"), U.values_of(W, "e4m3"), bx)
    ref = O.gelu_bwd(U.values_of(Hh, "bf16"), val, 1.0, bg)
    U.assert_close_stored(dH, ref, "e5m2", TOL, "gelu-grad epilogue")
    # dX = sqrt(1-tau) skip + sqrt(tau) beta_x G W^T, skip in f32 / bf16
    for skip_fmt, out_fmt in (("f32", "bf16"), ("bf16", "f32"), ("fp16", "fp16")):
        skip = synth.normal(4, 8, (b, m))
        out = U.empty(b, m, out_fmt)
        cs, cb = S.residual_coefficients(0.3)
        skip_t = U.to_device(skip, skip_fmt)
        ep = L.epilogue(skip=skip_t, skip_coef=float(cs), out_coef=float(cb))
        L.us_linear_bwd_x(U.to_device(G, "e5m2"), U.to_device(W, "e4m3"), float(bx), out, ws, ep)
        ref = O.weighted_add(U.values_of(skip, skip_fmt), val, cs, cb)
        U.assert_close_stored(out, ref, out_fmt, TOL, "residual epilogue")
    assert L.us_workspace_status(ws) == 0


def test_identity_weight_is_exact():
    """X I = X exactly for FP8 operands (products and float32 sums of one term are exact)."""
    L, synth = _lib()
    X = synth.normal(5, 0, (130, 256))
    out = U.empty(130, 256, "f32")
    ws = L.new_workspace()
    L.us_linear_fwd(U.to_device(X, "e4m3"), U.to_device(np.eye(256, dtype=np.float32), "e4m3"), 1.0, out, ws)
    assert np.array_equal(U.host_values(out), U.values_of(X, "e4m3"))


@pytest.mark.parametrize("op", ["fwd", "bwd_x", "bwd_w"])
def test_bert_large_shape_sampled(op):
    """Full-size GEMMs (8192 x 1024 x 4096): sampled rows and columns against fp64 dot products."""
    L, synth = _lib()
    b, m, n = 8192, 1024, 4096
    A, B, scale, ref_fn, oshape = _operands(op, b, m, n, 6, synth)
    fa, fb = _fp8_pair(op)
    out = U.empty(oshape[0], oshape[1], "f32")
    ws = L.new_workspace()
    getattr(L, "us_linear_" + op)(U.to_device(A, fa), U.to_device(B, fb), float(scale), out, ws)
    assert L.us_workspace_status(ws) == 0
    Av, Bv = U.values_of(A, fa), U.values_of(B, fb)
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([[0, 127, 128, oshape[0] - 1], rng.integers(0, oshape[0], 12)]))
    cols = np.unique(np.concatenate([[0, 255, 256, oshape[1] - 1], rng.integers(0, oshape[1], 12)]))
    got = U.host_values(out)
    if op == "fwd":
        r_ref, c_ref = ref_fn(Av[rows], Bv, scale), ref_fn(Av, Bv[:, cols], scale)
    elif op == "bwd_x":
        r_ref, c_ref = ref_fn(Av[rows], Bv, scale), ref_fn(Av, Bv[cols], scale)
    else:
        r_ref, c_ref = ref_fn(Av[:, rows], Bv, scale), ref_fn(Av, Bv[:, cols], scale)
    assert np.abs(got[rows] - r_ref).max() <= TOL
    assert np.abs(got[:, cols] - c_ref).max() <= TOL
    assert abs(got.std() - 1) < 0.02                      # unit variance at initialisation


def test_linear_argument_errors():
    L, _ = _lib()
    ws = L.new_workspace()
    X, W, Y = U.empty(32, 64, "e4m3"), U.empty(64, 48, "e4m3"), U.empty(32, 48, "f32")
    L.us_linear_fwd(X, W, 1.0, Y, ws)

    def status(fn, *a, **k):
        with pytest.raises(L.UnitScaleError) as e:
            fn(*a, **k)
        return e.value.status

    assert status(L.us_linear_fwd, X, U.empty(65, 48, "e4m3"), 1.0, Y, ws) == 1            # K mismatch
    assert status(L.us_linear_fwd, X, W, 1.0, U.empty(32, 47, "f32"), ws) == 1             # out shape
    assert status(L.us_linear_fwd, X, U.empty(64, 48, "bf16"), 1.0, Y, ws) == 2            # mixed classes
    assert status(L.us_linear_fwd, U.empty(32, 64, "f32"), U.empty(64, 48, "f32"), 1.0, Y, ws) == 2
    assert status(L.us_linear_fwd, U.empty(32, 72, "e4m3")[:, :64], W, 1.0, Y, ws) == 3    # pitch 72 bytes
    assert status(L.us_linear_fwd, X, W, 1.0, Y, torch.zeros(8, dtype=torch.uint8, device="cuda")) == 4
    ep = L.epilogue(act=L.US_ACT_GELU_GRAD)
    assert status(L.us_linear_fwd, X, W, 1.0, Y, ws, ep) == 1                              # aux required
    ep = L.epilogue(act=L.US_ACT_GELU, aux=U.empty(32, 48, "f32"))
    assert status(L.us_linear_fwd, X, W, 1.0, Y, ws, ep) == 2                              # aux must be 16 bit
    assert L.us_workspace_status(ws) == 0


@pytest.mark.parametrize("fn", ["relu", "tanh", "sigmoid"])
@pytest.mark.parametrize("shape", [(256, 128, 512), (200, 144, 336)])
def test_other_activations_as_epilogues(fn, shape):
    """relu / tanh / sigmoid fused like GELU: forward with the kept pre-activation, gradient from the stored one
    (table section "Activations"), against the oracle's activation_fwd / activation_bwd on the fp64 GEMM result."""
    L, synth = _lib()
    b, m, n = shape
    X, W, G = synth.linear_tensors(b, m, n, 8)
    a, bx, _ = S.linear_scales(b, m, n)
    alpha_f, beta_f = {"relu": S.relu_scales, "tanh": S.tanh_scales, "sigmoid": S.sigmoid_scales}[fn]()
    fwd_code = {"relu": L.US_ACT_RELU, "tanh": L.US_ACT_TANH, "sigmoid": L.US_ACT_SIGMOID}[fn]
    ws = L.new_workspace()
    val = O.linear_fwd(U.values_of(X, "e4m3"), U.values_of(W, "e4m3"), a)
    for out_fmt in ("e4m3", "bf16", "f32"):
        H = U.empty(b, n, "bf16")
        A = U.empty(b, n, out_fmt)
        ep = L.epilogue(act=fwd_code, act_in_scale=0.8, act_out_scale=float(alpha_f), aux=H)
        L.us_linear_fwd(U.to_device(X, "e4m3"), U.to_device(W, "e4m3"), float(a), A, ws, ep)
        U.assert_close_stored(H, val, "bf16", TOL, f"{fn}: stored pre-activation")
        U.assert_close_stored(A, O.activation_fwd(fn, val, 0.8, alpha_f), out_fmt, TOL * float(alpha_f), f"{fn} -> {out_fmt}")
    # gradient: dH = beta f'(s H) * (beta_x G W^T), H read back from its stored 16-bit form
    Hh = synth.normal(8, 7, (b, m))
    Hh[np.abs(Hh) < 1e-2] = 0.25                                # keep relu's kink away from rounding noise
    Ht = U.to_device(Hh, "bf16")
    gval = O.linear_bwd_x(U.values_of(G, "e5m2"), U.values_of(W, "e4m3"), bx)
    ref = O.activation_bwd(fn, U.values_of(Hh, "bf16"), gval, 1.0, beta_f)
    for out_fmt in ("e5m2", "bf16"):
        dH = U.empty(b, m, out_fmt)
        ep = L.epilogue(act=fwd_code + 1, act_in_scale=1.0, act_out_scale=float(beta_f), aux=Ht)
        L.us_linear_bwd_x(U.to_device(G, "e5m2"), U.to_device(W, "e4m3"), float(bx), dH, ws, ep)
        U.assert_close_stored(dH, ref, out_fmt, TOL * float(beta_f), f"{fn} gradient -> {out_fmt}")
    assert L.us_workspace_status(ws) == 0
