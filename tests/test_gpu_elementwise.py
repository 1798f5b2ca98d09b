"""Unfused scaled GELU forward/backward and the tau-weighted residual add against the oracle.

Tolerance: the kernels evaluate the normal tail Phi(-|z|) as 2^(degree-6 polynomial) in float32
(|error| <= 2.7e-7), so gelu / gelu' values carry an absolute error below 1e-6 at unit scale;
the checks allow 2e-6 absolute plus the rounding of the output format (1 ulp for 16-bit, one code
step for FP8)."""
import math

import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import scales as S
from tests import util as U

pytestmark = pytest.mark.gpu
ABS = 2e-6


def _lib():
    from paper_2303_11257_b200 import lib, synth
    return lib, synth


@pytest.mark.parametrize("in_fmt", ["f32", "bf16", "fp16"])
@pytest.mark.parametrize("out_fmt", ["f32", "bf16", "fp16", "e4m3", "e5m2"])
@pytest.mark.parametrize("shape,ld", [((257, 1000), None), ((33, 48), 64)])
def test_gelu_fwd_bwd(in_fmt, out_fmt, shape, ld):
    L, synth = _lib()
    ag, bg = S.gelu_scales()
    s_in = 0.875
    h = synth.normal(3, 0, shape, 1.5)
    h[0, :8] = [0.0, -0.0, 6.0, -6.0, 10.0, -10.0, 1e-8, -37.0]
    g = synth.normal(3, 1, shape)
    Ht, Gt = U.to_device(h, in_fmt, ld), U.to_device(g, in_fmt, ld)
    hv, gv = U.values_of(h, in_fmt), U.values_of(g, in_fmt)
    out = U.empty(shape[0], shape[1], out_fmt, ld)
    L.us_gelu_fwd(Ht, s_in, ag, out)
    U.assert_close_stored(out, O.gelu_fwd(hv, s_in, ag), out_fmt, ABS * ag, "gelu_fwd")
    L.us_gelu_bwd(Ht, Gt, s_in, bg, out)
    ref = O.gelu_bwd(hv, gv, s_in, bg)
    U.assert_close_stored(out, ref, out_fmt, ABS * bg * np.abs(gv).max(), "gelu_bwd")


@pytest.mark.parametrize("in_fmt", ["f32", "bf16", "fp16"])
@pytest.mark.parametrize("out_fmt", ["f32", "bf16", "fp16", "e4m3"])
@pytest.mark.parametrize("tau", [0.0, 0.25, 0.5, 1.0])
def test_residual_add(in_fmt, out_fmt, tau):
    L, synth = _lib()
    shape = (129, 515)
    a, b = synth.normal(4, 0, shape), synth.normal(4, 1, shape)
    out = U.empty(shape[0], shape[1], out_fmt)
    L.us_residual_add(U.to_device(a, in_fmt), U.to_device(b, in_fmt), tau, out)
    ref = O.residual_add(U.values_of(a, in_fmt), U.values_of(b, in_fmt), tau)
    U.assert_close_stored(out, ref, out_fmt, 1e-6, "residual")


def test_unit_variance_on_device():
    """alpha_g gelu(z) has unit std and beta_g gelu'(z) g unit std for unit-normal inputs."""
    L, synth = _lib()
    ag, bg = L.us_scales_gelu()
    assert abs(ag - S.gelu_scales()[0]) < 1e-6 and abs(bg - S.gelu_scales()[1]) < 1e-6
    z = torch.from_numpy(synth.normal(5, 0, (2048, 2048))).cuda()
    g = torch.from_numpy(synth.normal(5, 1, (2048, 2048))).cuda()
    out = torch.empty_like(z)
    L.us_gelu_fwd(z, 1.0, ag, out)
    assert abs(out.std().item() - 1) < 5e-3
    L.us_gelu_bwd(z, g, 1.0, bg, out)
    assert abs(out.std().item() - 1) < 5e-3


def test_elementwise_argument_errors():
    L, _ = _lib()
    a = torch.zeros((4, 8), device="cuda")
    with pytest.raises(L.UnitScaleError) as e:
        L.us_residual_add(a, a, 1.5, a)
    assert e.value.status == 1
    with pytest.raises(L.UnitScaleError) as e:
        L.us_gelu_fwd(U.empty(4, 8, "e4m3"), 1.0, 1.0, a)
    assert e.value.status == 2
    with pytest.raises(L.UnitScaleError) as e:
        L.us_gelu_bwd(a, torch.zeros((4, 7), device="cuda"), 1.0, 1.0, a)
    assert e.value.status == 1


@pytest.mark.parametrize("fn", ["relu", "tanh", "sigmoid", "gelu"])
@pytest.mark.parametrize("in_fmt,out_fmt", [("f32", "f32"), ("bf16", "bf16"), ("fp16", "e4m3"), ("bf16", "e5m2")])
@pytest.mark.parametrize("shape,ld", [((257, 1000), None), ((33, 48), 64)])
def test_activation_fwd_bwd(fn, in_fmt, out_fmt, shape, ld):
    """relu / tanh / sigmoid (and gelu through the same entry) with the table's scale factors.  exp goes
    through ex2.approx in float32: 1e-6 absolute for the bounded functions, times the scale factor."""
    L, synth = _lib()
    alpha, beta = L.us_scales_activation(fn)
    s_in = 0.875
    h = synth.normal(6, 0, shape, 1.5)
    h[0, :8] = [0.0, -0.0, 6.0, -6.0, 30.0, -30.0, 1e-8, -100.0]
    g = synth.normal(6, 1, shape)
    Ht, Gt = U.to_device(h, in_fmt, ld), U.to_device(g, in_fmt, ld)
    hv, gv = U.values_of(h, in_fmt), U.values_of(g, in_fmt)
    out = U.empty(shape[0], shape[1], out_fmt, ld)
    L.us_activation_fwd(fn, Ht, s_in, alpha, out)
    ref = O.activation_fwd(fn, hv, s_in, alpha)
    U.assert_close_stored(out, ref, out_fmt, ABS * alpha * max(1.0, float(np.abs(ref).max()) / alpha / 8), "act fwd " + fn)
    L.us_activation_bwd(fn, Ht, Gt, s_in, beta, out)
    refb = O.activation_bwd(fn, hv, gv, s_in, beta)
    U.assert_close_stored(out, refb, out_fmt, ABS * beta * np.abs(gv).max(), "act bwd " + fn)


def test_activation_gelu_entry_equals_gelu_calls_and_unit_scale():
    L, synth = _lib()
    z = torch.from_numpy(synth.normal(7, 0, (1024, 2048))).cuda()
    g = torch.from_numpy(synth.normal(7, 1, (1024, 2048))).cuda()
    a, b = torch.empty_like(z), torch.empty_like(z)
    L.us_activation_fwd("gelu", z, 1.0, 1.7, a); L.us_gelu_fwd(z, 1.0, 1.7, b)
    assert torch.equal(a, b)
    L.us_activation_bwd("gelu", z, g, 1.0, 1.48, a); L.us_gelu_bwd(z, g, 1.0, 1.48, b)
    assert torch.equal(a, b)
    for fn in ("relu", "tanh", "sigmoid"):
        alpha, beta = L.us_scales_activation(fn)
        L.us_activation_fwd(fn, z, 1.0, alpha, a)
        assert abs(a.std().item() - 1) < 5e-3, fn
        L.us_activation_bwd(fn, z, g, 1.0, beta, a)
        assert abs(a.std().item() - 1) < 5e-3, fn
    with pytest.raises(L.UnitScaleError) as e:
        L.us_activation_fwd(9, z, 1.0, 1.0, a)
    assert e.value.status == 1


@pytest.mark.parametrize("out_fmt", ["f32", "bf16", "e4m3"])
@pytest.mark.parametrize("shape,ld", [((129, 515), None), ((64, 1024), 1040), ((3, 16), None)])
def test_weighted_add_n(out_fmt, shape, ld):
    L, synth = _lib()
    fmts = ["f32", "bf16", "fp16"]
    xs = [synth.normal(8, i, shape) for i in range(3)]
    gammas = [1.0, 0.5, 2.0]
    alpha = float(np.float32(sum(g * g for g in gammas) ** -0.5))
    out = U.empty(shape[0], shape[1], out_fmt, ld)
    L.us_weighted_add([U.to_device(x, f, ld) for x, f in zip(xs, fmts)], gammas, alpha, out)
    # the device forms alpha * gamma_i in float32 first: mirror that rounding in the reference's coefficients
    coefs = [float(np.float32(alpha) * np.float32(g)) for g in gammas]
    ref = sum(c * U.values_of(x, f) for c, x, f in zip(coefs, xs, fmts))
    U.assert_close_stored(out, ref, out_fmt, 1e-6, "weighted_add")
    assert np.allclose(ref, O.weighted_add_n([U.values_of(x, f) for x, f in zip(xs, fmts)], gammas), rtol=1e-6, atol=1e-6)
    if out_fmt == "f32":
        assert abs(U.host_values(out).std() - 1) < 0.05 or shape[0] < 64
    with pytest.raises(L.UnitScaleError) as e:
        L.us_weighted_add([torch.zeros((4, 8), device="cuda")] * 9, [1.0] * 9, 1.0, torch.zeros((4, 8), device="cuda"))
    assert e.value.status == 1


@pytest.mark.parametrize("transport", ["e5m2", "e4m3", "bf16"])
@pytest.mark.parametrize("world", [3, 10])
def test_low_precision_gradient_exchange_arithmetic_on_device(transport, world):
    """The pack and sum steps of the token-sharded weight-gradient exchange (dp.exchange_weight_grads), run on one GPU over
    the partials of `world` stand-in ranks: packed codes bit-exact against the oracle's cast of scale * partial, the
    float32 sum in rank order against the oracle's sum of the decoded codes (more than eight ranks continue from the
    running sum)."""
    from oracle import formats as F
    from paper_2303_11257_b200 import dp, synth
    fmt = F.FORMATS[transport]
    rows, cols = 272, 304
    scale = dp.transport_scale(world)
    parts = [(synth.normal(71, r, (rows, cols)) * np.float32(world ** -0.5)).astype(np.float32) for r in range(world)]
    packed = [dp._pack_device(torch.from_numpy(p).cuda(), scale, dp._TRANSPORT[transport][0]) for p in parts]
    want_codes = [F.quantise_codes((p * np.float32(scale)).astype(np.float64), fmt) for p in parts]
    for got, want in zip(packed, want_codes):
        assert np.array_equal(U.codes_of(got), want)
    out = torch.empty(rows, cols, device="cuda")
    dp._sum_device(packed, 1.0 / scale, out)
    ref = sum(F.decode(c, fmt) for c in want_codes) / scale
    assert np.abs(out.cpu().numpy() - ref).max() <= 4e-7 * max(1.0, np.abs(ref).max()) * world
    # single-process form of the public call: no collective, same arithmetic
    res = torch.empty(rows, cols, device="cuda")
    dp.exchange_weight_grads([torch.from_numpy(parts[0]).cuda()], [res], transport=transport)
    assert np.abs(res.cpu().numpy() - F.decode(F.quantise_codes(parts[0].astype(np.float64), fmt), fmt)).max() <= 1e-6
