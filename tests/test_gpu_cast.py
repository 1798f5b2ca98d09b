"""us_cast_fp8 against the oracle quantiser: bit-exact codes."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from tests import util as U

pytestmark = pytest.mark.gpu


def _lib():
    from paper_2303_11257_b200 import lib
    return lib


def structured_fp32_patterns():
    hi = np.arange(1 << 16, dtype=np.uint32)
    lo = np.random.default_rng(4).integers(0, 1 << 16, size=256, dtype=np.uint32)
    lo[:4] = [0, 1, 0x8000, 0xFFFF]
    return (hi[:, None] << 16 | lo[None, :]).reshape(1 << 12, 1 << 12).view(np.float32)


def _assert_codes(got, want, fmt):
    nan_want = np.isnan(F.decode(want, fmt))
    nan_got = np.isnan(F.decode(got, fmt))
    assert np.array_equal(nan_want, nan_got)
    assert np.array_equal(got[~nan_want], want[~nan_want])


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_cast_structured_fp32_bit_patterns(fmt):
    L = _lib()
    x = structured_fp32_patterns()
    dst = U.empty(*x.shape, fmt)
    L.us_cast_fp8(torch.from_numpy(x).cuda(), 1.0, dst)
    _assert_codes(U.codes_of(dst), F.scaled_cast(x, 1.0, F.FORMATS[fmt]), F.FORMATS[fmt])


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
@pytest.mark.parametrize("src", ["bf16", "fp16"])
def test_cast_all_16bit_sources(fmt, src):
    L = _lib()
    codes = np.arange(1 << 16, dtype=np.uint16).reshape(256, 256)
    t = torch.from_numpy(codes.view(np.int16)).view(U.TORCH_OF[src]).cuda()
    vals = F.decode(codes, F.FORMATS[src])
    for scale in (1.0, 0.3, 2.0 ** -7):
        dst = U.empty(256, 256, fmt)
        L.us_cast_fp8(t, scale, dst)
        with np.errstate(over="ignore", invalid="ignore"):
            want = F.scaled_cast(vals.astype(np.float32), scale, F.FORMATS[fmt])
        _assert_codes(U.codes_of(dst), want, F.FORMATS[fmt])


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
@pytest.mark.parametrize("shape,ld", [((1, 1), None), ((3, 5), None), ((300, 257), None), ((64, 48), 64),
                                      ((37, 100), 112), ((2048, 4096), None)])
def test_cast_shapes_scales_and_saturation(fmt, shape, ld):
    from paper_2303_11257_b200 import synth
    L = _lib()
    for sigma, scale in ((1.0, 1.0), (256.0, 1.0), (2.0 ** -8, 1.0), (1.0, 1 / 3), (1.0, 1000.0)):
        x = synth.normal(11, 0, shape, sigma)
        src = U.to_device(x, "f32", ld)
        dst = U.empty(shape[0], shape[1], fmt, ld)
        L.us_cast_fp8(src, scale, dst)
        want = F.scaled_cast(x, scale, F.FORMATS[fmt])
        assert np.array_equal(U.codes_of(dst), want)
        if ld:   # padding untouched
            full = dst.as_strided((shape[0], ld), (ld, 1)).view(torch.uint8).cpu().numpy()
            assert not full[:, shape[1]:].any()


def test_cast_empty_and_errors():
    L = _lib()
    src = torch.zeros((0, 8), device="cuda")
    dst = torch.zeros((0, 8), dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn)
    L.us_cast_fp8(src, 1.0, dst)
    with pytest.raises(L.UnitScaleError) as e:
        L.us_cast_fp8(torch.zeros((4, 8), device="cuda"), 1.0, torch.zeros((4, 8), device="cuda", dtype=torch.bfloat16))
    assert e.value.status == 2
    with pytest.raises(L.UnitScaleError) as e:
        L.us_cast_fp8(torch.zeros((4, 8), device="cuda"), 1.0, U.empty(4, 9, "e4m3"))
    assert e.value.status == 1


def test_cast_multi_matches_oracle_and_single_casts():
    """Mixed source types, formats, scales and ragged sizes in one launch: codes equal the oracle's and
    those of separate us_cast_fp8 calls; neighbours of each destination stay untouched."""
    from paper_2303_11257_b200 import synth
    L = _lib()
    specs = [((64, 48), "f32", "e4m3", 1.0), ((1, 1), "f32", "e5m2", 0.5), ((300, 257), "bf16", "e5m2", 3.0),
             ((37, 19), "fp16", "e4m3", 2.0 ** -3), ((0, 8), "f32", "e4m3", 1.0), ((1024, 1024), "f32", "e4m3", 1 / 3),
             ((5, 16), "bf16", "e4m3", 1000.0), ((2, 7), "f32", "e5m2", 1.0)]
    srcs, dsts, wants, singles, scales = [], [], [], [], []
    for i, (shape, st, fmt, scale) in enumerate(specs):
        x = synth.normal(21 + i, 0, shape, 4.0)
        xs = F.quantise(x, F.FORMATS[st]).astype(np.float32) if st != "f32" else x
        srcs.append(U.to_device(xs, st) if x.size else torch.zeros(shape, device="cuda"))
        dsts.append(U.empty(shape[0], shape[1], fmt))
        singles.append(U.empty(shape[0], shape[1], fmt))
        wants.append(F.scaled_cast(xs, scale, F.FORMATS[fmt]))
        scales.append(scale)
    L.us_cast_fp8_multi(srcs, scales, dsts)
    for src, scale, one in zip(srcs, scales, singles):
        L.us_cast_fp8(src, scale, one)
    for dst, one, want in zip(dsts, singles, wants):
        assert np.array_equal(U.codes_of(dst), want)
        assert np.array_equal(U.codes_of(dst), U.codes_of(one))


def test_cast_multi_errors_launch_nothing():
    L = _lib()
    a, b = torch.ones((4, 16), device="cuda"), torch.ones((4, 16), device="cuda")
    da, db = U.empty(4, 16, "e4m3"), U.empty(4, 16, "e4m3")
    da.view(torch.uint8).zero_()
    padded = U.empty(4, 16, "e4m3", 32)
    with pytest.raises(L.UnitScaleError) as e:                       # row padding: not for the fused launch
        L.us_cast_fp8_multi([a, b], [1.0, 1.0], [da, padded])
    assert e.value.status == 2
    with pytest.raises(L.UnitScaleError) as e:                       # shape mismatch
        L.us_cast_fp8_multi([a, b], [1.0, 1.0], [da, U.empty(4, 8, "e4m3")])
    assert e.value.status == 1
    with pytest.raises(L.UnitScaleError) as e:                       # more tensors than one launch takes
        L.us_cast_fp8_multi([a] * 9, [1.0] * 9, [da] * 9)
    assert e.value.status == 1
    with pytest.raises(L.UnitScaleError) as e:                       # misaligned start
        L.us_cast_fp8_multi([a.view(-1)[1:33].view(2, 16)], [1.0], [U.empty(2, 16, "e4m3")])
    assert e.value.status == 3
    torch.cuda.synchronize()
    assert not da.view(torch.uint8).any()                            # the valid first tensor was not written either
