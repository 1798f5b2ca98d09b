"""us_quant_stats against the oracle: signal-to-noise ratio of a cast and exponent histogram."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from tests import util as U

pytestmark = pytest.mark.gpu
TORCH = {"e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2, "bf16": torch.bfloat16, "fp16": torch.float16}


def _mods():
    from paper_2303_11257_b200 import lib, synth
    return lib, synth


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2", "bf16", "fp16"])
@pytest.mark.parametrize("shape,ld,sigma", [((257, 1000), None, 1.0), ((64, 48), 64, 2.0 ** -10), ((1, 7), None, 300.0)])
def test_quant_stats_match_the_oracle(fmt, shape, ld, sigma):
    L, synth = _mods()
    x = synth.normal(61, 0, shape, sigma)
    x.flat[:4] = [0.0, -0.0, 1.0, -2.0][: min(4, x.size)]
    snr, s_sig, s_err, hist = L.us_quant_stats(U.to_device(x, "f32", ld), 1.0, TORCH[fmt], -20, 32)
    v = x.astype(np.float64)
    err = F.quantise(v, F.FORMATS[fmt]) - v
    assert abs(s_sig - np.sum(v * v)) <= 1e-12 * np.sum(v * v)
    assert abs(s_err - np.sum(err * err)) <= 1e-12 * np.sum(err * err) + 1e-300
    if s_err > 0:
        assert abs(snr - F.snr(v, F.FORMATS[fmt])) <= 1e-9 * snr
    assert hist == F.exponent_histogram(v, -20, 32).tolist()
    # a second call gives the same bits
    again = L.us_quant_stats(U.to_device(x, "f32", ld), 1.0, TORCH[fmt], -20, 32)
    assert again == (snr, s_sig, s_err, hist)


def test_snr_curve_is_flat_inside_the_range_and_four_per_mantissa_bit():
    """The figure "signal to noise ratio vs scale": a plateau over the scales where the format neither
    overflows nor underflows; one mantissa bit more is a factor of four (E4M3 vs E5M2)."""
    L, synth = _mods()
    x = torch.from_numpy(synth.normal(62, 0, (1024, 1024))).cuda()
    snr = {f: [L.us_quant_stats(x, 2.0 ** k, TORCH[f], -30, 60)[0] for k in (-4, 0, 4)] for f in ("e4m3", "e5m2")}
    for f in snr:
        assert max(snr[f]) / min(snr[f]) < 1.1
    assert 3.5 < snr["e4m3"][1] / snr["e5m2"][1] < 4.5
    assert L.us_quant_stats(x, 2.0 ** 12, TORCH["e4m3"], -30, 60)[0] < snr["e4m3"][1] / 10      # clipping
    assert L.us_quant_stats(x, 2.0 ** -14, TORCH["e4m3"], -30, 60)[0] < snr["e4m3"][1] / 10     # underflow
    # 16-bit input, scaled
    xb = x.to(torch.bfloat16)
    s = L.us_quant_stats(xb, 0.5, TORCH["e5m2"], -10, 12)
    v = xb.float().cpu().numpy().astype(np.float64) * 0.5
    assert abs(s[0] - F.snr(v, F.FORMATS["e5m2"])) <= 1e-9 * s[0] and s[3] == F.exponent_histogram(v, -10, 12).tolist()


def test_quant_stats_errors():
    L, _ = _mods()
    x = torch.zeros((4, 8), device="cuda")
    for bad in (dict(nbins=0), dict(nbins=65), dict(exp_lo=-127), dict(exp_lo=100, nbins=40)):
        kw = dict(exp_lo=-8, nbins=16); kw.update(bad)
        with pytest.raises(L.UnitScaleError) as e:
            L.us_quant_stats(x, 1.0, TORCH["e4m3"], kw["exp_lo"], kw["nbins"])
        assert e.value.status == 1
    with pytest.raises(L.UnitScaleError) as e:
        L.us_quant_stats(x, 1.0, torch.float32, -8, 16)
    assert e.value.status == 2
    snr, s_sig, s_err, hist = L.us_quant_stats(torch.zeros((0, 8), device="cuda"), 1.0, TORCH["e4m3"], -8, 16)
    assert s_sig == 0 and s_err == 0 and sum(hist) == 0
