"""The C-ABI library: builds, loads, exports every symbol the header declares; host-only calls work
without a GPU (scale helpers, status strings, argument validation that precedes any launch)."""
import ctypes as C
import math
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2303_11257_b200 import build
    build.build()
    from paper_2303_11257_b200 import lib as L
    return L


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "unitscale.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(us_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"us_linear_fwd", "us_linear_bwd_x", "us_linear_bwd_w", "us_gelu_fwd", "us_gelu_bwd",
            "us_residual_add", "us_cast_fp8"} <= set(names)
    raw = lib.raw()
    for n in names:
        assert hasattr(raw, n), n


def test_scale_helpers_match_closed_forms(lib):
    from oracle import scales as S
    for (b, m, n) in ((256, 128, 512), (8192, 1024, 4096), (8192, 4096, 1024), (7, 3, 5)):
        for constrained in (False, True):
            got = lib.us_scales_linear(b, m, n, constrained)
            want = S.linear_scales(b, m, n, constrained)
            for g, w in zip(got, want):
                assert g == C.c_float(w).value
    for constrained in (False, True):
        got = lib.us_scales_gelu(constrained)
        want = S.gelu_scales(constrained)
        for g, w in zip(got, want):
            assert abs(g - w) < 2e-7
    assert round(lib.us_scales_gelu()[0], 3) == 1.701 and round(lib.us_scales_gelu()[1], 3) == 1.481
    with pytest.raises(lib.UnitScaleError):
        lib.us_scales_linear(0, 1, 1)
    import math
    for fn, want in (("relu", S.relu_scales()), ("tanh", S.tanh_scales()), ("sigmoid", S.sigmoid_scales()), ("gelu", S.gelu_scales())):
        a, b = lib.us_scales_activation(fn)
        assert abs(a - want[0]) < 5e-7 * want[0] and abs(b - want[1]) < 5e-7 * want[1]
        c = lib.us_scales_activation(fn, True)
        assert abs(c[0] - math.sqrt(want[0] * want[1])) < 1e-6 and c[0] == c[1]
    with pytest.raises(lib.UnitScaleError):
        lib.us_scales_activation(7)


def test_status_strings_and_version(lib):
    assert lib.us_status_string(0) == "ok"
    assert "align" in lib.us_status_string(3)
    assert lib.us_version() >= 100
    assert lib.us_workspace_bytes() >= 4


def test_validation_happens_before_any_launch(lib):
    """Invalid descriptors are rejected on the host, so these calls are safe without a device."""
    raw = lib.raw()
    m = lib.us_mat(None, lib.US_F32, 4, 4, 4)
    assert raw.us_cast_fp8(C.byref(m), 1.0, C.byref(m), None) == 1          # null data pointer
    bad = lib.us_mat(0x1000, lib.US_E4M3, 4, 16, 8)
    assert raw.us_linear_fwd(C.byref(bad), C.byref(bad), 1.0, None, C.byref(bad), None, 0, None) == 1   # ld < cols
    a = lib.us_mat(0x1000, lib.US_E4M3, 16, 16, 16)
    o = lib.us_mat(0x2000, lib.US_F32, 16, 16, 16)
    assert raw.us_linear_fwd(C.byref(a), C.byref(a), 1.0, None, C.byref(o), None, 0, None) == 4         # no workspace
    a8 = lib.us_mat(0x1008, lib.US_E4M3, 16, 16, 16)
    assert raw.us_linear_fwd(C.byref(a8), C.byref(a), 1.0, None, C.byref(o), None, 0, None) == 3        # misaligned
    h = lib.us_mat(0x1000, lib.US_BF16, 16, 16, 16)
    assert raw.us_linear_fwd(C.byref(a), C.byref(h), 1.0, None, C.byref(o), None, 0, None) == 2         # mixed operands


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    import importlib
    from paper_2303_11257_b200 import lib as L
    monkeypatch.setattr(L, "library_path", lambda: str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        L._load()


def test_residual_and_attention_scale_helpers(lib):
    from oracle import scales as S
    for tau in (0.0, 0.3, 0.5, 1.0 / 7, 1.0):
        cs, cb = lib.us_scales_residual(tau)
        ws, wb = S.residual_coefficients(float(C.c_float(tau).value))
        assert cs == C.c_float(ws).value and cb == C.c_float(wb).value
        assert abs(cs * cs + cb * cb - 1) < 2e-7                   # unit variance of the sum of independent unit inputs
    with pytest.raises(lib.UnitScaleError):
        lib.us_scales_residual(1.5)
    for s, hd in ((512, 64), (128, 64), (80, 64), (272, 128)):
        a = lib.us_scales_attention(s, hd)
        f32 = lambda v: C.c_float(v).value
        assert a["alpha_s"] == a["beta_Q"] == a["beta_K"] == f32(hd ** -0.5)      # appendix: 1 / sqrt(d) in both passes
        assert a["sm"] == float(s)
        # the context matmul P[s x s] V[s x d_head] takes the ordinary matmul factors with batch = fan_in = s
        al, bx, bw = S.linear_scales(s, s, hd)
        assert (a["alpha_c"], a["beta_P"], a["beta_V"]) == (f32(al), f32(bx), f32(bw))
        c = lib.us_scales_attention(s, hd, True)
        alc, bxc, _ = S.linear_scales(s, s, hd, True)
        assert c["alpha_c"] == c["beta_P"] == f32(alc) and f32(bxc) == f32(alc)
    with pytest.raises(lib.UnitScaleError):
        lib.us_scales_attention(0, 64)
