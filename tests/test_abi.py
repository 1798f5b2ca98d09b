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


def test_attention_entry_points_validate_before_any_launch(lib):
    """Host checks of us_attention_fwd / us_attention_bwd (0 OK, 1 invalid argument, 2 unsupported, 3 alignment,
    4 workspace); nothing is launched, so fake device addresses are safe."""
    raw = lib.raw()
    M = lambda addr, dt, r, c, ld=None: lib.us_mat(addr, dt, r, c, ld or c)
    q, k, v = M(0x10000, lib.US_BF16, 128, 64), M(0x20000, lib.US_BF16, 256, 64), M(0x30000, lib.US_BF16, 256, 64)
    c, p = M(0x40000, lib.US_E4M3, 128, 64), M(0x50000, lib.US_BF16, 128, 256)
    bt = lib.attention_batch((1, 1), (0, 0), (0, 0), (0, 0), (0, 0))
    ws = (0x60000, 256)
    call = lambda Q, K, V, Cx, P, a=0.125, sm=256.0, w=ws, b=bt: raw.us_attention_fwd(
        C.byref(Q), C.byref(K), C.byref(V), a, sm, 0.0625, C.byref(Cx), C.byref(P) if P is not None else None, C.byref(b), w[0], w[1], None)
    assert call(q, k, M(0x30000, lib.US_BF16, 128, 64), c, p) == 1              # V rows differ from K rows
    assert call(q, k, v, M(0x40000, lib.US_E4M3, 64, 64), p) == 1               # context rows differ from query rows
    assert call(q, k, v, c, M(0x50000, lib.US_BF16, 128, 128)) == 1             # P is not s_q x s_k
    assert call(q, k, v, c, p, a=0.0) == 1                                      # scales must be positive
    assert call(q, k, v, c, M(0x50000, lib.US_F16, 128, 256)) == 2              # P in another format than the operands
    assert call(q, M(0x20000, lib.US_F16, 256, 64), v, c, p) == 2               # mixed operand formats
    w128 = lambda a: M(a, lib.US_BF16, 128, 128)
    assert call(w128(0x10000), w128(0x20000), w128(0x30000), w128(0x40000), None) == 2        # head width 128
    assert call(q, M(0x20000, lib.US_BF16, 1024, 64), M(0x30000, lib.US_BF16, 1024, 64), c, None) == 2   # more than 512 keys
    assert call(q, k, v, c, p, w=(None, 0)) == 4                                # no workspace
    assert call(M(0x10002, lib.US_BF16, 128, 64), k, v, c, p) == 3              # misaligned base address
    assert call(q, k, v, c, M(0x50000, lib.US_BF16, 128, 256, 260)) == 3        # row pitch of P not a multiple of 16 bytes
    many = lib.attention_batch((2, 2), (0, 64), (8192, 64), (8192, 64), (8192, 64), (65536, 32768))
    assert call(q, k, v, c, p, b=many) == 1                                     # zero stride with more than one problem
    assert call(M(0x10000, lib.US_BF16, 0, 64), k, v, M(0x40000, lib.US_E4M3, 0, 64), None) == 0   # no queries: nothing to do

    dc, ds, dq = M(0x70000, lib.US_BF16, 128, 64), M(0x80000, lib.US_BF16, 128, 256), M(0x90000, lib.US_BF16, 128, 64)
    btb = lib.attention_bwd_batch((1, 1), *[(0, 0)] * 6)
    bcall = lambda dC, P, K, V, dS, dQ, alpha=256.0: raw.us_attention_bwd(
        C.byref(dC), C.byref(P), C.byref(K), C.byref(V), 0.125, alpha, 256.0, 0.125, C.byref(dS), C.byref(dQ), C.byref(btb), ws[0], ws[1], None)
    assert bcall(dc, p, k, v, M(0x80000, lib.US_BF16, 128, 128), dq) == 1       # dS is not s_q x s_k
    assert bcall(dc, p, k, v, ds, dq, alpha=0.0) == 1
    assert bcall(dc, p, k, v, M(0x80000, lib.US_E5M2, 128, 256), dq) == 2       # 16-bit operands with an FP8 dS
    e5 = lambda a, r, cc: M(a, lib.US_E5M2, r, cc)
    e4 = lambda a, r, cc: M(a, lib.US_E4M3, r, cc)
    assert bcall(e5(0x70000, 128, 64), e5(0x50000, 128, 256), e4(0x20000, 256, 64), e4(0x30000, 256, 64), e5(0x80000, 128, 256), dq) == 2   # P must be E4M3


def test_ffn_hidden_validates_before_any_launch(lib):
    """Host checks of us_ffn_hidden (1 invalid argument, 2 unsupported, 3 alignment, 4 workspace): nothing is
    launched, so fake device addresses are safe."""
    raw = lib.raw()
    M = lambda addr, dt, r, c, ld=None: lib.us_mat(addr, dt, r, c, ld or c)
    E4, E5, BF = lib.US_E4M3, lib.US_E5M2, lib.US_BF16
    X, W1, G, W2 = M(0x10000, E4, 272, 144), M(0x20000, E4, 144, 400), M(0x30000, E5, 272, 208), M(0x40000, E4, 400, 208)
    A, dH = M(0x50000, E4, 272, 400), M(0x60000, E5, 272, 400)
    ws = (0x70000, 256)

    def call(X=X, W1=W1, G=G, W2=W2, A=A, dH=dH, H=None, h_dtype=BF, w=ws):
        return raw.us_ffn_hidden(C.byref(X), C.byref(W1), 1.0, C.byref(G), C.byref(W2), 1.0, 1.0, 1.7, 1.5, h_dtype,
                                 C.byref(H) if H is not None else None, C.byref(A), C.byref(dH), w[0], w[1], None)

    assert call(X=M(None, E4, 272, 144)) == 1                                   # null data pointer
    assert call(W1=M(0x20000, E4, 160, 400)) == 1                               # contraction lengths disagree
    assert call(G=M(0x30000, E5, 256, 208)) == 1                                # token counts disagree
    assert call(W2=M(0x40000, E4, 400, 224)) == 1                               # second contraction lengths disagree
    assert call(dH=M(0x60000, E5, 272, 384)) == 1                               # output shape
    assert call(h_dtype=lib.US_F32) == 1                                        # the kept format is BF16 or F16
    assert call(H=M(0x80000, lib.US_F16, 272, 400)) == 1                        # copy in another format than h_dtype
    assert call(w=(None, 0)) == 4                                               # no workspace
    assert call(X=M(0x10008, E4, 272, 144)) == 3                                # misaligned base address
    assert call(A=M(0x50000, E4, 272, 400, 408)) == 3                           # row pitch not a multiple of 16 bytes
    assert call(X=M(0x10000, BF, 272, 144)) == 2                                # 16-bit operands: use the separate calls
    assert call(dH=M(0x60000, BF, 272, 400)) == 2                               # outputs are 8-bit
    small = dict(X=M(0x10000, E4, 128, 144), G=M(0x30000, E5, 128, 208), A=M(0x50000, E4, 128, 400), dH=M(0x60000, E5, 128, 400))
    assert call(**small) == 2                                                   # at most 128 tokens: use the separate calls
    assert raw.us_test_ffn_hidden_starved(C.byref(X), C.byref(W1), C.byref(G), C.byref(W2), C.byref(A), C.byref(dH),
                                          ws[0], ws[1], 0, None) == 1           # wait limit out of range
