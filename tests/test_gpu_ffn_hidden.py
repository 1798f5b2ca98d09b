"""us_ffn_hidden: the first forward GEMM + scaled GELU and the second layer's input-gradient GEMM + GELU gradient in
one launch, against the oracle (section "Example", table row "gelu") and against the two separate entry points
(bit-identical: same accumulation order per tile, same rounding of the kept pre-activation)."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import ops as O
from oracle import scales as S
from tests import util as U

pytestmark = pytest.mark.gpu
US_ERR_INVALID_ARG, US_ERR_UNSUPPORTED, US_ERR_ALIGNMENT, US_ERR_TIMEOUT = 1, 2, 3, 6


def _mods():
    from paper_2303_11257_b200 import lib, synth
    return lib, synth


def _inputs(synth, b, m, f, n, seed, fx="e4m3", fg="e5m2"):
    X, W1 = synth.normal(seed, 0, (b, m)), synth.normal(seed, 1, (m, f))
    G, W2 = synth.normal(seed, 2, (b, n)), synth.normal(seed, 3, (f, n))
    dev = (U.to_device(X, fx), U.to_device(W1, "e4m3"), U.to_device(G, fg), U.to_device(W2, "e4m3"))
    val = (U.values_of(X, fx), U.values_of(W1, "e4m3"), U.values_of(G, fg), U.values_of(W2, "e4m3"))
    return dev, val


def _oracle(val, alpha, beta_x, s_in, ag, bg, h_fmt, a_fmt, d_fmt):
    Xv, W1v, Gv, W2v = val
    H = O.linear_fwd(Xv, W1v, alpha)
    A = O.gelu_fwd(H, s_in, ag)
    H16, _ = O.store(H, h_fmt)
    dH = O.gelu_bwd(H16, O.linear_bwd_x(Gv, W2v, beta_x), s_in, bg)
    return H, F.quantise_codes(A, F.FORMATS[a_fmt]), F.quantise_codes(dH, F.FORMATS[d_fmt])


CASES = [
    # b, m, f, n, h_fmt, a_fmt, d_fmt, s_in
    (256, 128, 512, 128, "bf16", "e4m3", "e5m2", 1.0),        # the small FFN configuration
    (200, 144, 336, 144, "bf16", "e4m3", "e5m2", 1.0),        # ragged rows, columns and contraction lengths
    (520, 272, 1040, 400, "fp16", "e4m3", "e5m2", 0.75),      # different contraction lengths, several tiles per pair, F16 kept H
    (300, 64, 304, 1040, "bf16", "e5m2", "e4m3", 1.0),        # the other output formats; a long second contraction
    (2304, 256, 4864, 256, "bf16", "e4m3", "e5m2", 1.0),      # 9 x 19 = 171 tiles on 74 pairs: up to three tiles per pair
]


@pytest.mark.parametrize("case", range(len(CASES)))
@pytest.mark.parametrize("keep_h", [False, True])
def test_ffn_hidden_matches_oracle_and_separate_calls(case, keep_h):
    L, synth = _mods()
    b, m, f, n, h_fmt, a_fmt, d_fmt, s_in = CASES[case]
    if keep_h and case in (3, 4):
        pytest.skip("the kept copy is covered by the other cases")
    dev, val = _inputs(synth, b, m, f, n, 300 + case)
    Xt, W1t, Gt, W2t = dev
    alpha, _, _ = S.linear_scales(b, m, f)
    _, beta_x, _ = S.linear_scales(b, f, n)
    ag, bg = S.gelu_scales()
    ws = L.new_workspace()
    A, dH = U.empty(b, f, a_fmt), U.empty(b, f, d_fmt)
    H = U.empty(b, f, h_fmt) if keep_h else None
    L.us_ffn_hidden(Xt, W1t, float(alpha), Gt, W2t, float(beta_x), s_in, float(ag), float(bg), A, dH, ws,
                    H=H, h_dtype=U.TORCH_OF[h_fmt])
    assert L.us_workspace_status(ws) == 0
    Href, A_codes, dH_codes = _oracle(val, alpha, beta_x, s_in, ag, bg, h_fmt, a_fmt, d_fmt)
    U.code_deltas(A, A_codes, a_fmt)
    U.code_deltas(dH, dH_codes, d_fmt)
    if keep_h:
        U.assert_close_stored(H, Href, h_fmt, 2e-3 * max(1.0, np.abs(Href).max() / 4), "kept pre-activation")
    # the two separate launches give the same bits
    A1, dH1, H1 = U.empty(b, f, a_fmt), U.empty(b, f, d_fmt), U.empty(b, f, h_fmt)
    L.us_linear_fwd(Xt, W1t, float(alpha), A1, ws,
                    L.epilogue(act=L.US_ACT_GELU, act_in_scale=s_in, act_out_scale=float(ag), aux=H1))
    L.us_linear_bwd_x(Gt, W2t, float(beta_x), dH1, ws,
                      L.epilogue(act=L.US_ACT_GELU_GRAD, act_in_scale=s_in, act_out_scale=float(bg), aux=H1))
    torch.cuda.synchronize()
    assert torch.equal(A.contiguous().view(torch.uint8), A1.contiguous().view(torch.uint8))
    assert torch.equal(dH.contiguous().view(torch.uint8), dH1.contiguous().view(torch.uint8))
    if keep_h:
        assert torch.equal(H.contiguous().view(torch.int16), H1.contiguous().view(torch.int16))
    assert L.us_workspace_status(ws) == 0


def test_ffn_hidden_padded_rows_and_repeat_launches():
    """Row pitches larger than the row length (views into wider allocations); launching twice gives the same bits
    and leaves the padding untouched."""
    L, synth = _mods()
    b, m, f, n = 272, 144, 400, 208
    X, W1 = synth.normal(41, 0, (b, m)), synth.normal(41, 1, (m, f))
    G, W2 = synth.normal(41, 2, (b, n)), synth.normal(41, 3, (f, n))
    Xt, W1t = U.to_device(X, "e4m3", ld=160), U.to_device(W1, "e4m3", ld=416)
    Gt, W2t = U.to_device(G, "e5m2", ld=224), U.to_device(W2, "e4m3", ld=208)
    val = (U.values_of(X, "e4m3"), U.values_of(W1, "e4m3"), U.values_of(G, "e5m2"), U.values_of(W2, "e4m3"))
    alpha, _, _ = S.linear_scales(b, m, f)
    _, beta_x, _ = S.linear_scales(b, f, n)
    ag, bg = S.gelu_scales()
    ws = L.new_workspace()
    outs = []
    for _ in range(2):
        A, dH = U.empty(b, f, "e4m3", ld=448), U.empty(b, f, "e5m2", ld=432)
        L.us_ffn_hidden(Xt, W1t, float(alpha), Gt, W2t, float(beta_x), 1.0, float(ag), float(bg), A, dH, ws)
        assert L.us_workspace_status(ws) == 0
        outs.append((A, dH))
    _, A_codes, dH_codes = _oracle(val, alpha, beta_x, 1.0, ag, bg, "bf16", "e4m3", "e5m2")
    U.code_deltas(outs[0][0], A_codes, "e4m3")
    U.code_deltas(outs[0][1], dH_codes, "e5m2")
    for k in range(2):
        full0 = torch.as_strided(outs[0][k].view(torch.uint8), (b, outs[0][k].stride(0)), (outs[0][k].stride(0), 1))
        full1 = torch.as_strided(outs[1][k].view(torch.uint8), (b, outs[1][k].stride(0)), (outs[1][k].stride(0), 1))
        assert torch.equal(full0, full1)
        assert int(full0[:, f:].max()) == 0                     # nothing written beyond the row length


def test_ffn_hidden_host_checks_launch_nothing():
    L, synth = _mods()
    ws = L.new_workspace()
    e = U.empty

    def status(**kw):
        a = dict(X=e(272, 144, "e4m3"), W1=e(144, 400, "e4m3"), G=e(272, 208, "e5m2"), W2=e(400, 208, "e4m3"),
                 A=e(272, 400, "e4m3"), dH=e(272, 400, "e5m2"), H=None, h_dtype=torch.bfloat16)
        a.update(kw)
        with pytest.raises(L.UnitScaleError) as err:
            L.us_ffn_hidden(a["X"], a["W1"], 1.0, a["G"], a["W2"], 1.0, 1.0, 1.0, 1.0, a["A"], a["dH"], ws, H=a["H"],
                            h_dtype=a["h_dtype"])
        return err.value.status

    assert status(W1=e(160, 400, "e4m3")) == US_ERR_INVALID_ARG            # contraction lengths disagree
    assert status(W2=e(384, 208, "e4m3")) == US_ERR_INVALID_ARG            # W2 rows != d_ff
    assert status(dH=e(272, 384, "e5m2")) == US_ERR_INVALID_ARG            # output shape
    assert status(H=e(272, 400, "fp16")) == US_ERR_INVALID_ARG             # kept copy of another format than h_dtype
    assert status(h_dtype=torch.float32) == US_ERR_INVALID_ARG
    assert status(X=e(272, 144, "bf16")) == US_ERR_UNSUPPORTED             # 16-bit operands: use the separate calls
    assert status(A=e(272, 400, "bf16")) == US_ERR_UNSUPPORTED             # outputs are 8-bit
    assert status(X=e(96, 144, "e4m3"), G=e(96, 208, "e5m2"), A=e(96, 400, "e4m3"), dH=e(96, 400, "e5m2")) == US_ERR_UNSUPPORTED
    assert status(X=e(272, 144, "e4m3", ld=152)) == US_ERR_ALIGNMENT       # row pitch not a multiple of 16 bytes
    assert L.us_workspace_status(ws) == 0


def test_ffn_hidden_starved_launch_times_out_and_the_next_call_is_correct():
    """The bounded waits of this kernel, exercised in the permitted form: no loads are issued, the waits of every role
    run out, the status word is raised, tensor memory is freed and the kernel returns by itself."""
    L, synth = _mods()
    b, m, f, n = 520, 272, 1040, 272
    dev, val = _inputs(synth, b, m, f, n, 77)
    Xt, W1t, Gt, W2t = dev
    ws = L.new_workspace()
    A, dH = U.empty(b, f, "e4m3"), U.empty(b, f, "e5m2")
    L.us_test_ffn_hidden_starved(Xt, W1t, Gt, W2t, A, dH, ws, wait_limit=2000)
    assert L.us_workspace_status(ws) == US_ERR_TIMEOUT
    ws.zero_()
    alpha, _, _ = S.linear_scales(b, m, f)
    _, beta_x, _ = S.linear_scales(b, f, n)
    ag, bg = S.gelu_scales()
    L.us_ffn_hidden(Xt, W1t, float(alpha), Gt, W2t, float(beta_x), 1.0, float(ag), float(bg), A, dH, ws)
    assert L.us_workspace_status(ws) == 0
    _, A_codes, dH_codes = _oracle(val, alpha, beta_x, 1.0, ag, bg, "bf16", "e4m3", "e5m2")
    U.code_deltas(A, A_codes, "e4m3")
    U.code_deltas(dH, dH_codes, "e5m2")
    for bad in (0, 1 << 17):
        with pytest.raises(L.UnitScaleError) as err:
            L.us_test_ffn_hidden_starved(Xt, W1t, Gt, W2t, A, dH, ws, wait_limit=bad)
        assert err.value.status == US_ERR_INVALID_ARG
