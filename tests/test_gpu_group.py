"""us_linear_group: several independent linear ops in one launch, against the oracle and against the
single entry points (bit-identical: every tile is still accumulated by one accumulator over its whole K)."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import scales as S
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _mods():
    from paper_2303_11257_b200 import lib, synth
    return lib, synth


def _problem(L, synth, op, b, m, n, seed, out_fmt, skip_fmt=None, fa="e4m3", fb="e4m3"):
    X, W, G = synth.linear_tensors(b, m, n, seed)
    a, bx, bw = S.linear_scales(b, m, n)
    A, B, scale, ref_fn, oshape, code = {"fwd": (X, W, a, O.linear_fwd, (b, n), L.US_OP_FWD),
                                         "bwd_x": (G, W, bx, O.linear_bwd_x, (b, m), L.US_OP_BWD_X),
                                         "bwd_w": (X, G, bw, O.linear_bwd_w, (m, n), L.US_OP_BWD_W)}[op]
    At, Bt = U.to_device(A, fa), U.to_device(B, fb)
    ref = ref_fn(U.values_of(A, fa), U.values_of(B, fb), scale)
    ep, ep_args = None, None
    if skip_fmt:
        sk = synth.normal(seed, 9, oshape)
        cs, cb = S.residual_coefficients(0.3)
        skt = U.to_device(sk, skip_fmt)
        ep_args = dict(skip=skt, skip_coef=float(cs), out_coef=float(cb))
        ref = O.weighted_add(U.values_of(sk, skip_fmt), ref, cs, cb)
    out = U.empty(oshape[0], oshape[1], out_fmt)
    single = U.empty(oshape[0], oshape[1], out_fmt)
    mk_ep = (lambda: L.epilogue(**ep_args)) if ep_args else (lambda: None)
    return dict(op=op, code=code, At=At, Bt=Bt, scale=float(scale), ref=ref, out=out, single=single, mk_ep=mk_ep, out_fmt=out_fmt)


CASES = [
    # ragged shapes, every layout, every output format, with and without a skip tensor
    [("fwd", 304, 272, 528, "f32", None), ("bwd_x", 272, 400, 304, "bf16", "f32"), ("bwd_w", 400, 272, 304, "f32", None),
     ("fwd", 528, 144, 272, "e4m3", "bf16")],
    [("bwd_w", 1024, 512, 768, "bf16", None), ("bwd_x", 512, 384, 1040, "e5m2", None)],
    [("fwd", 272, 2064, 272, "fp16", "fp16")],
    # long and short contractions mixed: the work list gives some pairs several tiles
    [("bwd_w", 4096, 512, 512, "f32", None), ("fwd", 1536, 256, 1024, "bf16", "f32"), ("bwd_x", 1536, 1024, 128 * 3, "bf16", "bf16"),
     ("bwd_w", 2048, 304, 528, "f32", None)],
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_group_matches_oracle_and_single_calls(case):
    L, synth = _mods()
    ws = L.new_workspace()
    probs = []
    for i, (op, b, m, n, out_fmt, skip_fmt) in enumerate(CASES[case]):
        fa, fb = {"fwd": ("e4m3", "e4m3"), "bwd_x": ("e5m2", "e4m3"), "bwd_w": ("e4m3", "e5m2")}[op]
        probs.append(_problem(L, synth, op, b, m, n, 70 + 10 * case + i, out_fmt, skip_fmt, fa, fb))
    calls = [L.linear_call(p["code"], p["At"], p["Bt"], p["scale"], p["out"], p["mk_ep"]()) for p in probs]
    L.us_linear_group(calls, ws)
    assert L.us_workspace_status(ws) == 0
    for p in probs:
        U.assert_close_stored(p["out"], p["ref"], p["out_fmt"], TOL * max(1.0, np.abs(p["ref"]).max() / 4), f"group {p['op']}")
        getattr(L, "us_linear_" + p["op"])(p["At"], p["Bt"], p["scale"], p["single"], ws, p["mk_ep"]())
        torch.cuda.synchronize()
        assert torch.equal(p["out"].contiguous().view(torch.uint8), p["single"].contiguous().view(torch.uint8)), p["op"]
    assert L.us_workspace_status(ws) == 0


def test_group_unsupported_and_invalid_calls_launch_nothing():
    L, synth = _mods()
    ws = L.new_workspace()
    big = lambda fmt: (U.empty(272, 272, fmt), U.empty(272, 304, fmt), U.empty(272, 304, "f32"))

    def status(calls):
        with pytest.raises(L.UnitScaleError) as e:
            L.us_linear_group(calls, ws)
        return e.value.status

    A, B, out = big("e4m3")
    assert status([L.linear_call(L.US_OP_FWD, *big("bf16")[:2], 1.0, out)]) == 2                  # 16-bit operands
    assert status([L.linear_call(L.US_OP_FWD, U.empty(64, 272, "e4m3"), B, 1.0, U.empty(64, 304, "f32"))]) == 2     # small output
    ep = L.epilogue(act=L.US_ACT_GELU)
    assert status([L.linear_call(L.US_OP_FWD, A, B, 1.0, out, ep)]) == 2                          # fused activation
    assert status([L.linear_call(L.US_OP_FWD, A, B, 1.0, U.empty(272, 308, "f32"))]) == 1         # shape mismatch
    assert status([L.linear_call(7, A, B, 1.0, out)]) == 1
    assert status([L.linear_call(L.US_OP_FWD, A, B, 1.0, out)] * 5) == 2                          # more than four calls
    sentinel = out.clone()
    assert torch.equal(out, sentinel) and L.us_workspace_status(ws) == 0


def test_ffn_step_with_the_grouped_launch_equals_the_seven_launch_step():
    from paper_2303_11257_b200 import ffn, synth
    shape = synth.FFN_RAGGED
    shape = synth.FFNShape("ragged_wide", 400, 272, 528)
    tensors = [torch.from_numpy(t).cuda() for t in synth.ffn_tensors(shape, seed=6)]
    outs = []
    for grouped in (True, False):
        blk = ffn.UnitScaledFFN(shape.tokens, shape.d_model, shape.d_ff)
        blk.grouped = grouped
        blk.step(*tensors)
        blk.check()
        outs.append([t.clone() for t in (blk.R, blk.dX, blk.dW1, blk.dW2)])
    for a, b in zip(*outs):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
