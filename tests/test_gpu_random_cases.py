"""Seeded random cases of the linear ops: op, shape (ragged and multi-tile), operand and output formats, row
padding of every tensor and the fused epilogue are drawn at random and compared with the oracle, one case at a
time.  Complements the hand-picked shapes of the other GEMM tests."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import scales as S
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3


@pytest.mark.parametrize("seed", [11, 12])
def test_random_linear_cases(seed):
    from paper_2303_11257_b200 import lib as L, synth
    rng = np.random.default_rng(seed)
    N = 60
    failures = []

    def dim(maxv, mult=16):
        k = int(rng.choice([16, 32, 48, 64, 96, 128, 144, 256, 272, 384, 512, 528, 1024, 1040])) if rng.random() < 0.5 \
            else int(rng.integers(1, maxv // mult + 1)) * mult
        return min(k, maxv)

    def ld_for(cols, e):
        unit = 16 // e                                   # rows must start 16-byte aligned
        base = (cols + unit - 1) // unit * unit
        return base + int(rng.choice([0, 0, unit, 2 * unit]))

    for case in range(N):
        op = rng.choice(["fwd", "bwd_x", "bwd_w"])
        operand = rng.choice(["fp8", "fp8", "e4e4", "bf16", "fp16"])
        b = int(rng.integers(1, 900 if op == "bwd_w" else 700))        # any number of rows; widths in multiples of 16
        m, n = dim(1100), dim(1100)
        out_fmt = rng.choice(["f32", "bf16", "fp16", "e4m3", "e5m2"])
        epi = rng.choice(["none", "none", "gelu", "gelu_grad", "skip", "gelu_skip"])
        X, W, G = synth.linear_tensors(b, m, n, 1000 * seed + case)
        a, bx, bw = S.linear_scales(b, m, n)
        if op == "fwd": A, B, scale, ref_fn, osh = X, W, a, O.linear_fwd, (b, n)
        elif op == "bwd_x": A, B, scale, ref_fn, osh = G, W, bx, O.linear_bwd_x, (b, m)
        else: A, B, scale, ref_fn, osh = X, G, bw, O.linear_bwd_w, (m, n)
        if operand == "fp8": fa, fb = {"fwd": ("e4m3", "e4m3"), "bwd_x": ("e5m2", "e4m3"), "bwd_w": ("e4m3", "e5m2")}[op]
        elif operand == "e4e4": fa, fb = "e4m3", "e4m3"
        else: fa = fb = operand
        es = 1 if fa.startswith("e") else 2
        desc = f"case {case}: {op} b={b} m={m} n={n} {fa}x{fb}->{out_fmt} epi={epi}"
        try:
            At, Bt = U.to_device(A, fa, ld_for(A.shape[1], es)), U.to_device(B, fb, ld_for(B.shape[1], es))
            oes = {"f32": 4, "bf16": 2, "fp16": 2, "e4m3": 1, "e5m2": 1}[out_fmt]
            out = U.empty(osh[0], osh[1], out_fmt, ld_for(osh[1], oes))
            ws = L.new_workspace()
            val = ref_fn(U.values_of(A, fa), U.values_of(B, fb), scale)
            ep = None; ref = val; extra = []
            if epi in ("gelu", "gelu_skip"):
                aux_fmt = rng.choice(["bf16", "fp16"])
                H = U.empty(osh[0], osh[1], aux_fmt, ld_for(osh[1], 2))
                kw = dict(act=L.US_ACT_GELU, act_in_scale=0.9, act_out_scale=1.7, aux=H)
                ref = O.gelu_fwd(val, 0.9, 1.7)
                if epi == "gelu_skip":
                    sk = synth.normal(77, case, osh); skt = U.to_device(sk, "bf16", ld_for(osh[1], 2))
                    kw.update(skip=skt, skip_coef=0.6, out_coef=0.8)
                    ref = 0.6000000238418579 * U.values_of(sk, "bf16") + 0.800000011920929 * ref
                ep = L.epilogue(**kw)
                extra.append((H, val, aux_fmt, "aux"))
            elif epi == "gelu_grad":
                Hh = synth.normal(78, case, osh); aux_fmt = rng.choice(["bf16", "fp16"])
                Ht = U.to_device(Hh, aux_fmt, ld_for(osh[1], 2))
                ep = L.epilogue(act=L.US_ACT_GELU_GRAD, act_in_scale=1.1, act_out_scale=1.48, aux=Ht)
                ref = O.gelu_bwd(U.values_of(Hh, aux_fmt), val, 1.1, 1.48)
            elif epi == "skip":
                sf = rng.choice(["f32", "bf16", "fp16"]); sk = synth.normal(79, case, osh)
                skt = U.to_device(sk, sf, ld_for(osh[1], 4 if sf == "f32" else 2))
                ep = L.epilogue(skip=skt, skip_coef=0.6, out_coef=0.8)
                ref = 0.6000000238418579 * U.values_of(sk, sf) + 0.800000011920929 * val
            getattr(L, "us_linear_" + op)(At, Bt, float(scale), out, ws, ep)
            torch.cuda.synchronize()
            assert L.us_workspace_status(ws) == 0, "timeout status"
            U.assert_close_stored(out, ref, out_fmt, TOL * max(1.0, float(np.abs(ref).max()) / 8), desc)
            for t, r, f, nm in extra:
                U.assert_close_stored(t, r, f, TOL, desc + " " + nm)
        except Exception as e:
            failures.append(f"{desc} :: {type(e).__name__} {str(e)[:200]}")
    assert not failures, "\n".join(failures)
