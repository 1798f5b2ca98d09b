"""Unit-scaled encoder layer (attention block + FFN block), forward and backward, against the
oracle's chain.

Each op is checked strictly on its own elsewhere (batched GEMMs, softmax, linear ops with fused
epilogues).  Here thirty launches are chained through 16-bit and FP8 intermediates: wherever the
device and the oracle round an intermediate to neighbouring codes (a near-tie decided by float32 vs
float64 arithmetic), everything downstream moves a little.  The chain is therefore compared with a
looser bound: the first GEMM strictly, later tensors to a few 16-bit ulps of their scale, with all
but a small fraction of the elements inside the strict bound."""
import numpy as np
import pytest
import torch

from oracle import encoder as E
from tests import util as U

pytestmark = pytest.mark.gpu


def _run(nseq, slen, d, nhead, f, seed, attention="bf16"):
    from paper_2303_11257_b200 import encoder, synth
    T = nseq * slen
    host = (synth.normal(seed, 0, (T, d)), synth.normal(seed, 1, (d, 3 * d)), synth.normal(seed, 2, (d, d)),
            synth.normal(seed, 3, (d, f)), synth.normal(seed, 4, (f, d)), synth.normal(seed, 5, (T, d)))
    layer = encoder.UnitScaledEncoderLayer(nseq, slen, d, nhead, f, attention=attention)
    layer.step(*[torch.from_numpy(t).cuda() for t in host])
    layer.check()
    return layer, host


def _close(got, ref, name):
    """Deep in the chain most elements carry the echo of some upstream rounding flip, so the check is
    statistical: small mean error relative to the tensor's scale, no error of the order of the tensor
    itself, and near-perfect correlation (a wiring, transposition or scale mistake fails all three)."""
    g = U.host_values(got)
    scale = max(1.0, float(np.abs(ref).std()))
    err = np.abs(g - ref) / scale
    assert err.mean() <= 5e-2, f"{name}: mean err {err.mean():.3e}"
    assert err.max() <= 0.5 + 0.02 * float(np.abs(ref).max()) / scale, f"{name}: max err {err.max():.3e}"
    corr = np.corrcoef(g.ravel(), ref.ravel())[0, 1]
    assert corr > 0.999, f"{name}: correlation {corr:.6f}"


def _mostly_strict(got, ref, name, frac):
    g = U.host_values(got)
    scale = max(1.0, float(np.abs(ref).std()))
    outside = np.abs(g - ref) / scale > 2e-3 + U.ulp_of(ref, "bf16") / scale
    assert outside.mean() <= frac, f"{name}: {outside.mean():.3%} of the elements beyond the strict bound"


@pytest.mark.parametrize("cfg", [(2, 128, 256, 4, 512), (3, 80, 192, 3, 400)])
def test_encoder_layer_small(cfg):
    nseq, slen, d, nhead, f = cfg
    layer, host = _run(nseq, slen, d, nhead, f, seed=41)
    r = E.encoder_layer(*host, nseq, slen, nhead)
    U.assert_close_stored(layer.QKV, r.QKV, "bf16", 2e-3, "QKV")                 # first GEMM: strict
    for name, got, ref in (("S", layer.S, r.S), ("P", layer.P, r.P), ("R1", layer.R1, r.R1), ("R2", layer.ffn.R, r.ffn.R),
                           ("dC", layer.dC, r.dC), ("dP", layer.dP, r.dP), ("dS", layer.dS, r.dS), ("dQKV", layer.dQKV, r.dQKV),
                           ("dX", layer.dX, r.dX), ("dWqkv", layer.dWqkv, r.dWqkv), ("dWo", layer.dWo, r.dWo),
                           ("dW1", layer.ffn.dW1, r.ffn.dW1), ("dW2", layer.ffn.dW2, r.ffn.dW2)):
        _close(got, ref, name)
    for name, got, ref in (("S", layer.S, r.S), ("P", layer.P, r.P), ("R1", layer.R1, r.R1)):
        _mostly_strict(got, ref, name, 0.02)                                 # early in the chain: nearly all strict
    from oracle import formats as Fm
    d_c = U.code_distance(U.codes_of(layer.Cq), Fm.quantise_codes(r.Cq, Fm.E4M3), "e4m3")
    assert (d_c > 0).mean() < 0.05                        # the FP8 context tensor: few codes differ ...
    _close(layer.Cq, r.Cq, "C")                          # ... and none by much in value


def test_encoder_layer_bert_large_shape_statistics():
    """Config 5 at full size (16 x 512 tokens, d = 1024, 16 heads): the layer runs, reports no timeout,
    and its tensors have the scale the oracle shows at a smaller size (unit-ish at initialisation)."""
    layer, _ = _run(16, 512, 1024, 16, 4096, seed=42)
    st = lambda t: t.float().std().item()
    assert abs(st(layer.QKV) - 1) < 0.03 and abs(st(layer.S) - 1) < 0.05
    assert abs(layer.P.float().mean().item() - 1) < 0.01
    for t in (layer.R1, layer.ffn.R, layer.dX, layer.dQKV, layer.dWqkv, layer.dWo, layer.ffn.dW1, layer.ffn.dW2):
        assert 0.5 < st(t) < 6.0
    assert torch.isfinite(layer.dX.float()).all().item()


@pytest.mark.parametrize("cfg", [(2, 128, 256, 4, 512), (3, 80, 192, 3, 400)])
def test_encoder_layer_fp8_attention(cfg):
    """FP8 operands for the attention matmuls (Q, K, V, P as E4M3; dC, dS, dQ, dK, dV as E5M2).  The first
    GEMM's FP8 output is within one code of the oracle's; the rest of the chain is compared statistically,
    with wider bounds than the 16-bit mode because a one-code difference is 6 % (E4M3) or 12 % (E5M2) of a value."""
    nseq, slen, d, nhead, f = cfg
    layer, host = _run(nseq, slen, d, nhead, f, seed=43, attention="fp8")
    r = E.encoder_layer(*host, nseq, slen, nhead, att="fp8")
    U.assert_close_stored(layer.QKV, r.QKV, "e4m3", 2e-3, "QKV")
    assert layer.dQKV is layer.dQKVq and layer.launches_per_step == 23 - (6 - layer.ffn.gemm_launches)

    def close(got, ref, name, mean_tol):
        g = U.host_values(got)
        scale = max(1.0, float(np.abs(ref).std()))
        err = np.abs(g - ref) / scale
        assert err.mean() <= mean_tol, f"{name}: mean err {err.mean():.3e}"
        assert np.corrcoef(g.ravel(), ref.ravel())[0, 1] > 0.995, name

    for name, got, ref in (("S", layer.S, r.S), ("P", layer.P, r.P), ("C", layer.Cq, r.Cq), ("R1", layer.R1, r.R1)):
        close(got, ref, name, 2e-2)
    for name, got, ref in (("R2", layer.ffn.R, r.ffn.R), ("dC", layer.dC, r.dC), ("dP", layer.dP, r.dP), ("dS", layer.dS, r.dS),
                           ("dQKV", layer.dQKV, r.dQKV), ("dX", layer.dX, r.dX), ("dWqkv", layer.dWqkv, r.dWqkv),
                           ("dWo", layer.dWo, r.dWo), ("dW1", layer.ffn.dW1, r.ffn.dW1), ("dW2", layer.ffn.dW2, r.ffn.dW2)):
        close(got, ref, name, 8e-2)
    # where the chain has not yet diverged the FP8 tensors agree code for code almost everywhere
    from oracle import formats as Fm
    d_p = U.code_distance(U.codes_of(layer.P), Fm.quantise_codes(r.P, Fm.E4M3), "e4m3")
    assert d_p.max() <= 2 and (d_p > 0).mean() < 0.08


@pytest.mark.parametrize("attention", ["bf16", "fp8"])
def test_encoder_layer_post_norm(attention):
    """Post-norm arrangement: a scaled layer norm after each residual sum, forward and backward."""
    from paper_2303_11257_b200 import encoder, synth
    nseq, slen, d, nhead, f = 2, 128, 256, 4, 512
    T = nseq * slen
    host = (synth.normal(44, 0, (T, d)), synth.normal(44, 1, (d, 3 * d)), synth.normal(44, 2, (d, d)),
            synth.normal(44, 3, (d, f)), synth.normal(44, 4, (f, d)), synth.normal(44, 5, (T, d)))
    ln_host = [(1 + 0.2 * synth.normal(44, 6, (1, d)))[0], (0.1 * synth.normal(44, 7, (1, d)))[0],
               (1 + 0.2 * synth.normal(44, 8, (1, d)))[0], (0.1 * synth.normal(44, 9, (1, d)))[0]]
    layer = encoder.UnitScaledEncoderLayer(nseq, slen, d, nhead, f, attention=attention, norm="post")
    layer.step(*[torch.from_numpy(t).cuda() for t in host], ln=[torch.from_numpy(v.astype(np.float32)).cuda() for v in ln_host])
    layer.check()
    r = E.encoder_layer(*host, nseq, slen, nhead, att=attention, norm="post", ln=[v.astype(np.float32) for v in ln_host])

    def close(got, ref, name, mean_tol):
        g = U.host_values(got)
        scale = max(1.0, float(np.abs(ref).std()))
        err = np.abs(g - ref) / scale
        assert err.mean() <= mean_tol, f"{name}: mean err {err.mean():.3e}"
        assert np.corrcoef(g.ravel(), ref.ravel())[0, 1] > 0.995, name

    tol_f, tol_b = (2e-2, 8e-2) if attention == "fp8" else (1e-2, 5e-2)
    for name, got, ref in (("U1", layer.U1, r.U1), ("R1", layer.R1, r.R1), ("U2", layer.ffn.R, r.ffn.R), ("R2", layer.R2, r.R2)):
        close(got, ref, name, tol_f)
    for name, got, ref in (("dU2", layer.dU2, r.dU2), ("dU1", layer.dU1, r.dU1), ("dX", layer.dX, r.dX), ("dWqkv", layer.dWqkv, r.dWqkv),
                           ("dW1", layer.ffn.dW1, r.ffn.dW1), ("dln2_w", layer.dln[2], r.dln2[0].reshape(-1)),
                           ("dln2_c", layer.dln[3], r.dln2[1].reshape(-1)), ("dln1_w", layer.dln[0], r.dln1[0].reshape(-1)),
                           ("dln1_c", layer.dln[1], r.dln1[1].reshape(-1))):
        close(got, ref, name, tol_b)
    # the second norm's backward pass sees the same U2 up to chain noise and an exact G: strict-ish on its bias gradient
    assert np.abs(layer.dln[3].cpu().numpy() - r.dln2[1].reshape(-1)).max() < 1e-4
    # the layer output is normalised: per token, (R2 - c2) / w2 has zero mean and unit variance
    z = (layer.R2.float().cpu().numpy() - ln_host[3]) / ln_host[2]
    assert np.abs(z.mean(axis=1)).max() < 0.03 and np.abs(z.std(axis=1) - 1).max() < 0.03
