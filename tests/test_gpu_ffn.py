"""The chained unit-scaled FFN block (forward + backward) against the oracle's chain."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import ops as O
from tests import util as U

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _mods():
    from paper_2303_11257_b200 import ffn, lib, synth
    return ffn, lib, synth


def _run(shape, operand, seed=0, sigma_x=1.0, io="bf16"):
    ffn, L, synth = _mods()
    X, W1, W2, G = synth.ffn_tensors(shape, seed, sigma_x)
    blk = ffn.UnitScaledFFN(shape.tokens, shape.d_model, shape.d_ff, operand=operand,
                            io_dtype=U.TORCH_OF[io])
    dev = [torch.from_numpy(t).cuda() for t in (X, W1, W2, G)]
    blk.step(*dev)
    blk.check()
    return blk, (X, W1, W2, G)


def _oracle(shape, tensors, operand, io="bf16"):
    sc = O.FFNScales.unconstrained(shape.tokens, shape.d_model, shape.d_ff)
    return O.ffn_block(*tensors, sc, operand=operand, io_dtype=io)


@pytest.mark.parametrize("shape_name", ["FFN_SMALL", "FFN_RAGGED"])
@pytest.mark.parametrize("operand", ["fp8", "bf16", "fp16"])
def test_ffn_block_full_compare(shape_name, operand):
    ffn, L, synth = _mods()
    shape = getattr(synth, shape_name)
    blk, tensors = _run(shape, operand)
    r = _oracle(shape, tensors, operand)
    act = "e4m3" if operand == "fp8" else operand
    grad = "e5m2" if operand == "fp8" else operand
    # casts of the same float32 values: bit-exact
    assert np.array_equal(U.codes_of(blk.Xq), F.quantise_codes(tensors[0], F.FORMATS[act]))
    assert np.array_equal(U.codes_of(blk.W1q), F.quantise_codes(tensors[1], F.FORMATS[act]))
    assert np.array_equal(U.codes_of(blk.Gq), F.quantise_codes(tensors[3], F.FORMATS[grad]))
    U.assert_close_stored(blk.H, r.H, "bf16", TOL, "H")
    if operand == "fp8":
        U.assert_close_stored(blk.Aq, r.Aq, act, TOL, "A")
        U.assert_close_stored(blk.dHq, r.dHq, grad, TOL, "dH")
    else:
        assert np.abs(U.host_values(blk.Aq) - r.Aq).max() <= TOL + np.abs(r.Aq).max() * 2.0 ** -8
        assert np.abs(U.host_values(blk.dHq) - r.dHq).max() <= TOL + np.abs(r.dHq).max() * 2.0 ** -8
    U.assert_close_stored(blk.R, r.R, "bf16", TOL, "R")
    U.assert_close_stored(blk.dX, r.dX, "bf16", TOL, "dX")
    U.assert_close_stored(blk.dW1, r.dW1, "f32", TOL, "dW1")
    U.assert_close_stored(blk.dW2, r.dW2, "f32", TOL, "dW2")


@pytest.fixture(scope="module")
def bert_large_fp8():
    ffn, L, synth = _mods()
    shape = synth.FFN_BERT_LARGE
    blk, tensors = _run(shape, "fp8", seed=0)
    return shape, blk, tensors


def test_ffn_bert_large_sampled_rows(bert_large_fp8):
    """Full BERT-large shape in the benchmark's launch configuration: the oracle chain is evaluated
    for a sample of token rows (forward and input gradient are row-wise independent given the
    weights) and for sampled rows of the weight gradients (which need all tokens of the stored
    activations: those come from a second, full oracle matmul on oracle-side tensors)."""
    shape, blk, (X, W1, W2, G) = bert_large_fp8
    T, d, f = shape.tokens, shape.d_model, shape.d_ff
    rng = np.random.default_rng(1)
    rows = np.unique(np.concatenate([[0, 127, 128, T - 1], rng.integers(0, T, 28)]))
    sc = O.FFNScales.unconstrained(T, d, f)
    r = O.ffn_block(X[rows], W1, W2, G[rows], sc, operand="fp8")
    g = lambda t: U.host_values(t[torch.from_numpy(rows).cuda()])
    U.assert_close_stored(blk.H[torch.from_numpy(rows).cuda()], r.H, "bf16", TOL, "H rows")
    d_codes = U.code_distance(U.codes_of(blk.Aq[torch.from_numpy(rows).cuda()]), r.Aq_codes, "e4m3")
    assert d_codes.max() <= 1 and (d_codes > 0).mean() < 2e-3
    U.assert_close_stored(blk.R[torch.from_numpy(rows).cuda()], r.R, "bf16", TOL, "R rows")
    d_codes = U.code_distance(U.codes_of(blk.dHq[torch.from_numpy(rows).cuda()]), r.dHq_codes, "e5m2")
    assert d_codes.max() <= 1 and (d_codes > 0).mean() < 2e-3
    U.assert_close_stored(blk.dX[torch.from_numpy(rows).cuda()], r.dX, "bf16", TOL, "dX rows")
    # statistics at initialisation (section "Unit Scaling": unit variance of activations and gradients)
    assert abs(blk.H.float().std().item() - 1) < 0.02
    assert abs(blk.Aq.float().std().item() - 1) < 0.03
    assert 0.9 < blk.dW1.std().item() < 1.2 and 0.9 < blk.dW2.std().item() < 1.2


def test_ffn_bert_large_weight_gradients(bert_large_fp8):
    shape, blk, (X, W1, W2, G) = bert_large_fp8
    T, d, f = shape.tokens, shape.d_model, shape.d_ff
    sc = O.FFNScales.unconstrained(T, d, f)
    r = O.ffn_block(X, W1, W2, G, sc, operand="fp8")          # full oracle chain (numpy fp64 matmuls)
    for got, ref in ((blk.dW1, r.dW1), (blk.dW2, r.dW2)):
        g = U.host_values(got)
        assert np.abs(g - ref).max() <= TOL
    U.assert_close_stored(blk.dX, r.dX, "bf16", TOL, "dX")
    U.assert_close_stored(blk.R, r.R, "bf16", TOL, "R")


@pytest.mark.parametrize("sigma", [2.0 ** 8, 2.0 ** -8])
def test_ffn_saturation_and_underflow_in_fused_cast(sigma):
    """X ~ N(0, sigma^2): sigma = 2^8 saturates part of q_E4(X) and of the fused A cast; sigma = 2^-8
    pushes X into E4M3's subnormal range.  Codes must still agree with the oracle's."""
    ffn, L, synth = _mods()
    shape = synth.FFN_SMALL
    blk, tensors = _run(shape, "fp8", seed=3, sigma_x=sigma)
    r = _oracle(shape, tensors, "fp8")
    want = F.quantise_codes(tensors[0], F.E4M3)
    assert np.array_equal(U.codes_of(blk.Xq), want)
    if sigma > 1:
        assert ((want & 0x7F) == 0x7E).mean() > 0.02           # some inputs clip to +-448
        assert ((r.Aq_codes & 0x7F) == 0x7E).mean() > 0.01     # and the fused GELU output saturates too
    else:
        assert ((want & 0x78) == 0).mean() > 0.5               # mostly subnormal / zero codes
    d = U.code_distance(U.codes_of(blk.Aq), r.Aq_codes, "e4m3")
    assert d.max() <= 1
    U.assert_close_stored(blk.dW2, r.dW2, "f32", TOL * max(1.0, np.abs(r.dW2).max()), "dW2")
