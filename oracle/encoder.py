"""Unit-scaled Transformer encoder layer, forward and backward (test infrastructure, fp64 NumPy).

Self-attention block followed by the FFN block of ops.py, both wrapped in fixed(tau) residuals
(section "Weighted addition"), without layer norm.  Scaled dot-product attention follows the
appendix "Unit scaling and attention" (scores scaled by 1 / sqrt(d_head) in both passes) and the
paragraph "Softmax (followed by matmul)" (softmax scaled by the row length s, then an ordinary
scaled matmul with alpha = s^-1/2).  Matmul inputs of the projections are FP8 (E4 activations and
weights, E5 gradients); the attention matmuls take 16-bit operands (att = "bf16" / "fp16") or, with
att = "fp8", FP8 operands like every other matmul (section "Experiments": all matmul inputs are
quantised): Q, K, V and the softmax output P as E4, the gradients dC, dS and dQ, dK, dV as E5, while
the softmax input S and the gradient dP of its output, which feed no matmul, stay in BF16.  Every
stored intermediate is rounded to the format it is stored in; with fused_scores the scores (and, in the
backward pass, the gradient of the softmax output) are not stored between the matmul that makes them and
the softmax (gradient) that consumes them, and therefore not rounded.

norm = "post" adds the post-norm arrangement of the appendix "Model architectures"
(res^PostNorm(f, z) = layernorm(interp(z, f(z)))): each of the two residual sums goes through a scaled
layer norm (table row layer_norm: alpha = 1, beta_x = 1, beta_w = beta_c = T^-1/2 for T tokens).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import ops as O
from . import scales as S


@dataclass
class EncoderResult:
    QKV: np.ndarray = None
    S: np.ndarray = None
    P: np.ndarray = None
    Cq: np.ndarray = None
    R1: np.ndarray = None
    ffn: O.FFNResult = None
    dC: np.ndarray = None
    dP: np.ndarray = None
    dS: np.ndarray = None
    dQKV: np.ndarray = None
    dX: np.ndarray = None
    dWqkv: np.ndarray = None
    dWo: np.ndarray = None
    # post-norm only: the residual sums before each layer norm, the layer output, and the gradients of the norms
    U1: np.ndarray = None
    R2: np.ndarray = None
    dU2: np.ndarray = None
    dU1: np.ndarray = None
    dln1: tuple = None          # (dw, dc) of the norm after the attention block
    dln2: tuple = None          # (dw, dc) of the norm after the FFN block


def _heads(M, nseq, slen, nhead, hd, which, d):
    """[T x 3d] (or [T x d] with which = 0) -> [nseq, nhead, slen, hd] view of one of Q / K / V."""
    o = which * d
    return M[:, o:o + nhead * hd].reshape(nseq, slen, nhead, hd).transpose(0, 2, 1, 3)


def _unheads(H, nseq, slen, nhead, hd):
    """[nseq, nhead, slen, hd] -> [T x d]."""
    return H.transpose(0, 2, 1, 3).reshape(nseq * slen, nhead * hd)


def encoder_layer(X, Wqkv, Wo, W1, W2, G, nseq, slen, nhead, tau=0.5, att="bf16", norm=None, ln=None,
                  eps=1e-5, fused_scores=False) -> EncoderResult:
    """norm = None: R2 = res(ffn, res(attention, X)), G = dL/dR2 (the FFN block's output r.ffn.R).
    norm = "post": ln = (w1, c1, w2, c2), each [d]; R1 = LN1(U1), R2 = LN2(U2) with U the residual sums.
    fused_scores: the scores S feed the softmax directly and are never stored, hence never rounded
    (ops.attention_fwd), and likewise the gradient dP of the weights in the backward pass
    (ops.attention_bwd_scores); r.S and r.dP then hold the unrounded values, and dQ, dK, dV are rounded once, to E5
    (the format of the one matmul operand they become), instead of first to the attention gradients' format."""
    T, d = X.shape
    hd = d // nhead
    f32 = lambda v: float(np.float32(v))
    r = EncoderResult()
    c_skip, c_branch = S.residual_coefficients(tau)
    a_qkv, b_qkv, b_w = d ** -0.5, (3 * d) ** -0.5, T ** -0.5
    a_o, b_o = d ** -0.5, d ** -0.5
    a_s = b_Q = b_K = hd ** -0.5
    a_c, b_P, b_V = slen ** -0.5, hd ** -0.5, slen ** -0.5
    sm = float(slen)
    # storage formats of the attention tensors: matmul operands (activations, gradients) and the rest
    f_act, f_grad, f_wide = ("e4m3", "e5m2", "bf16") if att == "fp8" else (att, att, att)

    Xq, _ = O.store(np.asarray(X), "e4m3")
    Wqkv_q, _ = O.store(np.asarray(Wqkv), "e4m3")
    Wo_q, _ = O.store(np.asarray(Wo), "e4m3")
    # ---- forward
    r.QKV, _ = O.store(O.linear_fwd(Xq, Wqkv_q, a_qkv), f_act)
    Q, K, V = (_heads(r.QKV, nseq, slen, nhead, hd, i, d) for i in range(3))
    if fused_scores:
        S4 = f32(a_s) * (Q @ K.transpose(0, 1, 3, 2))
        P4, C4 = O.attention_fwd(Q, K, V, a_s, sm, a_c, f_act)
    else:
        S4, _ = O.store(f32(a_s) * (Q @ K.transpose(0, 1, 3, 2)), f_wide)          # alpha Q K^T per (sequence, head)
        P4, _ = O.store(O.softmax_fwd(S4, sm), f_act)
        C4 = f32(a_c) * (P4 @ V)
    r.Cq, _ = O.store(_unheads(C4, nseq, slen, nhead, hd), "e4m3")
    r.S, r.P = S4.reshape(-1, slen), P4.reshape(-1, slen)
    ep = O.Epilogue(skip=np.asarray(X, np.float64), skip_coef=c_skip, out_coef=c_branch)
    r.R1, _, _ = O.apply_epilogue(O.linear_fwd(r.Cq, Wo_q, a_o), ep, "bf16")
    sc = O.FFNScales.unconstrained(T, d, W1.shape[1], tau)
    if norm == "post":
        w1, c1, w2, c2 = (np.asarray(v, np.float64).reshape(1, d) for v in ln)
        b_ln = f32(T ** -0.5)
        r.U1 = r.R1
        r.R1, _ = O.store(O.layer_norm_fwd(r.U1, w1, c1, f32(eps)), "bf16")
        fwd = O.ffn_block(r.R1, W1, W2, np.zeros_like(np.asarray(G, np.float64)), sc, operand="fp8")   # forward part only
        r.R2, _ = O.store(O.layer_norm_fwd(fwd.R, w2, c2, f32(eps)), "bf16")
        # ---- backward through the second norm, the FFN block, the first norm
        dU2, dw2, dc2 = O.layer_norm_bwd(fwd.R, w2, np.asarray(G, np.float64), f32(eps), 1.0, b_ln)
        r.dU2, _ = O.store(dU2, "bf16")
        r.dln2 = (O.store(dw2, "f32")[0], O.store(dc2, "f32")[0])
        r.ffn = O.ffn_block(r.R1, W1, W2, r.dU2, sc, operand="fp8")
        dU1, dw1, dc1 = O.layer_norm_bwd(r.U1, w1, r.ffn.dX, f32(eps), 1.0, b_ln)
        r.dU1, _ = O.store(dU1, "bf16")
        r.dln1 = (O.store(dw1, "f32")[0], O.store(dc1, "f32")[0])
        g1 = r.dU1
    else:
        r.ffn = O.ffn_block(r.R1, W1, W2, G, sc, operand="fp8")
        g1 = r.ffn.dX
    # ---- backward
    g1q, _ = O.store(g1, "e5m2")
    r.dC, _ = O.store(O.linear_bwd_x(g1q, Wo_q, b_o), f_grad)
    r.dWo, _ = O.store(O.linear_bwd_w(r.Cq, g1q, b_w), "f32")
    dC4 = _heads(r.dC, nseq, slen, nhead, hd, 0, d)
    dV4 = f32(b_V) * (P4.transpose(0, 1, 3, 2) @ dC4)                           # beta_2 X^T G with X = P
    if fused_scores:
        dP4 = f32(b_P) * (dC4 @ V.transpose(0, 1, 3, 2))                          # kept unrounded, like the scores
        dS4, dQ4 = O.attention_bwd_scores(dC4, P4, K, V, b_P, sm, sm, b_Q, f_grad)
    else:
        dP4, _ = O.store(f32(b_P) * (dC4 @ V.transpose(0, 1, 3, 2)), f_wide)       # beta_1 G W^T with W = V
        dS4, _ = O.store(O.softmax_bwd(P4, dP4, sm, sm), f_grad)
        dQ4 = f32(b_Q) * (dS4 @ K)
    dK4 = f32(b_K) * (dS4.transpose(0, 1, 3, 2) @ Q)
    r.dP, r.dS = dP4.reshape(-1, slen), dS4.reshape(-1, slen)
    dQKV = np.concatenate([_unheads(t, nseq, slen, nhead, hd) for t in (dQ4, dK4, dV4)], axis=1)
    # dQ, dK, dV feed only the QKV projection's backward matmuls, whose gradient operand is E5; with fused_scores they are
    # written once, in that format, instead of being stored in the attention gradients' format and cast afterwards
    r.dQKV, _ = O.store(dQKV, "e5m2" if fused_scores else f_grad)
    dQKVq, _ = O.store(r.dQKV, "e5m2")
    ep = O.Epilogue(skip=g1, skip_coef=c_skip, out_coef=c_branch)
    r.dX, _, _ = O.apply_epilogue(O.linear_bwd_x(dQKVq, Wqkv_q, b_qkv), ep, "bf16")
    r.dWqkv, _ = O.store(O.linear_bwd_w(Xq, dQKVq, b_w), "f32")
    return r
