"""Unit-scaled ops and the FFN block, forward and backward (test infrastructure, fp64).

Each function is the paper's definition of the op evaluated in float64 on
operands that have already been rounded to their storage format:

  * scaled ops f* = alpha f, f*_grad_i = beta_i f_grad_i   (section "Scaled ops");
  * matmul*, matmul*_grad_1, matmul*_grad_2                 (section "Example");
  * gelu(x) = x Phi(x) with its scale factors               ("Table of unit scaling factors");
  * fixed(tau) residual sqrt(1-tau) x + sqrt(tau) f(x) and the rewrite that
    moves the backward factor to the branch entry           (section "Weighted addition");
  * FP8 only on matmul inputs, E4 for activations / weights and E5 for
    gradients, outputs in higher precision                  (sections "Mixed precision",
    "Trade-offs of low-precision training").

Scale factors arrive as the float32 constants the device library receives and
are promoted to float64 before use.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
from scipy import special

from . import formats as F
from . import scales as S


def _f32(c) -> float:
    """The float32-rounded value of a scalar, as a Python float (double)."""
    return float(np.float32(c))


# --------------------------------------------------------------------------- linear

def linear_fwd(X, W, alpha):
    """matmul*(X, W) = alpha * X W;  X [b x m], W [m x n] -> [b x n]."""
    return _f32(alpha) * (np.asarray(X, np.float64) @ np.asarray(W, np.float64))


def linear_bwd_x(G, W, beta_x):
    """matmul*_grad(X, W, G)_1 = beta_1 * G W^T;  G [b x n], W [m x n] -> [b x m]."""
    return _f32(beta_x) * (np.asarray(G, np.float64) @ np.asarray(W, np.float64).T)


def linear_bwd_w(X, G, beta_w):
    """matmul*_grad(X, W, G)_2 = beta_2 * X^T G;  X [b x m], G [b x n] -> [m x n]."""
    return _f32(beta_w) * (np.asarray(X, np.float64).T @ np.asarray(G, np.float64))


# --------------------------------------------------------------------------- gelu

def _Phi(z):
    return 0.5 * special.erfc(-z / math.sqrt(2.0))      # = (1 + erf(z / sqrt 2)) / 2, accurate in the lower tail


def _phi(z):
    return np.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)


def gelu_fwd(H, s_in, alpha_g):
    """A = alpha_g * gelu(s_in * H), gelu(x) = x Phi(x)."""
    z = _f32(s_in) * np.asarray(H, np.float64)
    return _f32(alpha_g) * z * _Phi(z)


def gelu_bwd(H, dA, s_in, beta_g):
    """dH = beta_g * s_in * gelu'(s_in * H) * dA, gelu'(x) = Phi(x) + x phi(x)."""
    z = _f32(s_in) * np.asarray(H, np.float64)
    return _f32(beta_g) * _f32(s_in) * (_Phi(z) + z * _phi(z)) * np.asarray(dA, np.float64)


# --------------------------------------------------------------------------- other activations

def _act(fn: str):
    """(f, f') of a table activation ("Activations": relu, gelu, tanh, sigmoid), float64."""
    if fn == "relu":
        return (lambda z: np.maximum(z, 0.0)), (lambda z: (z > 0) * 1.0)
    if fn == "gelu":
        return (lambda z: z * _Phi(z)), (lambda z: _Phi(z) + z * _phi(z))
    if fn == "tanh":
        return np.tanh, (lambda z: 1.0 - np.tanh(z) ** 2)
    if fn == "sigmoid":
        from scipy.special import expit                              # (1 + e^-z)^-1 without overflow
        return expit, (lambda z: expit(z) * expit(-z))
    raise ValueError(fn)


def activation_fwd(fn, H, s_in, alpha):
    """A = alpha * f(s_in * H) for a table activation f."""
    f, _ = _act(fn)
    return _f32(alpha) * f(_f32(s_in) * np.asarray(H, np.float64))


def activation_bwd(fn, H, dA, s_in, beta):
    """dH = beta * s_in * f'(s_in * H) * dA."""
    _, df = _act(fn)
    z = _f32(s_in) * np.asarray(H, np.float64)
    return _f32(beta) * _f32(s_in) * df(z) * np.asarray(dA, np.float64)


# --------------------------------------------------------------------------- residual

def weighted_add(a, b, coef_a, coef_b):
    """coef_a * a + coef_b * b with float32-rounded coefficients."""
    return _f32(coef_a) * np.asarray(a, np.float64) + _f32(coef_b) * np.asarray(b, np.float64)


def residual_add(skip, branch, tau):
    """fixed(tau): sqrt(1 - tau) * skip + sqrt(tau) * branch.

    The same expression serves the backward pass: the branch output receives the
    incoming gradient unscaled, and the factor sqrt(tau) is applied where the
    branch's input gradient rejoins the skip gradient.
    """
    ca, cb = S.residual_coefficients(tau)
    return weighted_add(skip, branch, ca, cb)


def weighted_add_n(xs, gammas, alpha=None):
    """alpha * sum_i gamma_i x_i (table row "weighted_add": alpha = (sum_i gamma_i^2)^-1/2, which keeps
    unit variance for independent unit-variance inputs; beta_i = 1 / gamma_i makes every input's
    gradient the incoming gradient times alpha * gamma_i * beta_i = alpha)."""
    gam = [_f32(g) for g in gammas]
    if alpha is None:
        alpha = sum(g * g for g in gam) ** -0.5
    acc = np.zeros_like(np.asarray(xs[0], np.float64))
    for g, x in zip(gam, xs):
        acc = acc + g * np.asarray(x, np.float64)
    return _f32(alpha) * acc


# --------------------------------------------------------------------------- softmax

def softmax_fwd(S, alpha):
    """alpha * softmax over the last axis (table row "softmax": alpha = s for rows of s elements)."""
    S = np.asarray(S, np.float64)
    e = np.exp(S - S.max(axis=-1, keepdims=True))
    return _f32(alpha) * e / e.sum(axis=-1, keepdims=True)


def softmax_bwd(P, dP, alpha, beta):
    """beta * softmax_grad: dS_j = beta * p_j (dP_j - sum_k p_k dP_k), p = P / alpha = softmax(S).

    P is the forward pass's scaled output as stored; dP is the gradient with respect to it."""
    p = np.asarray(P, np.float64) / _f32(alpha)
    dP = np.asarray(dP, np.float64)
    return _f32(beta) * p * (dP - np.sum(p * dP, axis=-1, keepdims=True))


# --------------------------------------------------------------------------- scaled dot-product attention

def attention_fwd(Q, K, V, alpha_scores, softmax_scale, alpha_context, p_dtype: str):
    """Scaled dot-product attention of one (sequence, head) problem with the scores kept unrounded
    (appendix "Unit scaling and attention", paragraph "Softmax (followed by matmul)"):

        S = alpha_scores * Q K^T            Q [s_q x d], K [s_k x d]          (never stored)
        P = store(softmax_scale * softmax(S) over each row, p_dtype)          [s_q x s_k]
        C = alpha_context * P V             V [s_k x d]                       [s_q x d]

    P is a matmul input and is therefore rounded to its operand format before the second matmul; S
    feeds no matmul and no memory, so it is not rounded at all.  Returns (P as stored, C unrounded).
    Leading batch axes are allowed on all three operands."""
    Q, K, V = (np.asarray(t, np.float64) for t in (Q, K, V))
    S = _f32(alpha_scores) * (Q @ np.swapaxes(K, -1, -2))
    P, _ = store(softmax_fwd(S, softmax_scale), p_dtype)
    return P, _f32(alpha_context) * (P @ V)


def attention_bwd_scores(dC, P, K, V, beta_p, softmax_alpha, softmax_beta, beta_q, ds_dtype: str):
    """Backward of attention_fwd down to the queries, with the gradient of the weights kept unrounded:

        dP = beta_p * dC V^T                                  dC [s_q x d], V [s_k x d]      (never stored)
        dS = store(softmax_beta * p (dP - sum_k p_k dP_k), ds_dtype),  p = P / softmax_alpha   [s_q x s_k]
        dQ = beta_q * dS K                                    K [s_k x d]                      [s_q x d]

    (matmul*_grad_1 with W = V for dP and the forward matmul form with W = K for dQ, section "Example"; the softmax
    gradient of the table row "softmax").  P is the forward pass's stored output.  dS is a matmul input (of dQ here and
    of dK = beta dS^T Q elsewhere) and is rounded to its operand format; dP feeds no matmul and no memory.
    Returns (dS as stored, dQ unrounded).  Leading batch axes are allowed."""
    dC, P, K, V = (np.asarray(t, np.float64) for t in (dC, P, K, V))
    dP = _f32(beta_p) * (dC @ np.swapaxes(V, -1, -2))
    dS, _ = store(softmax_bwd(P, dP, softmax_alpha, softmax_beta), ds_dtype)
    return dS, _f32(beta_q) * (dS @ K)


# --------------------------------------------------------------------------- softmax cross-entropy

def softmax_xent_fwd(X, t):
    """softmax_xent(x, t) = log softmax(x)_t per row (table row "softmax_xent", alpha = 1):
    x_t - max(x) - log sum_j exp(x_j - max(x)).  t: integer class index per row."""
    X = np.asarray(X, np.float64)
    t = np.asarray(t, np.int64)
    m = X.max(axis=-1, keepdims=True)
    lse = np.log(np.exp(X - m).sum(axis=-1)) + m[..., 0]
    return np.take_along_axis(X, t[..., None], axis=-1)[..., 0] - lse


def softmax_xent_bwd(X, t, g, beta):
    """beta * g_i * d softmax_xent(x, t)_i / dx = beta * g_i * (onehot(t_i) - softmax(x_i));
    the table gives beta = s / sqrt(s - 1) for rows of s classes.  g: one incoming gradient per row."""
    X = np.asarray(X, np.float64)
    t = np.asarray(t, np.int64)
    e = np.exp(X - X.max(axis=-1, keepdims=True))
    p = e / e.sum(axis=-1, keepdims=True)
    onehot = np.zeros_like(p)
    np.put_along_axis(onehot, t[..., None], 1.0, axis=-1)
    return _f32(beta) * np.asarray(g, np.float64)[..., None] * (onehot - p)


# --------------------------------------------------------------------------- layer norm

def layer_norm_fwd(X, w, c, eps=0.0):
    """layer_norm(X, w, c)_ij = c_j + w_j (X_ij - mu_i) / sigma_i over the last axis, with
    mu_i the row mean and sigma_i^2 = mean_j X_ij^2 - mu_i^2 (table row "layer_norm"; alpha = 1).

    eps is added to sigma_i^2 (the table's formula has none: eps = 0 reproduces it)."""
    X = np.asarray(X, np.float64)
    mu = X.mean(axis=-1, keepdims=True)
    var = (X * X).mean(axis=-1, keepdims=True) - mu * mu
    xhat = (X - mu) / np.sqrt(var + eps)
    return np.asarray(c, np.float64) + np.asarray(w, np.float64) * xhat


def layer_norm_bwd(X, w, G, eps=0.0, beta_x=1.0, beta_wc=None):
    """Gradients of layer_norm for an incoming G = dL/dY, scaled as the table row "layer_norm" says:
    beta_x = 1 for the input, beta_w = beta_c = b^-1/2 for the b x n input's weight and bias
    (appendix: weights are cut-edges, so they may take their own factors).

        xhat = (X - mu) / sigma,  u = G * w
        dX_ij = beta_x / sigma_i * (u_ij - mean_j u_ij - xhat_ij mean_j(u_ij xhat_ij))
        dw_j  = beta_wc sum_i G_ij xhat_ij,   dc_j = beta_wc sum_i G_ij
    Returns (dX, dw, dc)."""
    X = np.asarray(X, np.float64)
    G = np.asarray(G, np.float64)
    w = np.asarray(w, np.float64)
    b = X.shape[0]
    if beta_wc is None:
        beta_wc = _f32(b ** -0.5)
    mu = X.mean(axis=-1, keepdims=True)
    var = (X * X).mean(axis=-1, keepdims=True) - mu * mu
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (X - mu) * rstd
    u = G * w
    dX = _f32(beta_x) * rstd * (u - u.mean(axis=-1, keepdims=True) - xhat * (u * xhat).mean(axis=-1, keepdims=True))
    dw = _f32(beta_wc) * (G * xhat).sum(axis=0)
    dc = _f32(beta_wc) * G.sum(axis=0)
    return dX, dw, dc


# --------------------------------------------------------------------------- storage rounding

def store(v, dtype: str):
    """Round float64 values to a storage format; returns (values float64, codes or None)."""
    if dtype == "f64":          # no rounding: used by exact-arithmetic checks
        return np.asarray(v, np.float64), None
    if dtype == "f32":
        with np.errstate(over="ignore"):
            return np.asarray(v, np.float64).astype(np.float32).astype(np.float64), None
    fmt = F.FORMATS[dtype]
    q = F.quantise(v, fmt)
    return q, F.encode(q, fmt)


# --------------------------------------------------------------------------- fused epilogue

@dataclass
class Epilogue:
    """What a linear call may fuse after the scaled accumulator.

    act: "none" | "gelu" | "gelu_grad".  For "gelu" the pre-activation is stored
    in `aux_dtype` (the copy the backward pass reads); for "gelu_grad" `aux`
    holds that stored pre-activation.  skip: optional tensor combined as
    skip_coef * skip + out_coef * value.
    """

    act: str = "none"
    act_in_scale: float = 1.0
    act_out_scale: float = 1.0
    aux: np.ndarray | None = None
    aux_dtype: str = "bf16"
    skip: np.ndarray | None = None
    skip_coef: float = 0.0
    out_coef: float = 1.0


def apply_epilogue(val, ep: Epilogue | None, out_dtype: str):
    """Chain scaled accumulator -> activation -> residual -> one rounding to out_dtype.

    Returns (out values, out codes or None, stored pre-activation values or None).
    """
    aux_saved = None
    if ep is not None:
        if ep.act == "gelu":
            aux_saved, _ = store(val, ep.aux_dtype)
            val = gelu_fwd(val, ep.act_in_scale, ep.act_out_scale)
        elif ep.act == "gelu_grad":
            val = gelu_bwd(ep.aux, val, ep.act_in_scale, ep.act_out_scale)
        elif ep.act != "none":
            raise ValueError(ep.act)
        if ep.skip is not None:
            val = weighted_add(ep.skip, val, ep.skip_coef, ep.out_coef)
    out, codes = store(val, out_dtype)
    return out, codes, aux_saved


# --------------------------------------------------------------------------- FFN block

@dataclass
class FFNScales:
    alpha1: float
    alpha2: float
    beta_x1: float
    beta_x2: float
    beta_w: float
    alpha_g: float
    beta_g: float
    s_in: float = 1.0
    tau: float = 0.5

    @staticmethod
    def unconstrained(T: int, d: int, f: int, tau: float = 0.5) -> "FFNScales":
        a1, bx1, bw = S.linear_scales(T, d, f)
        a2, bx2, _ = S.linear_scales(T, f, d)
        ag, bg = S.gelu_scales()
        return FFNScales(a1, a2, bx1, bx2, bw, ag, bg, 1.0, tau)

    @staticmethod
    def constrained(T: int, d: int, f: int, tau: float = 0.5) -> "FFNScales":
        """alpha = beta_X for both matmuls and for gelu (the residual makes X a non-cut edge)."""
        a1, bx1, bw = S.linear_scales(T, d, f, constrained=True)
        a2, bx2, _ = S.linear_scales(T, f, d, constrained=True)
        ag, bg = S.gelu_scales(constrained=True)
        return FFNScales(a1, a2, bx1, bx2, bw, ag, bg, 1.0, tau)


@dataclass
class FFNResult:
    Xq: np.ndarray = None
    W1q: np.ndarray = None
    W2q: np.ndarray = None
    Gq: np.ndarray = None
    H: np.ndarray = None        # stored pre-activation (values)
    Aq: np.ndarray = None       # q_E4(alpha_g gelu(H)) values
    Aq_codes: np.ndarray = None
    R: np.ndarray = None        # block output
    dA: np.ndarray = None       # beta_x2 q(G) q(W2)^T before the gelu-gradient factor (not stored on device)
    dHq: np.ndarray = None
    dHq_codes: np.ndarray = None
    dW2: np.ndarray = None
    dW1: np.ndarray = None
    dX: np.ndarray = None


def ffn_block(X, W1, W2, G, sc: FFNScales, *, operand: str = "fp8",
              h_dtype: str = "bf16", io_dtype: str = "bf16") -> FFNResult:
    """Unit-scaled Transformer FFN with a fixed(tau) residual, forward and backward.

    Forward:  H = alpha1 q(X) q(W1);  A = alpha_g gelu(s_in H);  Y = alpha2 q(A) q(W2);
              R = sqrt(1-tau) X + sqrt(tau) Y.
    Backward, G = dL/dR:  the branch output gradient is G itself;
              dA = beta_x2 q(G) q(W2)^T;  dH = beta_g s_in gelu'(s_in H) dA;
              dW2 = beta_w q(A)^T q(G);   dXb = beta_x1 q(dH) q(W1)^T;
              dW1 = beta_w q(X)^T q(dH);  dX = sqrt(1-tau) G + sqrt(tau) dXb.
    q is E4 for activations / weights and E5 for gradients when operand == "fp8";
    for "bf16" / "fp16" every matmul input is rounded to that format instead, and
    for "f64" nothing is rounded (pair it with h_dtype = io_dtype = "f64").
    """
    act_fmt = "e4m3" if operand == "fp8" else operand
    grad_fmt = "e5m2" if operand == "fp8" else operand
    r = FFNResult()
    r.Xq, _ = store(np.asarray(X), act_fmt)
    r.W1q, _ = store(np.asarray(W1), act_fmt)
    r.W2q, _ = store(np.asarray(W2), act_fmt)
    r.Gq, _ = store(np.asarray(G), grad_fmt)
    c_skip, c_branch = S.residual_coefficients(sc.tau)

    ep1 = Epilogue(act="gelu", act_in_scale=sc.s_in, act_out_scale=sc.alpha_g, aux_dtype=h_dtype)
    r.Aq, r.Aq_codes, r.H = apply_epilogue(linear_fwd(r.Xq, r.W1q, sc.alpha1), ep1, act_fmt)
    ep2 = Epilogue(skip=np.asarray(X, np.float64), skip_coef=c_skip, out_coef=c_branch)
    r.R, _, _ = apply_epilogue(linear_fwd(r.Aq, r.W2q, sc.alpha2), ep2, io_dtype)

    ep3 = Epilogue(act="gelu_grad", act_in_scale=sc.s_in, act_out_scale=sc.beta_g, aux=r.H)
    r.dA = linear_bwd_x(r.Gq, r.W2q, sc.beta_x2)
    r.dHq, r.dHq_codes, _ = apply_epilogue(r.dA, ep3, grad_fmt)
    r.dW2, _, _ = apply_epilogue(linear_bwd_w(r.Aq, r.Gq, sc.beta_w), None, "f32")
    ep5 = Epilogue(skip=np.asarray(G, np.float64), skip_coef=c_skip, out_coef=c_branch)
    r.dX, _, _ = apply_epilogue(linear_bwd_x(r.dHq, r.W1q, sc.beta_x1), ep5, io_dtype)
    r.dW1, _, _ = apply_epilogue(linear_bwd_w(r.Xq, r.dHq, sc.beta_w), None, "f32")
    return r


def ffn_flops(T: int, d: int, f: int) -> float:
    """Matmul FLOPs of one FFN block, forward + backward: two linear layers x 6 b m n."""
    return 2 * 6.0 * T * d * f
