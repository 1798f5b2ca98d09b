"""Unit-scaled Transformer encoder layer (self-attention block + FFN block), forward and backward,
as a sequence of libunitscale calls.  A driver only: buffers and call order; all arithmetic runs
in the library's kernels.

Layer (no layer norm; fixed(tau) residuals, section "Weighted addition"):
    QKV = alpha_qkv q(X) q(Wqkv)                          FP8 GEMM, 16-bit output [T x 3d]
    S   = alpha_s Q_h K_h^T   per (sequence, head)        batched, 16-bit operands, alpha_s = 1/sqrt(d_head)
    P   = s softmax(S)                                    scaled softmax (table row "softmax"), s = sequence length
    C   = alpha_c P V_h                                   batched, alpha_c = s^-1/2, stored as E4M3
    R1  = sqrt(1-tau) X + sqrt(tau) alpha_o C q(Wo)       FP8 GEMM + residual epilogue
    R2  = FFN block on R1                                 see ffn.py
Backward from G = dL/dR2: the FFN block's backward gives g1 = dL/dR1, then
    dC  = beta_o q(g1) q(Wo)^T ; dWo = beta_w C^T q(g1)
    dP  = beta_P dC_h V_h^T ; dV = beta_V P^T dC_h        batched
    dS  = s softmax_grad(P, dP)
    dQ  = beta_Q dS K_h ; dK = beta_K dS^T Q_h            batched
    dX  = sqrt(1-tau) g1 + sqrt(tau) beta_qkv q(dQKV) q(Wqkv)^T ; dWqkv = beta_w q(X)^T q(dQKV)
Scale factors are the unconstrained table values (alpha = fan_in^-1/2, beta_X = fan_out^-1/2,
beta_W = batch^-1/2 with the batch of an attention matmul = its sequence length).

attention = "bf16" / "fp16": the attention matmuls take 16-bit operands.  attention = "fp8": they take
FP8 operands like the projections (section "Experiments": all matmul inputs are quantised): the QKV
GEMM writes Q, K, V as E4M3, the softmax writes P as E4M3, the gradients dC and dS are written as E5M2
and the batched GEMMs write dQ, dK, dV straight into the E5M2 operand of the QKV backward GEMMs (one
cast launch fewer); S and dP, which feed no matmul, stay in BF16.
"""
from __future__ import annotations


import torch

from . import ffn as F
from . import lib as L

E4, E5 = torch.float8_e4m3fn, torch.float8_e5m2


class UnitScaledEncoderLayer:
    def __init__(self, nseq: int, slen: int, d: int, nhead: int, d_ff: int, tau: float = 0.5,
                 attention: str = "bf16", norm: str | None = None, eps: float = 1e-5, device="cuda",
                 fused_attention: bool = False):
        assert d % nhead == 0 and norm in (None, "post")
        self.attention, self.norm, self.eps = attention, norm, eps
        # fused_attention: scores, scaled softmax and context of the forward pass as one us_attention_fwd launch, and
        # dP, the softmax gradient and dQ of the backward pass as one us_attention_bwd launch (heads of 64, at most 512
        # tokens per sequence; 16-bit or FP8 attention operands); the scores and the gradient dP are then never stored
        self.fused_attention = fused_attention
        if fused_attention and not (d // nhead == 64 and slen <= 512):
            raise ValueError("fused attention needs heads of 64 and sequences of at most 512 tokens")
        if attention == "fp8":
            act_dt, grad_dt, wide_dt = E4, E5, torch.bfloat16
        else:
            act_dt = grad_dt = wide_dt = {"bf16": torch.bfloat16, "fp16": torch.float16}[attention]
        self.nseq, self.slen, self.d, self.nhead, self.hd, self.d_ff, self.tau = nseq, slen, d, nhead, d // nhead, d_ff, tau
        T = self.T = nseq * slen
        e = lambda r, c, dt: torch.empty((r, c), dtype=dt, device=device)
        self.Xq, self.Wqkv_q, self.Wo_q = e(T, d, E4), e(d, 3 * d, E4), e(d, d, E4)
        self.QKV = e(T, 3 * d, act_dt)
        self.S = None if fused_attention else e(nseq * nhead * slen, slen, wide_dt)
        self.P = e(nseq * nhead * slen, slen, act_dt)
        self.Cq = e(T, d, E4)
        self.R1 = e(T, d, torch.bfloat16)
        self.ffn = F.UnitScaledFFN(T, d, d_ff, scales=F.FFNScales.unit(T, d, d_ff, tau), device=device)
        self.g1q = e(T, d, E5)
        self.dC = e(T, d, grad_dt)
        self.dP = None if fused_attention else e(nseq * nhead * slen, slen, wide_dt)
        self.dS = e(nseq * nhead * slen, slen, grad_dt)
        self.dQKVq = e(T, 3 * d, E5)
        # dQ, dK, dV are consumed only as the E5M2 operand of the QKV projection's backward GEMMs: with FP8 attention
        # operands, and with the fused attention kernels, their producers write that format directly (no cast launch)
        self.dQKV = self.dQKVq if (attention == "fp8" or fused_attention) else e(T, 3 * d, grad_dt)
        self.dX = e(T, d, torch.bfloat16)
        self.dWqkv, self.dWo = e(d, 3 * d, torch.float32), e(d, d, torch.float32)
        self.ws = L.new_workspace(device)
        if norm == "post":
            # post-norm (appendix "Model architectures"): a scaled layer norm after each residual sum
            self.U1, self.R2 = e(T, d, torch.bfloat16), e(T, d, torch.bfloat16)
            self.dU1, self.dU2 = e(T, d, torch.bfloat16), e(T, d, torch.bfloat16)
            self.dln = [torch.empty(d, dtype=torch.float32, device=device) for _ in range(4)]      # dw1, dc1, dw2, dc2
            self.ln_ws = torch.empty(max(16, L.us_layer_norm_bwd_workspace_bytes(T, d)), dtype=torch.uint8, device=device)
            self.beta_ln = L.us_scales_linear(T, 1, 1)[2]          # b^-1/2 with b = all tokens
        self.c_skip, self.c_branch = L.us_scales_residual(tau)
        s, hd = slen, self.hd
        a_qkv, b_qkv, b_w = L.us_scales_linear(T, d, 3 * d)
        a_o, b_o, _ = L.us_scales_linear(T, d, d)
        self.sc = dict(alpha_qkv=a_qkv, beta_qkv=b_qkv, alpha_o=a_o, beta_o=b_o, beta_w=b_w, **L.us_scales_attention(s, hd))
        qkv = (slen * 3 * d, hd)          # (outer, inner) strides of a head slice of a [T x 3d] matrix
        sq = (nhead * slen * slen, slen * slen)
        td = (slen * d, hd)               # head slice of a [T x d] matrix
        n = (nseq, nhead)
        self.bt = dict(scores=L.batch(n, qkv, qkv, sq), ctx=L.batch(n, sq, qkv, td), dP=L.batch(n, td, qkv, sq),
                       dV=L.batch(n, sq, td, qkv), dQ=L.batch(n, sq, qkv, qkv), dK=L.batch(n, sq, qkv, qkv))
        # fused cast, attention forward, FFN forward + backward, attention backward (one cast fewer with FP8 attention)
        self._launches = 1 + (3 if fused_attention else 5) + 7 + ((10 if (attention == "fp8" or fused_attention) else 11) - (2 if fused_attention else 0)) + (7 if norm == "post" else 0)
        self.bt_fused = L.attention_batch(n, qkv, qkv, qkv, td, sq)
        self.bt_fused_bwd = L.attention_bwd_batch(n, td, sq, qkv, qkv, sq, qkv)

    @property
    def launches_per_step(self) -> int:
        """Kernel launches of one step (without layer norms the FFN block's six GEMMs go out in its grouped forms, as
        two or three launches, while those cover the shape)."""
        return self._launches - (6 - self.ffn.gemm_launches if self.norm is None else 0)

    def _heads(self, M, which):
        """Problem (0, 0) of a [T x 3d] matrix: rows of the first sequence, columns of head 0 of Q / K / V."""
        o = which * self.d
        return M[: self.slen, o:o + self.hd]

    def step(self, X, Wqkv, Wo, W1, W2, G, stream=None, ln=None):
        """One forward + backward pass.  G is the gradient of the layer output; with norm = "post",
        ln = (w1, c1, w2, c2) are the weights and biases of the two layer norms ([d] each)."""
        sc, ws, s = self.sc, self.ws, self.slen
        post = self.norm == "post"
        # ---- forward
        f = self.ffn
        # every tensor that is known when the step starts goes to FP8 in one launch (with post-norm the FFN
        # block's incoming gradient is produced by the second norm's backward pass and is cast there)
        L.us_cast_fp8_multi([Wqkv, Wo, X, W1, W2] + ([] if post else [G]), [1.0] * (5 if post else 6),
                            [self.Wqkv_q, self.Wo_q, self.Xq, f.W1q, f.W2q] + ([] if post else [f.Gq]), stream)
        L.us_linear_fwd(self.Xq, self.Wqkv_q, sc["alpha_qkv"], self.QKV, ws, None, stream)
        Q, K, V = (self._heads(self.QKV, i) for i in range(3))
        if self.fused_attention:
            L.us_attention_fwd(Q, K, V, sc["alpha_s"], sc["sm"], sc["alpha_c"], self.Cq[:s, : self.hd], self.P[:s],
                               self.bt_fused, ws, stream)
        else:
            L.us_linear_bwd_x_batched(Q, K, sc["alpha_s"], self.S[:s], self.bt["scores"], ws, stream)
            L.us_softmax_fwd(self.S, sc["sm"], self.P, stream)
            L.us_linear_fwd_batched(self.P[:s], V, sc["alpha_c"], self.Cq[:s, : self.hd], self.bt["ctx"], ws, stream)
        ep = L.epilogue(skip=X, skip_coef=self.c_skip, out_coef=self.c_branch)
        L.us_linear_fwd(self.Cq, self.Wo_q, sc["alpha_o"], self.U1 if post else self.R1, ws, ep, stream)
        if post:
            L.us_layer_norm_fwd(self.U1, ln[0], ln[1], self.eps, self.R1, stream)
        if post or not f.grouped:
            f.forward(self.R1, stream)
        # ---- backward
        if post:
            L.us_layer_norm_fwd(f.R, ln[2], ln[3], self.eps, self.R2, stream)
            L.us_layer_norm_bwd(f.R, ln[2], G, self.eps, 1.0, self.beta_ln, self.dU2, self.dln[2], self.dln[3], self.ln_ws, stream)
            f.backward(self.dU2, stream)                            # f.dX = dL/dR1
            L.us_layer_norm_bwd(self.U1, ln[0], f.dX, self.eps, 1.0, self.beta_ln, self.dU1, self.dln[0], self.dln[1], self.ln_ws, stream)
            g1 = self.dU1
        elif f.grouped:
            # G is known from the start, so the whole FFN block goes out as a cast of its input and three GEMM launches
            f._cast(self.R1, f.Xq, stream)
            f.step_from_casts(self.R1, G, stream)                   # f.R = layer output, f.dX = dL/dR1
            g1 = f.dX
        else:
            f.backward(G, stream, cast_g=False)                     # f.dX = dL/dR1
            g1 = f.dX
        # The weight-gradient GEMMs and one GEMM of each attention pair depend only on tensors that exist
        # already; with no explicit stream they go to a side stream (parallel branches under graph capture).
        par = stream is None and f.concurrent
        cur = torch.cuda.current_stream() if par else stream
        side = f._side_streams()[0] if par else stream

        def beside(fn):
            """Run fn on the side stream once everything issued so far on the main stream is done."""
            if par:
                ev = torch.cuda.Event()
                ev.record(cur)
                side.wait_event(ev)
            fn(side)

        L.us_cast_fp8(g1, 1.0, self.g1q, cur)
        beside(lambda st: L.us_linear_bwd_w(self.Cq, self.g1q, sc["beta_w"], self.dWo, ws, None, st))
        L.us_linear_bwd_x(self.g1q, self.Wo_q, sc["beta_o"], self.dC, ws, None, cur)
        dC_h = self.dC[:s, : self.hd]
        beside(lambda st: L.us_linear_bwd_w_batched(self.P[:s], dC_h, sc["beta_V"], self._heads(self.dQKV, 2), self.bt["dV"], ws, st))
        if self.fused_attention:
            L.us_attention_bwd(dC_h, self.P[:s], K, V, sc["beta_P"], sc["sm"], sc["sm"], sc["beta_Q"], self.dS[:s],
                               self._heads(self.dQKV, 0), self.bt_fused_bwd, ws, cur)
            beside(lambda st: L.us_linear_bwd_w_batched(self.dS[:s], Q, sc["beta_K"], self._heads(self.dQKV, 1), self.bt["dK"], ws, st))
        else:
            L.us_linear_bwd_x_batched(dC_h, V, sc["beta_P"], self.dP[:s], self.bt["dP"], ws, cur)
            L.us_softmax_bwd(self.P, self.dP, sc["sm"], sc["sm"], self.dS, cur)
            beside(lambda st: L.us_linear_bwd_w_batched(self.dS[:s], Q, sc["beta_K"], self._heads(self.dQKV, 1), self.bt["dK"], ws, st))
            L.us_linear_fwd_batched(self.dS[:s], K, sc["beta_Q"], self._heads(self.dQKV, 0), self.bt["dQ"], ws, cur)
        if par:
            cur.wait_stream(side)                                   # dQ, dK, dV all written
        if self.dQKV is not self.dQKVq:
            L.us_cast_fp8(self.dQKV, 1.0, self.dQKVq, cur)
        beside(lambda st: L.us_linear_bwd_w(self.Xq, self.dQKVq, sc["beta_w"], self.dWqkv, ws, None, st))
        ep = L.epilogue(skip=g1, skip_coef=self.c_skip, out_coef=self.c_branch)
        L.us_linear_bwd_x(self.dQKVq, self.Wqkv_q, sc["beta_qkv"], self.dX, ws, ep, cur)
        if par:
            cur.wait_stream(side)
        return self.dX

    def check(self) -> None:
        for ws in (self.ws, self.ffn.ws):
            st = L.us_workspace_status(ws)
            if st != L.US_OK:
                raise L.UnitScaleError("UnitScaledEncoderLayer", st)

    def flops(self) -> float:
        T, d, f, s, hd = self.T, self.d, self.d_ff, self.slen, self.hd
        proj = 6.0 * T * d * 3 * d + 6.0 * T * d * d
        att = 2 * 6.0 * (self.nseq * self.nhead) * s * s * hd
        return proj + att + 12.0 * T * d * f
