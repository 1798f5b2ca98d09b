"""Unit-scaled Transformer FFN block (forward + backward) as a sequence of libunitscale calls.

A driver only: it owns the device buffers and issues the C-ABI calls in order; every step
of the computation happens in the library's kernels.

Forward (Figure "PyTorch examples", scaled FFN; section "Weighted addition"):
    Xq = q(X); W1q = q(W1); W2q = q(W2)                                   us_cast_fp8 (step(): one us_cast_fp8_multi
                                                                          launch for these three and Gq)
    H  = alpha1 Xq W1q ; A = q(alpha_g gelu(s_in H)), H kept in 16 bit    us_linear_fwd + GELU epilogue
    R  = sqrt(1-tau) X + sqrt(tau) alpha2 A W2q                           us_linear_fwd + residual epilogue
Backward, G = dL/dR (the branch output receives G unscaled):
    Gq  = q(G)                                                            us_cast_fp8
    dH  = q(beta_g s_in gelu'(s_in H) * beta_x2 Gq W2q^T)                 us_linear_bwd_x + GELU-grad epilogue
    dW2 = beta_w A^T Gq                                                   us_linear_bwd_w
    dX  = sqrt(1-tau) G + sqrt(tau) beta_x1 dH W1q^T                      us_linear_bwd_x + residual epilogue
    dW1 = beta_w Xq^T dH                                                  us_linear_bwd_w
q is E4M3 for activations / weights and E5M2 for gradients in "fp8" mode; in "bf16" / "fp16"
mode the matmul inputs are rounded to that format instead (no loss scale, same fixed scales).

step() knows G when it starts.  In FP8 mode it therefore issues the two GEMMs that end in the hidden layer (H, A and
dH above) as one us_ffn_hidden launch, in which H stays on the SM, and the other four GEMMs as one us_linear_group
launch: three launches per step with the fused cast.  self.H is then written only with keep_h = True.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import lib as L


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
    def unit(T: int, d: int, f: int, tau: float = 0.5, constrained: bool = False, dp_world: int = 1) -> "FFNScales":
        """dp_world > 1: T tokens per rank of a token-sharded job; the weight-gradient factor then uses
        the global batch T * dp_world, and the ranks' weight gradients are summed afterwards (dp.py)."""
        a1, bx1, bw = L.us_scales_linear(T, d, f, constrained)
        if dp_world > 1:
            _, _, bw = L.us_scales_linear(T * dp_world, d, f, constrained)      # the batch of the weight gradient is global
        a2, bx2, _ = L.us_scales_linear(T, f, d, constrained)
        ag, bg = L.us_scales_gelu(constrained)
        return FFNScales(a1, a2, bx1, bx2, bw, ag, bg, 1.0, tau)


_OPERAND = {
    "fp8": (torch.float8_e4m3fn, torch.float8_e5m2),
    "bf16": (torch.bfloat16, torch.bfloat16),
    "fp16": (torch.float16, torch.float16),
}


class UnitScaledFFN:
    """Buffers + call sequence for one FFN block of T tokens, width d, hidden width f."""

    def __init__(self, T: int, d: int, f: int, scales: FFNScales | None = None, operand: str = "fp8",
                 h_dtype=torch.bfloat16, io_dtype=torch.bfloat16, device="cuda", keep_h: bool = False):
        self.T, self.d, self.f = T, d, f
        self.sc = scales or FFNScales.unit(T, d, f)
        self.operand = operand
        act_dt, grad_dt = _OPERAND[operand]
        e = lambda r, c, dt: torch.empty((r, c), dtype=dt, device=device)
        self.Xq, self.W1q, self.W2q, self.Gq = e(T, d, act_dt), e(d, f, act_dt), e(f, d, act_dt), e(T, d, grad_dt)
        self.H = e(T, f, h_dtype)
        self.Aq = e(T, f, act_dt)
        self.dHq = e(T, f, grad_dt)
        self.R, self.dX = e(T, d, io_dtype), e(T, d, io_dtype)
        self.dW1 = e(d, f, torch.float32)
        self.dW2 = e(f, d, torch.float32)
        self.ws = L.new_workspace(device)
        c_skip, c_branch = L.us_scales_residual(self.sc.tau)
        self._c = (c_skip, c_branch)
        # step() has all four tensors to quantise at hand when it starts, so in FP8 mode it casts them
        # with one launch; forward() / backward() on their own cast what they are given.
        self.fused_casts = operand == "fp8"
        # After the first GEMM, the second forward GEMM, the GELU-gradient GEMM and the first weight-gradient GEMM
        # depend on nothing but it, and the last two GEMMs only on the GELU-gradient one.  step() issues them on
        # three streams, so that the CTAs of one kernel fill the SMs another leaves idle in its last wave (64 or
        # 128 tiles on 74 CTA pairs); measured 6 % faster than one stream once the power cap holds the clock.
        self.concurrent = self.fused_casts
        self._side = None
        # FP8 operands: the four GEMMs that remain after the GELU-gradient GEMM are independent of one another and
        # go out as one us_linear_group launch (4 launches per step instead of 7).
        self.grouped = operand == "fp8"
        # FP8 operands and G known up front: the first GEMM + GELU and the GELU-gradient GEMM are one us_ffn_hidden
        # launch that keeps the pre-activation on the SM; keep_h = True also writes its 16-bit copy to self.H (the
        # separate launches always do, the backward one reads it from there).
        self.fused_hidden = operand == "fp8"
        self.keep_h = keep_h

    @property
    def gemm_launches(self) -> int:
        """Launches step_from_casts() makes for the six GEMMs."""
        return 6 - ((3 + (1 if self.fused_hidden else 0)) if self.grouped else 0)

    @property
    def launches_per_step(self) -> int:
        """Kernel launches of step(): the cast(s) plus gemm_launches in FP8 mode."""
        if self.fused_casts:
            return 1 + self.gemm_launches
        return 10

    def _cast(self, src, dst, stream):
        if dst.dtype in (torch.float8_e4m3fn, torch.float8_e5m2):
            L.us_cast_fp8(src, 1.0, dst, stream)
        else:
            # 16-bit operand mode: rounding fp32 -> bf16/fp16 is the residual kernel with tau = 0
            L.us_residual_add(src, src, 0.0, dst, stream)

    def stages(self, X, W1, W2, G, fused_casts: bool | None = None):
        """The launches of one pass, in order, as (name, kind, callable(stream)) triples.

        kind is "cast" or "gemm".  These are the unfused launches: step() runs exactly these (seven with the casts
        fused into one launch, ten otherwise) unless it takes the grouped forms (step_launches); forward() and
        backward() run the ones they need."""
        sc, (c_skip, c_branch) = self.sc, self._c
        fused = self.fused_casts if fused_casts is None else fused_casts
        ep1 = L.epilogue(act=L.US_ACT_GELU, act_in_scale=sc.s_in, act_out_scale=sc.alpha_g, aux=self.H)
        ep2 = L.epilogue(skip=X, skip_coef=c_skip, out_coef=c_branch)
        ep3 = L.epilogue(act=L.US_ACT_GELU_GRAD, act_in_scale=sc.s_in, act_out_scale=sc.beta_g, aux=self.H)
        ep5 = L.epilogue(skip=G, skip_coef=c_skip, out_coef=c_branch)
        ws = self.ws
        if fused:
            casts = [("cast_all", "cast", lambda st=None: L.us_cast_fp8_multi(
                [W1, W2, X, G], [1.0] * 4, [self.W1q, self.W2q, self.Xq, self.Gq], st))]
            cast_g = []
        else:
            casts = [("cast_W1", "cast", lambda st=None: self._cast(W1, self.W1q, st)),
                     ("cast_W2", "cast", lambda st=None: self._cast(W2, self.W2q, st)),
                     ("cast_X", "cast", lambda st=None: self._cast(X, self.Xq, st))]
            cast_g = [("cast_G", "cast", lambda st=None: self._cast(G, self.Gq, st))]
        return casts + [
            ("fwd1_gelu", "gemm", lambda st=None: L.us_linear_fwd(self.Xq, self.W1q, sc.alpha1, self.Aq, ws, ep1, st)),
            ("fwd2_residual", "gemm", lambda st=None: L.us_linear_fwd(self.Aq, self.W2q, sc.alpha2, self.R, ws, ep2, st)),
        ] + cast_g + [
            ("bwd_x2_gelu_grad", "gemm", lambda st=None: L.us_linear_bwd_x(self.Gq, self.W2q, sc.beta_x2, self.dHq, ws, ep3, st)),
            ("bwd_w2", "gemm", lambda st=None: L.us_linear_bwd_w(self.Aq, self.Gq, sc.beta_w, self.dW2, ws, None, st)),
            ("bwd_x1_residual", "gemm", lambda st=None: L.us_linear_bwd_x(self.dHq, self.W1q, sc.beta_x1, self.dX, ws, ep5, st)),
            ("bwd_w1", "gemm", lambda st=None: L.us_linear_bwd_w(self.Xq, self.dHq, sc.beta_w, self.dW1, ws, None, st)),
        ]

    def step_launches(self, X, W1, W2, G):
        """The launches step() makes, in order, as (name, kind, GEMMs in the launch, callable(stream)): with the
        grouped form the four GEMMs after the GELU-gradient GEMM are one entry of kind "group"."""
        st = self.stages(X, W1, W2, G)
        if not (self.grouped and self.fused_casts):
            return [(n, k, 1 if k == "gemm" else 0, fn) for n, k, fn in st]
        by = {n: (k, fn) for n, k, fn in st}
        head = [(n, by[n][0], 1 if by[n][0] == "gemm" else 0, by[n][1]) for n in ("cast_all", "fwd1_gelu", "bwd_x2_gelu_grad")]
        if self.fused_hidden:
            head = head[:1] + [("hidden_fwd1_gelu_bwd_x2_gelu_grad", "group", 2, lambda stream=None: self._hidden(stream))]
        return head + [("group_fwd2_bwd_w2_bwd_x1_bwd_w1", "group", 4,
                        lambda stream=None: L.us_linear_group(self.group_calls(X, G), self.ws, stream))]

    def group_calls(self, X, G):
        """The four GEMMs that follow the GELU-gradient GEMM, as the entries of one us_linear_group launch
        (same operands, scales and epilogues as the stages fwd2_residual, bwd_w2, bwd_x1_residual, bwd_w1)."""
        sc, (c_skip, c_branch) = self.sc, self._c
        ep2 = L.epilogue(skip=X, skip_coef=c_skip, out_coef=c_branch)
        ep5 = L.epilogue(skip=G, skip_coef=c_skip, out_coef=c_branch)
        return [L.linear_call(L.US_OP_BWD_W, self.Aq, self.Gq, sc.beta_w, self.dW2),
                L.linear_call(L.US_OP_BWD_W, self.Xq, self.dHq, sc.beta_w, self.dW1),
                L.linear_call(L.US_OP_FWD, self.Aq, self.W2q, sc.alpha2, self.R, ep2),
                L.linear_call(L.US_OP_BWD_X, self.dHq, self.W1q, sc.beta_x1, self.dX, ep5)]

    def _hidden(self, stream=None):
        """H, A and dH in one launch (us_ffn_hidden) from the quantised operands."""
        sc = self.sc
        L.us_ffn_hidden(self.Xq, self.W1q, sc.alpha1, self.Gq, self.W2q, sc.beta_x2, sc.s_in, sc.alpha_g, sc.beta_g,
                        self.Aq, self.dHq, self.ws, H=self.H if self.keep_h else None, h_dtype=self.H.dtype, stream=stream)

    def cast_weights(self, W1, W2, stream=None):
        self._cast(W1, self.W1q, stream)
        self._cast(W2, self.W2q, stream)

    def forward(self, X, stream=None):
        for name, _, fn in self.stages(X, None, None, None, fused_casts=False)[2:5]:
            fn(stream)
        return self.R

    def _side_streams(self):
        if self._side is None:
            self._side = (torch.cuda.Stream(), torch.cuda.Stream())
        return self._side

    def backward(self, G, stream=None, cast_g: bool = True):
        """Backward pass from G = dL/dR.  cast_g=False: self.Gq already holds q(G) (a caller that
        quantised G together with other tensors in one us_cast_fp8_multi launch).  With self.concurrent and
        no explicit stream the two weight-gradient GEMMs run on side streams beside the input-gradient ones."""
        st = self.stages(None, None, None, G, fused_casts=False)[5 if cast_g else 6:]
        if not (self.concurrent and stream is None):
            for name, _, fn in st:
                fn(stream)
            return self.dX, self.dW1, self.dW2
        by = {name: fn for name, _, fn in st}
        cur = torch.cuda.current_stream()
        s_b, s_c = self._side_streams()
        if cast_g:
            by["cast_G"](cur)
        s_b.wait_stream(cur)
        s_c.wait_stream(cur)
        by["bwd_w2"](s_c)
        by["bwd_x2_gelu_grad"](cur)
        have_dh = torch.cuda.Event()
        have_dh.record(cur)
        s_b.wait_event(have_dh)
        by["bwd_w1"](s_b)
        by["bwd_x1_residual"](cur)
        cur.wait_stream(s_b)
        cur.wait_stream(s_c)
        return self.dX, self.dW1, self.dW2

    def step(self, X, W1, W2, G, stream=None):
        """One pass of the whole path: casts, forward, backward (launches_per_step kernel launches).

        With self.concurrent and no explicit stream, independent GEMMs go to two side streams that fork from
        and join back into the current stream (this also records as parallel branches under graph capture)."""
        st = self.stages(X, W1, W2, G)
        if self.grouped and self.fused_casts:
            cast_all = next(fn for name, _, fn in st if name == "cast_all")
            cast_all(stream)
            return self.step_from_casts(X, G, stream)
        if not (self.concurrent and self.fused_casts and stream is None):
            for name, _, fn in st:
                fn(stream)
            return self.dX, self.dW1, self.dW2
        by = {name: fn for name, _, fn in st}
        cur = torch.cuda.current_stream()
        s_b, s_c = self._side_streams()
        by["cast_all"](cur)
        by["fwd1_gelu"](cur)
        s_b.wait_stream(cur)
        s_c.wait_stream(cur)
        by["bwd_x2_gelu_grad"](cur)
        have_dh = torch.cuda.Event()
        have_dh.record(cur)
        by["bwd_w1"](cur)
        by["fwd2_residual"](s_b)
        by["bwd_w2"](s_c)
        s_c.wait_event(have_dh)
        by["bwd_x1_residual"](s_c)
        cur.wait_stream(s_b)
        cur.wait_stream(s_c)
        return self.dX, self.dW1, self.dW2

    def step_from_casts(self, X, G, stream=None):
        """The GEMMs of one pass when self.Xq, W1q, W2q, Gq already hold the quantised operands (FP8 mode): two
        launches -- the hidden layer's two GEMMs with GELU and GELU gradient, the other four as one group -- or their
        separate forms where a shape is not covered.  X and G are the unquantised skip inputs of the two residual
        epilogues."""
        by = {name: fn for name, _, fn in self.stages(X, None, None, G)}
        fused = self.fused_hidden and self.grouped
        if fused:
            try:
                self._hidden(stream)
            except L.UnitScaleError as e:
                if e.status != L.US_ERR_UNSUPPORTED:
                    raise
                fused = self.fused_hidden = False            # at most 128 tokens or hidden units: nothing was launched
        if not fused:
            by["fwd1_gelu"](stream)
            by["bwd_x2_gelu_grad"](stream)
        if self.grouped:
            try:
                L.us_linear_group(self.group_calls(X, G), self.ws, stream)
                return self.dX, self.dW1, self.dW2
            except L.UnitScaleError as e:
                if e.status != L.US_ERR_UNSUPPORTED:
                    raise
                # a shape the grouped form does not cover (an output of at most 128 rows or columns): nothing was
                # launched; the four GEMMs go out one by one, now and in later steps
                self.grouped = False
        for name in ("fwd2_residual", "bwd_w2", "bwd_x1_residual", "bwd_w1"):
            by[name](stream)
        return self.dX, self.dW1, self.dW2

    def capture(self, X, W1, W2, G):
        """Records step() into a CUDA graph (run step() eagerly at least once before).  The graph
        reads X, W1, W2, G from the tensors given here; refill those in place between replays."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.step(X, W1, W2, G)
        return g

    def check(self) -> None:
        """Synchronise and raise if any kernel reported a timed-out wait."""
        st = L.us_workspace_status(self.ws)
        if st != L.US_OK:
            raise L.UnitScaleError("UnitScaledFFN", st)

    @staticmethod
    def flops(T: int, d: int, f: int) -> float:
        """Matmul FLOPs, forward + backward: 2 linear layers x 3 GEMMs x 2 T d f."""
        return 12.0 * T * d * f
