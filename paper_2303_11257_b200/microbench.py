"""Secondary measurements: the unfused elementwise kernels, the scaled softmax and layer norm against the HBM
roofline, and one encoder-layer step (config 5).  `python -m paper_2303_11257_b200.microbench`.

Each kernel is timed with CUDA events over graph replays that rotate among buffer sets larger than
the 126 MB L2; bandwidth = algorithmic bytes (inputs read once + outputs written once) / time.
"""
from __future__ import annotations

import json

import torch

from . import encoder, lib as L, synth


def _time_graph(fn, sets, iters=20):
    for s in sets:
        fn(*s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(iters):
            fn(*sets[i % len(sets)])
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    best = 1e30
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) * 1e-3 / iters)
    return best


def elementwise(rows=8192, cols=4096, nsets=4):
    dev = "cuda"
    f32 = lambda: torch.randn(rows, cols, device=dev)
    bf = lambda: torch.randn(rows, cols, device=dev).to(torch.bfloat16)
    e8 = lambda dt: torch.empty(rows, cols, device=dev, dtype=dt)
    n = rows * cols
    out = []
    cases = [
        ("us_cast_fp8 f32->e4m3", lambda a, o: L.us_cast_fp8(a, 1.0, o), lambda: (f32(), e8(torch.float8_e4m3fn)), 5),
        ("us_cast_fp8 bf16->e5m2", lambda a, o: L.us_cast_fp8(a, 1.0, o), lambda: (bf(), e8(torch.float8_e5m2)), 3),
        ("us_gelu_fwd bf16->e4m3", lambda a, o: L.us_gelu_fwd(a, 1.0, 1.7, o), lambda: (bf(), e8(torch.float8_e4m3fn)), 3),
        ("us_gelu_bwd bf16,bf16->e5m2", lambda a, b, o: L.us_gelu_bwd(a, b, 1.0, 1.48, o), lambda: (bf(), bf(), e8(torch.float8_e5m2)), 5),
        ("us_residual_add bf16,bf16->bf16", lambda a, b, o: L.us_residual_add(a, b, 0.5, o), lambda: (bf(), bf(), e8(torch.bfloat16)), 6),
        ("us_softmax_fwd bf16->bf16 (rows of 512)", lambda a, o: L.us_softmax_fwd(a, 512.0, o),
         lambda: (torch.randn(rows * 8, 512, device=dev).to(torch.bfloat16), torch.empty(rows * 8, 512, device=dev, dtype=torch.bfloat16)), 4),
        ("us_softmax_bwd bf16,bf16->bf16 (rows of 512)", lambda a, b, o: L.us_softmax_bwd(a, b, 512.0, 512.0, o),
         lambda: tuple(torch.randn(rows * 8, 512, device=dev).abs().to(torch.bfloat16) for _ in range(2)) + (torch.empty(rows * 8, 512, device=dev, dtype=torch.bfloat16),), 6),
        ("us_layer_norm_fwd bf16->bf16 (rows of 1024)", lambda a, w, c, o: L.us_layer_norm_fwd(a, w, c, 1e-5, o),
         lambda: (torch.randn(rows * 4, 1024, device=dev).to(torch.bfloat16), torch.ones(1024, device=dev), torch.zeros(1024, device=dev),
                  torch.empty(rows * 4, 1024, device=dev, dtype=torch.bfloat16)), 4),
        ("us_layer_norm_bwd bf16,bf16->bf16 (rows of 1024, two launches)",
         lambda a, w, g, o, dw, dc, ws: L.us_layer_norm_bwd(a, w, g, 1e-5, 1.0, (rows * 4) ** -0.5, o, dw, dc, ws),
         lambda: (torch.randn(rows * 4, 1024, device=dev).to(torch.bfloat16), torch.ones(1024, device=dev),
                  torch.randn(rows * 4, 1024, device=dev).to(torch.bfloat16), torch.empty(rows * 4, 1024, device=dev, dtype=torch.bfloat16),
                  torch.empty(1024, device=dev), torch.empty(1024, device=dev),
                  torch.empty(L.us_layer_norm_bwd_workspace_bytes(rows * 4, 1024), dtype=torch.uint8, device=dev)), 6),
    ]
    for name, fn, make, bytes_per_elt in cases:
        sets = [make() for _ in range(nsets)]
        t = _time_graph(fn, sets)
        out.append({"kernel": name, "us": t * 1e6, "gbs": n * bytes_per_elt / t / 1e9, "bytes_per_element": bytes_per_elt})
    return out


def encoder_step(nseq=16, slen=512, d=1024, nhead=16, d_ff=4096, iters=10, attention="bf16", norm=None):
    T = nseq * slen
    host = (synth.normal(0, 0, (T, d)), synth.normal(0, 1, (d, 3 * d)), synth.normal(0, 2, (d, d)),
            synth.normal(0, 3, (d, d_ff)), synth.normal(0, 4, (d_ff, d)), synth.normal(0, 5, (T, d)))
    dev = [torch.from_numpy(t).cuda() for t in host]
    layer = encoder.UnitScaledEncoderLayer(nseq, slen, d, nhead, d_ff, attention=attention, norm=norm)
    ln = [torch.ones(d, device="cuda"), torch.zeros(d, device="cuda")] * 2 if norm else None
    layer.step(*dev, ln=ln)
    layer.check()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        layer.step(*dev, ln=ln)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    layer.check()
    t = e0.elapsed_time(e1) * 1e-3 / iters
    return {"workload": f"encoder layer fwd+bwd 16x512 tokens, d=1024, 16 heads, d_ff=4096, {attention} attention operands" + (", post-norm" if norm else ""), "ms_per_step": t * 1e3,
            "tflops": layer.flops() / t / 1e12, "tokens_per_s": T / t, "launches": layer.launches_per_step}


if __name__ == "__main__":
    print(json.dumps({"elementwise": elementwise(), "encoder": encoder_step(),
                      "encoder_fp8_attention": encoder_step(attention="fp8"),
                      "encoder_fp8_attention_post_norm": encoder_step(attention="fp8", norm="post")}, indent=1))
