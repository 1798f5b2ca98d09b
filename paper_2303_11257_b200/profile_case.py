"""Runs a few eager passes of the FFN block so that a profiler can attach to individual launches.

    python -m paper_2303_11257_b200.profile_case [--tokens 8192] [--passes 2] [--operand fp8]
    python -m paper_2303_11257_b200.profile_case --case attention [--passes 2]
    python -m paper_2303_11257_b200.profile_case --case encoder [--passes 2] [--unfused] [--attention bf16|fp16|fp8]

Each pass is the launches of UnitScaledFFN.step (one fused cast, six GEMMs) at d_model = 1024, d_ff = 4096.  At the default
size the process holds well under 2 GB on the device and a pass lasts a fraction of a millisecond.
--case attention: passes of the fused attention forward launch (us_attention_fwd) at 16 sequences x 16 heads x 512
tokens x 64 (BF16 operands, E4M3 context, weights stored) followed by the fused backward launch (us_attention_bwd): about
0.5 GB on the device.  --case encoder: eager passes of the whole encoder-layer step (16 x 512 tokens, d = 1024, 16 heads,
d_ff = 4096, BF16 attention operands, fused attention kernels unless --unfused): about 1.5 GB on the device.
"""
from __future__ import annotations

import argparse

import torch

from . import encoder, ffn, lib as L, synth


def attention(passes: int):
    nseq, nhead, s, hd = 16, 16, 512, 64
    d, T = nhead * hd, nseq * s
    qkv = torch.from_numpy(synth.normal(0, 0, (T, 3 * d))).cuda().to(torch.bfloat16)
    P = torch.empty(nseq * nhead * s, s, device="cuda", dtype=torch.bfloat16)
    Cq = torch.empty(T, d, device="cuda", dtype=torch.uint8).view(torch.float8_e4m3fn)
    ws = L.new_workspace("cuda")
    st, td, sq = (s * 3 * d, hd), (s * d, hd), (nhead * s * s, s * s)
    bt = L.attention_batch((nseq, nhead), st, st, st, td, sq)
    sc = L.us_scales_attention(s, hd)
    dC = torch.from_numpy(synth.normal(0, 1, (T, d))).cuda().to(torch.bfloat16)
    dS = torch.empty_like(P)
    dQ = torch.empty(T, d, device="cuda", dtype=torch.bfloat16)
    btb = L.attention_bwd_batch((nseq, nhead), td, sq, st, st, sq, td)
    for _ in range(passes):
        L.us_attention_fwd(qkv[:s, 0:hd], qkv[:s, d:d + hd], qkv[:s, 2 * d:2 * d + hd], sc["alpha_s"], sc["sm"], sc["alpha_c"],
                           Cq[:s, :hd], P[:s], bt, ws)
        L.us_attention_bwd(dC[:s, :hd], P[:s], qkv[:s, d:d + hd], qkv[:s, 2 * d:2 * d + hd], sc["beta_P"], sc["sm"], sc["sm"],
                           sc["beta_Q"], dS[:s], dQ[:s, :hd], btb, ws)
    assert L.us_workspace_status(ws) == 0
    print("ok attention", passes)


def encoder_layer(passes: int, fused: bool, attention: str = "bf16"):
    nseq, slen, d, nhead, d_ff = 16, 512, 1024, 16, 4096
    T = nseq * slen
    host = (synth.normal(0, 0, (T, d)), synth.normal(0, 1, (d, 3 * d)), synth.normal(0, 2, (d, d)),
            synth.normal(0, 3, (d, d_ff)), synth.normal(0, 4, (d_ff, d)), synth.normal(0, 5, (T, d)))
    tensors = [torch.from_numpy(t).cuda() for t in host]
    layer = encoder.UnitScaledEncoderLayer(nseq, slen, d, nhead, d_ff, attention=attention, fused_attention=fused)
    for _ in range(passes):
        layer.step(*tensors, stream=torch.cuda.current_stream().cuda_stream)     # one stream: launches in issue order
    layer.check()
    print("ok encoder", passes, attention, "fused" if fused else "unfused")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, default=8192)
    ap.add_argument("--passes", type=int, default=2)
    ap.add_argument("--operand", default="fp8")
    ap.add_argument("--case", default="ffn", choices=["ffn", "attention", "encoder"])
    ap.add_argument("--unfused", action="store_true")
    ap.add_argument("--attention", default="bf16", choices=["bf16", "fp16", "fp8"])
    a = ap.parse_args()
    if a.case == "attention":
        return attention(a.passes)
    if a.case == "encoder":
        return encoder_layer(a.passes, not a.unfused, a.attention)
    shape = synth.FFNShape("profile", a.tokens, 1024, 4096)
    tensors = [torch.from_numpy(t).cuda() for t in synth.ffn_tensors(shape, seed=0)]
    blk = ffn.UnitScaledFFN(shape.tokens, shape.d_model, shape.d_ff, operand=a.operand)
    for _ in range(a.passes):
        blk.step(*tensors)
    blk.check()
    print("ok", a.tokens, a.passes)


if __name__ == "__main__":
    main()
