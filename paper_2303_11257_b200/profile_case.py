"""Runs a few eager passes of the FFN block so that a profiler can attach to individual launches.

    python -m paper_2303_11257_b200.profile_case [--tokens 8192] [--passes 2] [--operand fp8]

Each pass is the launches of UnitScaledFFN.step (one fused cast, six GEMMs) at d_model = 1024, d_ff = 4096.  At the default
size the process holds well under 2 GB on the device and a pass lasts a fraction of a millisecond.
"""
from __future__ import annotations

import argparse

import torch

from . import ffn, synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, default=8192)
    ap.add_argument("--passes", type=int, default=2)
    ap.add_argument("--operand", default="fp8")
    a = ap.parse_args()
    shape = synth.FFNShape("profile", a.tokens, 1024, 4096)
    tensors = [torch.from_numpy(t).cuda() for t in synth.ffn_tensors(shape, seed=0)]
    blk = ffn.UnitScaledFFN(shape.tokens, shape.d_model, shape.d_ff, operand=a.operand)
    for _ in range(a.passes):
        blk.step(*tensors)
    blk.check()
    print("ok", a.tokens, a.passes)


if __name__ == "__main__":
    main()
