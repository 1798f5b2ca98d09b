"""Token-sharded data parallelism for the unit-scaled linear layers: the one exchange of the path.

Each rank holds the same weights and its own shard of the tokens.  Forward and input-gradient GEMMs
are independent per shard; the weight gradient is a sum over all tokens, so the ranks add their partial
weight gradients (one all-reduce per weight), and the unit-scaling factor of that GEMM must use the
*global* batch: beta_w = (world * tokens_per_rank)^-1/2 (table row "matmul": beta_W = b^-1/2 with b
the number of rows of X), applied locally before the sum so that the reduced gradient is already
unit-scaled and the partial results stay well inside the range of a 16-bit or FP8 transport format.

Plumbing only: torch.distributed does the exchange (NCCL on GPUs, gloo in the CPU tests); the GEMMs
are the library's.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def global_beta_w(tokens_per_rank: int, world: int) -> float:
    """beta_W of a weight-gradient GEMM whose batch is sharded over `world` ranks."""
    return float(tokens_per_rank * world) ** -0.5


def allreduce_weight_grads(grads, group=None, async_op: bool = False):
    """Sum the ranks' partial weight gradients in place.  Each partial must have been computed with
    global_beta_w; returns the work handles when async_op is set (wait on them before reading)."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return []
    works = [dist.all_reduce(g, op=dist.ReduceOp.SUM, group=group, async_op=async_op) for g in grads]
    return works if async_op else []
