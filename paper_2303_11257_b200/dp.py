"""Token-sharded data parallelism for the unit-scaled linear layers: the one exchange of the path.

Each rank holds the same weights and its own shard of the tokens.  Forward and input-gradient GEMMs
are independent per shard; the weight gradient is a sum over all tokens, so the ranks add their partial
weight gradients, and the unit-scaling factor of that GEMM must use the *global* batch:
beta_w = (world * tokens_per_rank)^-1/2 (table row "matmul": beta_W = b^-1/2 with b the number of rows
of X), applied locally before the sum so that the reduced gradient is already unit-scaled.

Two forms of the exchange:

* allreduce_weight_grads: one float32 all-reduce per weight (torch.distributed; NCCL on GPUs).
* exchange_weight_grads: the partials travel in a low-precision format (appendix "Fusing scale factors":
  fixed scales keep partial results well inside the range of 16-bit or 8-bit formats, which suits
  distributed aggregation).  A rank's partial has standard deviation about world^-1/2; multiplied by
  the power of two nearest to world^1/2 it is unit-scaled and fits BF16 or FP8 without any range
  analysis.  Every rank all-gathers the packed partials and adds them itself in float32, in rank
  order, so all ranks hold bit-identical sums and the result does not depend on the collective's
  internal order.  Bytes received per rank and weight of S elements: (world - 1) S in FP8 and
  2 (world - 1) S in BF16, against about 8 S (world - 1) / world for a float32 ring all-reduce: FP8
  transport moves no more than the all-reduce up to eight ranks and a quarter of it on two.

Plumbing only: torch.distributed moves the bytes; packing and summing are the library's kernels
(us_cast_fp8 / us_weighted_add).  The pack and sum steps are arguments so that the host logic can be
exercised on CPU ranks (gloo) with stand-ins.
"""
from __future__ import annotations

import math

import torch
import torch.distributed as dist

_TRANSPORT = {"bf16": (torch.bfloat16, torch.uint8), "e4m3": (torch.float8_e4m3fn, torch.uint8),
              "e5m2": (torch.float8_e5m2, torch.uint8)}       # transport dtype, and the byte type the collective moves


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


def transport_scale(world: int) -> float:
    """Power of two nearest to sqrt(world): a partial of one of `world` ranks times this is unit-scaled."""
    return 2.0 ** round(0.5 * math.log2(world))


def _pack_device(partial: torch.Tensor, scale: float, dtype: torch.dtype) -> torch.Tensor:
    """q(scale * partial) in the transport format, by the library's kernels."""
    from . import lib as L
    out = torch.empty(partial.shape, dtype=dtype, device=partial.device)
    if dtype == torch.bfloat16:
        L.us_weighted_add([partial], [scale], 1.0, out)
    else:
        L.us_cast_fp8(partial, scale, out)
    return out


def _sum_device(packed, inv_scale: float, out: torch.Tensor) -> None:
    """out = inv_scale * (packed[0] + packed[1] + ...) in float32, in the order given (us_weighted_add takes
    up to eight tensors per call; more ranks continue from the running sum)."""
    from . import lib as L
    first = list(packed[:8])
    L.us_weighted_add(first, [1.0] * len(first), inv_scale, out)
    rest = list(packed[8:])
    while rest:
        chunk, rest = rest[:7], rest[7:]
        L.us_weighted_add([out] + chunk, [1.0] + [inv_scale] * len(chunk), 1.0, out)


def exchange_weight_grads(partials, outs, transport: str = "e5m2", group=None, pack=None, accumulate=None):
    """Sum the ranks' partial weight gradients with a low-precision transport.

    partials: this rank's float32 partial gradients (computed with global_beta_w); outs: float32 tensors of
    the same shapes that receive the sums (may be the partials themselves).  transport: "bf16", "e5m2" (the
    gradient format) or "e4m3".  pack(partial, scale, dtype) and accumulate(list of packed, inv_scale, out)
    default to the library's kernels."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    dtype, wire = _TRANSPORT[transport]
    pack = pack or _pack_device
    accumulate = accumulate or _sum_device
    scale = transport_scale(world)
    for partial, out in zip(partials, outs):
        mine = pack(partial, scale, dtype).contiguous()
        if world == 1:
            accumulate([mine], 1.0 / scale, out)
            continue
        rows = mine.shape[0]
        gathered = torch.empty((world * rows,) + tuple(mine.shape[1:]), dtype=dtype, device=mine.device)   # rank r's partial = rows [r * rows, (r + 1) * rows)
        # the collective moves plain integers: not every backend knows the 8-bit float types
        dist.all_gather_into_tensor(gathered.view(wire), mine.view(wire), group=group)
        accumulate([gathered[r * rows:(r + 1) * rows] for r in range(world)], 1.0 / scale, out)
    return outs
