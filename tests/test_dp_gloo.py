"""Token-sharded data parallelism on two gloo ranks (CPU): each rank forms its shard's weight gradient with
the global beta_w, the ranks add them, and the sum equals the single-process gradient over all tokens."""
import json
import os
import re
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np, torch
    import torch.distributed as dist
    from oracle import ops as O
    from paper_2303_11257_b200 import dp, synth
    dist.init_process_group(backend="gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    T, d, f = 64, 32, 48                         # tokens per rank, widths
    X = synth.normal(9, 0, (T * world, d)); G = synth.normal(9, 1, (T * world, f))
    Xq, Gq = O.store(X, "e4m3")[0], O.store(G, "e5m2")[0]
    beta = dp.global_beta_w(T, world)
    sl = slice(rank * T, (rank + 1) * T)
    part = torch.from_numpy(O.linear_bwd_w(Xq[sl], Gq[sl], beta))
    dp.allreduce_weight_grads([part])
    full = O.linear_bwd_w(Xq, Gq, (T * world) ** -0.5)
    err = float(np.abs(part.numpy() - full).max())
    handles = dp.allreduce_weight_grads([torch.ones(3)], async_op=True)
    for h in handles: h.wait()
    print(json.dumps({"rank": rank, "world": world, "err": err, "beta": beta, "std": float(full.std())}))
    dist.destroy_process_group()
""") % ROOT


def test_sharded_weight_gradient_equals_the_full_batch_gradient(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", MASTER_ADDR="127.0.0.1")
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
         "--master-addr", "127.0.0.1", "--master-port", "29741", str(script)],
        capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [json.loads(m) for m in re.findall(r"\{[^{}]*\}", out.stdout)]
    assert sorted(r["rank"] for r in rows) == [0, 1]
    for r in rows:
        assert r["err"] < 1e-12 and abs(r["beta"] - 128 ** -0.5) < 1e-15 and 0.7 < r["std"] < 1.3


def test_single_process_is_a_no_op():
    import torch
    from paper_2303_11257_b200 import dp
    g = torch.ones(4)
    assert dp.allreduce_weight_grads([g]) == [] and g.sum().item() == 4
    assert dp.global_beta_w(8192, 8) == (8192 * 8) ** -0.5


LOWP_WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np, torch
    import torch.distributed as dist
    from oracle import formats as F, ops as O
    from paper_2303_11257_b200 import dp, synth
    dist.init_process_group(backend="gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    T, d, f = 64, 32, 48
    X = synth.normal(9, 0, (T * world, d)); G = synth.normal(9, 1, (T * world, f))
    Xq, Gq = O.store(X, "e4m3")[0], O.store(G, "e5m2")[0]
    beta = dp.global_beta_w(T, world)
    parts = [O.linear_bwd_w(Xq[r * T:(r + 1) * T], Gq[r * T:(r + 1) * T], beta).astype(np.float32) for r in range(world)]
    full = O.linear_bwd_w(Xq, Gq, (T * world) ** -0.5)
    out = {}
    for transport in ("e5m2", "e4m3", "bf16"):
        fmt = F.FORMATS[transport]
        tdt = dp._TRANSPORT[transport][0]
        def pack(partial, scale, dtype, fmt=fmt):            # oracle stand-in for the device cast
            codes = F.quantise_codes((partial.numpy() * np.float32(scale)).astype(np.float64), fmt)
            return torch.from_numpy(codes.view(np.int16) if codes.dtype == np.uint16 else codes).view(dtype)
        def accumulate(packed, inv_scale, dst, fmt=fmt):      # oracle stand-in for the device sum, in the order given
            acc = np.zeros(dst.shape, np.float64)
            for t in packed:
                raw = t.contiguous().view(torch.int16).numpy().view(np.uint16) if t.element_size() == 2 else t.contiguous().view(torch.uint8).numpy()
                acc += F.decode(raw, fmt)
            dst.copy_(torch.from_numpy((acc * inv_scale).astype(np.float32)))
        res = torch.zeros(d, f)
        dp.exchange_weight_grads([torch.from_numpy(parts[rank])], [res], transport=transport, pack=pack, accumulate=accumulate)
        s = dp.transport_scale(world)
        want = sum(F.quantise((p * np.float32(s)).astype(np.float64), fmt) for p in parts) / s     # every rank's packed partial, rank order
        out[transport + "_exact"] = float(np.abs(res.numpy() - want.astype(np.float32)).max())
        out[transport + "_vs_full"] = float(np.abs(res.numpy() - full).max())
        out[transport + "_digest"] = float(res.double().sum())
    print(json.dumps({"rank": rank, "world": world, "scale": dp.transport_scale(world), **out}))
    dist.destroy_process_group()
""") % ROOT


def test_low_precision_exchange_on_two_ranks(tmp_path):
    """The packed partials of all ranks arrive in rank order on every rank, are summed in that order, and the sum is
    the sum of the individually quantised partials (exactly), close to the full-batch gradient (to the format's step)."""
    script = tmp_path / "worker_lowp.py"
    script.write_text(LOWP_WORKER)
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", MASTER_ADDR="127.0.0.1")
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
         "--master-addr", "127.0.0.1", "--master-port", "29743", str(script)],
        capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [json.loads(m) for m in re.findall(r"\{[^{}]*\}", out.stdout)]   # ranks may interleave their lines
    assert sorted(r["rank"] for r in rows) == [0, 1]
    for r in rows:
        assert r["scale"] == 1.0 or r["scale"] == 2.0            # power of two nearest sqrt(2)
        for transport, step in (("e5m2", 2.0 ** -2), ("e4m3", 2.0 ** -3), ("bf16", 2.0 ** -7)):
            assert r[transport + "_exact"] < 1e-6
            assert r[transport + "_vs_full"] < 4.5 * step        # |partial| < 4.5 at this size, two roundings of half a step each
    for transport in ("e5m2", "e4m3", "bf16"):
        assert rows[0][transport + "_digest"] == rows[1][transport + "_digest"]       # bit-identical on both ranks


def test_transport_scale_is_a_power_of_two_near_sqrt_world():
    import math
    from paper_2303_11257_b200 import dp
    assert dp.transport_scale(1) == 1.0 and dp.transport_scale(4) == 2.0 and dp.transport_scale(16) == 4.0 and dp.transport_scale(64) == 8.0
    for w in (2, 3, 8, 32, 48):
        s = dp.transport_scale(w)
        assert s == 2.0 ** round(math.log2(s)) and 2 ** -0.5 - 1e-9 <= s / w ** 0.5 <= 2 ** 0.5 + 1e-9
