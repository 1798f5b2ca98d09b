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
