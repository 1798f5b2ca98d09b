"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, barrier + max-over-ranks timing,
whole-job aggregation under weak scaling, and the reference arm's rank-0-only rule."""
import json
import re
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import bench
    rank, world, local = bench.dist_setup(2)
    bench.barrier(world)
    elapsed = 1.0 + rank            # rank 1 is the slow one
    mx = bench.max_over_ranks(elapsed, world)
    total = bench.aggregate_throughput(10.0, world, mx)
    bench.barrier(world)
    print(json.dumps({"rank": rank, "world": world, "max": mx, "total": total}))
    import torch.distributed as dist
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_reduce_time_and_aggregate(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", MASTER_ADDR="127.0.0.1")
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
         "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)],
        capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [json.loads(m) for m in re.findall(r"\{[^{}]*\}", out.stdout)]   # ranks may interleave their lines
    assert sorted(r["rank"] for r in rows) == [0, 1]
    for r in rows:
        assert r["world"] == 2 and r["max"] == 2.0 and r["total"] == 10.0 * 2 / 2.0


def test_single_process_helpers():
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.aggregate_throughput(8.0, 4, 2.0) == 16.0
    p = bench.load_peaks()
    assert p["hbm_gbs"] > 0 and p["bf16_tflops_sustained"] > 0
