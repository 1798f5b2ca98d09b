"""Benchmark of the unit-scaled FFN block (forward + backward) at the BERT-large shape.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole path over one batch: FP8 casts of X, W1, W2 and the
upstream gradient, the six scaled GEMMs with their fused GELU / GELU-gradient / residual
epilogues (10 kernel launches, replayed as one CUDA graph).  Prints ONE JSON line.

  value      matmul TFLOP/s (12 T d f FLOP per step) with all inputs resident in HBM,
             K steps timed with CUDA events after W warm-ups, max over ranks.
  e2e        same metric through the public call with host buffers: every step copies
             X, W1, W2, G from pinned host memory and reads R, dX, dW1, dW2 back (copies of
             neighbouring steps overlap the compute on separate streams).
  roofline   the GEMM kernel: achieved FLOP/s per launch (timing events between the launches of
             the step graph, separate pass) against the measured tensor peak.
  cpu_baseline / --impl reference: the fp64 NumPy oracle on the host cores, on a bounded
             sample of the same workload.

With N > 1 (torchrun, one rank per GPU) every rank runs its own replica of the block on
its own batch (weak scaling, no data-path collective); ranks meet only at the timing barriers.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "unit-scaled FFN fwd+bwd TFLOP/s at BERT-large shape"
NOMINAL_FP8_TFLOPS = 4500.0      # B200 dense FP8, public figure
NOMINAL_HBM_GBS = 7700.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--operand", default="fp8", choices=["fp8", "bf16", "fp16"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dp", action="store_true", help="token-sharded data parallelism: global beta_w and an all-reduce of the weight gradients every step (default: independent replicas)")
    ap.add_argument("--one-stream", action="store_true", help="issue the step's GEMMs on one stream (no overlap of independent launches)")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


# ----------------------------------------------------------------------------- distributed plumbing

def dist_setup(n_gpus: int):
    """Returns (rank, world, local_rank); initialises torch.distributed when launched by torchrun."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch
        import torch.distributed as dist
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend)
    return rank, world, local


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Largest value over all ranks (the slowest rank sets the job's time)."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, world: int, elapsed_s_max: float) -> float:
    """Whole-job throughput under weak scaling: every rank processed units_per_rank."""
    return units_per_rank * world / elapsed_s_max


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed regions run."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu_index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, windows):
        """windows: list of (t0, t1) wall-clock intervals of the timed regions."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        for ts, line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                clk, mx, pw = float(parts[1]), float(parts[2]), float(parts[3])
            except ValueError:
                continue
            smax.append(mx)
            if any(t0 <= ts <= t1 + 0.06 for t0, t1 in windows):
                sm.append(clk)
                power.append(pw)
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        return {
            "sm_mhz": statistics.median(sm) if sm else None,
            "sm_max_mhz": max(smax) if smax else None,
            "power_w_max": max(power) if power else None,
            "samples_under_load": len(sm),
            "reasons": sorted(reasons),
        }


# ----------------------------------------------------------------------------- oracle legs (host cores)

def _oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def _oracle_sample_step(tensors, shape, tokens: int, width: int):
    """The oracle's FFN block on the first `tokens` tokens and the first `width` hidden units."""
    from oracle import ops as O
    X, W1, W2, G = tensors
    sc = O.FFNScales.unconstrained(shape.tokens, shape.d_model, shape.d_ff)
    t0 = time.perf_counter()
    O.ffn_block(X[:tokens], W1[:, :width], W2[:width], G[:tokens], sc, operand="fp8")
    return time.perf_counter() - t0


def gemm_traffic_mb():
    """DRAM bytes per GEMM launch from the committed ncu capture, or None when the kernel sources
    have changed since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "gemm_kernel_ffn_bert_large_fp8_traffic.json")
    try:
        with open(path) as fh:
            rec = json.load(fh)
        h = hashlib.sha256()
        for f in rec["source_files"]:
            with open(os.path.join(ROOT, f), "rb") as src:
                h.update(src.read())
        return rec["mean_mb"] if h.hexdigest() == rec["source_sha256"] else None
    except (OSError, KeyError, ValueError):
        return None


def cpu_baseline(shape, seed: int = 0, tokens: int = 1024):
    """The oracle as it stands, timed once on a bounded sample (about 10-30 s of host work):
    the first 1024 tokens, and the whole batch instead when that took under three seconds."""
    from paper_2303_11257_b200 import synth
    tensors = synth.ffn_tensors(shape, seed)
    dt = _oracle_sample_step(tensors, shape, tokens, shape.d_ff)
    if dt < 3.0 and tokens < shape.tokens:
        tokens = shape.tokens
        dt = _oracle_sample_step(tensors, shape, tokens, shape.d_ff)
    flops = 12.0 * tokens * shape.d_model * shape.d_ff
    return {
        "value": flops / dt / 1e12, "unit": "TFLOP/s", "cores": _oracle_threads(), "kind": "oracle",
        "sample": f"first {tokens} of {shape.tokens} tokens, full d_model x d_ff weights, fp64 NumPy, {dt:.1f} s",
    }


def run_reference(args, rank: int, world: int):
    """--impl reference: times the CPU oracle, each step a bounded sample of the workload."""
    if rank != 0:
        return
    from paper_2303_11257_b200 import synth
    shape = synth.FFN_BERT_LARGE
    tensors = synth.ffn_tensors(shape, 0)
    # size the per-step sample so that warmup + steps finish in about two and a half minutes
    budget = 150.0 / max(1, args.steps + args.warmup)
    ladder = [(1024, 4096), (512, 4096), (256, 2048), (128, 1024), (64, 512), (32, 256), (16, 128)]
    probe = _oracle_sample_step(tensors, shape, 16, 128)
    probe_cost = 16 * 128 + 16 * shape.d_model + 2 * shape.d_model * 128      # elements touched ~ time driver
    tokens, width = ladder[-1]
    for tk, wd in ladder:
        cost = tk * wd * 4 + tk * shape.d_model * 4 + 2 * shape.d_model * wd
        if probe * cost / probe_cost <= budget:
            tokens, width = tk, wd
            break
    for _ in range(args.warmup):
        _oracle_sample_step(tensors, shape, tokens, width)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        _oracle_sample_step(tensors, shape, tokens, width)
    dt = time.perf_counter() - t0
    flops = 12.0 * tokens * shape.d_model * width * args.steps
    value = flops / dt / 1e12
    sample = f"per step: first {tokens} of {shape.tokens} tokens x first {width} of {shape.d_ff} hidden units"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "ffn_bert_large fwd+bwd (T=8192, d_model=1024, d_ff=4096), CPU oracle sample",
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": _oracle_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- GPU arm

def run_ours(args, rank: int, world: int, local: int):
    import torch

    from paper_2303_11257_b200 import dp, ffn, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks = load_peaks()
    shape = synth.FFN_BERT_LARGE
    T, d, f = shape.tokens, shape.d_model, shape.d_ff
    flops_step = ffn.UnitScaledFFN.flops(T, d, f)

    # two rotating input sets per rank (seed differs per rank and set); weights shared
    host = [synth.ffn_tensors(shape, seed=1000 * rank + i) for i in range(2)]
    pinned = [[torch.from_numpy(t).pin_memory() for t in tensors] for tensors in host]
    sets = [[p.to(dev, non_blocking=True) for p in tensors] for tensors in pinned]
    dp_on = args.dp and world > 1
    scales = ffn.FFNScales.unit(T, d, f, dp_world=world) if dp_on else None
    blocks = [ffn.UnitScaledFFN(T, d, f, scales=scales, operand=args.operand, device=dev) for _ in sets]
    if args.one_stream:
        for b in blocks:
            b.concurrent = False
    torch.cuda.synchronize()
    for blk, tensors in zip(blocks, sets):            # eager pass: first-call set-up happens here
        blk.step(*tensors)
        blk.check()
    graphs = [blk.capture(*tensors) for blk, tensors in zip(blocks, sets)]
    torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
    windows = []

    # ---- device-resident timing: exactly K steps between two events
    for i in range(args.warmup):
        graphs[i % 2].replay()
    torch.cuda.synchronize()
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    e0.record()
    for i in range(args.steps):
        graphs[i % 2].replay()
        if dp_on:
            dp.allreduce_weight_grads([blocks[i % 2].dW1, blocks[i % 2].dW2])
    e1.record()
    torch.cuda.synchronize()
    windows.append((w0, time.time()))
    barrier(world)
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
    for blk in blocks:
        blk.check()
    ms_per_step = ms_total / args.steps
    value = aggregate_throughput(flops_step * args.steps, world, ms_total * 1e-3) / 1e12

    # ---- per-launch timing pass: the same launches captured in one graph with a timing event
    #      (event-record node) between consecutive launches, replayed after a warm-up
    blk, tensors = blocks[0], sets[0]
    stage_list = blk.stages(*tensors)
    evs = [torch.cuda.Event(enable_timing=True, external=True) for _ in range(len(stage_list) + 1)]
    timed_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(timed_graph):
        evs[0].record()
        for j, (_, _, fn) in enumerate(stage_list):
            fn(None)
            evs[j + 1].record()
    n_prof = max(3, min(args.steps, 200))
    for _ in range(5):
        graphs[1].replay()
        timed_graph.replay()
    torch.cuda.synchronize()
    sums = [0.0] * len(stage_list)
    w0 = time.time()
    for it in range(n_prof):
        graphs[1].replay()                 # the other buffer set in between, as in the timed loop
        timed_graph.replay()
        torch.cuda.synchronize()
        for j in range(len(stage_list)):
            sums[j] += evs[j].elapsed_time(evs[j + 1])
    windows.append((w0, time.time()))
    stage_graphs = [(name, kind, None) for name, kind, _ in stage_list]
    per_launch_us = {name: sums[j] / n_prof * 1e3 for j, (name, _, _) in enumerate(stage_list)}
    gemm_names = [n for n, k, _ in stage_graphs if k == "gemm"]
    cast_names = [n for n, k, _ in stage_graphs if k == "cast"]
    gemm_us = statistics.mean(per_launch_us[n] for n in gemm_names)
    flops_launch = 2.0 * T * d * f
    operand_ratio = 2.0 if args.operand == "fp8" else 1.0
    tensor_peak = peaks["bf16_tflops_sustained"] * operand_ratio
    achieved = flops_launch / (gemm_us * 1e-6) / 1e12
    roofline = {
        "kernel": "gemm_kernel (6 launches per step, mean)", "bound": "tensor", "achieved": achieved,
        "peak": tensor_peak, "unit": "TFLOP/s", "frac": achieved / tensor_peak,
        "traffic": (gemm_traffic_mb() * 1e6 if args.operand == "fp8" and gemm_traffic_mb() is not None else None),
        "traffic_unit": "bytes per launch (ncu dram read + write, mean of the six launches)",
        "peak_source": f"{peaks['_source']} bf16 sustained x {operand_ratio:g} (nominal dtype ratio)",
        "flops_per_launch": flops_launch, "us_per_launch": gemm_us,
    }
    cast_bytes = {"cast_W1": d * f * 5, "cast_W2": d * f * 5, "cast_X": T * d * 5, "cast_G": T * d * 5}
    cast_bytes["cast_all"] = sum(cast_bytes.values())
    if args.operand != "fp8":
        cast_bytes = {k: v // 5 * 6 for k, v in cast_bytes.items()}
    kernels = []
    for n in gemm_names:
        kernels.append({"name": n, "us": per_launch_us[n], "tflops": flops_launch / per_launch_us[n] / 1e6,
                        "frac_of_peak": flops_launch / per_launch_us[n] / 1e6 / tensor_peak})
    for n in cast_names:
        gbs = cast_bytes[n] / per_launch_us[n] / 1e3
        kernels.append({"name": n, "us": per_launch_us[n], "gbs": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"]})

    # ---- end to end: host buffers in, results out, every step
    n_e2e = max(3, min(args.steps, 30))
    outs = [[torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in (b.R, b.dX, b.dW1, b.dW2)] for b in blocks]
    h2d = sum(t.numel() * t.element_size() for t in pinned[0])
    d2h = sum(t.numel() * t.element_size() for t in outs[0])

    # Three streams pipeline the steps: while step i computes, step i+1's inputs are being copied
    # in and step i-1's results are being read back (two buffer sets; events keep a set's copies
    # and its graph replay in order).
    cur = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in sets]      # inputs of the set are on the device
    ev_done = [torch.cuda.Event() for _ in sets]    # the set's step has finished
    ev_out = [torch.cuda.Event() for _ in sets]     # the set's results have been read back

    def e2e_step(i):
        s = i % 2
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_done[s])             # the previous step on this set no longer reads its inputs
            for dst, src in zip(sets[s], pinned[s]):
                dst.copy_(src, non_blocking=True)
            ev_in[s].record(s_in)
        cur.wait_event(ev_in[s])
        cur.wait_event(ev_out[s])                   # its previous results have been copied out
        graphs[s].replay()
        ev_done[s].record(cur)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[s])
            for dst, src in zip(outs[s], (blocks[s].R, blocks[s].dX, blocks[s].dW1, blocks[s].dW2)):
                dst.copy_(src, non_blocking=True)
            ev_out[s].record(s_out)

    for ev in ev_done + ev_out:
        ev.record(cur)
    for i in range(4):
        e2e_step(i)
    torch.cuda.synchronize()
    barrier(world)
    w0 = time.time()
    e0.record()
    for i in range(n_e2e):
        e2e_step(i)
    cur.wait_stream(s_out)
    e1.record()
    torch.cuda.synchronize()
    windows.append((w0, time.time()))
    barrier(world)
    ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev)
    e2e_value = aggregate_throughput(flops_step * n_e2e, world, ms_e2e * 1e-3) / 1e12

    clocks = sampler.stop(windows) if sampler else None
    if rank != 0:
        return
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": {"fp8": "fp8_e4m3/e5m2 (fp32 accumulate)", "bf16": "bf16", "fp16": "fp16"}[args.operand],
        "data": "synthetic",
        "config": {"workload": "ffn_bert_large fwd+bwd: T=8192 tokens (16x512), d_model=1024, d_ff=4096, tau=0.5",
                   "operand": args.operand, "replicas": world, "weight_gradient_allreduce": dp_on,
                   "l2": "two rotating input/buffer sets, ~0.45 GB touched per step (> 126 MB L2)",
                   "launch": f"one CUDA graph of {blocks[0].launches_per_step} kernels per step, "
                             + ("GEMMs after the first on three streams" if blocks[0].concurrent else "one stream")},
        "tokens_per_s": T * world / (ms_per_step * 1e-3),
        "pct_of_nominal_fp8_peak": 100.0 * value / world / NOMINAL_FP8_TFLOPS,
        "pct_of_measured_tensor_peak": 100.0 * value / world / tensor_peak,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": n_e2e, "ms_per_step": ms_e2e / n_e2e},
        "gpu_launches": blocks[0].launches_per_step * args.steps,
        "roofline": roofline,
        "kernels": kernels,
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(shape)
    elif world > 1:
        line["cpu_baseline"] = None
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    rank, world, local = dist_setup(args.gpus)
    try:
        if args.impl == "reference":
            run_reference(args, rank, world)
        else:
            run_ours(args, rank, world, local)
    finally:
        if world > 1:
            import torch.distributed as dist
            if dist.is_initialized():
                dist.destroy_process_group()


if __name__ == "__main__":
    main()
