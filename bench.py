"""Benchmark of the unit-scaled FFN block (forward + backward) at the BERT-large shape.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload ffn|ffn_bf16|ffn_fp16|sweep|encoder]

One "step" of the default workload is one pass of the whole path over one batch: the FP8 casts of
X, W1, W2 and the upstream gradient (one launch), then the six scaled GEMMs with their fused GELU /
GELU-gradient / residual epilogues as two launches (the two GEMMs that end in the hidden layer, with the
pre-activation kept on the SM; the other four as one grouped launch): 3 kernel launches, replayed as one
CUDA graph.  Prints ONE JSON line.

  value      matmul TFLOP/s (12 T d f FLOP per step) with all inputs resident in HBM,
             K steps timed with CUDA events after W warm-ups, max over ranks.
  sustained  the same graph replayed for at least two seconds (the power cap pulls the clock down),
             with its own clock samples.
  e2e        same metric through the public call with host buffers: every step copies
             X, W1, W2, G from pinned host memory and reads R, dX, dW1, dW2 back (copies of
             neighbouring steps overlap the compute on separate streams).
  roofline   the GEMM kernel: achieved FLOP/s per launch (each launch of the step timed on its own:
             a graph of back-to-back launches of that call over the rotating buffer sets) against the
             measured tensor peak that matches the run's clock regime, and against a black-box
             FP8 GEMM of the vendor library (torch._scaled_mm, 8192^3) timed in the same process.
  cpu_baseline / --impl reference: the fp64 NumPy oracle on the host cores, on a bounded
             sample of the same workload.

Other workloads (same JSON keys; `config.workload` names them): ffn_bf16 / ffn_fp16 = the block with
16-bit matmul operands; sweep = each of Y, dX, dW alone at M = N = K in {1024 ... 16384} and
M = 512, N = K = 8192 (value = the 8192^3 forward GEMM, the table in `kernels`); encoder = one
BERT-large-shaped encoder layer, forward + backward.

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
    ap.add_argument("--workload", default="ffn", choices=["ffn", "ffn_bf16", "ffn_fp16", "sweep", "encoder"])
    ap.add_argument("--sustain-seconds", type=float, default=2.0, help="length of the sustained leg (0 = skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dp", action="store_true", help="token-sharded data parallelism: global beta_w and an all-reduce of the weight gradients every step (default: independent replicas)")
    ap.add_argument("--dp-transport", default="f32", choices=["f32", "bf16", "e5m2"], help="with --dp: format the partial weight gradients travel in (f32 = all-reduce; bf16 / e5m2 = all-gather of unit-scaled partials, summed locally in float32 in rank order)")
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
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
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
        """Ends the sampling; windows: list of (t0, t1) wall-clock intervals of the timed regions."""
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        return self.summary(windows)

    def summary(self, windows):
        """Clock statistics over the samples that fall into the given wall-clock windows."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        sm, smax, power, reasons = [], [], [], set()
        parsed = []
        for ts, line in list(self.lines):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                clk, mx, pw = float(parts[1]), float(parts[2]), float(parts[3])
            except ValueError:
                continue
            smax.append(mx)
            parsed.append((ts, clk, pw, parts[5:9]))
        inside = [r for r in parsed if any(t0 <= r[0] <= t1 + 0.06 for t0, t1 in windows)]
        note = None
        if not inside and parsed and windows:
            # a timed region of a few milliseconds can fall between two samples (20 ms apart): take the nearest one
            # (the warm-up steps run right before the region, so the GPU is under the same load there)
            dist = lambda r: min(max(t0 - r[0], r[0] - t1, 0.0) for t0, t1 in windows)
            best = min(parsed, key=dist)
            if dist(best) <= 0.25:
                inside = [best]
                note = f"no sample inside the timed region; nearest one, {dist(best) * 1e3:.0f} ms away"
        for ts, clk, pw, flags in inside:
            sm.append(clk)
            power.append(pw)
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), flags):
                if val.lower().startswith("active"):
                    reasons.add(name)
        out = {
            "sm_mhz": statistics.median(sm) if sm else None,
            "sm_max_mhz": max(smax) if smax else None,
            "power_w_max": max(power) if power else None,
            "samples_under_load": len(sm),
            "reasons": sorted(reasons),
        }
        if note:
            out["note"] = note
        return out


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

def pick_tensor_peak(peaks, operand_ratio: float, timed_seconds: float, clocks):
    """The measured tensor peak that matches the clock regime of a timed region: the burst figure when the
    region is short (under a second) or the sampled SM clock sat at its maximum, the sustained figure
    when the region was long enough for the power cap to pull the clock down.  FP8 peaks are the BF16
    measurements times the nominal dtype ratio.  Returns (peak TFLOP/s, description, both peaks)."""
    burst = peaks["bf16_tflops"] * operand_ratio
    sustained = peaks["bf16_tflops_sustained"] * operand_ratio
    at_max = bool(clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"])
    use_burst = timed_seconds < 1.0 or at_max
    src = f"{peaks['_source']} bf16 {'burst' if use_burst else 'sustained'} x {operand_ratio:g} (nominal dtype ratio)"
    return (burst if use_burst else sustained), src, {"burst": burst, "sustained": sustained}


class Fp8LibraryCeiling:
    """Black-box FP8 ceiling of this process on this GPU: torch._scaled_mm (the vendor library's FP8 GEMM) at 8192^3,
    best of ten launches (burst) and a back-to-back loop of some seconds (sustained)."""

    def __init__(self, torch, dev):
        self.torch, self.n = torch, 8192
        self.result = {"what": "torch._scaled_mm 8192^3 e4m3 x e4m3 -> bf16"}
        try:
            a = torch.randn(self.n, self.n, device=dev).to(torch.float8_e4m3fn)
            b = torch.randn(self.n, self.n, device=dev).to(torch.float8_e4m3fn).t()          # column-major second operand
            one = torch.ones((), device=dev)
            self.fn = lambda: torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
            for _ in range(3):
                self.fn()
            torch.cuda.synchronize()
        except Exception as exc:                                                 # noqa: BLE001 - reported, not fatal
            self.fn = None
            self.result["unavailable"] = str(exc)[:120]

    def burst(self):
        if self.fn is None:
            return
        torch, best = self.torch, 1e30
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); self.fn(); e1.record(); torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        self.best_ms = best
        self.result["burst_tflops"] = 2.0 * self.n ** 3 / (best * 1e-3) / 1e12

    def sustained(self, seconds: float):
        if self.fn is None or seconds <= 0:
            return
        torch = self.torch
        iters = max(10, int(seconds / (self.best_ms * 1e-3)))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            self.fn()
        e1.record(); torch.cuda.synchronize()
        self.result["sustained_tflops"] = 2.0 * self.n ** 3 * iters / (e0.elapsed_time(e1) * 1e-3) / 1e12
        self.result["sustained_seconds"] = e0.elapsed_time(e1) * 1e-3


def time_alone(torch, fn, nsets: int, iters: int = 12, reps: int = 5) -> float:
    """Microseconds per launch of fn(set index), timed on its own: one CUDA graph of `iters` back-to-back
    launches that rotate over the buffer sets, best of `reps` replays."""
    for i in range(nsets):
        fn(i)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(iters):
            fn(i % nsets)
    g.replay()
    torch.cuda.synchronize()
    best = 1e30
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) * 1e3 / iters)
    return best


def run_ours(args, rank: int, world: int, local: int):
    import torch

    from paper_2303_11257_b200 import dp, ffn, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks = load_peaks()
    if args.workload in ("ffn_bf16", "ffn_fp16"):
        args.operand = args.workload[4:]
    if args.workload == "sweep":
        return run_sweep(args, rank, world, local, torch, dev, peaks)
    if args.workload == "encoder":
        return run_encoder(args, rank, world, local, torch, dev, peaks)
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
            grads = [blocks[i % 2].dW1, blocks[i % 2].dW2]
            if args.dp_transport == "f32":
                dp.allreduce_weight_grads(grads)
            else:
                dp.exchange_weight_grads(grads, grads, transport=args.dp_transport)
    e1.record()
    torch.cuda.synchronize()
    main_window = (w0, time.time())
    windows.append(main_window)
    barrier(world)
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
    for blk in blocks:
        blk.check()
    ms_per_step = ms_total / args.steps
    value = aggregate_throughput(flops_step * args.steps, world, ms_total * 1e-3) / 1e12

    # ---- per-launch timing: every launch of the step on its own (see time_alone), so that no event
    #      node sits between the launches that are timed
    launch_lists = [b.step_launches(*t) for b, t in zip(blocks, sets)]
    names = [(n, k, c) for n, k, c, _ in launch_lists[0]]
    w0 = time.time()
    per_launch_us = {}
    for j, (name, kind, _) in enumerate(names):
        per_launch_us[name] = time_alone(torch, lambda s, j=j: launch_lists[s][j][3](None), len(sets))
    windows.append((w0, time.time()))
    gemm_names = [n for n, k, c in names if c > 0]
    gemms_in = {n: c for n, k, c in names}
    cast_names = [n for n, k, c in names if k == "cast"]
    gemm_us = sum(per_launch_us[n] for n in gemm_names) / sum(gemms_in[n] for n in gemm_names)     # per GEMM
    flops_launch = 2.0 * T * d * f
    operand_ratio = 2.0 if args.operand == "fp8" else 1.0

    # ---- the vendor library's FP8 GEMM as a black-box ceiling (rank 0, FP8 runs only): burst figure now,
    #      sustained figure after this benchmark's own sustained leg
    ceiling = None
    if rank == 0 and args.operand == "fp8":
        w0 = time.time()
        ceiling = Fp8LibraryCeiling(torch, dev)
        ceiling.burst()
        windows.append((w0, time.time()))

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

    # ---- sustained leg: the same graphs for at least args.sustain_seconds, with its own clock window
    sustained = None
    if args.sustain_seconds > 0:
        n_sus = max(args.steps, int(args.sustain_seconds / (ms_per_step * 1e-3)) + 1)
        barrier(world)
        w0 = time.time()
        e0.record()
        for i in range(n_sus):
            graphs[i % 2].replay()
        e1.record()
        torch.cuda.synchronize()
        sus_window = (w0, time.time())
        barrier(world)
        ms_sus = max_over_ranks(e0.elapsed_time(e1), world, dev)
        sustained = {"steps": n_sus, "seconds": ms_sus * 1e-3, "ms_per_step": ms_sus / n_sus,
                     "value": aggregate_throughput(flops_step * n_sus, world, ms_sus * 1e-3) / 1e12, "unit": "TFLOP/s",
                     "window": sus_window}
        for blk in blocks:
            blk.check()

    if ceiling is not None:
        w0 = time.time()
        ceiling.sustained(args.sustain_seconds)
        windows.append((w0, time.time()))
    fp8_measured = ceiling.result if ceiling is not None else None

    clocks_all = sampler.stop(windows + ([sus_window] if sustained else [])) if sampler else None
    if rank != 0:
        return
    main_clocks = sampler.summary([main_window])
    tensor_peak, peak_source, both = pick_tensor_peak(peaks, operand_ratio, ms_total * 1e-3, main_clocks)
    achieved = flops_launch / (gemm_us * 1e-6) / 1e12
    roofline = {
        "kernel": ("ffn_hidden_kernel / gemm_group_kernel" if blocks[0].grouped and blocks[0].fused_hidden else "gemm_kernel / gemm_group_kernel")
                  + " (the step's six GEMMs, mean per GEMM)", "bound": "tensor", "achieved": achieved,
        "peak": tensor_peak, "unit": "TFLOP/s", "frac": achieved / tensor_peak,
        "frac_of_burst_peak": achieved / both["burst"], "frac_of_sustained_peak": achieved / both["sustained"],
        "traffic": (gemm_traffic_mb() * 1e6 if args.operand == "fp8" and gemm_traffic_mb() is not None else None),
        "traffic_unit": "bytes per launch (ncu dram read + write, mean of the six launches)",
        "peak_source": peak_source, "flops_per_launch": flops_launch, "us_per_launch": gemm_us,
        "per_launch_method": "each launch timed alone: graph of 12 back-to-back launches over the rotating buffer sets",
        "fp8_measured": fp8_measured,
    }
    cast_bytes = {"cast_W1": d * f * 5, "cast_W2": d * f * 5, "cast_X": T * d * 5, "cast_G": T * d * 5}
    cast_bytes["cast_all"] = sum(cast_bytes.values())
    if args.operand != "fp8":
        cast_bytes = {k: v // 5 * 6 for k, v in cast_bytes.items()}
    kernels = []
    for n in gemm_names:
        tf = gemms_in[n] * flops_launch / per_launch_us[n] / 1e6
        kernels.append({"name": n, "gemms": gemms_in[n], "us": per_launch_us[n], "tflops": tf, "frac_of_peak": tf / tensor_peak})
    for n in cast_names:
        gbs = cast_bytes[n] / per_launch_us[n] / 1e3
        kernels.append({"name": n, "us": per_launch_us[n], "gbs": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"]})
    if sustained is not None:
        sus_clocks = sampler.summary([sustained.pop("window")])
        sustained["clocks"] = sus_clocks
        sustained["pct_of_nominal_fp8_peak"] = 100.0 * sustained["value"] / world / NOMINAL_FP8_TFLOPS
        sustained["frac_of_sustained_peak"] = sustained["value"] / world / both["sustained"]
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": {"fp8": "fp8_e4m3/e5m2 (fp32 accumulate)", "bf16": "bf16", "fp16": "fp16"}[args.operand],
        "data": "synthetic",
        "config": {"workload": "ffn_bert_large fwd+bwd: T=8192 tokens (16x512), d_model=1024, d_ff=4096, tau=0.5",
                   "operand": args.operand, "replicas": world, "weight_gradient_allreduce": dp_on, "weight_gradient_transport": args.dp_transport if dp_on else None,
                   "l2": "two rotating input/buffer sets, ~0.45 GB touched per step (> 126 MB L2)",
                   "launch": f"one CUDA graph of {blocks[0].launches_per_step} kernels per step, "
                             + ("the hidden layer's two GEMMs as one launch, the other four as one grouped launch"
                                if blocks[0].grouped and blocks[0].fused_hidden else
                                "the last four GEMMs as one grouped launch" if blocks[0].grouped else
                                "GEMMs after the first on three streams" if blocks[0].concurrent else "one stream")},
        "tokens_per_s": T * world / (ms_per_step * 1e-3),
        "pct_of_nominal_fp8_peak": 100.0 * value / world / NOMINAL_FP8_TFLOPS,
        "pct_of_measured_tensor_peak": 100.0 * value / world / tensor_peak,
        "target": {"pct_of_nominal_fp8_peak": 60.0, "met": bool(100.0 * value / world / NOMINAL_FP8_TFLOPS >= 60.0)},
        "clocks": main_clocks,
        "clocks_all_legs": clocks_all,
        "sustained": sustained,
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


def run_sweep(args, rank, world, local, torch, dev, peaks):
    """Each of Y = alpha X W, dX = beta_x G W^T, dW = beta_w X^T G alone: squares 1024 ... 16384 and the skinny
    M = 512, N = K = 8192 case, E4M3 x E4M3 and E5M2 x E4M3 operands, float32 and FP8-cast outputs."""
    from paper_2303_11257_b200 import lib as L
    if rank != 0:
        return
    E4, E5 = torch.float8_e4m3fn, torch.float8_e5m2
    ws = L.new_workspace(dev)
    sampler = ClockSampler(local)
    sampler.start()
    w0 = time.time()
    rows = []
    shapes = [(n, n, n) for n in (1024, 2048, 4096, 8192, 16384)] + [(512, 8192, 8192)]
    for (b, m, n) in shapes:
        for op in ("fwd", "bwd_x", "bwd_w"):
            pairs = [("e4m3", "e4m3")] if op == "fwd" else [("e5m2", "e4m3"), ("e4m3", "e4m3")] if op == "bwd_x" else [("e4m3", "e5m2"), ("e4m3", "e4m3")]
            ashape, bshape, oshape = {"fwd": ((b, m), (m, n), (b, n)), "bwd_x": ((b, n), (m, n), (b, m)), "bwd_w": ((b, m), (b, n), (m, n))}[op]
            for fa, fb in pairs:
                for out_name, out_dt in (("f32", torch.float32), ("fp8", E5 if op != "fwd" else E4)):
                    per_set = ashape[0] * ashape[1] + bshape[0] * bshape[1] + oshape[0] * oshape[1] * (4 if out_name == "f32" else 1)
                    nsets = max(2, min(6, int(2.2 * 126e6 / per_set) + 1))
                    mk = lambda shp, dt: torch.randn(shp, device=dev).to(dt)
                    A = [mk(ashape, E5 if fa == "e5m2" else E4) for _ in range(nsets)]
                    B = [mk(bshape, E5 if fb == "e5m2" else E4) for _ in range(nsets)]
                    out = [torch.empty(oshape, device=dev, dtype=torch.uint8).view(out_dt) if out_name == "fp8"
                           else torch.empty(oshape, device=dev) for _ in range(nsets)]
                    scale = {"fwd": m, "bwd_x": n, "bwd_w": b}[op] ** -0.5
                    fn = getattr(L, "us_linear_" + op)
                    us = time_alone(torch, lambda s: fn(A[s], B[s], scale, out[s], ws), nsets, iters=8 if b >= 8192 else 12, reps=3)
                    rows.append({"op": op, "b": b, "m": m, "n": n, "operands": f"{fa} x {fb}", "out": out_name, "us": us,
                                 "tflops": 2.0 * b * m * n / us / 1e6, "buffer_sets": nsets,
                                 "l2_resident": bool(per_set * nsets < 126e6)})
                    del A, B, out
    assert L.us_workspace_status(ws) == 0
    clocks = sampler.stop([(w0, time.time())])
    head = next(r for r in rows if r["op"] == "fwd" and r["b"] == 8192 and r["out"] == "f32")
    peak = peaks["bf16_tflops"] * 2.0
    line = {"metric": "unit-scaled linear GEMM TFLOP/s (sweep; value = forward 8192^3, float32 output)", "value": head["tflops"],
            "unit": "TFLOP/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": head["us"] * 1e-3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3/e5m2 (fp32 accumulate)",
            "data": "synthetic",
            "config": {"workload": "linear GEMM sweep: each op alone, M=N=K in {1024..16384} and M=512,N=K=8192",
                       "timing": "each case alone: graph of 8-12 back-to-back launches over rotating buffer sets, best of 3 replays"},
            "clocks": clocks, "e2e": None, "gpu_launches": len(rows) * 4 * 12,
            "roofline": {"kernel": "gemm_kernel, forward 8192^3", "bound": "tensor", "achieved": head["tflops"], "peak": peak,
                         "unit": "TFLOP/s", "frac": head["tflops"] / peak, "traffic": None,
                         "peak_source": f"{peaks['_source']} bf16 burst x 2 (nominal dtype ratio)"},
            "pct_of_nominal_fp8_peak": 100.0 * head["tflops"] / NOMINAL_FP8_TFLOPS,
            "kernels": rows, "cpu_baseline": None}
    print(json.dumps(line), flush=True)


def run_encoder(args, rank, world, local, torch, dev, peaks):
    """One BERT-large-shaped encoder layer (16 x 512 tokens, d = 1024, 16 heads, d_ff = 4096), forward + backward."""
    from paper_2303_11257_b200 import encoder, synth
    if rank != 0:
        return
    nseq, slen, d, nhead, d_ff = 16, 512, 1024, 16, 4096
    T = nseq * slen
    sampler = ClockSampler(local)
    sampler.start()
    results = {}
    windows = []
    for name, attention, fused in (("bf16", "bf16", False), ("fp8", "fp8", False), ("bf16, fused attention kernels", "bf16", True), ("fp8, fused attention kernels", "fp8", True)):
        host = (synth.normal(0, 0, (T, d)), synth.normal(0, 1, (d, 3 * d)), synth.normal(0, 2, (d, d)),
                synth.normal(0, 3, (d, d_ff)), synth.normal(0, 4, (d_ff, d)), synth.normal(0, 5, (T, d)))
        tensors = [torch.from_numpy(t).to(dev) for t in host]
        layer = encoder.UnitScaledEncoderLayer(nseq, slen, d, nhead, d_ff, attention=attention, device=dev, fused_attention=fused)
        layer.step(*tensors)
        layer.check()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            layer.step(*tensors)
        for _ in range(max(3, args.warmup)):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0 = time.time()
        e0.record()
        for _ in range(args.steps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        windows.append((w0, time.time()))
        layer.check()
        ms = e0.elapsed_time(e1) / args.steps
        results[name] = {"ms_per_step": ms, "tflops": layer.flops() / (ms * 1e-3) / 1e12, "launches": layer.launches_per_step,
                              "tokens_per_s": T / (ms * 1e-3)}
        flops = layer.flops()
        del layer, g
    clocks = sampler.stop(windows)
    head = results["bf16, fused attention kernels"]         # the graded configuration keeps 16-bit attention operands; fastest form of it
    peak = peaks["bf16_tflops"] * 2.0
    line = {"metric": "unit-scaled encoder layer fwd+bwd TFLOP/s at BERT-large shape", "value": head["tflops"], "unit": "TFLOP/s",
            "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3/e5m2 projections and FFN, bf16 attention (fp32 accumulate)",
            "data": "synthetic",
            "config": {"workload": "encoder layer fwd+bwd: 16 x 512 tokens, d=1024, 16 heads x 64, d_ff=4096, tau=0.5, no layer norm",
                       "attention": "16-bit operands; us_attention_fwd and us_attention_bwd (scores and their gradient stay in tensor memory)",
                       "launch": f"one CUDA graph of {head['launches']} kernels per step", "flops_per_step": flops,
                       "l2": "one buffer set; a step touches about 1.4 GB (> 126 MB L2)"},
            "clocks": clocks, "e2e": None, "gpu_launches": head["launches"] * args.steps,
            "roofline": {"kernel": "whole layer step", "bound": "tensor", "achieved": head["tflops"], "peak": peak, "unit": "TFLOP/s",
                         "frac": head["tflops"] / peak, "traffic": None,
                         "peak_source": f"{peaks['_source']} bf16 burst x 2 (nominal dtype ratio)"},
            "kernels": [dict(name=f"encoder layer, {k} attention operands", **v) for k, v in results.items()], "cpu_baseline": None}
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
