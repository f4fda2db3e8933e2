#!/usr/bin/env python
"""Benchmark of the tensorized-attention forward on B200 (tokens per second at 128k tokens).

One step = one whole forward pass (every hop of Algorithm 1) over one batch of synthetic
Llama-8B-shaped q, k, v: causal, B=1, H=32, H_kv=8, D=128, N=131072 viewed as 32x64x64, bf16.
Prints ONE JSON line (rank 0).  `value` is device-timed throughput with inputs resident in
HBM; `e2e` goes through ta_forward_host with pinned host buffers (copies inside the timed
region); `roofline` is the hop kernel against the measured HBM bandwidth; `cpu_baseline` is
the fp64 oracle on a bounded sample of the same workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 4]

With N > 1 (launched by torch.distributed.run) every rank runs the same workload on its own
GPU -- heads and batches are independent, so there is no data-path collective (weak scaling);
the step time is the max over ranks.  `--impl reference` times the CPU oracle instead (rank 0
only): it is a deliberately slow program, reported for context.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2410_20926_b200 import inputs as ta_inputs  # noqa: E402

METRIC = "tensorized_attention_forward_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per token per launch of the hop kernel, from
# the ncu capture of config 3 summarised in profiles/hop_pipe_kernel_config3_ncu_full.md
# (mean of the three hops, 758.8 MB for 32768 tokens); traffic is proportional to the tokens.
NCU_TRAFFIC_BYTES_PER_TOKEN_PER_LAUNCH = 757.9e6 / 32768


# ------------------------------------------------------------------ roofline arithmetic
def hop_bytes(cfg, hop_index: int) -> int:
    """Algorithmic HBM bytes of one hop: read Q (H heads), K (H_kv), the value tensor in
    (V with H_kv heads for the first hop, else H heads) and write the value tensor out (H)."""
    e = 2 if cfg.dtype == "bf16" else 4
    vin = cfg.H_kv if hop_index == 0 else cfg.H
    return e * cfg.B * cfg.N * cfg.D * (cfg.H + cfg.H_kv + vin + cfg.H)


def real_hops(cfg):
    return [i for i, n in enumerate(cfg.dims) if n > 1]


def step_bytes(cfg) -> int:
    return sum(hop_bytes(cfg, j) for j, _ in enumerate(real_hops(cfg)))


def step_flops(cfg, causal_useful: bool = True) -> float:
    f = 0.0
    for i in real_hops(cfg):
        n = cfg.dims[i]
        f += 4.0 * cfg.B * cfg.H * cfg.N * cfg.D * ((n + 1) / 2 if (cfg.causal and causal_useful) else n)
    return f


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json)", d
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s)", {}


# ------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        self.index = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ CPU oracle timing
def oracle_sample(cfg, inp, min_seconds: float = 0.0):
    """Times the fp64 oracle on ONE head of the workload (all N tokens, every hop) and scales
    to the whole batch: tokens/s = B*N / (t_head * B*H)."""
    import oracle
    t0 = time.perf_counter()
    reps = 0
    while True:
        oracle.forward(inp["q"], inp["k"], inp["v"], list(cfg.dims), cfg.causal, heads=[(0, reps % cfg.H)])
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds:
            break
    t_head = dt / reps
    value = cfg.B * cfg.N / (t_head * cfg.B * cfg.H)
    return {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{reps} single-head passes over the workload's heads (all {cfg.N} tokens, all hops; "
                      f"the batch has {cfg.B * cfg.H} heads), {dt:.1f} s, scaled to the batch"}, t_head


# ------------------------------------------------------------------ distributed plumbing
def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            import torch
            backend = "nccl" if torch.cuda.is_available() else "gloo"
            dist.init_process_group(backend=backend)
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float, world: int, device=None) -> float:
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate(tokens_per_rank: int, world: int, ms_max: float, steps: int) -> float:
    """Whole-job tokens/s: every rank processed `tokens_per_rank` tokens per step."""
    return tokens_per_rank * world * steps / (ms_max * 1e-3)


# ------------------------------------------------------------------ arms
def run_reference(args, cfg):
    rank, world, _ = dist_setup(args.gpus)
    if rank != 0:
        return
    inp = ta_inputs.make_config_inputs(cfg)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(cfg, inp)
    times = []
    info = None
    for _ in range(args.steps):
        info, t_head = oracle_sample(cfg, inp)
        times.append(t_head)
    t_head = sum(times) / len(times)
    value = cfg.B * cfg.N / (t_head * cfg.B * cfg.H)
    info["value"] = value
    info["sample"] = (f"each step = 1 of {cfg.B * cfg.H} heads of the workload (all {cfg.N} tokens, all hops), "
                      f"scaled to the batch; {len(times)} steps")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_head * cfg.B * cfg.H * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(cfg, world),
            "cpu_baseline": info,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_config(cfg, world):
    return {"workload": f"config {cfg.index}: causal fwd, B={cfg.B}, H={cfg.H}, H_kv={cfg.H_kv}, D={cfg.D}, "
                        f"N={cfg.N} as {'x'.join(map(str, cfg.dims))}, {cfg.dtype}, q/k/v ~ N(0,1) seeded",
            "B": cfg.B, "H": cfg.H, "H_kv": cfg.H_kv, "D": cfg.D, "N": cfg.N, "dims": list(cfg.dims),
            "causal": cfg.causal, "per_gpu_batch": cfg.B, "replicas": world,
            "l2": "inputs (%.2f GB per step) exceed the 126 MB L2; no flush needed" % (step_bytes(cfg) / 1e9)}


def run_ours(args, cfg):
    import torch
    import paper_2410_20926_b200 as ta

    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ta.load()

    inp = ta_inputs.make_config_inputs(cfg)
    host = {}
    for name in ("q", "k", "v"):
        t = torch.from_numpy(inp[name + "_bits"].view(np.int16)).view(torch.bfloat16)
        host[name] = t.pin_memory()
    host["out"] = torch.empty((cfg.B, cfg.H, cfg.N, cfg.D), dtype=torch.bfloat16).pin_memory()
    q, k, v = (host[n].to(dev, non_blocking=True) for n in ("q", "k", "v"))
    out = torch.empty((cfg.B, cfg.H, cfg.N, cfg.D), dtype=torch.bfloat16, device=dev)
    dims = list(cfg.dims)
    stream = torch.cuda.current_stream()

    def step():
        if args.rope_base > 0:
            ta.ta_forward_ex(q, k, v, out, cfg.B, cfg.H, cfg.H_kv, cfg.N, cfg.D, dims, cfg.causal,
                             rope_base=args.rope_base, stream=stream)
        else:
            ta.ta_forward(q, k, v, out, cfg.B, cfg.H, cfg.H_kv, cfg.N, cfg.D, dims, cfg.causal, stream=stream)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    ta.ta_device_status()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier(world)
    torch.cuda.synchronize()
    launches0 = ta.ta_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize()
    barrier(world)
    launches = ta.ta_launch_count() - launches0
    ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
    if rank == 0:
        time.sleep(0.2)
    clocks = sampler.stop() if rank == 0 else None
    ta.ta_device_status()
    value = aggregate(cfg.B * cfg.N, world, ms, args.steps)

    # ---- end to end: host buffers in, host buffer out, copies inside the timed region
    e2e_steps = max(1, min(args.steps, 10))
    for _ in range(2):
        ta.ta_forward_host(host["q"], host["k"], host["v"], host["out"], cfg.B, cfg.H, cfg.H_kv, cfg.N, cfg.D,
                           dims, cfg.causal, stream=stream)
    torch.cuda.synchronize()
    barrier(world)
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        ta.ta_forward_host(host["q"], host["k"], host["v"], host["out"], cfg.B, cfg.H, cfg.H_kv, cfg.N, cfg.D,
                           dims, cfg.causal, stream=stream)
    e1.record(stream)
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - t0) * 1e3
    e2e_ms = max_over_ranks(max(e0.elapsed_time(e1), wall_ms), world, dev)
    barrier(world)
    e2e_value = aggregate(cfg.B * cfg.N, world, e2e_ms, e2e_steps)
    h2d = sum(host[n].numel() * 2 for n in ("q", "k", "v"))
    d2h = host["out"].numel() * 2
    # the e2e result must be the same bits as the device-resident run (the host entry point
    # takes no positional encoding, so there is nothing to compare with --rope-base)
    same = bool(torch.equal(host["out"], out.cpu())) if args.rope_base == 0 else None

    if rank != 0:
        return
    # ---- roofline of the hop kernel (all launches of a step are the same kernel)
    peak, peak_src, _ = measured_peaks()
    n_launch = len(real_hops(cfg))
    bytes_per_launch = step_bytes(cfg) / n_launch
    launch_ms = ms / (args.steps * n_launch)
    achieved = bytes_per_launch / (launch_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC_BYTES_PER_TOKEN_PER_LAUNCH * cfg.B * cfg.N,
                "traffic_source": "ncu capture of config 3 scaled by tokens (profiles/)", "peak_source": peak_src,
                "kernel": "hop_pipe_kernel<128, false, false>", "algorithmic_bytes_per_launch": bytes_per_launch,
                "launches_per_step": n_launch, "avg_launch_ms": launch_ms,
                "useful_tflops": step_flops(cfg) / (ms / args.steps * 1e-3) / 1e12}
    cpu, _ = oracle_sample(cfg, inp, min_seconds=args.cpu_seconds)

    cfg_desc = workload_config(cfg, world)
    if args.rope_base > 0:
        cfg_desc["workload"] += f", tensorized positional encoding fused (RoPE base {args.rope_base:g})"
        cfg_desc["rope_base"] = args.rope_base
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": cfg_desc, "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps, "matches_device_run": same},
            "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4, help="workload: index into the five configurations")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="CPU time budget of the oracle sample")
    ap.add_argument("--rope-base", type=float, default=0.0,
                    help="> 0: time the forward with the fused tensorized positional encoding (not the "
                         "headline workload; device-timed value only)")
    args = ap.parse_args()
    cfg = ta_inputs.CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)
    try:
        import torch.distributed as dist
        if dist.is_available() and dist.is_initialized():
            dist.destroy_process_group()
    except Exception:
        pass


if __name__ == "__main__":
    main()
