#!/usr/bin/env python
"""Benchmark of the LOT attention forward hot path (costs, two Sinkhorn solves, apply).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--n 16384]

A step is one lot_attention_fwd_ex call over one batch of synthetic input of the headline
workload (B=1 per GPU, H=16, n=16384, d=64, r=64, bf16, eps=0.1, T=10).  `value` is tokens/s
(B*n per call, all ranks) with inputs resident in HBM; `e2e` is the same call fed from pinned
host buffers with the host<->device copies inside the timed region.  L2 is flushed between
timed steps (a 512 MiB buffer is overwritten) and each step is timed with its own CUDA event
pair on the launching stream, so the flush is outside the timed span.

`--impl reference` times the float64 CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "lot_attn_fwd_tokens_per_s"
UNIT = "tokens/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--n", type=int, default=16384)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--iters", type=int, default=None,
                    help="Sinkhorn iterations (default: the configuration's 10); for profiling single phases, e.g. 0 = apply passes only")
    args = ap.parse_args()
    global ITERS
    ITERS = args.iters
    return args


ITERS = None


def workload(n, rank=0):
    from paper_2509_23436_b200 import synth
    return synth.config(4, n=n, variant=rank, iters=ITERS)


def algorithmic_bytes(B, H, n, d, r, s_in, s_out):
    """Compulsory HBM bytes of one forward call: Q, K, V read once, out written once, Z and beta."""
    return B * H * n * d * (3 * s_in + s_out) + H * r * (d + 1) * 4


# --------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while running."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, cuda_index):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(cuda_index).uuid)
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                bits = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.004)

    def finish(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


# --------------------------------------------------------------------------- CPU oracle timing
def time_oracle(x, reps, threads=0):
    """Best wall time of `reps` runs of the oracle over the whole workload; returns (seconds, threads)."""
    from oracle import lot_oracle as O
    d = x.f64()
    best, used = None, 0
    for _ in range(reps):
        t0 = time.perf_counter()
        _, _, _, used = O.attention_fwd(d["q"], d["k"], d["v"], d["z"], d["beta"], x.eps, x.iters,
                                        key_len=d["key_len"], threads=threads, return_potentials=True)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best, used


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    x = workload(args.n)
    B, H, n, d, r = x.shape
    # one step = the oracle over a bounded sample of the workload: as many heads as keep a step ~1 s
    heads = H if n <= 16384 else max(1, H * 16384 // n)
    from paper_2509_23436_b200 import synth
    xs = synth.config(4, n=n, H=heads)
    for _ in range(min(args.warmup, 1)):
        time_oracle(xs, 1)
    steps = max(1, min(args.steps, 5))
    t0 = time.perf_counter()
    used = 0
    for _ in range(steps):
        _, used = time_oracle(xs, 1)
    dt = (time.perf_counter() - t0) / steps
    # tokens/s of the full workload = B*n tokens per (all H heads); a step covered heads/H of it
    val = B * n / (dt * H / heads)
    sample = f"{heads} of {H} heads of cfg4 n={n} per step, {steps} steps, float64"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3 * H / heads,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": x.name, "B": B, "H": H, "n": n, "d": d, "r": r, "eps": x.eps, "iters": x.iters},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- our arm

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2509_23436_b200 import binding as lot

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    x = workload(args.n, rank)
    B, H, n, d, r = x.shape
    q, k, v = x.q.to(dev), x.k.to(dev), x.v.to(dev)
    z, beta = x.z.to(dev), x.beta.to(dev)
    out = torch.empty_like(q)
    code = lot.LOT_BF16 if q.dtype == torch.bfloat16 else lot.LOT_F32
    ws = torch.empty(lot.lot_workspace_bytes(B, H, n, d, r, code), device=dev, dtype=torch.uint8)
    flush = torch.empty(512 << 20, device=dev, dtype=torch.uint8)
    stream = torch.cuda.current_stream()

    def step():
        lot.lot_attention_fwd_ex(q, k, v, z, beta, None, x.eps, x.iters, out=out, ws=ws, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        flush.fill_(1)
        step()
    barrier()
    if lot.lot_device_status(ws) != 0:
        raise SystemExit("device status flagged during warm-up")

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for a, b in evs:
        flush.fill_(0)
        a.record(stream)
        step()
        b.record(stream)
    barrier()
    clocks = sampler.finish() if sampler else None
    times = [a.elapsed_time(b) for a, b in evs]           # ms
    total_ms = float(sum(times))
    if world > 1:
        tt = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())
    ms_per_step = total_ms / args.steps
    tokens_per_step = B * n * world
    value = tokens_per_step / (ms_per_step * 1e-3)

    # ---- end to end: pinned host buffers in, host buffer out, copies inside the timed region
    hq, hk, hv = x.q.pin_memory(), x.k.pin_memory(), x.v.pin_memory()
    hz, hb = x.z.pin_memory(), x.beta.pin_memory()
    hout = torch.empty_like(x.q).pin_memory()

    def e2e_step():
        q.copy_(hq, non_blocking=True); k.copy_(hk, non_blocking=True); v.copy_(hv, non_blocking=True)
        z.copy_(hz, non_blocking=True); beta.copy_(hb, non_blocking=True)
        step()
        hout.copy_(out, non_blocking=True)

    e2e_steps = max(3, min(args.steps, 30))
    for _ in range(3):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    if world > 1:
        tt = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        e2e_ms = float(tt.item())
    e2e_val = tokens_per_step * e2e_steps / (e2e_ms * 1e-3)
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hz, hb))
    d2h = hout.numel() * hout.element_size()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the call (all its kernels together): algorithmic bytes = Q, K, V read once, out written once, pivots
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = 6650.0, "fallback"
    s_el = q.element_size()
    fused = lot.lot_launch_count(code, d, r, x.iters) == 2
    abytes = algorithmic_bytes(B, H, n, d, r, s_el, s_el)
    per_call_ms = sum(times) / len(times)
    achieved = abytes / (per_call_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": 251.2e6 if (n == 16384 and fused and ITERS is None) else None, "peak_source": peak_src,
                "algorithmic_bytes": abytes,
                "kernel": "fused_forward_kernel (persistent; the call is this kernel plus a 3 us pivot preparation)"
                          if fused else "whole lot_attention_fwd_ex call (all launches)"}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        secs, used = time_oracle(workload(args.n), 3)
        cpu = {"value": B * n / secs, "unit": UNIT, "cores": used, "kind": "oracle",
               "sample": f"whole workload ({H} heads, n={n}), best of 3 runs, float64"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32" , "data": "synthetic",
            "config": {"workload": x.name, "B_per_gpu": B, "H": H, "n": n, "d": d, "r": r, "eps": x.eps,
                       "iters": x.iters, "tensor_dtype": str(q.dtype).replace("torch.", ""),
                       "l2": "flushed between timed steps (512 MiB overwrite)",
                       "parallelism": f"independent batches x{world}"},
            "clocks": clocks, "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d,
                                      "d2h_bytes_per_step": d2h},
            "gpu_launches": lot.lot_launch_count(code, d, r, x.iters) * args.steps,
            "roofline": roofline, "cpu_baseline": cpu,
            "ms_per_step_min": min(times), "ms_per_step_median": sorted(times)[len(times) // 2]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
