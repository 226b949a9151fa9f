#!/usr/bin/env python
"""Benchmark of the LOT attention forward hot path (costs, two Sinkhorn solves, apply).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg2|cfg3|cfg4|cfg5] [--n N] [--r R] [--iters T] [--eps E] [--dtype bf16|f32]
                    [--shard batch|heads]

A step is one lot_attention_fwd_ex call over one batch of synthetic input.  The default workload is the
headline one (config 4: B=1 per GPU, H=16, n=16384, d=64, r=64, bf16, eps=0.1, T=10); the other
configurations are reachable with --workload and keep their own shapes unless overridden.  `value` is
tokens/s (B*n per call, all ranks) with inputs resident in HBM; `e2e` is the same call fed from pinned
host buffers with the host<->device copies inside the timed region.  L2 is flushed between timed steps
(a 512 MiB buffer is overwritten) and each step is timed with its own CUDA event pair on the launching
stream, so the flush is outside the timed span.

With N > 1 ranks, `--shard batch` (default) gives every rank its own batch of the workload (weak
scaling); `--shard heads` splits the (batch, head) slices of ONE workload over the ranks through
paper_2509_23436_b200.shard (strong scaling).  Neither has a data-path collective.

`--impl reference` times the float64 CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import hashlib
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
CFG = {"cfg2": 2, "cfg3": 3, "cfg4": 4, "cfg5": 5}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(CFG))
    ap.add_argument("--n", type=int, default=None)
    ap.add_argument("--r", type=int, default=None)
    ap.add_argument("--B", type=int, default=None)
    ap.add_argument("--eps", type=float, default=None)
    ap.add_argument("--dtype", default=None, choices=["bf16", "f32"])
    ap.add_argument("--shard", default="batch", choices=["batch", "heads"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--path", default="auto", choices=["auto", "general", "streamed", "resident"],
                    help="kernel path the library takes where it can run (default: the library's own choice)")
    ap.add_argument("--op", default="fwd", choices=["fwd", "bwd"],
                    help="bwd: time lot_attention_bwd (gradients of q, k, v, z, beta; one GPU) instead of the forward")
    ap.add_argument("--iters", type=int, default=None,
                    help="Sinkhorn iterations (default: the configuration's); 0 = apply passes only")
    return ap.parse_args()


def workload(args, variant=0, **over):
    import torch
    from paper_2509_23436_b200 import synth
    dt = {None: None, "bf16": torch.bfloat16, "f32": torch.float32}[args.dtype]
    kw = dict(dtype=dt, n=args.n, r=args.r, iters=args.iters, eps=args.eps, B=args.B, variant=variant)
    kw.update(over)
    return synth.config(CFG[args.workload], **kw)


def algorithmic_bytes(B, H, n, d, r, s_in, s_out, masked):
    """Compulsory HBM bytes of one forward call: Q, K, V read once, out written once, Z, beta, key lengths."""
    return B * H * n * d * (3 * s_in + s_out) + H * r * (d + 1) * 4 + (B * 4 if masked else 0)


def source_digest():
    """Digest of the CUDA sources: a stored DRAM-traffic figure only describes the kernel it was taken from."""
    h = hashlib.sha256()
    src = os.path.join(ROOT, "paper_2509_23436_b200", "csrc")
    for name in sorted(os.listdir(src)):
        with open(os.path.join(src, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()[:16]


def stored_traffic(key):
    """DRAM bytes per call of the dominant kernel from profiles/traffic.json (written beside the ncu summary it
    comes from), or None when there is no entry for this workload or the sources have changed since."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None, None
    ent = json.load(open(path)).get(key)
    if not ent or ent.get("source_digest") != source_digest():
        return None, None
    return float(ent["dram_bytes_per_call"]), ent.get("summary")


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
ORACLE_SEC_PER_ENTRY = 7e-8      # float64 oracle, one core: seconds per (token, pivot) entry and pass, order of magnitude


def oracle_sample(x, budget_s=15.0):
    """A bounded sample of workload x for the CPU oracle: the first `heads` heads of the first `batch` batch rows,
    sized so that one run takes about budget_s on the host cores.  Returns (inputs dict, slices, total slices)."""
    B, H, n, d, r = x.shape
    cores = os.cpu_count() or 1
    per_slice = 2.0 * n * (r * (x.iters + 2) + 2 * d * r) * ORACLE_SEC_PER_ENTRY
    want = max(1, min(B * H, int(cores * max(1.0, budget_s / max(per_slice, 1e-9)))))
    heads = min(H, want)
    batch = max(1, min(B, want // heads))
    f = x.f64()
    kl = None if f["key_len"] is None else f["key_len"][:batch]
    sub = dict(q=f["q"][:batch, :heads], k=f["k"][:batch, :heads], v=f["v"][:batch, :heads], z=f["z"][:heads],
               beta=f["beta"][:heads], key_len=kl)
    return sub, batch * heads, B * H


def time_oracle(sub, x, reps, threads=0):
    """Best wall time of `reps` runs of the oracle over the sample; returns (seconds, threads used)."""
    import numpy as np
    from oracle import lot_oracle as O
    c = np.ascontiguousarray
    best, used = None, 0
    for _ in range(reps):
        t0 = time.perf_counter()
        _, _, _, used = O.attention_fwd(c(sub["q"]), c(sub["k"]), c(sub["v"]), sub["z"], sub["beta"], x.eps, x.iters,
                                        key_len=sub["key_len"], threads=threads, return_potentials=True)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best, used


def config_of(x, extra=None):
    B, H, n, d, r = x.shape
    c = {"workload": x.name, "B": B, "H": H, "n": n, "d": d, "r": r, "eps": x.eps, "iters": x.iters,
         "tensor_dtype": str(x.q.dtype).replace("torch.", ""), "key_mask": x.key_len is not None}
    c.update(extra or {})
    return c


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    x = workload(args)
    B, H, n, d, r = x.shape
    sub, ns, total = oracle_sample(x, budget_s=8.0)
    warm = min(args.warmup, 1)
    for _ in range(warm):
        time_oracle(sub, x, 1)
    steps = max(1, min(args.steps, 5))
    t0 = time.perf_counter()
    used = 0
    for _ in range(steps):
        _, used = time_oracle(sub, x, 1)
    dt = (time.perf_counter() - t0) / steps
    # tokens/s of the full workload: B*n tokens per pass over all slices; a step covered ns of the total slices
    full_s = dt * total / ns
    val = B * n / full_s
    sample = f"{ns} of {total} (batch, head) slices of {x.name} per step, {steps} steps, float64"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": full_s * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(x),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- our arm
PATH_NAMES = {0: "general path (cost, T+1 Sinkhorn passes, two apply kernels)",
              1: "fused_forward_kernel (persistent, Gibbs kernel streamed from L2; plus the pivot preparation)",
              2: "resident_forward_kernel (persistent, Gibbs kernel resident in shared memory and TMEM)",
              3: "slice_forward_kernel (one thread block per slice, logits and Gibbs kernel in float32 registers)"}
ARITH = {0: {"bfloat16": "f32", "float32": "f64"},
         1: {"bfloat16": "bf16 operands, f32 accumulate, bf16 stored Gibbs kernel"},
         2: {"bfloat16": "bf16 operands, f32 accumulate, bf16 resident Gibbs kernel"},
         3: {"bfloat16": "bf16 operands, f32 accumulate, f32 Gibbs kernel in registers"}}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2509_23436_b200 import binding as lot
    from paper_2509_23436_b200 import shard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "WARN")
        dist.init_process_group("nccl", device_id=dev)

    if args.shard == "heads" and world > 1:
        # one workload for the whole job; this rank takes its rectangle of (batch, head) slices
        x = workload(args)
        gB, gH, n, d, r = x.shape
        blk, qs, ks, vs, zs, bs, kl = shard.shard_inputs(x.q, x.k, x.v, x.z, x.beta, x.key_len, world, rank)
        hq, hk, hv, hz, hb = (t.contiguous() for t in (qs, ks, vs, zs, bs))
        hkl = None if kl is None else kl.contiguous()
        tokens_per_step = gB * n
        scaling, par = "strong", f"(batch, head) slices of one workload split over {world} ranks"
    else:
        x = workload(args, variant=rank)
        gB, gH, n, d, r = x.shape
        hq, hk, hv, hz, hb, hkl = x.q, x.k, x.v, x.z, x.beta, x.key_len
        tokens_per_step = gB * n * world
        scaling, par = "weak", f"independent batches x{world}"
    B, H = hq.shape[0], hq.shape[1]
    empty = B == 0 or H == 0
    q, k, v, z, beta = (t.to(dev) for t in (hq, hk, hv, hz, hb))
    key_len = None if hkl is None else hkl.to(dev)
    out = torch.empty_like(q)
    code = lot.LOT_BF16 if q.dtype == torch.bfloat16 else lot.LOT_F32
    if args.path != "auto":          # before the workspace is sized: its size follows the path
        lot.lot_debug_hook(4, {"general": 0, "streamed": 1, "resident": 2}[args.path])
    ws = torch.empty(max(256, lot.lot_workspace_bytes(B, H, n, d, r, code)), device=dev, dtype=torch.uint8)
    flush = torch.empty(512 << 20, device=dev, dtype=torch.uint8)
    stream = torch.cuda.current_stream()

    def step():
        if not empty:
            lot.lot_attention_fwd_ex(q, k, v, z, beta, key_len, x.eps, x.iters, out=out, ws=ws, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warm = max(args.warmup, 3)
    for _ in range(warm):
        flush.fill_(1)
        step()
    barrier()
    if not empty and lot.lot_device_status(ws) != 0:
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
    value = tokens_per_step / (ms_per_step * 1e-3)

    # ---- end to end: pinned host buffers in, host buffer out, copies inside the timed region
    pq, pk, pv, pz, pb = (t.pin_memory() for t in (hq, hk, hv, hz, hb))
    pkl = None if hkl is None else hkl.pin_memory()
    hout = torch.empty_like(hq).pin_memory()

    def e2e_step():
        q.copy_(pq, non_blocking=True); k.copy_(pk, non_blocking=True); v.copy_(pv, non_blocking=True)
        z.copy_(pz, non_blocking=True); beta.copy_(pb, non_blocking=True)
        if pkl is not None:
            key_len.copy_(pkl, non_blocking=True)
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
    h2d = sum(t.numel() * t.element_size() for t in (pq, pk, pv, pz, pb)) + (0 if pkl is None else pkl.numel() * 4)
    d2h = hout.numel() * hout.element_size()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the call: algorithmic bytes = Q, K, V read once, out written once, pivots, key lengths
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = 6650.0, "fallback"
    s_el = q.element_size()
    path = lot.lot_path(code, B, H, n, d, r, x.iters)
    tdt = str(q.dtype).replace("torch.", "")
    abytes = algorithmic_bytes(B, H, n, d, r, s_el, s_el, key_len is not None)
    per_call_ms = sum(times) / len(times)
    achieved = abytes / (per_call_ms * 1e-3) / 1e9
    traffic, traffic_src = stored_traffic(f"{args.workload}:{tdt}:B{B}:H{H}:n{n}:d{d}:r{r}:T{x.iters}")
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "traffic_source": traffic_src, "peak_source": peak_src,
                "algorithmic_bytes": abytes, "kernel": PATH_NAMES.get(path, "?"),
                "note": "achieved = algorithmic bytes / CUDA-event time of the whole call (every launch of it)"}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        sub, ns, total = oracle_sample(x)
        secs, used = time_oracle(sub, x, 2)
        cpu = {"value": gB * n / (secs * total / ns), "unit": UNIT, "cores": used, "kind": "oracle",
               "sample": f"{ns} of {total} (batch, head) slices of {x.name}, best of 2 runs, float64, scaled to all slices"}

    launches = lot.lot_launch_count(code, B, H, n, d, r, x.iters)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": scaling, "vs_baseline": None, "dtype": ARITH.get(path, {}).get(tdt, tdt), "data": "synthetic",
            "config": config_of(x, {"B_per_gpu": B, "H_per_gpu": H,
                                    "l2": "flushed between timed steps (512 MiB overwrite)", "parallelism": par}),
            "clocks": clocks, "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d,
                                      "d2h_bytes_per_step": d2h},
            "gpu_launches": launches * args.steps,
            "roofline": roofline, "cpu_baseline": cpu,
            "ms_per_step_min": min(times), "ms_per_step_median": sorted(times)[len(times) // 2]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_backward(args):
    """The backward pass (Section "Learning") timed like the forward: CUDA events, L2 flushed between steps."""
    import torch
    from paper_2509_23436_b200 import binding as lot
    from paper_2509_23436_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    x = workload(args)
    B, H, n, d, r = x.shape
    q, k, v, z, beta = (t.to(dev) for t in (x.q, x.k, x.v, x.z, x.beta))
    key_len = None if x.key_len is None else x.key_len.to(dev)
    dout = synth.cotangent(x).to(dev)
    code = lot.LOT_BF16 if q.dtype == torch.bfloat16 else lot.LOT_F32
    ws = torch.empty(max(256, lot.lot_bwd_workspace_bytes(B, H, n, d, r, code, x.iters)), device=dev, dtype=torch.uint8)
    out = torch.empty_like(q)
    fws = torch.empty(max(256, lot.lot_workspace_bytes(B, H, n, d, r, code)), device=dev, dtype=torch.uint8)
    flush = torch.empty(512 << 20, device=dev, dtype=torch.uint8)
    stream = torch.cuda.current_stream()

    def bwd():
        lot.lot_attention_bwd(q, k, v, z, beta, key_len, dout, x.eps, x.iters, ws=ws, stream=stream)

    def fwd():
        lot.lot_attention_fwd_ex(q, k, v, z, beta, key_len, x.eps, x.iters, out=out, ws=fws, stream=stream)

    def timed(fn, steps):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        torch.cuda.synchronize()
        for a, b in evs:
            flush.fill_(0)
            a.record(stream)
            fn()
            b.record(stream)
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    warm = max(args.warmup, 3)
    for _ in range(warm):
        flush.fill_(1)
        bwd()
        fwd()
    torch.cuda.synchronize()
    if lot.lot_device_status(ws) != 0:
        raise SystemExit("device status flagged during warm-up")
    sampler = ClockSampler(0)
    sampler.start()
    tb = timed(bwd, args.steps)
    clocks = sampler.finish()
    tf = timed(fwd, args.steps)
    ms = sum(tb) / len(tb)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = 6650.0, "fallback"
    s_el = q.element_size()
    abytes = B * H * n * d * 7 * s_el + 2 * H * r * (d + 1) * 4 + (B * 4 if key_len is not None else 0)
    achieved = abytes / (ms * 1e-3) / 1e9
    tdt = str(q.dtype).replace("torch.", "")
    line = {"metric": "lot_attn_bwd_tokens_per_s", "value": B * n / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": ARITH[0][tdt], "data": "synthetic",
            "config": config_of(x, {"l2": "flushed between timed steps (512 MiB overwrite)",
                                    "op": "backward (forward recomputed inside, materialised similarities)"}),
            "clocks": clocks, "gpu_launches": (2 * x.iters + 15) * args.steps,
            "forward_ms_per_step": sum(tf) / len(tf), "backward_over_forward": ms / (sum(tf) / len(tf)),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": None, "peak_source": peak_src, "algorithmic_bytes": abytes,
                         "note": "q, k, v, dout read once; dq, dk, dv written once; z, beta, dz, dbeta"}}
    print(json.dumps(line), flush=True)


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    elif args.op == "bwd":
        run_backward(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
