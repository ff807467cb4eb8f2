#!/usr/bin/env python
"""Benchmark of the BRA forward hot path (pool -> route -> routed attention + LCE).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

A step is one `bra_forward` call on one batch of synthetic Q, K, V of the
BiFormer-T stage-1 shape (B=64, 56x56, C=64, 2 heads, S=7, topk=1, bf16; the
shape the headline metric is quoted on).  Prints ONE JSON line.

  value      queries/s (spatial tokens through the whole forward per second),
             inputs resident in HBM, timed with CUDA events, max over ranks
  e2e        same metric with Q, K, V copied from pinned host memory and O
             copied back inside the timed region of every step (copies and
             kernels of neighbouring steps overlap on three streams)
  roofline   dominant kernel (routed attention + LCE): algorithmic bytes of
             one launch / its mean duration from CUDA events, against the
             measured HBM copy bandwidth
  cpu_baseline  the fp64 CPU oracle timed on a bounded sample (rank 0, N=1)

`--impl reference` times the CPU oracle instead (the paper ships no code).
With N > 1 (torchrun) every rank runs its own batch: the path has no
collective in the forward pass (weak scaling).
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

METRIC = "BRA fwd queries/s per shape on 1 B200; % of HBM/tensor roofline"
UNIT = "queries/s"
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 1024 * 1024


FALLBACK_BF16_TFLOPS = 1590.0


def measured_peaks():
    """(HBM GB/s, dense bf16 TFLOP/s burst, 'measured' | 'fallback')."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops", FALLBACK_BF16_TFLOPS)), "measured"
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.lines = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ts, line in self.lines:
            if t0 is not None and not (t0 - 0.05 <= ts <= t1 + 0.1):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def oracle_sample(cfg, images: int, seed: int):
    """Time the CPU oracle's forward on the first `images` images of the workload."""
    from oracle import bra_oracle as orc
    from paper_2303_08810_b200 import synthetic
    small = synthetic.with_batch(cfg, images)
    x = synthetic.make_inputs(small, seed=seed)
    t0 = time.perf_counter()
    orc.bra_forward(x["Q"], x["K"], x["V"], x["w"], cfg.heads, cfg.S, cfg.topk)
    dt = time.perf_counter() - t0
    return small.B * small.N / dt, dt


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def run_reference(args, cfg):
    """The reference arm: the paper ships no code, so this is the CPU oracle as it stands."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    images = args.sample_images
    import numpy as np  # noqa: F401  (BLAS pools exist once numpy is loaded)
    for _ in range(args.warmup):
        oracle_sample(cfg, 1, 999)
    times = []
    for s in range(args.steps):
        qps, dt = oracle_sample(cfg, images, 2000 + s)
        times.append(dt)
    total = sum(times)
    value = args.steps * images * cfg.N / total
    sample = f"{images} of {cfg.B} images per step, oracle.bra_forward (fp64 NumPy)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(cfg, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(cfg, args, extra=None):
    c = {"workload": f"config {args.config}: {cfg.name}", "B": cfg.B, "H": cfg.H, "W": cfg.W,
         "C": cfg.C, "heads": cfg.heads, "S": cfg.S, "topk": cfg.topk, "io_dtype": cfg.dtype,
         "lce": "off" if getattr(args, "no_lce", False) else "5x5 depthwise fused",
         "parallelism": f"batch-sharded x{args.gpus}, no collective"}
    if extra:
        c.update(extra)
    return c


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", default="auto", choices=["auto", "simt", "mma", "tc", "img"])
    ap.add_argument("--sample-images", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-lce", action="store_true", help="attention term only (lce_ksize = 0)")
    args = ap.parse_args()

    from paper_2303_08810_b200 import synthetic
    cfg = synthetic.CONFIGS[args.config]
    if args.sample_images <= 0:
        # about 10-30 s of oracle time at ~10-20 k queries/s
        args.sample_images = max(1, min(cfg.B, 200_000 // cfg.N))
    if args.impl == "reference":
        if args.steps == 200:
            args.steps, args.warmup = 3, 1
        return run_reference(args, cfg)

    import numpy as np
    import torch
    import paper_2303_08810_b200 as bra

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    bra.load_library()

    impl = {"auto": 0, "simt": 1, "mma": 2, "tc": 3, "img": 4}[args.kernel]
    p = bra.make_problem(cfg.B, cfg.H, cfg.W, cfg.C, cfg.heads, cfg.S, cfg.topk, cfg.dtype, impl=impl,
                         lce=not args.no_lce)
    tdtype = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    esize = 2 if cfg.dtype == "bf16" else 4
    tensor_bytes = cfg.B * cfg.N * cfg.C * esize
    index_bytes = cfg.B * cfg.heads * cfg.R * cfg.topk * 4

    # rotate over enough input/output sets that a step never finds its inputs in L2
    nsets = max(2, -(-3 * L2_BYTES // (4 * tensor_bytes)))
    sets = []
    host = synthetic.make_inputs(cfg, seed=1000 + args.config + 97 * rank)
    w = torch.from_numpy(host["w"]).to(dev)
    for s in range(nsets):
        if s == 0:
            q, k, v = (torch.from_numpy(host[n]).to(dev).to(tdtype) for n in ("Q", "K", "V"))
        else:
            g = torch.Generator(device=dev)
            g.manual_seed(1234 + s + 131 * rank)
            q, k, v = (torch.randn(cfg.B, cfg.H, cfg.W, cfg.C, device=dev, generator=g).to(tdtype)
                       for _ in range(3))
        sets.append((q, k, v, torch.empty_like(q)))
    ws = bra.workspace(p, dev)
    index = torch.empty(cfg.B, p.heads_i, cfg.R, cfg.topk, dtype=torch.int32, device=dev)

    def step(i):
        q, k, v, o = sets[i % nsets]
        bra.bra_forward(p, q, k, v, w, None, O=o, index=index, ws=ws, want_lse=False)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    launches_per_step = bra.last_launch_count()
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    ev0.record()
    for i in range(args.steps):
        step(i)
    ev1.record()
    barrier()
    t_wall1 = time.time()
    ms = ev0.elapsed_time(ev1)

    # per-kernel split with the same launches: route and attend called one after the other
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    for i in range(args.steps):
        q, k, v, o = sets[i % nsets]
        evs[i][0].record()
        bra.bra_route(p, q, k, index=index, ws=ws, want_means=False)
        evs[i][1].record()
        bra.bra_attend(p, q, k, v, index, w, None, O=o, ws=ws, want_lse=False)
        evs[i][2].record()
    torch.cuda.synchronize()
    clocks = sampler.stop(t_wall0, time.time()) if rank == 0 else None
    route_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    attend_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps
    assert bra.bra_device_status(ws) == 0

    # end to end: pinned host -> device, forward, device -> host, every step.  Three streams and two
    # sets of device buffers, so that the copies of neighbouring steps overlap the kernels (PCIe moves
    # both ways at once); every copy of every step is inside the timed region.
    hq, hk, hv = (sets[0][j].cpu().pin_memory() for j in range(3))
    ho = [torch.empty_like(hq).pin_memory() for _ in range(2)]
    dbuf = [[torch.empty_like(sets[0][0]) for _ in range(4)] for _ in range(2)]     # q, k, v, o
    e2e_steps = max(3, min(args.steps, 20))
    s_in, s_run, s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
    ev_in = [torch.cuda.Event() for _ in range(2)]       # inputs of the buffer set have arrived
    ev_run = [torch.cuda.Event() for _ in range(2)]      # forward on the buffer set is done
    ev_out = [torch.cuda.Event() for _ in range(2)]      # its result has left the device

    def e2e_step(i):
        sel = i & 1
        dq, dk, dv, do = dbuf[sel]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_run[sel])                 # the forward two steps back has read these buffers
            dq.copy_(hq, non_blocking=True)
            dk.copy_(hk, non_blocking=True)
            dv.copy_(hv, non_blocking=True)
            ev_in[sel].record(s_in)
        with torch.cuda.stream(s_run):
            s_run.wait_event(ev_in[sel])
            s_run.wait_event(ev_out[sel])                # the result two steps back has been copied out
            bra.bra_forward(p, dq, dk, dv, w, None, O=do, index=index, ws=ws, want_lse=False)
            ev_run[sel].record(s_run)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_run[sel])
            ho[sel].copy_(do, non_blocking=True)
            ev_out[sel].record(s_out)

    torch.cuda.synchronize()
    for i in range(4):
        e2e_step(i)
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    s_in.wait_event(e0); s_run.wait_event(e0); s_out.wait_event(e0)
    for i in range(e2e_steps):
        e2e_step(i)
    cur = torch.cuda.current_stream()
    cur.wait_stream(s_in); cur.wait_stream(s_run); cur.wait_stream(s_out)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    # training configs: the backward pass for the fixed routing index, timed the same way
    bwd_ms = None
    if cfg.backward:
        q, k, v, o = sets[0]
        lse = torch.empty(cfg.B, cfg.heads, cfg.N, dtype=torch.float32, device=dev)
        bra.bra_forward(p, q, k, v, w, None, O=o, index=index, lse=lse, ws=ws)
        g = torch.Generator(device=dev)
        g.manual_seed(77 + rank)
        d_o = torch.randn(cfg.B, cfg.H, cfg.W, cfg.C, device=dev, generator=g).to(tdtype)
        grads = [torch.empty_like(q) for _ in range(3)]
        d_w = torch.empty(cfg.C, 5, 5, dtype=torch.float32, device=dev)
        bsteps = max(3, min(args.steps, 20))
        for _ in range(3):
            bra.bra_backward(p, q, k, v, index, w, lse, d_o, *grads, d_lce_w=d_w, ws=ws)
        bwd_launches = bra.last_launch_count()
        barrier()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record()
        for _ in range(bsteps):
            bra.bra_backward(p, q, k, v, index, w, lse, d_o, *grads, d_lce_w=d_w, ws=ws)
        b1.record()
        barrier()
        bwd_ms = b0.elapsed_time(b1) / bsteps
        assert bra.bra_device_status(ws) == 0

    from paper_2303_08810_b200 import sharding
    ms = sharding.max_over_ranks(ms, dev)
    e2e_ms = sharding.max_over_ranks(e2e_ms, dev)
    if bwd_ms is not None:
        bwd_ms = sharding.max_over_ranks(bwd_ms, dev)
    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    queries = cfg.B * cfg.N
    value = world * queries * args.steps / (ms * 1e-3)
    e2e_value = world * queries * e2e_steps / (e2e_ms * 1e-3)
    peak, peak_tf, peak_kind = measured_peaks()
    algo_bytes = 4 * tensor_bytes + index_bytes          # Q, K, V read + O written once, plus the index
    achieved = algo_bytes / (attend_ms * 1e-3) / 1e9
    fwd_achieved = algo_bytes / (ms / args.steps * 1e-3) / 1e9
    flops = 4.0 * cfg.B * cfg.N * cfg.topk * cfg.n_r * cfg.C
    def roofline_of(t_ms, kernel):
        # the slower of (minimum HBM bytes / bandwidth) and (routed-attention FLOPs / tensor peak) bounds the shape
        t_hbm, t_tensor = algo_bytes / (peak * 1e9), flops / (peak_tf * 1e12)
        if t_tensor > t_hbm:
            ach = flops / (t_ms * 1e-3) / 1e12
            return {"bound": "tensor", "kernel": kernel, "achieved": ach, "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": ach / peak_tf, "peak_kind": f"of {peak_kind} (burst)", "traffic": None,
                    "algorithmic_flops_per_launch": flops, "us_per_launch": 1e3 * t_ms}
        ach = algo_bytes / (t_ms * 1e-3) / 1e9
        return {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "peak_kind": f"of {peak_kind}", "traffic": None, "algorithmic_bytes_per_launch": algo_bytes,
                "us_per_launch": 1e3 * t_ms}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": workload_config(cfg, args, {
            "kernel": args.kernel,
            "l2": f"inputs larger than L2: rotating {nsets} input/output sets "
                  f"({nsets * 4 * tensor_bytes / 2**20:.0f} MiB > 126 MiB L2)"}),
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 3 * tensor_bytes,
                "d2h_bytes_per_step": tensor_bytes, "steps": e2e_steps},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline_of(attend_ms, "routed attention + LCE (bra_attend)"),
        "roofline_forward": {"bound": "hbm", "achieved": fwd_achieved, "peak": peak, "unit": "GB/s",
                             "frac": fwd_achieved / peak, "us_per_call": 1e3 * ms / args.steps,
                             "route_us": 1e3 * route_ms, "attend_us": 1e3 * attend_ms,
                             "routed_tflops": flops / (ms / args.steps * 1e-3) / 1e12},
    }
    if bwd_ms is not None:
        bwd_bytes = 7 * tensor_bytes + cfg.B * cfg.heads * cfg.N * 4 + index_bytes   # Q,K,V,dO in; dQ,dK,dV out; lse
        line["backward"] = {"us_per_call": 1e3 * bwd_ms, "gpu_launches_per_call": bwd_launches,
                            "algorithmic_bytes": bwd_bytes, "achieved_gbs": bwd_bytes / (bwd_ms * 1e-3) / 1e9,
                            "frac_of_hbm_peak": bwd_bytes / (bwd_ms * 1e-3) / 1e9 / peak,
                            "note": "fixed routing index; dQ, dK, dV, d_lce_w; L2 state as left by the previous call"}
    traffic_file = os.path.join(ROOT, "profiles", "attend_traffic.json")
    if os.path.exists(traffic_file):
        with open(traffic_file) as f:
            tr = json.load(f)
        line["roofline"]["traffic"] = tr.get(f"config{args.config}_{args.kernel}")
    if not args.no_cpu_baseline and world == 1:
        qps, dt = oracle_sample(cfg, args.sample_images, 1000 + args.config)
        line["cpu_baseline"] = {
            "value": qps, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"first {args.sample_images} of {cfg.B} images, one oracle.bra_forward call "
                      f"(fp64 NumPy, {dt:.1f} s)"}
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
