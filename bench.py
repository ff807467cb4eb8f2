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
             one launch / its mean duration from CUDA events (a loop of
             bra_attend calls), against the measured HBM copy bandwidth
  per_shape  the other benchmark shapes (configs 3, 4, 5 and the config-5
             backward) and the Appendix-D ViT-adaptation shape (config 6, head
             dim 64), timed in the same process
  cpu_baseline  the fp64 CPU oracle timed on a bounded sample (rank 0, N=1):
             one thread, and the same sample split over all host cores

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
    """Time the CPU oracle's forward on the first `images` images of the workload, in this
    process, on one thread (BLAS pools limited to 1)."""
    from oracle import bra_oracle as orc
    from paper_2303_08810_b200 import synthetic
    small = synthetic.with_batch(cfg, images)
    x = synthetic.make_inputs(small, seed=seed)
    try:
        from threadpoolctl import threadpool_limits
        limit = threadpool_limits(limits=1)
    except Exception:
        limit = None
    t0 = time.perf_counter()
    orc.bra_forward(x["Q"], x["K"], x["V"], x["w"], cfg.heads, cfg.S, cfg.topk)
    dt = time.perf_counter() - t0
    if limit is not None:
        limit.restore_original_limits()
    return small.B * small.N / dt, dt


def _oracle_worker(job):
    """One process of the all-cores leg: the oracle's forward on its share of the images."""
    config, images, seed = job
    from paper_2303_08810_b200 import synthetic
    qps, dt = oracle_sample(synthetic.CONFIGS[config], images, seed)
    return images * synthetic.CONFIGS[config].N, dt


def oracle_all_cores(config: int, images: int, seed: int):
    """The same oracle, the sample's images split over one process per host core."""
    import multiprocessing as mp
    procs = max(1, min(os.cpu_count() or 1, images))
    share = [images // procs + (1 if i < images % procs else 0) for i in range(procs)]
    jobs = [(config, n, seed + 10 * i) for i, n in enumerate(share) if n > 0]
    ctx = mp.get_context("spawn")
    t0 = time.perf_counter()
    with ctx.Pool(len(jobs)) as pool:
        done = pool.map(_oracle_worker, jobs)
    dt = time.perf_counter() - t0
    return sum(q for q, _ in done) / dt, dt, len(jobs)


def run_reference(args, cfg):
    """The reference arm: the paper ships no code, so this is the CPU oracle as it stands."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    images = args.sample_images
    for _ in range(args.warmup):
        oracle_sample(cfg, 1, 999)
    times = []
    for s in range(args.steps):
        qps, dt = oracle_sample(cfg, images, 2000 + s)
        times.append(dt)
    total = sum(times)
    value = args.steps * images * cfg.N / total
    sample = f"{images} of {cfg.B} images per step, oracle.bra_forward (fp64 NumPy), one process, one thread"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(cfg, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
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


IMPL = {"auto": 0, "simt": 1, "mma": 2, "tc": 3, "img": 4, "one-launch": 5}
NOMINAL_HBM_GBS = 8000.0


class Workload:
    """Device tensors of one benchmark config: enough rotating (Q, K, V, O) sets that a step never
    finds its inputs in L2, LCE weights, scratch, index."""

    def __init__(self, number, rank, dev, kernel="auto", lce=True, host_set=False):
        import torch
        import paper_2303_08810_b200 as bra
        from paper_2303_08810_b200 import synthetic
        self.bra, self.torch = bra, torch
        self.number, self.cfg = number, synthetic.CONFIGS[number]
        cfg = self.cfg
        self.p = bra.make_problem(cfg.B, cfg.H, cfg.W, cfg.C, cfg.heads, cfg.S, cfg.topk, cfg.dtype,
                                  impl=IMPL[kernel], lce=lce)
        self.tdtype = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
        esize = 2 if cfg.dtype == "bf16" else 4
        self.tensor_bytes = cfg.B * cfg.N * cfg.C * esize
        self.index_bytes = cfg.B * cfg.heads * cfg.R * cfg.topk * 4
        self.algo_bytes = 4 * self.tensor_bytes + self.index_bytes      # Q, K, V read + O written once, plus the index
        self.flops = 4.0 * cfg.B * cfg.N * cfg.topk * cfg.n_r * cfg.C    # routed attention, 2 flops per MAC
        self.nsets = max(2, -(-3 * L2_BYTES // (4 * self.tensor_bytes)))
        self.sets = []
        g = torch.Generator(device=dev)
        for s in range(self.nsets):
            if s == 0 and host_set:
                host = synthetic.make_inputs(cfg, seed=1000 + number + 97 * rank)
                q, k, v = (torch.from_numpy(host[n]).to(dev).to(self.tdtype) for n in ("Q", "K", "V"))
                self.w = torch.from_numpy(host["w"]).to(dev)
            else:
                g.manual_seed(1234 + s + 131 * rank + 7 * number)
                q, k, v = (torch.randn(cfg.B, cfg.H, cfg.W, cfg.C, device=dev, generator=g).to(self.tdtype)
                           for _ in range(3))
            self.sets.append((q, k, v, torch.empty_like(q)))
        if not host_set:
            g.manual_seed(99 + number)
            self.w = 0.02 * torch.randn(cfg.C, 5, 5, device=dev, generator=g)
        self.ws = bra.workspace(self.p, dev)
        self.index = torch.empty(cfg.B, self.p.heads_i, cfg.R, cfg.topk, dtype=torch.int32, device=dev)
        self.dev = dev

    def forward(self, i):
        q, k, v, o = self.sets[i % self.nsets]
        self.bra.bra_forward(self.p, q, k, v, self.w, None, O=o, index=self.index, ws=self.ws, want_lse=False)

    def route(self, i):
        q, k, _, _ = self.sets[i % self.nsets]
        self.bra.bra_route(self.p, q, k, index=self.index, ws=self.ws, want_means=False)

    def attend(self, i):
        q, k, v, o = self.sets[i % self.nsets]
        self.bra.bra_attend(self.p, q, k, v, self.index, self.w, None, O=o, ws=self.ws, want_lse=False)

    def loop_ms(self, fn, steps):
        """Device time of `steps` back-to-back calls, CUDA events on the launching stream."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            fn(i)
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1)

    def bound(self, peak_gbs, peak_tf):
        t_hbm, t_tensor = self.algo_bytes / (peak_gbs * 1e9), self.flops / (peak_tf * 1e12)
        return ("tensor", t_tensor) if t_tensor > t_hbm else ("hbm", t_hbm)

    def backward_setup(self, rank):
        torch, cfg, bra = self.torch, self.cfg, self.bra
        q, k, v, o = self.sets[0]
        self.lse = torch.empty(cfg.B, cfg.heads, cfg.N, dtype=torch.float32, device=self.dev)
        bra.bra_forward(self.p, q, k, v, self.w, None, O=o, index=self.index, lse=self.lse, ws=self.ws)
        g = torch.Generator(device=self.dev)
        g.manual_seed(77 + rank)
        self.d_o = torch.randn(cfg.B, cfg.H, cfg.W, cfg.C, device=self.dev, generator=g).to(self.tdtype)
        self.grads = [torch.empty_like(q) for _ in range(3)]
        self.d_w = torch.empty(cfg.C, 5, 5, dtype=torch.float32, device=self.dev)
        self.bwd_bytes = 7 * self.tensor_bytes + cfg.B * cfg.heads * cfg.N * 4 + self.index_bytes

    def backward(self, i):
        q, k, v, _ = self.sets[0]
        self.bra.bra_backward(self.p, q, k, v, self.index, self.w, self.lse, self.d_o, *self.grads,
                              d_lce_w=self.d_w, ws=self.ws)


def shape_report(wl, steps, reps, peak, peak_tf, peak_kind, rank):
    """Forward (and backward for training configs) of one more shape: median over `reps` loops."""
    for i in range(5):
        wl.forward(i)
    ms = statistics.median(wl.loop_ms(wl.forward, steps) for _ in range(reps)) / steps
    kind, t_bound = wl.bound(peak, peak_tf)
    cfg = wl.cfg
    out = {"workload": f"config {wl.number}: {cfg.name}", "us_per_call": 1e3 * ms,
           "queries_per_s": cfg.B * cfg.N / (ms * 1e-3), "bound": kind,
           "roofline_frac": t_bound / (ms * 1e-3), "peak_kind": f"of {peak_kind}",
           "gpu_launches_per_call": wl.bra.last_launch_count()}
    if cfg.backward:
        wl.backward_setup(rank)
        for i in range(3):
            wl.backward(i)
        bms = statistics.median(wl.loop_ms(wl.backward, max(3, steps // 2)) for _ in range(reps)) / max(3, steps // 2)
        out["backward"] = {"us_per_call": 1e3 * bms, "gpu_launches_per_call": wl.bra.last_launch_count(),
                           "algorithmic_bytes": wl.bwd_bytes,
                           "frac_of_hbm_peak": wl.bwd_bytes / (bms * 1e-3) / 1e9 / peak}
    assert wl.bra.bra_device_status(wl.ws) == 0
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", default="auto", choices=sorted(IMPL))
    ap.add_argument("--reps", type=int, default=5, help="repetitions of the timed loop; the headline is their median")
    ap.add_argument("--sample-images", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-shape", action="store_true", help="skip the other benchmark shapes")
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
    peak, peak_tf, peak_kind = measured_peaks()

    wl = Workload(args.config, rank, dev, kernel=args.kernel, lce=not args.no_lce, host_set=True)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        wl.forward(i)
    launches_per_step = bra.last_launch_count()
    barrier()

    # ---- the timed region: EXACTLY --steps forward calls, bracketed by barrier + synchronize ----
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    barrier()
    t_wall0 = time.time()
    ms = wl.loop_ms(wl.forward, args.steps)
    barrier()
    # repetitions of the same loop (same steps): the headline value is the median, less noisy than one loop
    rep_ms = [ms] + [wl.loop_ms(wl.forward, args.steps) for _ in range(max(0, args.reps - 1))]
    # per-kernel split: loops of the two halves of the forward, each back to back on the same stream
    wl.route(0)
    route_ms = wl.loop_ms(wl.route, args.steps) / args.steps
    attend_ms = wl.loop_ms(wl.attend, args.steps) / args.steps
    torch.cuda.synchronize()
    clocks = sampler.stop(t_wall0, time.time()) if rank == 0 else None
    assert bra.bra_device_status(wl.ws) == 0

    # ---- end to end: pinned host -> device, forward, device -> host, every step.  Three streams and two
    # sets of device buffers, so that the copies of neighbouring steps overlap the kernels (PCIe moves
    # both ways at once); every copy of every step is inside the timed region.
    hq, hk, hv = (wl.sets[0][j].cpu().pin_memory() for j in range(3))
    ho = [torch.empty_like(hq).pin_memory() for _ in range(2)]
    dbuf = [[torch.empty_like(wl.sets[0][0]) for _ in range(4)] for _ in range(2)]     # q, k, v, o
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
            bra.bra_forward(wl.p, dq, dk, dv, wl.w, None, O=do, index=wl.index, ws=wl.ws, want_lse=False)
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
    del dbuf, ho, hq, hk, hv

    # ---- training configs: the backward pass for the fixed routing index, timed the same way ----
    bwd_ms = None
    if cfg.backward:
        wl.backward_setup(rank)
        bsteps = max(3, min(args.steps, 20))
        for i in range(3):
            wl.backward(i)
        bwd_launches = bra.last_launch_count()
        barrier()
        bwd_ms = wl.loop_ms(wl.backward, bsteps) / bsteps
        barrier()
        assert bra.bra_device_status(wl.ws) == 0

    # ---- the other shapes of the metric ("per shape"), same process, rank 0 ----
    per_shape = None
    if not args.no_per_shape and args.config == 2 and rank == 0:
        per_shape = []
        for number in (3, 4, 5, 6):
            other = Workload(number, rank, dev)
            per_shape.append(shape_report(other, 50, 3, peak, peak_tf, peak_kind, rank))
            del other
            torch.cuda.empty_cache()

    from paper_2303_08810_b200 import sharding
    ms = sharding.max_over_ranks(ms, dev)
    med_ms = sharding.max_over_ranks(statistics.median(rep_ms), dev)
    e2e_ms = sharding.max_over_ranks(e2e_ms, dev)
    if bwd_ms is not None:
        bwd_ms = sharding.max_over_ranks(bwd_ms, dev)
    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    queries = cfg.B * cfg.N
    step_ms = med_ms / args.steps                      # median loop: the headline
    value = world * queries / (step_ms * 1e-3)
    e2e_value = world * queries * e2e_steps / (e2e_ms * 1e-3)
    algo_bytes, flops = wl.algo_bytes, wl.flops
    kind, _ = wl.bound(peak, peak_tf)

    def roofline_of(t_ms, kernel):
        # the slower of (minimum HBM bytes / bandwidth) and (routed-attention FLOPs / tensor peak) bounds the shape
        if kind == "tensor":
            ach = flops / (t_ms * 1e-3) / 1e12
            return {"bound": "tensor", "kernel": kernel, "achieved": ach, "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": ach / peak_tf, "peak_kind": f"of {peak_kind} (burst)", "traffic": None,
                    "algorithmic_flops_per_launch": flops, "us_per_launch": 1e3 * t_ms}
        ach = algo_bytes / (t_ms * 1e-3) / 1e9
        return {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
                "peak_kind": f"of {peak_kind}", "traffic": None, "algorithmic_bytes_per_launch": algo_bytes,
                "us_per_launch": 1e3 * t_ms}

    fwd_achieved = algo_bytes / (step_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": workload_config(cfg, args, {
            "kernel": args.kernel,
            "l2": f"inputs larger than L2: rotating {wl.nsets} input/output sets "
                  f"({wl.nsets * 4 * wl.tensor_bytes / 2**20:.0f} MiB > 126 MiB L2)"}),
        "clocks": clocks,
        "timing": {"first_loop_ms_per_step": ms / args.steps, "loops": len(rep_ms),
                   "loops_ms_per_step": [m / args.steps for m in rep_ms],
                   "note": "value and ms_per_step are the median over the loops of --steps calls"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 3 * wl.tensor_bytes,
                "d2h_bytes_per_step": wl.tensor_bytes, "steps": e2e_steps},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline_of(attend_ms, "routed attention + LCE (bra_attend)"),
        "roofline_forward": {"bound": "hbm", "achieved": fwd_achieved, "peak": peak, "unit": "GB/s",
                             "frac": fwd_achieved / peak, "frac_of_nominal_8TBs": fwd_achieved / NOMINAL_HBM_GBS,
                             "us_per_call": 1e3 * step_ms,
                             "route_us": 1e3 * route_ms, "attend_us": 1e3 * attend_ms,
                             "routed_tflops": flops / (step_ms * 1e-3) / 1e12},
    }
    if bwd_ms is not None:
        line["backward"] = {"us_per_call": 1e3 * bwd_ms, "gpu_launches_per_call": bwd_launches,
                            "algorithmic_bytes": wl.bwd_bytes, "achieved_gbs": wl.bwd_bytes / (bwd_ms * 1e-3) / 1e9,
                            "frac_of_hbm_peak": wl.bwd_bytes / (bwd_ms * 1e-3) / 1e9 / peak,
                            "note": "fixed routing index; dQ, dK, dV, d_lce_w; L2 state as left by the previous call"}
    if per_shape is not None:
        line["per_shape"] = per_shape
    traffic_file = os.path.join(ROOT, "profiles", "attend_traffic.json")
    if os.path.exists(traffic_file):
        with open(traffic_file) as f:
            tr = json.load(f)
        line["roofline"]["traffic"] = tr.get(f"config{args.config}_{args.kernel}")
    if not args.no_cpu_baseline and world == 1:
        # about 10 s of oracle time: calls on the sample's images until then (at most 8 calls)
        calls, spent = 0, 0.0
        while calls < 8 and spent < 10.0:
            _, dt = oracle_sample(cfg, args.sample_images, 1000 + args.config + calls)
            calls, spent = calls + 1, spent + dt
        qps = calls * args.sample_images * cfg.N / spent
        line["cpu_baseline"] = {
            "value": qps, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{calls} oracle.bra_forward calls on {args.sample_images} of {cfg.B} images each "
                      f"(fp64 NumPy, one process, one thread, {spent:.1f} s)"}
        try:
            qps_all, dt_all, procs = oracle_all_cores(args.config, args.sample_images, 1000 + args.config)
            line["cpu_baseline"]["all_cores"] = {
                "value": qps_all, "unit": UNIT, "cores": procs,
                "sample": f"the same {args.sample_images} images split over {procs} processes ({dt_all:.1f} s wall)"}
        except Exception as exc:                          # the single-thread figure stands on its own
            line["cpu_baseline"]["all_cores"] = {"unavailable": repr(exc)[:200]}
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
