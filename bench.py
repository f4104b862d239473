#!/usr/bin/env python
"""Benchmark of the TWA subspace step on B200.

One "step" is one fused subspace iteration (project the gradient, update the
coefficients, lift the weights) through the C-ABI call twa_step on a basis built and
quantised by the library from synthetic correlated candidates; the basis build and the
quantisation are timed once and reported beside the step throughput.

    python bench.py --gpus N --steps K --warmup W [--workload vitb16] [--bits 8]
    python bench.py --impl reference ...     # the float64 CPU oracle on a bounded sample

Prints one JSON line (rank 0).  With N > 1 every rank runs an independent replica of the
workload on its own GPU (the path has no exchange step); value is the sum over ranks.
"""

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "twa_fused_step_GBps_int8"
UNIT = "GB/s"


def step_bytes(D, n, bits, g_bytes):
    """Algorithmic bytes of one fused step: P~ read by the projection and again by the lift,
    g read once, w_bar read once, w written once."""
    p = n * ((D * bits + 7) // 8)
    return 2 * p + D * g_bytes + 4 * D + 4 * D


def kernel_bytes(D, n, bits, g_bytes):
    p = n * ((D * bits + 7) // 8)
    return {"project": p + D * g_bytes, "lift": p + 8 * D}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def read_traffic(key):
    """DRAM bytes per launch from profiles/traffic.md, or None when there is no entry or the
    kernel sources changed since the counters were taken."""
    import hashlib
    import re
    path = os.path.join(ROOT, "profiles", "traffic.md")
    if not os.path.exists(path):
        return None
    h = hashlib.sha256()
    for name in ("twa_stream_mma.cu", "twa_mma.cuh", "twa_common.cuh"):
        with open(os.path.join(ROOT, "paper_2205_13104_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    digest = h.hexdigest()[:16]
    with open(path) as f:
        for line in f:
            m = re.match(r"^(\S+) = (\d+) \| ([0-9a-f]{16})\s*$", line)
            if m and m.group(1) == key:
                return int(m.group(2)) if m.group(3) == digest else None
    return None


def max_over_ranks(values, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group):
    a job is as slow as its slowest replica."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_gbps(world, bytes_per_step_per_rank, ms_per_step):
    """Throughput of the whole job: every rank runs its own replica of the workload (the path has
    no exchange step), so the bytes add up and the time is the slowest rank's."""
    return world * bytes_per_step_per_rank / (ms_per_step * 1e-3) / 1e9


class ClockSampler:
    """nvidia-smi samples of one GPU's clocks and throttle reasons while a region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 8:
                    continue
                try:
                    sm.append(float(parts[0]))
                    mx.append(float(parts[1]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[4:8]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "samples": len(sm),
                "reasons": sorted(reasons)}


def oracle_sample_run(wl, bits, sample_rows, steps, warmup):
    """The float64 oracle's fused step on the first `sample_rows` rows of the workload
    (candidates -> float32 basis by the oracle's CGS2 is NOT timed; only the step is)."""
    import numpy as np
    import torch
    from oracle import twa_oracle as orc
    from paper_2205_13104_b200 import inputs
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = 1
    D, n = sample_rows, wl.n
    rng = np.random.default_rng(0)
    # a random orthonormal-scale basis is enough for timing: the oracle's cost does not depend on values
    P32 = (rng.standard_normal((n, D)) / np.sqrt(D)).astype(np.float32).T
    codes, s = orc.quantize(P32, bits)
    wbar = rng.standard_normal(D).astype(np.float32)
    alpha = np.zeros(n)
    gdt = torch.bfloat16 if wl.g_dtype == "bf16" else torch.float32
    times = []
    for t in range(warmup + steps):
        g = inputs.gradient(D, wl.g_std, wl.seed, t, gdt, "cpu").float().numpy()
        t0 = time.perf_counter()
        alpha, w, c = orc.step(codes, s, g, alpha, wbar, 0.1, 0.0)
        dt = time.perf_counter() - t0
        if t >= warmup:
            times.append(dt)
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    gbps = step_bytes(D, n, bits, g_bytes) / (sum(times) / len(times)) / 1e9
    return gbps, cores, sum(times) / len(times)


def run_reference(args):
    from paper_2205_13104_b200 import inputs
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = inputs.WORKLOADS[args.workload]
    sample_rows = min(wl.D, args.reference_rows)
    gbps, cores, sec = oracle_sample_run(wl, args.bits, sample_rows, args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbps, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3 * wl.D / sample_rows,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": f"{wl.name}: D={wl.D} n={wl.n} int{args.bits} P, {wl.g_dtype} g",
                   "sample": f"first {sample_rows} rows of D; ms_per_step scaled to full D"},
        "cpu_baseline": {"value": gbps, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"fused step on the first {sample_rows} of {wl.D} rows, all {wl.n} columns"},
        "e2e": {"value": gbps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2205_13104_b200 import inputs, twa

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    twa.load()
    wl = inputs.WORKLOADS[args.workload]
    import dataclasses
    if args.rows:
        wl = dataclasses.replace(wl, name=f"{wl.name}[rows={args.rows}]", D=args.rows)
    D, n, bits = wl.D, wl.n, args.bits
    gdt = torch.bfloat16 if wl.g_dtype == "bf16" else torch.float32
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    ctx = twa.twa_create(local)
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_DEQUANT_PATH, args.dequant_path)
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_LIFT_VECTORS, args.lift_vectors)
    ws = twa.new_workspace(dev)

    # ---- basis build and quantisation, timed once each -------------------------------
    wbar = torch.empty(D, dtype=torch.float32, device=dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    if args.random_basis:
        wl = dataclasses.replace(wl, chunked_build=False)
        # profiling aid: skip the Gram-Schmidt launches; the step kernels do the same work on any values
        W = torch.randn((n, inputs.padded_ld(D, 128)), device=dev) / (D ** 0.5)
        twa.twa_mean(ctx, W, D, wbar)
        torch.cuda.synchronize()
        ev[0].record()
        P32 = twa.basis_from_tensor(W, D)
    elif wl.chunked_build:
        # The candidates (4*n*D bytes) do not fit beside P~: every row chunk is regenerated from
        # its seed once per pass and fed to the chunked build.  Library time = CUDA events around
        # the feed calls only; generating the chunks is not counted.
        if bits == 32:
            raise SystemExit("the chunked workload has no resident float32 basis; use --bits 8 or 4")
        bws = torch.empty(twa.twa_build_workspace_bytes(n), dtype=torch.uint8, device=dev)
        Pq = twa.new_quantised_basis(D, n, bits, dev)
        buf = torch.empty((n, inputs.CHUNK_ROWS), dtype=torch.float32, device=dev)
        pairs = []
        twa.twa_build_begin(ctx, D, n, wbar, bws)
        for p in range(4):
            for r0 in range(0, D, inputs.CHUNK_ROWS):
                rows = min(inputs.CHUNK_ROWS, D - r0)
                inputs.trajectory_rows(D, n, wl.step, wl.drift, wl.seed, dev, row0=r0, rows=rows,
                                       out=buf[:, :rows])
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                twa.twa_build_feed(ctx, p, buf, r0, rows, Pq=Pq if p == 3 else None)
                if r0 + rows == D:
                    twa.twa_build_end_pass(ctx, p, bits if p == 2 else 0, Pq if p == 2 else None)
                b.record()
                pairs.append((a, b))
        torch.cuda.synchronize()
        build_ms, quant_ms = sum(a.elapsed_time(b) for a, b in pairs), 0.0
        del buf, bws, pairs
        W = P32 = None
    else:
        W = wl.candidates(dev, ld=inputs.padded_ld(D, 128))
        torch.cuda.synchronize()
        ev[0].record()
        P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
    if not wl.chunked_build or args.random_basis:
        ev[1].record()
        Pq = twa.twa_quantize_basis(ctx, P32, bits, ws) if bits != 32 else P32
        ev[2].record()
        torch.cuda.synchronize()
        build_ms, quant_ms = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"basis build failed: {twa.twa_strerror(code)} column {detail}")
    if bits != 32:
        del W, P32
        torch.cuda.empty_cache()

    # ---- per-step inputs: a pool of distinct gradients, cycled ------------------------
    g_pool = args.g_pool if D * g_bytes * args.g_pool <= 8e9 else max(2, int(8e9 // (D * g_bytes)))
    pool = [wl.gradient(t, dev) for t in range(g_pool)]
    alpha = torch.zeros(n, dtype=torch.float32, device=dev)
    w = torch.empty(D, dtype=torch.float32, device=dev)
    lr, lam = 0.1, 0.0

    def step(t):
        twa.twa_step(ctx, Pq, pool[t % len(pool)], lr, lam, alpha, wbar, w, ws)

    for t in range(args.warmup):
        step(t)
    barrier()
    twa.twa_profile_enable(ctx, args.steps)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for t in range(args.steps):
        step(args.warmup + t)
    e1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = e0.elapsed_time(e1)
    proj_ms, lift_ms, rec = twa.twa_profile_read(ctx)
    twa.twa_profile_enable(ctx, 0)
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"step failed: {twa.twa_strerror(code)}")

    # ---- end to end: gradient from pinned host memory, weights back to the host --------
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    g_host = [p.cpu().pin_memory() for p in pool[:2]]
    w_host = torch.empty(D, dtype=torch.float32).pin_memory()
    g_stage = torch.empty(D, dtype=gdt, device=dev)
    alpha2 = torch.zeros(n, dtype=torch.float32, device=dev)
    for t in range(2):
        twa.twa_step_host(ctx, Pq, g_host[t % 2], lr, lam, alpha2, wbar, w, w_host, g_stage, ws)
    barrier()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for t in range(e2e_steps):
        twa.twa_step_host(ctx, Pq, g_host[t % 2], lr, lam, alpha2, wbar, w, w_host, g_stage, ws)
    t1.record()
    barrier()
    e2e_ms = t0.elapsed_time(t1) / e2e_steps

    # ---- max over ranks ------------------------------------------------------------------
    total_ms, e2e_ms, proj_ms, lift_ms, build_ms, quant_ms = max_over_ranks(
        [total_ms, e2e_ms, proj_ms, lift_ms, build_ms, quant_ms], dev)

    if rank == 0:
        peak, peak_kind = load_peaks()
        sb = step_bytes(D, n, bits, g_bytes)
        kb = kernel_bytes(D, n, bits, g_bytes)
        ms_per_step = total_ms / args.steps
        value = whole_job_gbps(world, sb, ms_per_step)
        suffix = "_mma" if args.dequant_path == 0 and bits != 32 else ""
        dom = "project" if proj_ms >= lift_ms else "lift"
        dom_ms = (proj_ms if dom == "project" else lift_ms) / max(rec, 1)
        achieved = kb[dom] / (dom_ms * 1e-3) / 1e9
        other = "lift" if dom == "project" else "project"
        other_ms = (lift_ms if dom == "project" else proj_ms) / max(rec, 1)
        traffic = read_traffic(f"{wl.name}_int{bits}_{dom}") if args.dequant_path == 0 else None
        # CPU baseline: the oracle on a bounded sample (rank 0, N = 1 only)
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            rows = min(D, args.reference_rows)
            gbps, cores, sec = oracle_sample_run(wl, bits if bits != 32 else 8, rows, 2, 1)
            cpu = {"value": gbps, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"fused step on the first {rows} of {D} rows, all {n} columns, 2 timed steps"}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{wl.name}: D={D} n={n} int{bits} P, {wl.g_dtype} g, lr={lr} lambda={lam}",
                       "l2": f"inputs larger than L2: P~ is {n * ((D * bits + 7) // 8) / 1e6:.0f} MB per pass",
                       "gradients": f"{len(pool)} distinct gradients generated before the timed region, cycled",
                       "dequant_path": "tensor-pipe integer dot products" if args.dequant_path == 0 else "float32 FMA",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "bytes_per_step": sb,
            "frac_of_hbm_peak": value / world / peak,
            "frac_of_8TBps": value / world / 8000.0,
            "basis_build_ms": None if args.random_basis else build_ms,
            "quantize_ms": None if wl.chunked_build else quant_ms,
            "basis_build": ("row-chunked Gram-form build incl. quantisation, 4 passes, chunk generation not counted"
                            if wl.chunked_build else "resident classical Gram-Schmidt with re-orthogonalisation"),
            "roofline": {"bound": "hbm", "kernel": f"twa_{dom}{suffix}_kernel", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "traffic": traffic, "bytes_per_launch": kb[dom], "ms_per_launch": dom_ms,
                         "other_kernel": {"kernel": f"twa_{other}{suffix}_kernel", "ms_per_launch": other_ms,
                                          "achieved": kb[other] / (other_ms * 1e-3) / 1e9,
                                          "bytes_per_launch": kb[other]}},
            "cpu_baseline": cpu,
            "e2e": {"value": world * sb / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
                    "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "h2d_bytes_per_step": D * g_bytes, "d2h_bytes_per_step": 4 * D},
            "gpu_launches": 2 * args.steps,
            "clocks": clocks,
        }
        print(json.dumps(line))
    twa.twa_destroy(ctx)
    if world > 1:
        dist.destroy_process_group()


def run_layered(args):
    """The paper's default construction: per-layer centred and normalised basis, per-layer affine
    B-bit codes, layer-wise step (one coefficient vector per layer)."""
    import dataclasses
    import torch
    import torch.distributed as dist
    from paper_2205_13104_b200 import inputs, twa

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    twa.load()
    wl = inputs.WORKLOADS[args.workload]
    if args.bits == 32:
        raise SystemExit("the layer-wise step runs on 8- or 4-bit codes")
    layers = inputs.layer_offsets(args.workload, args.rows or None)
    if args.rows:
        wl = dataclasses.replace(wl, name=f"{wl.name}[rows={args.rows}]", D=args.rows)
    D, n, bits, L = wl.D, wl.n, args.bits, len(layers) - 1
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    ctx = twa.twa_create(local)
    wbar = torch.empty(D, dtype=torch.float32, device=dev)
    lws = twa.new_layered_workspace(layers, n, dev)
    chunked = wl.chunked_build and not args.rows
    if chunked:
        # The candidates do not fit beside P~: every row chunk is regenerated from its seed once per
        # pass and fed to the row-chunked build.  Library time = CUDA events around the feed calls.
        lb = twa.twa_layered_build_begin(ctx, D, n, layers, bits, lws, dev)
        buf = torch.empty((n, inputs.CHUNK_ROWS), dtype=torch.float32, device=dev)
        pairs = []
        for p in range(3):
            for r0 in range(0, D, inputs.CHUNK_ROWS):
                rows = min(inputs.CHUNK_ROWS, D - r0)
                inputs.trajectory_rows(D, n, wl.step, wl.drift, wl.seed, dev, row0=r0, rows=rows, out=buf[:, :rows])
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                twa.twa_layered_build_feed(ctx, lb, p, buf, r0, rows, wbar, lws)
                if r0 + rows == D:
                    twa.twa_layered_build_end_pass(ctx, lb, p, lws)
                b.record()
                pairs.append((a, b))
        torch.cuda.synchronize()
        build_ms, quant_ms = sum(a.elapsed_time(b) for a, b in pairs), 0.0
        del buf, pairs
    else:
        W = wl.candidates(dev, ld=inputs.padded_ld(D, 128))
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        torch.cuda.synchronize()
        ev[0].record()
        P32 = twa.twa_build_centered(ctx, W, D, layers, wbar, lws)
        ev[1].record()
        lb = twa.twa_quantize_affine(ctx, P32, layers, bits, lws)
        ev[2].record()
        torch.cuda.synchronize()
        build_ms, quant_ms = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])
        del W, P32
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"layer-wise build failed: {twa.twa_strerror(code)} layer {detail}")
    torch.cuda.empty_cache()

    g_pool = args.g_pool if D * g_bytes * args.g_pool <= 8e9 else max(2, int(8e9 // (D * g_bytes)))
    pool = [wl.gradient(t, dev) for t in range(g_pool)]
    beta = torch.zeros((L, n), dtype=torch.float32, device=dev)
    c = torch.empty((L, n), dtype=torch.float32, device=dev)
    w = torch.empty(D, dtype=torch.float32, device=dev)
    sws = twa.new_layered_step_workspace(lb)
    lr, lam = 0.1, 0.0

    def timed(fn, steps):
        for t in range(args.warmup):
            fn(t)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for t in range(steps):
            fn(args.warmup + t)
        e1.record()
        barrier()
        return e0.elapsed_time(e1)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    total_ms = timed(lambda t: twa.twa_layered_step(ctx, lb, pool[t % len(pool)], lr, lam, beta, wbar, w, sws),
                     args.steps)
    clocks = sampler.stop() if rank == 0 else None
    # the two streaming launches apart (each call also runs its small per-layer kernel)
    part_steps = max(1, args.steps // 4)
    proj_ms = timed(lambda t: twa.twa_layered_project(ctx, lb, pool[t % len(pool)], c, sws), part_steps) / part_steps
    lift_ms = timed(lambda t: twa.twa_layered_lift(ctx, lb, beta, wbar, w, sws), part_steps) / part_steps
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"layer-wise step failed: {twa.twa_strerror(code)} layer {detail}")
    total_ms, proj_ms, lift_ms, build_ms, quant_ms = max_over_ranks(
        [total_ms, proj_ms, lift_ms, build_ms, quant_ms], dev)
    if rank == 0:
        peak, peak_kind = load_peaks()
        sb = step_bytes(D, n, bits, g_bytes)
        kb = kernel_bytes(D, n, bits, g_bytes)
        ms_per_step = total_ms / args.steps
        value = whole_job_gbps(world, sb, ms_per_step)
        dom = "project" if proj_ms >= lift_ms else "lift"
        dom_ms = proj_ms if dom == "project" else lift_ms
        line = {
            "metric": METRIC.replace("int8", f"int{bits}") + "_layerwise", "value": value, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{wl.name}: D={D} n={n} L={L} layers, per-layer affine int{bits} P, "
                                   f"{wl.g_dtype} g, lr={lr} lambda={lam}",
                       "l2": f"inputs larger than L2: P~ is {n * ((D * bits + 7) // 8) / 1e6:.0f} MB per pass",
                       "gradients": f"{len(pool)} distinct gradients generated before the timed region, cycled",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "bytes_per_step": sb,
            "frac_of_hbm_peak": value / world / peak,
            "frac_of_8TBps": value / world / 8000.0,
            "basis_build_ms": build_ms, "quantize_ms": quant_ms,
            "basis_build": ("row-chunked: mean + norms, min-max, codes in three fed passes, chunk generation not counted"
                            if chunked else "per-layer centring and normalisation of the candidates, per-layer min-max codes"),
            "roofline": {"bound": "hbm", "kernel": f"layered_{dom}_kernel", "achieved": kb[dom] / (dom_ms * 1e-3) / 1e9,
                         "peak": peak, "unit": "GB/s", "frac": kb[dom] / (dom_ms * 1e-3) / 1e9 / peak,
                         "peak_kind": f"of {peak_kind}", "traffic": None, "bytes_per_launch": kb[dom],
                         "ms_per_launch": dom_ms, "timing": "separate loop of that call alone",
                         "project_ms": proj_ms, "lift_ms": lift_ms},
            "cpu_baseline": None,
            "gpu_launches": 4 * args.steps,
            "clocks": clocks,
        }
        print(json.dumps(line))
    twa.twa_destroy(ctx)
    if world > 1:
        dist.destroy_process_group()


def run_project_batch(args):
    """Projection of --project-batch gradients per call (P~ read once per group) beside the same
    number of single-gradient calls, on the workload's column shape; D may be cut with --rows."""
    import dataclasses
    import torch
    from paper_2205_13104_b200 import inputs, twa

    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    twa.load()
    wl = inputs.WORKLOADS[args.workload]
    if args.rows:
        wl = dataclasses.replace(wl, name=f"{wl.name}[rows={args.rows}]", D=args.rows)
    D, n, bits, B = wl.D, wl.n, args.bits, args.project_batch
    gdt = torch.bfloat16 if wl.g_dtype == "bf16" else torch.float32
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    ctx = twa.twa_create(0)
    ws = twa.new_workspace(dev)
    # the projection does the same work on any values: codes of a random matrix
    if 4 * n * D > 120e9:
        raise SystemExit("the float32 matrix to quantise does not fit: cut D with --rows")
    W = torch.randn((n, inputs.padded_ld(D, 128)), device=dev) / (D ** 0.5)
    Pq = twa.twa_quantize_basis(ctx, twa.basis_from_tensor(W, D), bits, ws)
    del W
    torch.cuda.empty_cache()
    ld = inputs.padded_ld(D, 8)
    G = torch.empty((B, ld), dtype=gdt, device=dev)
    for b in range(B):
        G[b, :D] = wl.gradient(b, dev)
    C = torch.empty((B, n), dtype=torch.float32, device=dev)
    c1 = torch.empty(n, dtype=torch.float32, device=dev)

    def timed(fn):
        for _ in range(args.warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    def singles():
        for b in range(B):
            twa.twa_project(ctx, Pq, G[b, :D], c1, ws)

    sampler = ClockSampler(0)
    sampler.start()
    batch_ms = timed(lambda: twa.twa_project_batch(ctx, Pq, G, C, ws))
    clocks = sampler.stop()
    single_ms = timed(singles)
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"projection failed: {twa.twa_strerror(code)} {detail}")
    group = twa.twa_project_batch_group(ctx, Pq, gdt)
    p_bytes = n * ((D * bits + 7) // 8)
    moved = -(-B // group) * p_bytes + B * D * g_bytes
    peak, peak_kind = load_peaks()
    print(json.dumps({
        "metric": f"twa_project_batch_gradients_per_s_int{bits}", "value": B / (batch_ms * 1e-3), "unit": "gradients/s",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": batch_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{wl.name}: D={D} n={n} int{bits} P, {wl.g_dtype} g, {B} gradients per call, "
                               f"groups of {group}", "l2": f"inputs larger than L2: P~ is {p_bytes / 1e6:.0f} MB"},
        "single_calls_ms": single_ms, "speedup_over_single_calls": single_ms / batch_ms,
        "roofline": {"bound": "hbm", "kernel": "twa_project_batch_kernel", "achieved": moved / (batch_ms * 1e-3) / 1e9,
                     "peak": peak, "unit": "GB/s", "frac": moved / (batch_ms * 1e-3) / 1e9 / peak,
                     "peak_kind": f"of {peak_kind}", "traffic": None, "bytes_per_launch": moved // -(-B // group)},
        "cpu_baseline": None, "gpu_launches": -(-B // group) * args.steps, "clocks": clocks}))
    twa.twa_destroy(ctx)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vitb16")
    ap.add_argument("--bits", type=int, default=8, choices=[32, 8, 4])
    ap.add_argument("--g-pool", type=int, default=8)
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--reference-rows", type=int, default=1 << 21)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--lift-vectors", type=int, default=0, choices=[0, 1, 2, 3],
                    help="TWA_TUNE_LIFT_VECTORS: how base and output travel in the 8/4-bit lift (0 = built-in choice)")
    ap.add_argument("--dequant-path", type=int, default=0, choices=[0, 1],
                    help="0: integer dot products on the tensor pipe (default); 1: float32 FMA path")
    ap.add_argument("--rows", type=int, default=0, help="override D (smaller cases for profiler captures)")
    ap.add_argument("--random-basis", action="store_true",
                    help="profiling aid: quantise a random matrix instead of building the basis")
    ap.add_argument("--layered", action="store_true",
                    help="the layer-wise construction with per-layer affine codes instead of the default workload")
    ap.add_argument("--project-batch", type=int, default=0,
                    help="time the projection of this many gradients per call instead of the fused step")
    args = ap.parse_args()
    if args.project_batch and args.impl == "ours":
        run_project_batch(args)
    elif args.layered and args.impl == "ours":
        run_layered(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
