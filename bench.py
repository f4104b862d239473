#!/usr/bin/env python
"""Benchmark of the TWA subspace step on B200.

One "step" is one fused subspace iteration (project the gradient, update the
coefficients, lift the weights) through the C-ABI call twa_step on a basis built and
quantised by the library from synthetic correlated candidates; the basis build and the
quantisation are timed once and reported beside the step throughput.

    python bench.py --gpus N --steps K --warmup W [--workload vitb16] [--bits 8]
    python bench.py --impl reference ...     # the float64 CPU oracle on a bounded sample

Prints one JSON line (rank 0).  The headline (metric, value, config) is the ViT-B/16-sized
workload with int8 codes; the same line carries, under "configs", the step throughput of
every other synthetic workload and storage width (--no-configs leaves them out).  The K-step
timed region is repeated until about a second of device time has been measured, so that the
number does not depend on how long the clocks take to settle; the series is in the line.
With N > 1 every rank runs an independent replica of the workload on its own GPU (the path
has no exchange step); value is the sum over ranks.
"""

import argparse
import dataclasses
import datetime
import json
import math
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
LR, LAM = 0.1, 0.0
L2_BYTES = 126e6


def step_bytes(D, n, bits, g_bytes):
    """Algorithmic bytes of one fused step: P~ read by the projection and again by the lift,
    g read once, w_bar read once, w written once."""
    p = n * ((D * bits + 7) // 8)
    return 2 * p + D * g_bytes + 4 * D + 4 * D


def kernel_bytes(D, n, bits, g_bytes):
    p = n * ((D * bits + 7) // 8)
    return {"project": p + D * g_bytes, "lift": p + 8 * D}


def workload_label(wl, D, bits):
    """The one string both arms (library and oracle) put in config.workload."""
    kind = "float32" if bits == 32 else f"int{bits}"
    return f"{wl.name}: D={D} n={wl.n} {kind} P, {wl.g_dtype} g, lr={LR} lambda={LAM}"


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


def series_stats(ms_list):
    """Mean, median and minimum of a per-repeat series of ms/step."""
    s = sorted(ms_list)
    k = len(s)
    med = s[k // 2] if k % 2 else 0.5 * (s[k // 2 - 1] + s[k // 2])
    return {"mean": sum(s) / k, "median": med, "min": s[0], "max": s[-1]}


class ClockSampler:
    """nvidia-smi samples of one GPU's clocks and throttle reasons while a region runs (read-only
    queries; nothing is set)."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index, period_ms=20):
        self.index, self.period_ms = index, period_ms
        self.proc = None
        self.path = None
        self.samples = []

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        return self

    def stop(self):
        """Ends the sampling; self.samples = [(unix time, sm MHz, max MHz, watts, [reasons])]."""
        if self.proc is None:
            return self
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    sm, mx, watts = float(parts[1]), float(parts[2]), float(parts[3])
                except ValueError:
                    continue
                reasons = [n for n, v in zip(self.NAMES, parts[5:9]) if v.lower().startswith("active")]
                self.samples.append((ts, sm, mx, watts, reasons))
        os.unlink(self.path)
        self.proc = None
        return self

    def summary(self, t0=None, t1=None):
        """Median SM clock and the reasons seen between two time.time() stamps (all samples if
        none given)."""
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0,
                    "reasons": ["nvidia-smi gave no samples"]}
        sel = [s for s in self.samples if (t0 is None or s[0] >= t0) and (t1 is None or s[0] <= t1)]
        if not sel and t0 is not None:
            mid = 0.5 * (t0 + t1)
            sel = [min(self.samples, key=lambda s: abs(s[0] - mid))]
        sm = sorted(s[1] for s in sel)
        reasons = sorted({r for s in sel for r in s[4]})
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(s[2] for s in sel), "samples": len(sel),
                "power_w_max": max(s[3] for s in sel), "reasons": reasons}


def host_record():
    """Host the CPU baseline ran on: logical cores, CPU model, RAM."""
    model, ram = None, None
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemTotal"):
                    ram = round(int(line.split()[1]) / 1048576.0, 1)
                    break
    except OSError:
        pass
    return {"host_cores": os.cpu_count(), "cpu_model": model, "ram_gib": ram}


# --------------------------------------------------------------------------------------
# the oracle, timed (CPU baseline and reference arm)
# --------------------------------------------------------------------------------------
def oracle_timed_steps(codes, scales, wbar, gradients, steps, warmup, threads):
    """orc.step on host arrays, `steps` timed calls after `warmup`, with the numerical libraries
    limited to `threads` threads (None = their default).  Returns the list of seconds."""
    import numpy as np
    from oracle import twa_oracle as orc
    try:
        from threadpoolctl import threadpool_limits
    except Exception:                                  # pragma: no cover
        threadpool_limits = None
    alpha = np.zeros(codes.shape[1])
    times = []

    def run():
        nonlocal alpha
        for t in range(warmup + steps):
            g = gradients[t % len(gradients)]
            t0 = time.perf_counter()
            alpha, _, _ = orc.step(codes, scales, g, alpha, wbar, LR, LAM)
            dt = time.perf_counter() - t0
            if t >= warmup:
                times.append(dt)
    if threadpool_limits is not None and threads is not None:
        with threadpool_limits(limits=threads):
            run()
    else:
        run()
    return times


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:                                  # pragma: no cover
        return 1


def oracle_sample_host(wl, bits, rows):
    """A sample basis for the oracle when no GPU-built basis is at hand (reference arm): the
    oracle's own quantiser on the first `rows` rows of the workload's candidates, centred on
    their mean (orthonormalising them is not part of the timed step and is left out)."""
    import numpy as np
    import torch
    from oracle import twa_oracle as orc
    from paper_2205_13104_b200 import inputs
    cols = []
    for r0 in range(0, rows, inputs.CHUNK_ROWS):
        nr = min(inputs.CHUNK_ROWS, rows - r0)
        part = inputs.trajectory_rows(max(rows, r0 + nr), wl.n, wl.step, wl.drift, wl.seed, "cpu",
                                      row0=r0, rows=nr)
        cols.append(part.numpy())
    A = np.concatenate(cols, axis=1).T                                  # (rows, n) float32
    wbar = orc.mean(A).astype(np.float32)
    P32 = np.asfortranarray(((A - wbar[:, None]) / np.sqrt(rows)).astype(np.float32))
    codes, s = orc.quantize(P32, bits)
    gdt = torch.bfloat16 if wl.g_dtype == "bf16" else torch.float32
    grads = [inputs.gradient(rows, wl.g_std, wl.seed, t, gdt, "cpu").float().numpy() for t in range(4)]
    return codes, s, wbar, grads


def cpu_baseline_record(wl, D, bits, codes, scales, wbar, grads, steps, warmup):
    """The oracle's fused step on a sample of the workload's rows: all cores the numerical
    libraries use by default, then one thread."""
    rows, n = codes.shape
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    sb = step_bytes(rows, n, bits, g_bytes)
    t_all = oracle_timed_steps(codes, scales, wbar, grads, steps, warmup, None)
    t_one = oracle_timed_steps(codes, scales, wbar, grads, max(2, steps // 2), 1, 1)
    mean_all, mean_one = sum(t_all) / len(t_all), sum(t_one) / len(t_one)
    rec = {"value": sb / mean_all / 1e9, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
           "sample": f"fused step of the float64 oracle on the first {rows} of {D} rows, all {n} columns, "
                     f"{len(t_all)} timed steps after {warmup} warm-up",
           "seconds_per_sample_step": mean_all, "timed_seconds": sum(t_all) + sum(t_one),
           "single_thread": {"value": sb / mean_one / 1e9, "unit": UNIT, "threads": 1,
                             "seconds_per_sample_step": mean_one, "steps": len(t_one)},
           "ms_per_full_step_extrapolated": mean_all * 1e3 * D / rows,
           "note": "cores = threads the numerical libraries may use; the oracle is a loop of vector "
                   "operations (convert a column, dot product or axpy), which keeps one core busy at a time"}
    rec.update(host_record())
    return rec


def run_reference(args):
    from paper_2205_13104_b200 import inputs
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = inputs.WORKLOADS[args.workload]
    bits = args.bits if args.bits != 32 else 8
    rows = min(wl.D, args.reference_rows)
    codes, s, wbar, grads = oracle_sample_host(wl, bits, rows)
    steps = max(1, min(args.steps, args.reference_max_steps))
    rec = cpu_baseline_record(wl, wl.D, bits, codes, s, wbar, grads, steps, min(args.warmup, 2))
    line = {
        "impl": "reference", "metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": rec["ms_per_full_step_extrapolated"],
        "ms_per_step_note": f"extrapolated from the sample to all {wl.D} rows; the run itself timed "
                            f"{steps} sample steps in {rec['timed_seconds']:.1f} s",
        "timed_seconds": rec["timed_seconds"], "sample_steps_timed": steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": workload_label(wl, wl.D, bits),
                   "sample": f"first {rows} rows of D; quantised by the oracle from the workload's candidates"},
        "cpu_baseline": rec,
        "e2e": {"value": rec["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------------
# the library, timed
# --------------------------------------------------------------------------------------
class Env:
    """Process-wide plumbing of one rank: device, process group, barrier."""

    def __init__(self):
        import torch
        import torch.distributed as dist
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if self.world > 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{self.local}"))
        self.dev = torch.device(f"cuda:{self.local}")
        torch.cuda.set_device(self.dev)

    def barrier(self):
        import torch
        import torch.distributed as dist
        if self.world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def close(self):
        import torch.distributed as dist
        if self.world > 1:
            dist.destroy_process_group()


def timed_regions(env, step_fn, steps, warmup, min_total_ms, max_repeats=400):
    """`warmup` untimed steps, then the region of exactly `steps` steps, bracketed by a barrier and
    a device synchronisation on both sides and timed with CUDA events on the launch stream,
    repeated until `min_total_ms` of device time is covered (the count is fixed from the first
    region, the same on every rank).  Returns (ms per region, max over ranks; wall stamps)."""
    import torch
    t = 0
    for _ in range(warmup):
        step_fn(t)
        t += 1
    regions, walls = [], []
    repeats = 1
    k = 0
    while k < repeats:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        env.barrier()
        w0 = time.time()
        e0.record()
        for _ in range(steps):
            step_fn(t)
            t += 1
        e1.record()
        env.barrier()
        w1 = time.time()
        ms = max_over_ranks([e0.elapsed_time(e1)], env.dev)[0]
        regions.append(ms)
        walls.append((w0, w1))
        if k == 0:
            repeats = max(1, min(max_repeats, int(math.ceil(min_total_ms / max(ms, 1e-3)))))
        k += 1
    return regions, walls


def gradient_pool(wl, D, dev, count):
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    count = count if D * g_bytes * count <= 8e9 else max(2, int(8e9 // (D * g_bytes)))
    return [wl.gradient(t, dev) for t in range(count)]


def build_resident(ctx, wl, dev, ws, bits_list, twa, inputs, random_basis=False):
    """Candidates -> float32 basis (timed) -> one quantised basis per width (each timed, output buffers
    allocated beforehand), then once more from fresh candidates through the one-call form
    twa_build_quantized (timed; same buffers, same bytes).
    Returns ({bits: basis}, wbar, build_ms, {bits: quantise ms}, fused build+quantise ms or None)."""
    import torch
    D, n = wl.D, wl.n
    wbar = torch.empty(D, dtype=torch.float32, device=dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    low = [b for b in bits_list if b != 32]
    outs = {b: twa.new_quantised_basis(D, n, b, dev) for b in low}
    if random_basis:
        # profiling aid: skip the Gram-Schmidt launches; the step kernels do the same work on any values
        W = torch.randn((n, inputs.padded_ld(D, 128)), device=dev) / (D ** 0.5)
        twa.twa_mean(ctx, W, D, wbar)
        P32 = twa.basis_from_tensor(W, D)
        build_ms = None
    else:
        W = wl.candidates(dev, ld=inputs.padded_ld(D, 128))
        torch.cuda.synchronize()
        ev[0].record()
        P32 = twa.twa_build_basis(ctx, W, D, wbar, ws)
        ev[1].record()
        torch.cuda.synchronize()
        build_ms = ev[0].elapsed_time(ev[1])
    bases, quant_ms = {}, {}
    for bits in bits_list:
        if bits == 32:
            bases[32], quant_ms[32] = P32, 0.0
            continue
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        bases[bits] = twa.twa_quantize_basis(ctx, P32, bits, ws, out=outs[bits])
        b.record()
        torch.cuda.synchronize()
        quant_ms[bits] = a.elapsed_time(b)
    fused_ms = None
    if low and not random_basis:
        keep32 = 32 in bits_list
        if not keep32:
            del P32, W
            torch.cuda.empty_cache()
        W2 = wl.candidates(dev, ld=inputs.padded_ld(D, 128))
        torch.cuda.synchronize()
        ev[0].record()
        P32b, _ = twa.twa_build_quantized(ctx, W2, D, wbar, low, ws, out=[outs[b] for b in low])
        ev[1].record()
        torch.cuda.synchronize()
        fused_ms = ev[0].elapsed_time(ev[1])
        del W2, P32b
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"basis build failed: {twa.twa_strerror(code)} column {detail}")
    return bases, wbar, build_ms, quant_ms, fused_ms


def build_chunked(ctx, wl, dev, bits_list, twa, inputs):
    """The candidates (4*n*D bytes) do not fit beside P~: every row chunk is regenerated from its seed
    once per pass and fed to the row-chunked build; the codes of every width in bits_list come out of
    the same four passes.  Library time = CUDA events around the feed calls only (generating the
    chunks is not counted).  Returns ({bits: basis}, wbar, build_ms)."""
    import torch
    D, n = wl.D, wl.n
    wbar = torch.empty(D, dtype=torch.float32, device=dev)
    bws = torch.empty(twa.twa_build_workspace_bytes(n), dtype=torch.uint8, device=dev)
    bases = {bits: twa.new_quantised_basis(D, n, bits, dev) for bits in bits_list}
    buf = torch.empty((n, inputs.CHUNK_ROWS), dtype=torch.float32, device=dev)
    pairs = []
    twa.twa_build_begin(ctx, D, n, wbar, bws)
    for p in range(4):
        for r0 in range(0, D, inputs.CHUNK_ROWS):
            rows = min(inputs.CHUNK_ROWS, D - r0)
            inputs.trajectory_rows(D, n, wl.step, wl.drift, wl.seed, dev, row0=r0, rows=rows, out=buf[:, :rows])
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            if p < 3:
                twa.twa_build_feed(ctx, p, buf, r0, rows)
            else:
                # the chunk's rows of Q are formed once and encoded for every width (two at a time)
                todo = [bases[bits] for bits in bits_list]
                for i in range(0, len(todo), 2):
                    twa.twa_build_feed_codes(ctx, buf, r0, rows, todo[i:i + 2])
            if r0 + rows == D:
                if p == 2:
                    for bits in bits_list:
                        twa.twa_build_end_pass(ctx, p, bits, bases[bits])
                else:
                    twa.twa_build_end_pass(ctx, p, 0, None)
            b.record()
            pairs.append((a, b))
    torch.cuda.synchronize()
    build_ms = sum(a.elapsed_time(b) for a, b in pairs)
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"chunked build failed: {twa.twa_strerror(code)} column {detail}")
    return bases, wbar, build_ms


def measure_steps(env, ctx, twa, wl, basis, wbar, ws, pool, steps, warmup, min_total_ms, sampler):
    """Times twa_step on one basis.  Returns a dict: per-repeat ms/step series and its statistics,
    the two kernels' mean durations (events recorded inside twa_step), the clocks seen."""
    import torch
    D, n, bits = wl.D, wl.n, basis.bits
    alpha = torch.zeros(n, dtype=torch.float32, device=env.dev)
    w = torch.empty(D, dtype=torch.float32, device=env.dev)

    def step(t):
        twa.twa_step(ctx, basis, pool[t % len(pool)], LR, LAM, alpha, wbar, w, ws)

    twa.twa_profile_enable(ctx, min(65536, steps * 401 + warmup))
    for t in range(warmup):
        step(t)
    twa.twa_profile_read(ctx)                           # drop the warm-up steps from the series
    regions, walls = timed_regions(env, step, steps, 0, min_total_ms)
    proj_ms, lift_ms, rec = twa.twa_profile_read(ctx)
    twa.twa_profile_enable(ctx, 0)
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"step failed: {twa.twa_strerror(code)}")
    proj_ms, lift_ms = max_over_ranks([proj_ms / max(rec, 1), lift_ms / max(rec, 1)], env.dev)
    series = [r / steps for r in regions]
    out = {"series_ms_per_step": series, "stats": series_stats(series), "repeats": len(series),
           "project_ms": proj_ms, "lift_ms": lift_ms, "launches": 2 * steps * len(series),
           "walls": walls}
    del w
    return out


def graph_replay_ms(env, twa, wl, basis, wbar, pool, steps, min_total_ms):
    """The same K steps captured once into a CUDA graph (a context of its own on a side stream: the
    default stream cannot be captured) and replayed: ms per step, max over ranks.  For the small
    workloads, where a step is two launches of tens of microseconds."""
    import torch
    D, n = wl.D, wl.n
    stream = torch.cuda.Stream(device=env.dev)
    stream.wait_stream(torch.cuda.current_stream(env.dev))
    with torch.cuda.stream(stream):
        ctx = twa.twa_create(env.local, stream=stream)
        ws = twa.new_workspace(env.dev)
        alpha = torch.zeros(n, dtype=torch.float32, device=env.dev)
        w = torch.empty(D, dtype=torch.float32, device=env.dev)
        twa.twa_step(ctx, basis, pool[0], LR, LAM, alpha, wbar, w, ws)          # raises the kernels' limits
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for t in range(steps):
                twa.twa_step(ctx, basis, pool[t % len(pool)], LR, LAM, alpha, wbar, w, ws)
        for _ in range(3):
            graph.replay()
        stream.synchronize()
        regions, repeats, k = [], 1, 0
        while k < repeats:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            env.barrier()
            e0.record(stream)
            graph.replay()
            e1.record(stream)
            stream.synchronize()
            env.barrier()
            ms = max_over_ranks([e0.elapsed_time(e1)], env.dev)[0]
            regions.append(ms)
            if k == 0:
                repeats = max(1, min(400, int(math.ceil(min_total_ms / max(ms, 1e-3)))))
            k += 1
        code, _ = twa.twa_get_status(ctx)
        del graph
        twa.twa_destroy(ctx)
    torch.cuda.current_stream(env.dev).wait_stream(stream)
    if code != 0:
        raise RuntimeError(f"replayed step failed: {twa.twa_strerror(code)}")
    return sum(regions) / len(regions) / steps


def optimiser_entries(env, ctx, twa, inputs, wl, basis, wbar, ws, pool, steps, min_total_ms, peak):
    """Two more calls of the library on this workload, as "configs" entries: the fused step with Adam
    and a cosine schedule on the coefficients, and a fixed-weight average of the candidates."""
    import torch
    D, n, bits = wl.D, wl.n, basis.bits
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    alpha = torch.zeros(n, dtype=torch.float32, device=env.dev)
    m1 = torch.zeros(n, dtype=torch.float32, device=env.dev)
    m2 = torch.zeros(n, dtype=torch.float32, device=env.dev)
    w = torch.empty(D, dtype=torch.float32, device=env.dev)

    def adam_step(t):
        lr = twa.twa_cosine_lr(0.01, t % 1000, 1000)
        twa.twa_step_adam(ctx, basis, pool[t % len(pool)], lr, t + 1, alpha, m1, m2, wbar, w, ws, weight_decay=0.01)

    regions, _ = timed_regions(env, adam_step, steps, 3, min_total_ms)
    ms = sum(regions) / len(regions) / steps
    sb = step_bytes(D, n, bits, g_bytes)
    out = [{"mode": "fused step with Adam (decoupled decay) and a cosine schedule on the coefficients (twa_step_adam)",
            "workload": workload_label(wl, D, bits), "bits": bits, "ms_per_step": ms, "repeats": len(regions),
            "GBps": sb / (ms * 1e-3) / 1e9, "frac_of_measured_copy_peak": sb / (ms * 1e-3) / 1e9 / peak,
            "frac_of_8TBps": sb / (ms * 1e-3) / 1e9 / 8000.0, "bytes_per_step": sb}]
    W = wl.candidates(env.dev, ld=inputs.padded_ld(D, 128))
    weights = torch.full((n,), 1.0 / n, dtype=torch.float32, device=env.dev)

    def average(t):
        twa.twa_weighted_average(ctx, W, D, weights, w, ws)

    regions, _ = timed_regions(env, average, steps, 3, min_total_ms)
    ms = sum(regions) / len(regions) / steps
    ab = 4 * D * (n + 1)
    out.append({"mode": "fixed-weight average of the n candidates (twa_weighted_average: SWA, LAWA, EMA by the weights)",
                "workload": f"{wl.name}: D={D} n={n} float32 candidates", "bits": 32, "ms_per_call": ms,
                "repeats": len(regions), "GBps": ab / (ms * 1e-3) / 1e9,
                "frac_of_measured_copy_peak": ab / (ms * 1e-3) / 1e9 / peak, "frac_of_8TBps": ab / (ms * 1e-3) / 1e9 / 8000.0,
                "bytes_per_call": ab})
    code, _ = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"optimiser entries failed: {twa.twa_strerror(code)}")
    del W, w
    return out


def clock_fields(sampler, walls, series):
    """The clocks over all repeats, and per repeat the sampled SM clock with ms x MHz (how the
    time follows the clock, without touching any clock)."""
    if sampler is None:
        return None, None
    clocks = sampler.summary(walls[0][0], walls[-1][1])
    per = []
    for (w0, w1), ms in zip(walls, series):
        mhz = sampler.summary(w0, w1)["sm_mhz"]
        per.append({"ms_per_step": ms, "sm_mhz": mhz, "ms_x_mhz": None if mhz is None else ms * mhz})
    return clocks, per


def fused_record(fused_ms, widths):
    """What twa_build_quantized took: mean, basis and every low-bit width in one call."""
    low = [b for b in widths if b != 32]
    if fused_ms is None or not low:
        return None
    return {"ms": fused_ms, "widths": low,
            "call": "twa_build_quantized: the column maxima are taken while the build writes its last pass, "
                    "so each width costs one encoding pass"}


def config_entry(wl, bits, m, peak, build_ms, quant_ms, clocks, fused_ms=None, widths=(), note=None):
    """One element of the line's "configs" array."""
    D, n = wl.D, wl.n
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    sb, kb = step_bytes(D, n, bits, g_bytes), kernel_bytes(D, n, bits, g_bytes)
    ms = m["stats"]["mean"]
    gbps = sb / (ms * 1e-3) / 1e9
    p_bytes = n * ((D * bits + 7) // 8)
    e = {"workload": workload_label(wl, D, bits), "bits": bits, "ms_per_step": ms,
         "ms_per_step_median": m["stats"]["median"], "ms_per_step_min": m["stats"]["min"],
         "repeats": m["repeats"], "GBps": gbps, "frac_of_measured_copy_peak": gbps / peak,
         "frac_of_8TBps": gbps / 8000.0, "bytes_per_step": sb,
         "project_ms": m["project_ms"], "lift_ms": m["lift_ms"],
         "project_GBps": kb["project"] / (m["project_ms"] * 1e-3) / 1e9,
         "lift_GBps": kb["lift"] / (m["lift_ms"] * 1e-3) / 1e9,
         "sm_mhz": None if clocks is None else clocks["sm_mhz"],
         "clock_reasons": None if clocks is None else clocks["reasons"],
         "basis_build_ms": build_ms, "quantize_ms": quant_ms,
         "build_and_quantize_one_call": fused_record(fused_ms, widths),
         "l2": ("P~ (%.0f MB) fits the 126 MB L2 wholly or in good part: not an HBM fraction" % (p_bytes / 1e6))
               if p_bytes < 2.5 * L2_BYTES else "inputs larger than L2"}
    if note:
        e["note"] = note
    return e


def run_ours(args):
    import torch
    from paper_2205_13104_b200 import inputs, twa

    env = Env()
    dev, world, rank = env.dev, env.world, env.rank
    twa.load()
    wl = inputs.WORKLOADS[args.workload]
    if args.rows:
        wl = dataclasses.replace(wl, name=f"{wl.name}[rows={args.rows}]", D=args.rows, chunked_build=False)
    D, n, bits = wl.D, wl.n, args.bits
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    gdt = torch.bfloat16 if wl.g_dtype == "bf16" else torch.float32
    ctx = twa.twa_create(env.local)
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_DEQUANT_PATH, args.dequant_path)
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_LIFT_VECTORS, args.lift_vectors)
    twa.twa_set_tuning(ctx, twa.TWA_TUNE_TILE_SEGMENTS, args.tile_segments)
    ws = twa.new_workspace(dev)
    peak, peak_kind = load_peaks()
    with_configs = (not args.no_configs and args.workload == "vitb16" and bits == 8 and not args.rows
                    and not args.random_basis and args.dequant_path == 0 and args.tile_segments == 0)

    # ---- basis build and quantisation, timed once each -------------------------------
    extra_bits = [4] if with_configs else []
    if wl.chunked_build and not args.random_basis:
        if bits == 32:
            raise SystemExit("the chunked workload has no resident float32 basis; use --bits 8 or 4")
        bases, wbar, build_ms = build_chunked(ctx, wl, dev, [bits] + extra_bits, twa, inputs)
        quant_ms, fused_ms = {b: None for b in bases}, None
    else:
        bases, wbar, build_ms, quant_ms, fused_ms = build_resident(ctx, wl, dev, ws, [bits] + extra_bits, twa, inputs,
                                                                   args.random_basis)
    Pq = bases[bits]
    if bits != 32:
        bases.pop(32, None)
    torch.cuda.empty_cache()

    # ---- per-step inputs: a pool of distinct gradients, cycled ------------------------
    pool = gradient_pool(wl, D, dev, args.g_pool)
    sampler = ClockSampler(env.local).start() if rank == 0 else None
    m = measure_steps(env, ctx, twa, wl, Pq, wbar, ws, pool, args.steps, args.warmup, args.min_timed_ms, sampler)

    # ---- end to end: gradient from pinned host memory, weights back to the host --------
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    g_host = [p.cpu().pin_memory() for p in pool[:2]]
    w_host = torch.empty(D, dtype=torch.float32).pin_memory()
    g_stage = torch.empty(D, dtype=gdt, device=dev)
    w = torch.empty(D, dtype=torch.float32, device=dev)
    alpha2 = torch.zeros(n, dtype=torch.float32, device=dev)

    def host_step(t):
        twa.twa_step_host(ctx, Pq, g_host[t % 2], LR, LAM, alpha2, wbar, w, w_host, g_stage, ws)

    e2e_regions, _ = timed_regions(env, host_step, e2e_steps, 2, args.min_timed_ms / 2)
    e2e_series = [r / e2e_steps for r in e2e_regions]
    e2e_ms = series_stats(e2e_series)["mean"]
    if sampler is not None:
        sampler.stop()
    del g_host, w_host, g_stage, w
    build_ms_all, = max_over_ranks([build_ms or 0.0], dev)
    qm = quant_ms.get(bits)
    quant_ms_all, = max_over_ranks([qm or 0.0], dev)

    # ---- the other workloads and widths (rank 0's record; every rank runs them) ------------
    configs = []
    clocks, per_repeat = clock_fields(sampler, m["walls"], m["series_ms_per_step"])
    cpu = None
    if with_configs:
        if 4 in bases:
            s4 = ClockSampler(env.local).start() if rank == 0 else None
            m4 = measure_steps(env, ctx, twa, wl, bases[4], wbar, ws, pool, args.steps, args.warmup,
                               args.configs_min_ms, s4)
            c4 = s4.stop().summary(m4["walls"][0][0], m4["walls"][-1][1]) if s4 is not None else None
            configs.append(config_entry(wl, 4, m4, peak, build_ms_all, quant_ms.get(4), c4, fused_ms, [bits] + extra_bits))
    # CPU baseline: the oracle on the first rows of THIS basis (rank 0, N = 1 only)
    if rank == 0 and world == 1 and not args.no_cpu_baseline and bits != 32:
        rows = min(D, args.reference_rows)
        seg = 512 * 8 // bits
        rows = max(seg, rows - rows % seg) if rows < D else D
        codes_d, s_d = twa.twa_basis_export(ctx, twa.basis_view(Pq, row0=0, rows=rows))
        from oracle import twa_oracle as orc
        codes_h = orc.unpack_codes(codes_d.cpu().numpy(), rows, bits)
        grads_h = [p[:rows].float().cpu().numpy() for p in pool[:4]]
        cpu = cpu_baseline_record(wl, D, bits, codes_h, s_d.cpu().numpy(), wbar[:rows].cpu().numpy(), grads_h, 5, 1)
        del codes_d, codes_h
    del bases, Pq, pool
    torch.cuda.empty_cache()
    if with_configs:
        configs += other_configs(env, ctx, twa, inputs, ws, args, peak)

    if rank == 0:
        sb = step_bytes(D, n, bits, g_bytes)
        kb = kernel_bytes(D, n, bits, g_bytes)
        ms_per_step = m["stats"]["mean"]
        value = whole_job_gbps(world, sb, ms_per_step)
        suffix = "_mma" if args.dequant_path == 0 and bits != 32 else ""
        dom = "project" if m["project_ms"] >= m["lift_ms"] else "lift"
        other = "lift" if dom == "project" else "project"
        dom_ms, other_ms = m[f"{dom}_ms"], m[f"{other}_ms"]
        achieved = kb[dom] / (dom_ms * 1e-3) / 1e9
        traffic = read_traffic(f"{wl.name}_int{bits}_{dom}") if args.dequant_path == 0 else None
        p_bytes = n * ((D * bits + 7) // 8)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_label(wl, D, bits),
                       "l2": f"inputs larger than L2: P~ is {p_bytes / 1e6:.0f} MB per pass"
                             if p_bytes > 2.5 * L2_BYTES else f"P~ is {p_bytes / 1e6:.0f} MB: partly L2-resident",
                       "gradients": f"{args.g_pool} distinct gradients generated before the timed region, cycled",
                       "dequant_path": "tensor-pipe integer dot products" if args.dequant_path == 0 else "float32 FMA",
                       "timed_region": f"{args.steps} steps between barriers, repeated {m['repeats']} times "
                                       f"(about {args.min_timed_ms:.0f} ms of device time); ms_per_step and value "
                                       "are the mean over all repeats",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "ms_per_step_median": m["stats"]["median"], "ms_per_step_min": m["stats"]["min"],
            "repeats": m["repeats"], "series": per_repeat,
            "bytes_per_step": sb,
            "frac_of_hbm_peak": value / world / peak,
            "frac_of_hbm_peak_note": f"of the {peak_kind} copy bandwidth ({peak:.0f} GB/s, half read, half written): "
                                     "not an upper bound for these read-dominated streams",
            "frac_of_8TBps": value / world / 8000.0,
            "basis_build_ms": None if args.random_basis else build_ms_all,
            "quantize_ms": None if wl.chunked_build else quant_ms_all,
            "build_and_quantize_one_call": fused_record(fused_ms, [bits] + extra_bits),
            "basis_build": ("row-chunked Gram-form build incl. quantisation, 4 passes, chunk generation not counted"
                            if wl.chunked_build else
                            "resident block Gram-Schmidt with re-orthogonalisation: panels of 8 columns, "
                            "Gram-form inside a panel (same factor as column-by-column classical Gram-Schmidt)"),
            "roofline": {"bound": "hbm", "kernel": f"twa_{dom}{suffix}_kernel", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": f"of {peak_kind} (copy bandwidth; a read-dominated stream can exceed it)",
                         "frac_of_8TBps": achieved / 8000.0,
                         "traffic": traffic, "bytes_per_launch": kb[dom], "ms_per_launch": dom_ms,
                         "other_kernel": {"kernel": f"twa_{other}{suffix}_kernel", "ms_per_launch": other_ms,
                                          "achieved": kb[other] / (other_ms * 1e-3) / 1e9,
                                          "bytes_per_launch": kb[other]}},
            "cpu_baseline": cpu,
            "e2e": {"value": world * sb / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
                    "ms_per_step": e2e_ms, "steps": e2e_steps, "repeats": len(e2e_series),
                    "h2d_bytes_per_step": D * g_bytes, "d2h_bytes_per_step": 4 * D},
            "gpu_launches": m["launches"],
            "clocks": clocks,
            "configs": configs if with_configs else None,
        }
        print(json.dumps(line))
    twa.twa_destroy(ctx)
    env.close()


def other_configs(env, ctx, twa, inputs, ws, args, peak):
    """Step throughput of the remaining synthetic workloads and widths, each with its own build, a
    clock record and at least --configs-min-ms of timed device time."""
    import torch
    dev = env.dev
    out = []
    plan = [("tiny", [32]), ("resnet18", [32, 8]), ("resnet50", [8]), ("decoder1p3b", [8, 4])]
    for name, widths in plan:
        wl = inputs.WORKLOADS[name]
        if wl.chunked_build:
            bases, wbar, build_ms = build_chunked(ctx, wl, dev, widths, twa, inputs)
            quant_ms, fused_ms = {b: None for b in widths}, None
        else:
            bases, wbar, build_ms, quant_ms, fused_ms = build_resident(ctx, wl, dev, ws, widths, twa, inputs)
        pool = gradient_pool(wl, wl.D, dev, args.g_pool)
        for bits in widths:
            sampler = ClockSampler(env.local).start() if env.rank == 0 else None
            m = measure_steps(env, ctx, twa, wl, bases[bits], wbar, ws, pool, args.steps, args.warmup,
                              args.configs_min_ms, sampler)
            clocks = None
            if sampler is not None:
                sampler.stop()
                clocks = sampler.summary(m["walls"][0][0], m["walls"][-1][1])
            entry = config_entry(wl, bits, m, peak, build_ms, quant_ms.get(bits), clocks, fused_ms, widths)
            if wl.n * ((wl.D * bits + 7) // 8) < 2.5 * L2_BYTES or name == "resnet18":
                entry["cuda_graph_replay_ms_per_step"] = graph_replay_ms(env, twa, wl, bases[bits], wbar, pool,
                                                                         args.steps, args.configs_min_ms / 2)
            out.append(entry)
        if name == "resnet50":
            out.extend(optimiser_entries(env, ctx, twa, inputs, wl, bases[8], wbar, ws, pool, args.steps,
                                         args.configs_min_ms / 2, peak))
        del bases, wbar, pool
        torch.cuda.empty_cache()
    # a basis of more than 2^31 rows: the 1.3 B-sized workload's recipe stretched to 2^31 + 3 * 2^22 + 70,001 rows
    # (row-chunked build, int8); the step walks it in three slabs of 2^30 rows
    large_rows = not args.no_large_rows
    if large_rows:
        import dataclasses
        wl = dataclasses.replace(inputs.WORKLOADS["decoder1p3b"], name="decoder-recipe rows > 2^31",
                                 D=(1 << 31) + 3 * (1 << 22) + 70_001)
        torch.cuda.empty_cache()
        free_bytes, _ = torch.cuda.mem_get_info(dev)
        free_bytes = -max_over_ranks([-float(free_bytes)], dev)[0]       # every rank takes the same decision
        need = wl.n * wl.D + 2 * 2 * wl.D + 3 * 4 * wl.D + (2 << 30)      # codes, two gradients, w-bar, w, slack
        if free_bytes < need:
            out.append({"workload": workload_label(wl, wl.D, 8), "bits": 8,
                        "skipped": "%.0f GB free on the device, %.0f GB needed" % (free_bytes / 1e9, need / 1e9)})
            large_rows = False
    if large_rows:
        bases, wbar, build_ms = build_chunked(ctx, wl, dev, [8], twa, inputs)
        pool = gradient_pool(wl, wl.D, dev, 2)
        sampler = ClockSampler(env.local).start() if env.rank == 0 else None
        m = measure_steps(env, ctx, twa, wl, bases[8], wbar, ws, pool, args.steps, args.warmup,
                          args.configs_min_ms, sampler)
        clocks = None
        if sampler is not None:
            sampler.stop()
            clocks = sampler.summary(m["walls"][0][0], m["walls"][-1][1])
        out.append(config_entry(wl, 8, m, peak, build_ms, None, clocks,
                                note="three slabs of 2^30 rows per kernel; the projection's slab sums are added in float64"))
        del bases, wbar, pool
        torch.cuda.empty_cache()
    # the other modes of the library, each through its own benchmark routine, condensed
    for name, bits in (("vitb16", 8), ("vitb16", 4), ("decoder1p3b", 4)):
        line = layered_line(env, args, name, bits, args.configs_min_ms)
        if line is not None:
            r = line["roofline"]
            out.append({"mode": "layer-wise construction, per-layer affine codes (the paper's default; B = 4 its default width)",
                        "workload": line["config"]["workload"], "bits": bits, "ms_per_step": line["ms_per_step"],
                        "ms_per_step_median": line["ms_per_step_median"], "repeats": line["repeats"],
                        "GBps": line["value"], "frac_of_measured_copy_peak": line["frac_of_hbm_peak"],
                        "frac_of_8TBps": line["frac_of_8TBps"], "bytes_per_step": line["bytes_per_step"],
                        "project_ms": r["project_ms"], "lift_ms": r["lift_ms"],
                        "sm_mhz": line["clocks"]["sm_mhz"] if line["clocks"] else None,
                        "clock_reasons": line["clocks"]["reasons"] if line["clocks"] else None,
                        "basis_build_ms": line["basis_build_ms"], "quantize_ms": line["quantize_ms"]})
    for bits in ((8, 4) if env.world == 1 else ()):
        line = project_batch_line(env, args, "vitb16", bits, 8, args.configs_min_ms)
        r = line["roofline"]
        out.append({"mode": "8 gradients per projection (twa_project_batch)", "workload": line["config"]["workload"],
                    "bits": bits, "ms_per_call": line["ms_per_step"], "gradients_per_s": line["value"],
                    "GBps": r["achieved"], "frac_of_measured_copy_peak": r["frac"], "frac_of_8TBps": r["achieved"] / 8000.0,
                    "single_calls_ms": line["single_calls_ms"], "speedup_over_single_calls": line["speedup_over_single_calls"],
                    "sm_mhz": line["clocks"]["sm_mhz"], "clock_reasons": line["clocks"]["reasons"]})
    return out


def run_layered(args):
    env = Env()
    line = layered_line(env, args, args.workload, args.bits, args.min_timed_ms)
    if env.rank == 0:
        print(json.dumps(line))
    env.close()


def layered_line(env, args, workload, bits, min_timed_ms):
    """The paper's default construction: per-layer centred and normalised basis, per-layer affine
    B-bit codes, layer-wise step (one coefficient vector per layer).  Returns the JSON line (rank 0)."""
    import torch
    from paper_2205_13104_b200 import inputs, twa

    dev, world, rank = env.dev, env.world, env.rank
    twa.load()
    wl = inputs.WORKLOADS[workload]
    if bits == 32:
        raise SystemExit("the layer-wise step runs on quantised codes")
    layers = inputs.layer_offsets(workload, args.rows or None)
    if args.rows:
        wl = dataclasses.replace(wl, name=f"{wl.name}[rows={args.rows}]", D=args.rows)
    D, n, L = wl.D, wl.n, len(layers) - 1
    if bits == 16 and n > 64:
        raise SystemExit("16-bit codes are stored as two 8-bit planes: at most 64 candidates")
    slot = {16: 16, 8: 8, 4: 4, 3: 4, 2: 2, 1: 1}[bits]   # bits of device memory per code
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    ctx = twa.twa_create(env.local)
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
        mem = torch.empty(twa.twa_layered_basis_bytes(layers, n, bits), dtype=torch.uint8, device=dev)
        torch.cuda.synchronize()
        ev[0].record()
        P32 = twa.twa_build_centered(ctx, W, D, layers, wbar, lws)
        ev[1].record()
        lb = twa.twa_quantize_affine(ctx, P32, layers, bits, lws, mem=mem)
        ev[2].record()
        torch.cuda.synchronize()
        build_ms, quant_ms = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])
        del W, P32
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"layer-wise build failed: {twa.twa_strerror(code)} layer {detail}")
    torch.cuda.empty_cache()

    pool = gradient_pool(wl, D, dev, args.g_pool)
    beta = torch.zeros((L, n), dtype=torch.float32, device=dev)
    c = torch.empty((L, n), dtype=torch.float32, device=dev)
    w = torch.empty(D, dtype=torch.float32, device=dev)
    sws = twa.new_layered_step_workspace(lb)

    sampler = ClockSampler(env.local).start() if rank == 0 else None
    regions, walls = timed_regions(
        env, lambda t: twa.twa_layered_step(ctx, lb, pool[t % len(pool)], LR, LAM, beta, wbar, w, sws),
        args.steps, args.warmup, min_timed_ms)
    if sampler is not None:
        sampler.stop()
    series = [r / args.steps for r in regions]
    # the two streaming launches apart (each call also runs its small per-layer kernel)
    part_steps = max(1, args.steps // 2)
    pr, _ = timed_regions(env, lambda t: twa.twa_layered_project(ctx, lb, pool[t % len(pool)], c, sws),
                          part_steps, args.warmup, min_timed_ms / 4)
    lr_, _ = timed_regions(env, lambda t: twa.twa_layered_lift(ctx, lb, beta, wbar, w, sws),
                           part_steps, args.warmup, min_timed_ms / 4)
    proj_ms, lift_ms = sum(pr) / len(pr) / part_steps, sum(lr_) / len(lr_) / part_steps
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"layer-wise step failed: {twa.twa_strerror(code)} layer {detail}")
    build_ms, quant_ms = max_over_ranks([build_ms, quant_ms], dev)
    line = None
    if rank == 0:
        peak, peak_kind = load_peaks()
        sb = step_bytes(D, n, slot, g_bytes)
        kb = kernel_bytes(D, n, slot, g_bytes)
        stats = series_stats(series)
        ms_per_step = stats["mean"]
        value = whole_job_gbps(world, sb, ms_per_step)
        dom = "project" if proj_ms >= lift_ms else "lift"
        dom_ms = proj_ms if dom == "project" else lift_ms
        clocks, per_repeat = clock_fields(sampler, walls, series)
        line = {
            "metric": METRIC.replace("int8", f"int{bits}") + "_layerwise", "value": value, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "ms_per_step_median": stats["median"], "ms_per_step_min": stats["min"], "repeats": len(series),
            "series": per_repeat,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{wl.name}: D={D} n={n} L={L} layers, per-layer affine int{bits} P, "
                                   f"{wl.g_dtype} g, lr={LR} lambda={LAM}",
                       "l2": f"inputs larger than L2: P~ is {n * ((D * slot + 7) // 8) / 1e6:.0f} MB per pass "
                             f"({slot} bits of device memory per code)",
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
                         "peak_kind": f"of {peak_kind} (copy bandwidth)", "traffic": None, "bytes_per_launch": kb[dom],
                         "ms_per_launch": dom_ms, "timing": "separate loop of that call alone",
                         "project_ms": proj_ms, "lift_ms": lift_ms},
            "cpu_baseline": None,
            "gpu_launches": 4 * args.steps * len(series),
            "clocks": clocks,
        }
    twa.twa_destroy(ctx)
    del lb, sws, pool, w, wbar
    torch.cuda.empty_cache()
    return line if rank == 0 else None


def run_project_batch(args):
    env = Env()
    line = project_batch_line(env, args, args.workload, args.bits, args.project_batch, args.min_timed_ms)
    if env.rank == 0:
        print(json.dumps(line))
    env.close()


def project_batch_line(env, args, workload, bits, B, min_timed_ms):
    """Projection of B gradients per call (P~ read once per group) beside the same number of
    single-gradient calls, on the workload's column shape; D may be cut with --rows."""
    import torch
    from paper_2205_13104_b200 import inputs, twa

    dev = env.dev
    twa.load()
    wl = inputs.WORKLOADS[workload]
    if args.rows:
        wl = dataclasses.replace(wl, name=f"{wl.name}[rows={args.rows}]", D=args.rows)
    D, n = wl.D, wl.n
    gdt = torch.bfloat16 if wl.g_dtype == "bf16" else torch.float32
    g_bytes = 2 if wl.g_dtype == "bf16" else 4
    ctx = twa.twa_create(env.local)
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

    def singles(_):
        for b in range(B):
            twa.twa_project(ctx, Pq, G[b, :D], c1, ws)

    sampler = ClockSampler(env.local).start()
    br, walls = timed_regions(env, lambda _: twa.twa_project_batch(ctx, Pq, G, C, ws), args.steps, args.warmup,
                              min_timed_ms)
    sampler.stop()
    sr, _ = timed_regions(env, singles, max(1, args.steps // 4), args.warmup, min_timed_ms / 4)
    batch_ms = sum(br) / len(br) / args.steps
    single_ms = sum(sr) / len(sr) / max(1, args.steps // 4)
    code, detail = twa.twa_get_status(ctx)
    if code != 0:
        raise RuntimeError(f"projection failed: {twa.twa_strerror(code)} {detail}")
    group = twa.twa_project_batch_group(ctx, Pq, gdt)
    p_bytes = n * ((D * bits + 7) // 8)
    moved = -(-B // group) * p_bytes + B * D * g_bytes
    peak, peak_kind = load_peaks()
    line = {
        "metric": f"twa_project_batch_gradients_per_s_int{bits}", "value": B / (batch_ms * 1e-3), "unit": "gradients/s",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": batch_ms, "repeats": len(br),
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{wl.name}: D={D} n={n} int{bits} P, {wl.g_dtype} g, {B} gradients per call, "
                               f"groups of {group}", "l2": f"inputs larger than L2: P~ is {p_bytes / 1e6:.0f} MB"},
        "single_calls_ms": single_ms, "speedup_over_single_calls": single_ms / batch_ms,
        "roofline": {"bound": "hbm", "kernel": "twa_project_batch_kernel", "achieved": moved / (batch_ms * 1e-3) / 1e9,
                     "peak": peak, "unit": "GB/s", "frac": moved / (batch_ms * 1e-3) / 1e9 / peak,
                     "peak_kind": f"of {peak_kind} (copy bandwidth)", "traffic": None,
                     "bytes_per_launch": moved // -(-B // group)},
        "cpu_baseline": None, "gpu_launches": -(-B // group) * args.steps * len(br),
        "clocks": sampler.summary(walls[0][0], walls[-1][1])}
    twa.twa_destroy(ctx)
    del Pq, G, C
    torch.cuda.empty_cache()
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vitb16")
    ap.add_argument("--bits", type=int, default=8, choices=[32, 16, 8, 4, 3, 2, 1],
                    help="storage width of P: 32 / 8 / 4 for the per-column path; the layer-wise path (--layered)\n"
                         "takes every width of the paper's ablation: 16, 8, 4, 3, 2, 1")
    ap.add_argument("--g-pool", type=int, default=8)
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--min-timed-ms", type=float, default=1000.0,
                    help="the K-step region is repeated until this much device time is covered")
    ap.add_argument("--configs-min-ms", type=float, default=400.0,
                    help="the same, for each entry of the configs array")
    ap.add_argument("--no-configs", action="store_true",
                    help="headline workload only: leave out the other workloads and widths")
    ap.add_argument("--reference-rows", type=int, default=1 << 21)
    ap.add_argument("--reference-max-steps", type=int, default=20,
                    help="the oracle arm times at most this many sample steps (bounded run)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--lift-vectors", type=int, default=0, choices=[0, 1, 2, 3],
                    help="TWA_TUNE_LIFT_VECTORS: how base and output travel in the 8/4-bit lift (0 = built-in choice)")
    ap.add_argument("--tile-segments", type=int, default=0, choices=[0, 1, 2, 4],
                    help="TWA_TUNE_TILE_SEGMENTS: 512-byte segments of a column per tile (0 = built-in choice)")
    ap.add_argument("--dequant-path", type=int, default=0, choices=[0, 1],
                    help="0: integer dot products on the tensor pipe (default); 1: float32 FMA path")
    ap.add_argument("--rows", type=int, default=0, help="override D (smaller cases for profiler captures)")
    ap.add_argument("--no-large-rows", action="store_true",
                    help="leave the basis of more than 2^31 rows (about 95 GB on the device) out of the configs array")
    ap.add_argument("--random-basis", action="store_true",
                    help="profiling aid: quantise a random matrix instead of building the basis")
    ap.add_argument("--layered", action="store_true",
                    help="the layer-wise construction with per-layer affine codes instead of the default workload")
    ap.add_argument("--project-batch", type=int, default=0,
                    help="time the projection of this many gradients per call instead of the fused step")
    args = ap.parse_args()
    if args.steps < 1:
        raise SystemExit("--steps must be at least 1")
    if args.bits in (16, 3, 2, 1) and not (args.layered and args.impl == "ours"):
        raise SystemExit("widths 16, 3, 2 and 1 exist for the layer-wise construction only: add --layered")
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
