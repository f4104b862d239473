"""Host logic of the N > 1 benchmark path on CPU: two gloo ranks, max-over-ranks timing, whole-job
throughput of independent replicas, and the reference arm staying silent on ranks other than 0."""

import io
import os
import socket
import sys
from contextlib import redirect_stdout

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 5.0 - rank, 1.0]                      # rank 1 is slower on the first entry only
    got = bench.max_over_ranks(mine, "cpu")
    dist.barrier()
    out.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_two_gloo_ranks():
    import bench
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0] == results[1] == [11.0, 5.0, 1.0]
    # two replicas of 18 GB per step, the slower one takes 3 ms: 12,000 GB/s for the job
    assert abs(bench.whole_job_gbps(2, 18e9, 3.0) - 12000.0) < 1e-9
    assert bench.whole_job_gbps(1, 18e9, 3.0) * 2 == bench.whole_job_gbps(2, 18e9, 3.0)


def test_without_a_process_group_the_reduction_is_the_identity():
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu") == [1.5, 2.5]


def test_reference_arm_prints_only_on_rank_zero(monkeypatch):
    import argparse
    import bench
    monkeypatch.setenv("RANK", "1")
    args = argparse.Namespace(workload="tiny", bits=8, steps=2, warmup=0, gpus=2, reference_rows=4096,
                              reference_max_steps=20)
    buf = io.StringIO()
    with redirect_stdout(buf):
        bench.run_reference(args)
    assert buf.getvalue() == ""
    monkeypatch.setenv("RANK", "0")
    with redirect_stdout(buf):
        bench.run_reference(args)
    import json
    line = json.loads(buf.getvalue())
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    # the record says what really ran: seconds timed, threads used, one-thread figure, the host
    cpu = line["cpu_baseline"]
    assert cpu["timed_seconds"] > 0 and cpu["single_thread"]["threads"] == 1 and cpu["host_cores"] >= 1
    assert line["config"]["workload"] == bench.workload_label(bench_inputs().WORKLOADS["tiny"], 1048576, 8)


def bench_inputs():
    from paper_2205_13104_b200 import inputs
    return inputs


def test_series_statistics_and_clock_windows():
    import bench
    st = bench.series_stats([3.0, 1.0, 2.0, 10.0])
    assert st == {"mean": 4.0, "median": 2.5, "min": 1.0, "max": 10.0}
    s = bench.ClockSampler(0)
    s.samples = [(10.0, 1900.0, 1965.0, 900.0, []), (10.5, 1500.0, 1965.0, 1000.0, ["sw_power_cap"]),
                 (11.0, 1600.0, 1965.0, 990.0, ["sw_power_cap"])]
    assert s.summary(10.4, 11.1)["sm_mhz"] == 1600.0 and s.summary(10.4, 11.1)["reasons"] == ["sw_power_cap"]
    assert s.summary(9.0, 10.1) == {"sm_mhz": 1900.0, "sm_max_mhz": 1965.0, "samples": 1, "power_w_max": 900.0,
                                    "reasons": []}
    assert s.summary(20.0, 21.0)["sm_mhz"] == 1600.0           # no sample inside: the nearest one


def test_step_byte_accounting():
    import bench
    # 2 passes over P~, the gradient, w_bar and w
    assert bench.step_bytes(1000, 10, 8, 2) == 2 * 10 * 1000 + 2000 + 8000
    assert bench.step_bytes(1001, 3, 4, 4) == 2 * 3 * 501 + 4004 + 8008
    kb = bench.kernel_bytes(1000, 10, 8, 2)
    assert kb["project"] + kb["lift"] == bench.step_bytes(1000, 10, 8, 2)
