"""The N > 1 path of bench.py on CPU: two gloo ranks, replicas only (no data-path collective)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from workloads import configs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + rank, 3.0 - rank, 1.0]
    got = bench.max_over_ranks(mine, torch.device("cpu"), world)
    dist.barrier()
    out.put((rank, got))
    dist.destroy_process_group()


def test_timings_are_reduced_with_max_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0] == results[1] == [11.0, 3.0, 1.0]


def test_whole_job_value_counts_every_replica():
    one = bench.whole_job_value(1, 1000, 10, 5.0)
    assert bench.whole_job_value(4, 1000, 10, 5.0) == 4 * one == 4 * 1000 * 10 / 5e-3


def test_steps_group_trace_events_by_completed_update():
    cfg = configs.LARGE_SOFTSYNC
    steps = bench.step_events(cfg, 25)
    assert len(steps) == 25
    for evs in steps:
        assert sum(k == 1 for k, _ in evs) == cfg.c and evs[-1][0] == 1
    assert bench.algorithmic_bytes(60965224, 4, 4) == 60965224 * 32


def test_traffic_is_reported_only_for_the_captured_kernel_instantiation():
    v, src = bench.traffic_for("large_softsync", "vector", "fp32", 4, 1, 0, False, False)
    assert v == 1.9124e9 and os.path.exists(os.path.join(os.path.dirname(bench.__file__), src))
    for other in (("large_softsync", "bulk", "fp32", 4, 1, 0, False, False),        # another kernel
                  ("large_softsync", "vector", "fp32", 4, 1, 256, False, False),    # another block size
                  ("large_softsync", "vector", "fp32", 4, 1, 0, True, False),       # with the bf16 mirror
                  ("large_softsync@flat16777216", "vector", "fp32", 4, 1, 0, False, False)):
        v, why = bench.traffic_for(*other)
        assert v is None and "no ncu capture" in why


def test_repeats_are_summarised_by_their_median():
    stat = bench.summarise([{"ms": 30.0}, {"ms": 10.0}, {"ms": 20.0}], 10)
    assert stat == {"median": 2.0, "min": 1.0, "max": 3.0}
