"""N > 1 path of the benchmark on CPU: two gloo ranks, replicas only (no data-path collective)."""
import os
import socket
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2509_23410_b200 import replicas
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        secs = 1.0 + rank                       # rank 1 is the slow one
        slowest = replicas.max_over_ranks(secs)
        agg = replicas.aggregate_throughput(10.0, secs)
        dist.barrier()
        out.put((rank, slowest, agg))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_slowest_time_and_summed_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, agg in results:
        assert slowest == 2.0                    # max over ranks, known to every rank
        assert agg == pytest.approx(2 * 10.0 / 2.0)   # all ranks' units / slowest time


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    from paper_2509_23410_b200 import replicas
    assert replicas.max_over_ranks(0.25) == 0.25
    assert replicas.aggregate_throughput(8.0, 2.0) == 4.0
