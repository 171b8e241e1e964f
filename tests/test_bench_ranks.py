"""The multi-rank bookkeeping of bench.py (replicas, slowest-rank timing, whole-job aggregate),
run as two gloo ranks on the CPU."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    local_ms = 2.0 + rank                       # rank 1 is the slow one
    job_ms = bench.slowest_rank_ms(local_ms, dist, "cpu")
    dist.barrier()
    gbs = bench.whole_job_gbs(world, 6.4e9, job_ms)
    out.put((rank, job_ms, gbs))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    for rank, job_ms, gbs in got:
        assert job_ms == 3.0
        assert gbs == pytest.approx(2 * 6.4e9 / 3e-3 / 1e9)


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.slowest_rank_ms(1.5, None, "cpu") == 1.5
    assert bench.whole_job_gbs(1, 6.4e9, 2.0) == pytest.approx(3200.0)
    assert bench.quantize_bytes(25_000_000, 4, 2048) == 100_000_000 + 12_500_000 + 4 * 12_208
    assert bench.server_bytes(25_000_000, 8, 2048, 8) == 8 * (25_000_000 + 4 * 12_208) + 200_000_000
