"""The multi-rank bookkeeping of bench.py with two gloo ranks on CPU: every rank runs its own replica, the timing is the
maximum over ranks, the value is the whole-job aggregate."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + 5.0 * rank, 2.0 - rank]          # rank 1 is slower on the first, faster on the second
        got = bench.max_over_ranks(mine, dist, torch.device("cpu"))
        ms_per_step, value = bench.whole_job_value(got[0], 5, 1000, world)
        out.put((rank, got, ms_per_step, value))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_max_and_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, ms_per_step, value in res:
        assert got == [15.0, 2.0]                        # the maximum over ranks, on every rank
        assert ms_per_step == 3.0
        assert abs(value - 2 * 1000 / 3.0e-3) < 1e-6     # two replicas' worth of units per step


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], None, None) == [1.5, 2.5]
    assert bench.whole_job_value(20.0, 10, 500, 1) == (2.0, 500 / 2.0e-3)
