"""The sharded layout's integer bookkeeping with two (and three) gloo ranks on CPU: ownership maps and exchange lists of
every rank against lists derived from the oracle's partitioning by their definitions."""
import os
import socket
import sys

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _case():
    sys.path.insert(0, ROOT)
    from oracle import sat_ref as orc
    from sat_synth import make_workload
    wl = make_workload("medium", shrink=32, with_dense=False)
    part = orc.contig_blocks(wl.n, wl.M)
    return wl, part, orc.build_partition(wl.rowptr, wl.col, part, wl.M)


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    # the package's binding needs the CUDA library; the plan module is plain numpy and is loaded on its own
    import importlib.util
    spec = importlib.util.spec_from_file_location("sat_shard", os.path.join(ROOT, "paper_2308_13466_b200", "shard.py"))
    shard = importlib.util.module_from_spec(spec)
    sys.modules["sat_shard"] = shard
    spec.loader.exec_module(shard)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl, part, P = _case()
        plan = shard.local_plan(rank, world, wl.M, part, P.slot, lambda m: P.halo_gid[m])
        shard.exchange_plan(plan, dist)
        out.put((rank, plan.parts, plan.slot_owner.tolist(), plan.owned_slots.tolist(), plan.need_slots.tolist(),
                 {q: v.tolist() for q, v in plan.recv.items()}, {q: v.tolist() for q, v in plan.send.items()}, plan.pull_rows()))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_ownership_and_exchange_lists(world):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = {}
    for _ in procs:
        r = out.get(timeout=300)
        res[r[0]] = r
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl, part, P = _case()
    # from the definitions: the owner of a slot is the rank of the partition its node is an inner node of
    node_of_slot = np.nonzero(P.slot >= 0)[0]
    want_owner = [int(part[v]) % world for v in node_of_slot]
    total_pull = 0
    for rank in range(world):
        _, parts, slot_owner, owned, need, recv, send, pull_rows = res[rank]
        assert parts == [m for m in range(wl.M) if m % world == rank]
        assert slot_owner == want_owner
        assert owned == [s for s, o in enumerate(want_owner) if o == rank]
        # every owned slot is pushed by one of this rank's partitions, and by no other rank's
        pushed = sorted(int(s) for m in parts for s in P.push_slot[m])
        assert pushed == owned
        want_need = sorted({int(P.slot[u]) for m in parts for u in P.halo_gid[m]})
        assert need == want_need
        for q in range(world):
            if q == rank:
                assert q not in recv and q not in send
                continue
            assert recv[q] == [s for s in want_need if want_owner[s] == q]
            # what rank `rank` sends to q is what q receives from `rank`
            assert send[q] == res[q][5][rank]
        assert pull_rows == sum(len(v) for v in recv.values())
        total_pull += pull_rows
    # fewer rows cross between GPUs than there are halo rows: co-located partitions share pulled rows and read their
    # neighbours' slots locally
    assert 0 < total_pull <= sum(P.halo_gid[m].shape[0] for m in range(wl.M))
