"""World-size-2 CPU (gloo) test of the multi-GPU host logic: the unit partition is a disjoint
cover, and the bench's aggregation takes the max time over ranks."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_13612_b200 import shard


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, B, Hkv, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = shard.shard_units(B, Hkv, world, rank)
    # every rank learns every rank's unit ids
    ids = torch.full((B * Hkv,), -1, dtype=torch.int64)
    for n, (b, h) in enumerate(mine):
        ids[n] = b * Hkv + h
    gathered = [torch.empty_like(ids) for _ in range(world)]
    dist.all_gather(gathered, ids)
    # timing: max over ranks
    t = torch.tensor([0.010 * (rank + 1)], dtype=torch.float64)
    dist.barrier()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    done = torch.tensor([float(len(mine))], dtype=torch.float64)
    all_done = [torch.empty_like(done) for _ in range(world)]
    dist.all_gather(all_done, done)
    thr = shard.aggregate_throughput([float(x.item()) for x in all_done], float(t.item()))
    if rank == 0:
        q.put(([g[g >= 0].tolist() for g in gathered], float(t.item()), thr))
    dist.destroy_process_group()


def test_unit_partition_and_max_time_over_two_ranks():
    B, Hkv, world = 3, 5, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, B, Hkv, q)) for r in range(world)]
    for p in procs:
        p.start()
    got, tmax, thr = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    flat = sorted(x for g in got for x in g)
    assert flat == list(range(B * Hkv))                 # disjoint cover
    assert abs(len(got[0]) - len(got[1])) <= 1          # balanced
    assert abs(tmax - 0.020) < 1e-12                    # slowest rank decides
    assert abs(thr - (B * Hkv) / 0.020) < 1e-6


def test_partition_edge_cases():
    assert shard.shard_units(1, 1, 4, 3) == []
    assert shard.shard_units(2, 2, 1, 0) == [(0, 0), (0, 1), (1, 0), (1, 1)]
