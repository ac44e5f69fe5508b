"""The N > 1 plumbing of bench.py (replicas, MAX over ranks) on CPU with gloo, world size 2."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_14952_b200 import replicas


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ids = replicas.member_ids(rank, 4)
    ms = 100.0 + 50.0 * rank                      # rank 1 is the slow one
    mx = replicas.max_over_ranks(ms, torch.device("cpu"), world)
    dist.barrier()
    out.put((rank, ids, mx, replicas.aggregate_throughput(10.0, 5, world, mx)))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_disjoint_members():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ids0, mx0, agg0), (r1, ids1, mx1, agg1) = res
    assert ids0 == [0, 1, 2, 3] and ids1 == [4, 5, 6, 7] and not set(ids0) & set(ids1)
    assert mx0 == mx1 == 150.0                     # MAX over ranks, seen by both
    assert agg0 == agg1 == 2 * 10.0 * 5 / 0.150    # whole-job units per second


def test_single_rank_is_the_identity():
    assert replicas.max_over_ranks(12.5, torch.device("cpu"), 1) == 12.5
    assert replicas.member_ids(0, 2) == [0, 1]
