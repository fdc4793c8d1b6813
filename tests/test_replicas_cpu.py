"""The N > 1 path is replicas with user-hash placement and no data-path collective: its host logic (placement,
max-over-ranks timing, whole-job throughput) on two gloo ranks on the CPU."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

from paper_2601_01712_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    users = list(range(1000))
    mine = replicas.users_of_rank(users, rank, world)
    seconds = 0.5 + 0.25 * rank                        # rank 1 is the slow replica
    t = replicas.max_over_ranks(seconds, dist)
    thr = replicas.job_throughput(float(len(mine)), seconds, dist)
    dist.barrier()
    out.put((rank, mine, t, thr))
    dist.destroy_process_group()


def test_two_replicas_partition_users_and_agree_on_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, u0, t0, thr0), (_, u1, t1, thr1) = res
    assert sorted(u0 + u1) == list(range(1000)) and not set(u0) & set(u1)      # every user has exactly one owner
    assert 350 < len(u0) < 650                                                  # and the hash spreads them
    assert t0 == t1 == 0.75
    assert thr0 == thr1 == 1000 / 0.75


def test_placement_is_stable_and_single_rank_is_identity():
    assert all(replicas.owner_rank(u, 1) == 0 for u in range(50))
    assert [replicas.owner_rank(u, 8) for u in (1, 2, 3)] == [replicas.owner_rank(u, 8) for u in (1, 2, 3)]
    counts = np.bincount([replicas.owner_rank(u, 8) for u in range(8000)], minlength=8)
    assert counts.min() > 800 and counts.max() < 1200
    assert replicas.max_over_ranks(3.0) == 3.0 and replicas.job_throughput(10.0, 2.0) == 5.0
