"""World-size-2 check (gloo, CPU) of the replica aggregation used by bench.py under torchrun."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2609_35465_b200 import ranks
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 1.0 + rank                     # rank 1 is the slow one
    worst = ranks.max_over_ranks(ms)
    rate = ranks.aggregate_rate(10.0, ms)
    dist.barrier()
    out.put((rank, worst, rate))
    dist.destroy_process_group()


def test_replica_aggregation_two_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, worst, rate in got:
        assert worst == 2.0                       # the slowest rank's time
        assert rate == 2 * 10.0 / 2.0             # both ranks' work over that time


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2609_35465_b200 import ranks
    assert ranks.max_over_ranks(3.5) == 3.5
    assert ranks.aggregate_rate(7.0, 2.0) == 3.5
