"""world_size-2 check (gloo, CPU) of the only cross-rank step of a multi-GPU run: the max-over-ranks timing
reduction and the whole-job rate computed from it.  The attention path itself shards by request without any
collective."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2502_05431_b200 import dist_util


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    import torch.distributed as td
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    td.init_process_group("gloo", rank=rank, world_size=world)
    mine = [1.0 + rank, 5.0 - rank, 2.0]            # per-rank phase times (ms)
    td.barrier()
    red = dist_util.max_over_ranks(mine)
    out.put((rank, red, dist_util.replica_seed(7, rank)))
    td.barrier()
    td.destroy_process_group()


def test_max_over_ranks_two_processes():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0][1] == got[1][1] == [2.0, 5.0, 2.0]
    assert got[0][2] != got[1][2]                   # replicas are seeded differently


def test_single_process_is_identity_and_rate():
    assert dist_util.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert dist_util.whole_job_rate(10.0, 4, 2.0) == 4 * 10.0 / 2e-3
