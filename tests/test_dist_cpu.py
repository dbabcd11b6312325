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


# ---- context-sharded attend: the sharding table and the all-gather layout ------------------------------------------

def test_shard_contexts_is_a_balanced_partition():
    lens = [256] * 37 + [1000, 3, 0, 512, 512, 77]
    for world in (1, 2, 3, 8):
        table = dist_util.shard_contexts(lens, world)
        assert sorted(i for t in table for i in t) == list(range(len(lens)))          # every context exactly once
        loads = [sum(lens[i] for i in t) for t in table]
        assert max(loads) - min(loads) <= max(lens)                                    # longest-first greedy bound
    assert dist_util.shard_contexts([], 4) == [[], [], [], []]


def _gather_worker(rank: int, world: int, port: int, out):
    import torch.distributed as td
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    td.init_process_group("gloo", rank=rank, world_size=world)
    rows, H, d = 3, 2, 4
    o = torch.full((rows, H, d), float(rank + 1))
    l = torch.full((rows, H), float(10 * (rank + 1)))
    o_all, l_all = dist_util.gather_context_partials(o, l)
    table = dist_util.shard_contexts([5, 9, 2, 7, 7], world)
    out.put((rank, tuple(o_all.shape), o_all[:, 0, 0, 0].tolist(), tuple(l_all.shape), l_all[:, 0, 0].tolist(), table))
    td.barrier()
    td.destroy_process_group()


def test_gather_context_partials_two_processes():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gather_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, o_shape, o_vals, l_shape, l_vals, table in got:
        assert o_shape == (2, 3, 2, 4) and l_shape == (2, 3, 2)
        assert o_vals == [1.0, 2.0] and l_vals == [10.0, 20.0]                       # shard-major, rank r at index r
    assert got[0][5] == got[1][5]                                                    # every rank derives the same table


def test_gather_without_a_process_group_is_one_shard():
    o, l = torch.zeros(2, 3, 4), torch.zeros(2, 3)
    o_all, l_all = dist_util.gather_context_partials(o, l)
    assert tuple(o_all.shape) == (1, 2, 3, 4) and tuple(l_all.shape) == (1, 2, 3)
