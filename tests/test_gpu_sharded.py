"""Context-sharded attend on one GPU: the shards of a multi-GPU run are planned and launched one after the other on the
same device (no kernel waits for another), their context partials are stacked the way an all-gather leaves them, and
ape_merge_shards must give what the oracle gives for the attend over ALL contexts."""
import pytest
import torch

from paper_2502_05431_b200 import dist_util, libape, workloads as wl
from paper_2502_05431_b200.workloads import Batch, Request
from tests.gpu_util import handle, gpu_attend, oracle_attend, compare

pytestmark = pytest.mark.gpu
LLAMA = dict(H_q=32, H_kv=8, d=128)


def _sharded(b: Batch, mode: int, world: int, kv_extra: int = 0):
    dev = torch.device("cuda:0")
    h = handle()
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    rows = q.shape[0]
    o_parts, l_parts, oth = [], [], None
    tables = [dist_util.shard_contexts([l for _, l in rq.ctx], world) for rq in b.requests]
    for rank in range(world):
        reqs = [Request(rq.q_start, rq.q_len, rq.prefix, [rq.ctx[i] for i in tables[r][rank]], rq.query_kv, rq.query_kv_capacity)
                for r, rq in enumerate(b.requests)]
        scratch = torch.empty_like(q)
        plan = h.attend_plan(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=scratch, requests=reqs, mode=mode)
        ws = plan.alloc_workspace()
        o_c = torch.full((rows, b.H_q, b.d), float("nan"), dtype=torch.float32, device=dev)
        l_c = torch.full((rows, b.H_q), float("nan"), dtype=torch.float32, device=dev)
        o_o, l_o = torch.full_like(o_c, float("nan")), torch.full_like(l_c, float("nan"))
        plan.attend_partial(b.T, ws, o_c, l_c, o_o, l_o, kv_extra=kv_extra)
        torch.cuda.synchronize()
        plan.close()
        o_parts.append(o_c); l_parts.append(l_c)
        if oth is None:
            oth = (o_o, l_o)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((rows, b.H_q), float("nan"), dtype=torch.float32, device=dev)
    libape.merge_shards(h, H_q=b.H_q, H_kv=b.H_kv, d=b.d, o_ctx_all=torch.stack(o_parts).contiguous(),
                        lse_ctx_all=torch.stack(l_parts).contiguous(), o_oth=oth[0], lse_oth=oth[1], S=b.S, out=out, lse=lse)
    torch.cuda.synchronize()
    assert h.get_status() == 0
    return out.cpu(), lse.cpu()


@pytest.mark.parametrize("world", [1, 2, 3])
def test_sharded_prefill_matches_the_oracle(world):
    b = wl.make_batch(**LLAMA, l_P=20, ctx_lens=[[256, 64, 130, 7, 300], [77]], l_q=33, l_k=40, seed=51, T=0.7, S=0.8,
                      name=f"sharded_prefill_w{world}")
    out, lse = _sharded(b, libape.APE_PREFILL, world)
    for r, rq in enumerate(b.requests):
        ref = oracle_attend(b, r)
        compare(out[rq.q_start:rq.q_start + rq.q_len], ref.out.float(), f"{b.name} req {r}")
        assert (lse[rq.q_start:rq.q_start + rq.q_len].double() - ref.lse).abs().max().item() < 2e-3


@pytest.mark.parametrize("world", [2, 4])
def test_sharded_decode_matches_the_oracle_and_the_single_plan(world):
    b = wl.make_batch(**LLAMA, l_P=64, ctx_lens=[[256] * 9, [512, 100, 1]], l_q=1, l_k=30, capacity=40, seed=52, T=0.9, S=1.1,
                      name=f"sharded_decode_w{world}")
    for t in (0, 10):
        out, lse = _sharded(b, libape.APE_DECODE, world, kv_extra=t)
        one, _, _ = gpu_attend(b, libape.APE_DECODE, kv_extra=t)
        assert (out.float() - one.float()).abs().max().item() <= 2e-2
        for r, rq in enumerate(b.requests):
            ref = oracle_attend(b, r, l_k=rq.query_kv[1] + t)
            compare(out[rq.q_start:rq.q_start + 1], ref.out.float(), f"{b.name} step {t} req {r}")


def test_a_shard_without_contexts_and_more_shards_than_contexts():
    b = wl.make_batch(H_q=8, H_kv=2, d=64, l_P=5, ctx_lens=[[100, 30]], l_q=4, seed=53, T=0.9, S=0.6, name="sharded_sparse")
    out, lse = _sharded(b, libape.APE_PREFILL, 4)                     # two of the four shards hold no context
    ref = oracle_attend(b, 0)
    compare(out, ref.out.float(), "sharded_sparse")
    assert (lse.double() - ref.lse).abs().max().item() < 2e-3


def test_partial_is_refused_for_per_context_plans_and_bad_arguments():
    b = wl.make_batch(**LLAMA, l_P=8, ctx_lens=[[64, 64]], l_q=1, l_k=4, seed=54)
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.empty_like(q)
    plan = handle().attend_plan(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests,
                                mode=libape.APE_DECODE, per_context=True)
    ws = plan.alloc_workspace()
    o = torch.zeros(1, 32, 128, device=dev); l = torch.zeros(1, 32, device=dev)
    with pytest.raises(libape.ApeError) as e:
        plan.attend_partial(0.9, ws, o, l, o.clone(), l.clone())
    assert e.value.code == -10
    with pytest.raises(libape.ApeError) as e:
        libape.merge_shards(handle(), H_q=32, H_kv=8, d=128, o_ctx_all=o.unsqueeze(0), lse_ctx_all=l.unsqueeze(0), o_oth=o, lse_oth=l,
                            S=-1.0, out=out)
    assert e.value.code == -4


def _rank_requests(b: Batch, world: int, rank: int):
    tables = [dist_util.shard_contexts([l for _, l in rq.ctx], world) for rq in b.requests]
    return [Request(rq.q_start, rq.q_len, rq.prefix, [rq.ctx[i] for i in tables[r][rank]], rq.query_kv, rq.query_kv_capacity)
            for r, rq in enumerate(b.requests)]


@pytest.mark.parametrize("mode,world", [(libape.APE_PREFILL, 1), (libape.APE_PREFILL, 3), (libape.APE_DECODE, 2)])
def test_the_multi_rank_entry_point_itself(mode, world):
    """dist_util.attend_context_sharded -- the call a rank of a multi-GPU job makes -- run for every rank in turn on one
    GPU.  The all-gather is replaced by a function that hands each rank the partials all ranks produced (collected in a
    first pass through the same entry point), in the layout the collective leaves them; everything else is the real path:
    ape_attend_partial, the gather hook, ape_merge_shards.  Every rank must end up with the oracle's result."""
    l_q = 1 if mode == libape.APE_DECODE else 33
    b = wl.make_batch(**LLAMA, l_P=20, ctx_lens=[[256, 64, 130, 7, 300], [77, 500]], l_q=l_q, l_k=40, seed=55, T=0.7, S=0.8,
                      name=f"sharded_entry_w{world}")
    dev = torch.device("cuda:0")
    h = handle()
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    plans, parts = [], []
    for rank in range(world):
        out = torch.full_like(q, float("nan"))
        plan = h.attend_plan(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=out, requests=_rank_requests(b, world, rank), mode=mode)
        plans.append((plan, plan.alloc_workspace(), out))

    def collect(o_c, l_c):                       # first pass: every rank's own partials, kept as the collective would see them
        parts.append((o_c.clone(), l_c.clone()))
        return dist_util.gather_context_partials(o_c, l_c)

    for plan, ws, out in plans:
        dist_util.attend_context_sharded(h, plan, H_q=b.H_q, H_kv=b.H_kv, d=b.d, T=b.T, S=b.S, workspace=ws, out=out, gather=collect)
    torch.cuda.synchronize()
    o_all = torch.stack([p[0] for p in parts]).contiguous()
    l_all = torch.stack([p[1] for p in parts]).contiguous()
    for plan, ws, out in plans:                  # second pass: what each rank computes once the gather has delivered all shards
        out.fill_(float("nan"))
        lse = torch.full((q.shape[0], b.H_q), float("nan"), dtype=torch.float32, device=dev)
        dist_util.attend_context_sharded(h, plan, H_q=b.H_q, H_kv=b.H_kv, d=b.d, T=b.T, S=b.S, workspace=ws, out=out, lse=lse,
                                         gather=lambda o_c, l_c: (o_all, l_all))
        torch.cuda.synchronize()
        assert h.get_status() == 0
        for r, rq in enumerate(b.requests):
            ref = oracle_attend(b, r)
            sl = slice(rq.q_start, rq.q_start + rq.q_len)
            compare(out[sl].cpu(), ref.out.float(), f"{b.name} req {r}")
            assert (lse[sl].cpu().double() - ref.lse).abs().max().item() < 2e-3
        plan.close()


_NCCL_WORLD1 = r"""
import os, sys, torch, torch.distributed as td
sys.path.insert(0, os.environ["APE_ROOT"])
from paper_2502_05431_b200 import dist_util, libape, workloads as wl
os.environ.setdefault("MASTER_ADDR", "127.0.0.1"); os.environ.setdefault("MASTER_PORT", os.environ["APE_PORT"])
torch.cuda.set_device(0)
td.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda:0"))
b = wl.make_batch(H_q=32, H_kv=8, d=128, l_P=20, ctx_lens=[[256, 64, 130]], l_q=17, seed=56, T=0.7, S=0.8)
dev = torch.device("cuda:0")
h = libape.Handle(0)
q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
one, two = torch.zeros_like(q), torch.zeros_like(q)
plan = h.attend_plan(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=one, requests=b.requests, mode=libape.APE_PREFILL)
ws = plan.alloc_workspace()
plan.attend(b.T, b.S, ws)
plan2 = h.attend_plan(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=two, requests=b.requests, mode=libape.APE_PREFILL)
dist_util.attend_context_sharded(h, plan2, H_q=32, H_kv=8, d=128, T=b.T, S=b.S, workspace=ws, out=two)
torch.cuda.synchronize()
assert h.get_status() == 0
err = (one.float() - two.float()).abs().max().item()
td.destroy_process_group()
assert err <= 2e-2, err
print("NCCL_WORLD1_OK", err)
"""


def test_the_entry_point_over_a_real_nccl_group_of_one_rank():
    """The same entry point with its own all-gather (NCCL, all_gather_into_tensor) in a process group of one rank, in a
    child process so that the process group does not outlive the test."""
    import os, socket, subprocess, sys
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, APE_ROOT=root, APE_PORT=str(port), NCCL_NVLS_ENABLE="0")
    r = subprocess.run([sys.executable, "-c", _NCCL_WORLD1], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and "NCCL_WORLD1_OK" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
