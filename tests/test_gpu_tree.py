"""GPU parity of the context-tree form (ape_attend_plan_tree) against the oracle's ape_oracle_attend_tree, which is itself
pinned on the CPU (tests/test_tree_pins.py)."""
import pytest
import torch

from oracle import ape_oracle as orc
from paper_2502_05431_b200 import libape
from paper_2502_05431_b200 import workloads as wl
from tests.gpu_util import compare, gpu_attend, handle

pytestmark = pytest.mark.gpu
LLAMA = dict(H_q=32, H_kv=8, d=128)


def _check(b, mode, parents, scaled=None, kv_extra=0):
    out, lse, n = gpu_attend(b, mode, tree=(parents, scaled), kv_extra=kv_extra)
    assert n == (4 if mode == libape.APE_PREFILL else 2)      # prefill: statistics pass, biases, biased prefill, merge
    for r, rq in enumerate(b.requests):
        q, p, c, k = b.views(r)
        if kv_extra:
            s0 = rq.query_kv[0]
            k = (b.k_pool[s0:s0 + rq.query_kv[1] + kv_extra], b.v_pool[s0:s0 + rq.query_kv[1] + kv_extra])
        ref = orc.attend_tree(q, p, c, k, b.T, b.S, parents[r], None if scaled is None else scaled[r])
        sl = slice(rq.q_start, rq.q_start + rq.q_len)
        compare(out[sl], ref.out.float(), f"{b.name} req {r}")
        assert (lse[sl].double() - ref.lse).abs().max().item() < 2e-3
    return out


TREES = [
    # node lengths per request, parents per request, scaled per request (None: roots)
    ([[300, 0, 130, 64, 200, 1, 77]], [[-1, 0, 1, 1, 0, -1, 5]], None),
    ([[300, 0, 130, 64, 200, 1, 77]], [[-1, 0, 1, 1, 0, -1, 5]], [[0, 1, 0, 1, 1, 1, 0]]),
    ([[0, 256, 256, 256], [40, 500]], [[-1, 0, 0, 0], [-1, 0]], None),
    ([[100, 90, 80, 70, 60]], [[-1, 0, 1, 2, 3]], [[1, 1, 1, 1, 1]]),                    # a chain, S at every level
    ([[0, 0, 0, 129, 0, 65]], [[-1, 0, 1, 2, 0, 4]], [[1, 0, 1, 0, 0, 1]]),              # grouping nodes, leaves at depth 3 and 2
]


@pytest.mark.parametrize("mode", [libape.APE_PREFILL, libape.APE_DECODE])
@pytest.mark.parametrize("tree", range(len(TREES)))
def test_tree_form_matches_the_oracle(mode, tree):
    lens, parents, scaled = TREES[tree]
    l_q = 1 if mode == libape.APE_DECODE else 33
    b = wl.make_batch(**LLAMA, l_P=20, ctx_lens=lens, l_q=l_q, l_k=40, capacity=44, gap=2, seed=60 + tree, T=0.8, S=0.7, name=f"tree{tree}")
    _check(b, mode, parents, scaled, kv_extra=3 if mode == libape.APE_DECODE else 0)


def test_the_two_ends_of_the_family():
    """One node per context = the per-context plan; one tree over all contexts = the ordinary plan (Eq. 5)."""
    b = wl.make_batch(**LLAMA, l_P=32, ctx_lens=[[256] * 6], l_q=64, seed=70, T=0.9, S=0.7, name="tree_ends")
    forest = _check(b, libape.APE_PREFILL, [[-1] * 6])
    per_ctx, _, _ = gpu_attend(b, libape.APE_PREFILL, per_context=True)
    assert (forest.float() - per_ctx.float()).abs().max().item() <= 1e-2
    one = _check(b, libape.APE_PREFILL, [[-1, 0, 0, 1, 1, 2]])
    flat, _, _ = gpu_attend(b, libape.APE_PREFILL)
    assert (one.float() - flat.float()).abs().max().item() <= 1e-2
    assert (forest.float() - flat.float()).abs().max().item() > 1e-3


def test_tree_with_many_nodes_and_deep_levels_small_d():
    g = torch.Generator().manual_seed(71)
    n = 60
    parent = [-1] + [int(torch.randint(max(0, i - 4), i, (1,), generator=g)) if i % 7 else -1 for i in range(1, n)]
    depth = [0] * n
    for i in range(1, n):
        depth[i] = 0 if parent[i] < 0 else depth[parent[i]] + 1
        if depth[i] > 14:
            parent[i], depth[i] = -1, 0
    lens = [int(x) for x in torch.randint(0, 150, (n,), generator=g)]
    scaled = [int(x) for x in torch.randint(0, 2, (n,), generator=g)]
    b = wl.make_batch(H_q=8, H_kv=2, d=64, l_P=5, ctx_lens=[lens], l_q=70, l_k=80, seed=72, T=0.7, S=0.8, name="tree_many")
    _check(b, libape.APE_PREFILL, [parent], [scaled])


def test_malformed_trees_are_refused():
    b = wl.make_batch(**LLAMA, l_P=8, ctx_lens=[[64, 64, 64]], l_q=4, seed=73)
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.empty_like(q)
    kw = dict(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, mode=libape.APE_PREFILL)
    for parents in ([[0, 0, 0]], [[-1, 1, 0]], [[-1, 0, 7]], [[-2, 0, 0]]):
        with pytest.raises(libape.ApeError) as e:
            handle().attend_plan(tree=(parents, None), **kw)
        assert e.value.code == -1
    deep = wl.make_batch(**LLAMA, l_P=8, ctx_lens=[[8] * 18], l_q=4, seed=74)
    with pytest.raises(libape.ApeError) as e:
        handle().attend_plan(H_q=32, H_kv=8, d=128, k_pool=deep.k_pool.to(dev), v_pool=deep.v_pool.to(dev), q=q, out=out,
                             requests=deep.requests, mode=libape.APE_PREFILL, tree=([[-1] + list(range(17))], None))
    assert e.value.code == -1
    plan = handle().attend_plan(tree=([[-1, 0, 0]], None), **kw)
    ws = plan.alloc_workspace()
    o = torch.zeros(4, 32, 128, device=dev); l = torch.zeros(4, 32, device=dev)
    with pytest.raises(libape.ApeError) as e:          # the sharded hand-out is defined for Eq. 5 only
        plan.attend_partial(0.9, ws, o, l, o.clone(), l.clone())
    assert e.value.code == -10


def test_more_nodes_than_shared_memory_holds():
    """1,900 one- to three-token contexts, every one a marked top-level node (Eq. 11-12): the walk over the nodes between the
    two passes then keeps its per-node arrays in global memory instead of shared memory."""
    import random
    rnd = random.Random(5)
    lens = [rnd.randint(1, 3) for _ in range(1900)]
    b = wl.make_batch(H_q=8, H_kv=2, d=64, l_P=4, ctx_lens=[lens], l_q=9, seed=41, T=0.9, S=0.8, name="many_nodes")
    out, lse, n = gpu_attend(b, libape.APE_PREFILL, per_context=True)
    assert n == 4
    q, p, c, k = b.views(0)
    ref = orc.attend(q, p, c, k, b.T, b.S, per_context=True)
    compare(out, ref.out.float(), "many nodes")
    assert (lse.double() - ref.lse).abs().max().item() < 2e-3
