"""Seeded random shapes through every plan kind of the attention path, each request checked against the fp64 oracle.

The fixed cases of the other GPU tests are chosen by hand for what they exercise; these are drawn: head layout (G = 1 .. 16,
d = 64 / 128), prefix, context counts and lengths (empty, one token, ragged, several tiles), gaps between spans, query rows,
extra cached keys, T and S on both sides of 1.  One plan kind per case: Eq. 5 prefill / decode, the per-context form,
context trees, a decode batch that shares its contexts.
"""
import random

import pytest

from oracle import ape_oracle as orc
from paper_2502_05431_b200 import libape
from paper_2502_05431_b200 import workloads as wl
from tests.gpu_util import compare, gpu_attend, oracle_attend

pytestmark = pytest.mark.gpu

HEADS = [(4, 4, 64), (8, 2, 64), (32, 8, 128), (16, 1, 128), (8, 8, 128), (4, 1, 64), (16, 4, 128)]


def _draw(seed):
    rnd = random.Random(seed)
    H_q, H_kv, d = rnd.choice(HEADS)
    n_req = rnd.choice([1, 1, 2, 3])
    lens = []
    for _ in range(n_req):
        n_ctx = rnd.choice([0, 1, 2, 3, 5, 9])
        lens.append([rnd.choice([0, 1, 7, 64, 100, 128, 129, 255, 300, 700]) for _ in range(n_ctx)])
    kw = dict(H_q=H_q, H_kv=H_kv, d=d, l_P=rnd.choice([0, 1, 16, 64, 130]), ctx_lens=lens, gap=rnd.choice([0, 0, 3]),
              T=rnd.choice([0.5, 0.9, 1.0, 1.3]), S=rnd.choice([0.6, 0.9, 1.0, 1.2]), seed=1000 + seed,
              shuffle_ctx=rnd.random() < 0.3, name=f"random{seed}")
    return rnd, kw


def _check_all(b, out, lse, ref_fn):
    for r, rq in enumerate(b.requests):
        ref = ref_fn(r)
        sl = slice(rq.q_start, rq.q_start + rq.q_len)
        compare(out[sl], ref.out.float(), f"{b.name} req {r}")
        assert (lse[sl].double() - ref.lse).abs().max().item() < 2e-3


@pytest.mark.parametrize("seed", range(12))
def test_random_prefill_and_per_context(seed):
    rnd, kw = _draw(seed)
    l_q = rnd.choice([1, 5, 33, 64, 65, 200])
    b = wl.make_batch(l_q=l_q, l_k=l_q + rnd.choice([0, 0, 3, 70]), **kw)
    out, lse, _ = gpu_attend(b, libape.APE_PREFILL)
    _check_all(b, out, lse, lambda r: oracle_attend(b, r))
    out, lse, _ = gpu_attend(b, libape.APE_PREFILL, per_context=True)
    _check_all(b, out, lse, lambda r: orc.attend(*b.views(r), b.T, b.S, per_context=True))


@pytest.mark.parametrize("seed", range(12, 20))
def test_random_decode_and_growth(seed):
    rnd, kw = _draw(seed)
    l_k = rnd.choice([1, 2, 63, 64, 65, 200])
    b = wl.make_batch(l_q=1, l_k=l_k, capacity=l_k + 9, **kw)
    for t in (0, rnd.choice([1, 5, 9])):
        out, lse, _ = gpu_attend(b, libape.APE_DECODE, kv_extra=t)
        _check_all(b, out, lse, lambda r: oracle_attend(b, r, l_k=b.requests[r].query_kv[1] + t))
    out, lse, _ = gpu_attend(b, libape.APE_DECODE, per_context=True)
    _check_all(b, out, lse, lambda r: orc.attend(*b.views(r), b.T, b.S, per_context=True))


@pytest.mark.parametrize("seed", range(20, 28))
def test_random_trees(seed):
    rnd, kw = _draw(seed)
    kw["shuffle_ctx"] = False                      # node i is the request's i-th context
    parents, scaled = [], []
    for lens in kw["ctx_lens"]:
        par = [(-1 if (i == 0 or rnd.random() < 0.3) else rnd.randrange(0, i)) for i in range(len(lens))]
        # keep the depth within what the decode-side merge holds (16 levels)
        depth = []
        for i, pp in enumerate(par):
            depth.append(0 if pp < 0 else depth[pp] + 1)
            if depth[i] > 12:
                par[i], depth[i] = -1, 0
        parents.append(par)
        scaled.append([rnd.random() < 0.5 for _ in lens])
    use_scaled = scaled if rnd.random() < 0.7 else None
    mode = rnd.choice([libape.APE_PREFILL, libape.APE_DECODE])
    l_q = 1 if mode == libape.APE_DECODE else rnd.choice([3, 40, 70])
    b = wl.make_batch(l_q=l_q, l_k=l_q + rnd.choice([0, 4]), **kw)
    out, lse, _ = gpu_attend(b, mode, tree=(parents, use_scaled))
    _check_all(b, out, lse, lambda r: orc.attend_tree(*b.views(r), b.T, b.S, parents[r], None if use_scaled is None else use_scaled[r]))


@pytest.mark.parametrize("seed", range(28, 36))
def test_random_shared_context_batches(seed):
    rnd, kw = _draw(seed)
    n_req = rnd.choice([1, 2, 7, 16, 33])
    lens = kw.pop("ctx_lens")[0]
    kw.pop("shuffle_ctx")
    l_k = rnd.choice([1, 9, 70])
    b = wl.share_contexts(wl.make_batch(ctx_lens=[lens] * n_req, l_q=1, l_k=l_k, capacity=l_k + 4, **kw))
    t = rnd.choice([0, 3])
    out, lse, _ = gpu_attend(b, libape.APE_DECODE, shared=True, kv_extra=t)
    _check_all(b, out, lse, lambda r: oracle_attend(b, r, l_k=b.requests[r].query_kv[1] + t))


@pytest.mark.parametrize("seed", range(36, 46))
def test_random_encode(seed):
    """Context encoding with drawn prefixes (tails that do and do not share a tile with the contexts) and context sets
    (enough contexts in some cases for every thread block to get several row blocks of several (context, head) pairs)."""
    from tests.test_gpu_parity import _check_encode
    rnd = random.Random(seed)
    H_q, H_kv, d = rnd.choice(HEADS)
    n_ctx = rnd.choice([1, 3, 8, 40])
    lens = [rnd.choice([0, 1, 9, 63, 64, 65, 128, 200, 256, 257, 400]) for _ in range(n_ctx)]
    b = wl.make_batch(H_q=H_q, H_kv=H_kv, d=d, l_P=rnd.choice([0, 3, 8, 64, 72, 128, 200]), ctx_lens=[lens], l_q=1,
                      gap=rnd.choice([0, 0, 2]), seed=2000 + seed, with_encode_q=True, name=f"random_encode{seed}")
    _check_encode(b)
