"""GPU parity of the shared-context decode plan (a batch of queries over ONE set of cached contexts, read once) against
the fp64 oracle, request by request, through the C ABI."""
import pytest
import torch

from paper_2502_05431_b200 import libape, workloads as wl
from tests.gpu_util import handle, gpu_attend, oracle_attend, compare

pytestmark = pytest.mark.gpu
LLAMA = dict(H_q=32, H_kv=8, d=128)


def _check(b, kv_extra=0, lse_tol=2e-3):
    out, lse, n = gpu_attend(b, libape.APE_DECODE, shared=True, kv_extra=kv_extra)
    has_ctx = any(l > 0 for _, l in b.requests[0].ctx)
    assert n == (3 if has_ctx else 2)
    for r, rq in enumerate(b.requests):
        ref = oracle_attend(b, r, l_k=(rq.query_kv[1] + kv_extra) if kv_extra else None)
        compare(out[rq.q_start:rq.q_start + 1], ref.out.float(), f"{b.name} req {r} O")
        d = (lse[rq.q_start:rq.q_start + 1].double() - ref.lse).abs().max().item()
        assert d < lse_tol, f"{b.name} req {r}: LSE error {d}"
    return out


@pytest.mark.parametrize("kw,n_req", [
    (dict(**LLAMA, l_P=16, ctx_lens=[64, 200, 1, 130], l_k=5, T=0.9, S=0.9), 3),
    (dict(**LLAMA, l_P=7, ctx_lens=[300], l_k=66, T=0.6, S=1.2, gap=2), 16),
    (dict(H_q=8, H_kv=8, d=64, l_P=3, ctx_lens=[100, 100], l_k=9, T=0.9, S=0.5), 5),        # G = 1, d = 64
    (dict(H_q=16, H_kv=1, d=128, l_P=64, ctx_lens=[256] * 3, l_k=65, T=1.1, S=0.9), 20),    # G = 16: two row blocks
    (dict(**LLAMA, l_P=4, ctx_lens=[], l_k=3, T=0.9, S=0.9), 2),                            # no contexts at all
    (dict(**LLAMA, l_P=0, ctx_lens=[129], l_k=1, T=0.8, S=0.7), 70),                        # 70 x 4 rows: two row blocks, ragged
    (dict(**LLAMA, l_P=5, ctx_lens=[100], l_k=2, T=0.9, S=0.9), 32),                        # 128 rows exactly, one tile: one half idle
    (dict(**LLAMA, l_P=5, ctx_lens=[100, 700], l_k=2, T=0.9, S=0.9), 33),                   # 132 rows: one 256-row block again
    (dict(**LLAMA, l_P=9, ctx_lens=[128 * 5], l_k=2, T=0.7, S=0.8), 9),                     # an odd number of whole tiles
])
def test_shared_context_decode(kw, n_req):
    lens = kw.pop("ctx_lens")
    b = wl.share_contexts(wl.make_batch(ctx_lens=[lens] * n_req, l_q=1, seed=21, name="shared", **kw))
    _check(b)


def test_shared_plan_agrees_with_the_per_request_plan_and_grows():
    b = wl.share_contexts(wl.make_batch(**LLAMA, l_P=32, ctx_lens=[[256] * 6] * 4, l_q=1, l_k=40, capacity=60, seed=22,
                                        T=0.9, S=0.9, name="shared_grow"))
    for t in (0, 1, 20):
        out = _check(b, kv_extra=t)
        ref, _, _ = gpu_attend(b, libape.APE_DECODE, kv_extra=t)                # ordinary decode plan on the same requests
        assert (out.float() - ref.float()).abs().max().item() <= 2e-2


def test_shared_plan_rejects_requests_that_do_not_share():
    b = wl.make_batch(**LLAMA, l_P=8, ctx_lens=[[64], [64]], l_q=1, l_k=4, seed=23)     # two different context sets
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.empty_like(q)
    with pytest.raises(libape.ApeError) as e:
        handle().attend_plan(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests,
                             mode=libape.APE_DECODE, shared=True)
    assert e.value.code == -1
    s = wl.share_contexts(b)
    s.requests[1].q_start = 0                                                          # rows not consecutive
    with pytest.raises(libape.ApeError) as e:
        handle().attend_plan(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=s.requests,
                             mode=libape.APE_DECODE, shared=True)
    assert e.value.code == -1


def test_shared_decode_at_the_benchmark_size_sampled_requests():
    """16 requests over one set of 500 x 256 cached context tokens behind a 64-token prefix, the shape bench.py times;
    the oracle checks sampled requests at the first and a late decode step."""
    lens = [[256] * 500] + [[]] * 15                      # only request 0 owns contexts in the pool; the others borrow them
    b = wl.share_contexts(wl.make_batch(**LLAMA, l_P=64, ctx_lens=lens, l_q=1, l_k=257, capacity=257 + 255, seed=31,
                                        T=0.9, S=0.9, name="shared_128k"))
    for t in (0, 255):
        out, lse, n = gpu_attend(b, libape.APE_DECODE, shared=True, kv_extra=t)
        assert n == 3
        for r in (0, 7, 15):
            rq = b.requests[r]
            ref = oracle_attend(b, r, l_k=rq.query_kv[1] + t)
            compare(out[r:r + 1], ref.out.float(), f"shared 128K step {t} req {r}")
            assert (lse[r:r + 1].double() - ref.lse).abs().max().item() < 2e-3
