"""GPU tests of the C-ABI boundary itself: error codes that only a live handle can reach, the device the caller had
current, the stream-ordered status read, and the SM budget (a different split of the key/value stream over thread
blocks must not change the result: a race between partials or a slot that the merge reads but nobody wrote shows up
as a difference between budgets)."""
import ctypes as C

import pytest
import torch

from paper_2502_05431_b200 import libape
from paper_2502_05431_b200 import workloads as wl
from tests.gpu_util import compare, gpu_attend, handle, oracle_attend

pytestmark = pytest.mark.gpu
LLAMA = dict(H_q=32, H_kv=8, d=128)


def _dev_batch(**kw):
    b = wl.make_batch(**kw)
    dev = torch.device("cuda:0")
    return b, b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)


def test_misaligned_pointers_and_strides_are_refused():
    b, q, k, v = _dev_batch(**LLAMA, l_P=8, ctx_lens=[[64]], l_q=4, seed=31)
    out = torch.empty_like(q)
    plan_kw = dict(H_q=32, H_kv=8, d=128, requests=b.requests, mode=libape.APE_PREFILL)
    # a Q tensor that starts 2 bytes into an allocation
    q_off = torch.empty(q.numel() + 8, dtype=torch.bfloat16, device=q.device)[1:1 + q.numel()].view(q.shape)
    with pytest.raises(libape.ApeError) as e:
        handle().attend_plan(k_pool=k, v_pool=v, q=q_off, out=out, **plan_kw)
    assert e.value.code == -3
    # a head stride that is not a multiple of 8 elements (rows of 129 elements)
    wide = torch.empty(q.shape[0], 32, 129, dtype=torch.bfloat16, device=q.device)[:, :, :128]
    with pytest.raises(libape.ApeError) as e:
        handle().attend_plan(k_pool=k, v_pool=v, q=q, out=wide, **plan_kw)
    assert e.value.code == -3
    # an LSE pointer that is not float-aligned
    lse_raw = torch.empty(q.shape[0] * 32 * 4 + 8, dtype=torch.uint8, device=q.device)
    lse_bad = lse_raw[2:2 + q.shape[0] * 32 * 4]
    with pytest.raises(libape.ApeError) as e:
        handle().attend_plan(k_pool=k, v_pool=v, q=q, out=out, lse=lse_bad, **plan_kw)
    assert e.value.code == -3
    # the KV pool
    k_off = torch.empty(k.numel() + 8, dtype=torch.bfloat16, device=q.device)[4:4 + k.numel()].view(k.shape)
    with pytest.raises(libape.ApeError) as e:
        handle().attend_plan(k_pool=k_off, v_pool=k_off, q=q, out=out, **plan_kw)
    assert e.value.code == -3


def test_a_pool_too_large_for_the_copy_engine_is_refused():
    """Token coordinates are 32-bit: a pool of 2^31 tokens cannot be described (APE_ERR_LAYOUT).  Only the descriptor says
    so; no such memory exists or is touched, planning stops at the check."""
    b, q, k, v = _dev_batch(**LLAMA, l_P=8, ctx_lens=[[64]], l_q=4, seed=32)
    out = torch.empty_like(q)
    lib = libape.load()
    shape = libape.ape_shape_t(32, 8, 128, 0.0)
    pool = libape.ape_kv_pool_t(k.data_ptr(), v.data_ptr(), 1 << 31, k.stride(0), k.stride(1))
    qr, orows = libape._rows(q), libape._rows(out)
    arr, _keep = libape._request_array(b.requests)
    p = C.c_void_p()
    rc = lib.ape_attend_plan(handle()._h, C.byref(shape), C.byref(pool), C.byref(qr), C.byref(orows), None, arr, 1,
                             libape.APE_PREFILL, C.byref(p))
    assert rc == -5 and not p.value
    big_rows = libape.ape_rows_t(q.data_ptr(), 1 << 31, q.stride(0), q.stride(1))
    pool = libape._pool(k, v)
    rc = lib.ape_attend_plan(handle()._h, C.byref(shape), C.byref(pool), C.byref(big_rows), C.byref(big_rows), None, arr, 1,
                             libape.APE_PREFILL, C.byref(p))
    assert rc == -5 and not p.value


def test_the_callers_current_device_is_kept():
    before = torch.cuda.current_device()
    b = wl.make_batch(**LLAMA, l_P=8, ctx_lens=[[64]], l_q=1, l_k=4, seed=33, T=0.9, S=0.9)
    gpu_attend(b, libape.APE_DECODE)
    assert torch.cuda.current_device() == before


def test_status_read_in_stream_order():
    h = handle()
    s = torch.cuda.Stream()
    assert h.get_status_stream(s) == 0
    h.selftest_timeout(stream=s)               # a bounded wait that runs out (about a second), enqueued on s
    assert h.get_status_stream(s) == -8        # waits for s only, reports, clears in stream order
    assert h.get_status_stream(s) == 0
    assert h.get_status() == 0


@pytest.mark.parametrize("budget", [1, 37, 101])
def test_sm_budget_changes_the_split_not_the_result(budget):
    """The same three workloads planned for 1, 37 and 101 thread blocks instead of 148: other chunk boundaries of the
    stream-K split, other partial slots, another merge order.  Each against the oracle and against the full-device plan."""
    h = handle()
    cases = [
        (libape.APE_PREFILL, wl.make_batch(**LLAMA, l_P=64, ctx_lens=[[512] * 9], l_q=320, seed=41, T=0.9, S=0.9, name="budget_prefill")),
        (libape.APE_PREFILL, wl.make_batch(**LLAMA, l_P=7, ctx_lens=[[130, 1, 255], [77]], l_q=33, l_k=50, gap=5, seed=42, T=0.6, S=0.7,
                                           name="budget_ragged")),
        (libape.APE_DECODE, wl.make_batch(**LLAMA, l_P=64, ctx_lens=[[256] * 40, [512] * 11], l_q=1, l_k=100, capacity=170, seed=43,
                                          T=0.9, S=0.9, name="budget_decode")),
    ]
    for mode, b in cases:
        full, lse_full, _ = gpu_attend(b, mode)
        try:
            h.set_sm_budget(budget)
            out, lse, _ = gpu_attend(b, mode)
        finally:
            h.set_sm_budget(0)
        assert (out.float() - full.float()).abs().max().item() <= 2e-2
        assert (lse - lse_full).abs().max().item() < 2e-3
        for r, rq in enumerate(b.requests):
            ref = oracle_attend(b, r)
            compare(out[rq.q_start:rq.q_start + rq.q_len], ref.out.float(), f"{b.name} budget {budget} req {r}")
    with pytest.raises(libape.ApeError) as e:
        h.set_sm_budget(100000)
    assert e.value.code == -1


def test_shared_context_plan_under_a_budget():
    h = handle()
    b = wl.share_contexts(wl.make_batch(**LLAMA, l_P=16, ctx_lens=[[256, 100, 300]] * 5, l_q=1, l_k=9, capacity=12, seed=44,
                                        T=0.9, S=0.8, name="budget_shared"))
    try:
        h.set_sm_budget(29)
        out, lse, n = gpu_attend(b, libape.APE_DECODE, shared=True, kv_extra=2)
    finally:
        h.set_sm_budget(0)
    assert n == 3
    for r, rq in enumerate(b.requests):
        ref = oracle_attend(b, r, l_k=rq.query_kv[1] + 2)
        compare(out[r:r + 1], ref.out.float(), f"budget_shared req {r}")


@pytest.mark.parametrize("budget", [5, 148])
def test_two_pass_forms_under_another_split(budget):
    """The per-context form in prefill (two passes: node statistics, biased prefill) with the context run cut into few and
    into many items: a node's tiles never straddle two items, long nodes included (one context of 40 tiles), and the
    result does not depend on where the cuts fall."""
    from oracle import ape_oracle as orc
    h = handle()
    b = wl.make_batch(**LLAMA, l_P=20, ctx_lens=[[5000, 130, 1, 255, 700, 64, 64, 64]], l_q=70, l_k=90, seed=45, T=0.8, S=0.7,
                      name="two_pass_split")
    try:
        h.set_sm_budget(budget)
        out, lse, n = gpu_attend(b, libape.APE_PREFILL, per_context=True)
    finally:
        h.set_sm_budget(0)
    assert n == 4
    q, p, c, k = b.views(0)
    ref = orc.attend(q, p, c, k, b.T, b.S, per_context=True)
    compare(out, ref.out.float(), f"two-pass per-context, budget {budget}")
    assert (lse.double() - ref.lse).abs().max().item() < 2e-3


@pytest.mark.parametrize("mode", [libape.APE_PREFILL, libape.APE_DECODE])
def test_attend_once_is_plan_launch_and_cleanup_in_one_call(mode):
    l_q = 40 if mode == libape.APE_PREFILL else 1
    b = wl.make_batch(**LLAMA, l_P=16, ctx_lens=[[64, 200, 130], [300]], l_q=l_q, l_k=l_q + 6, seed=46, T=0.8, S=0.9, name="once")
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.zeros_like(q)
    lse = torch.zeros(q.shape[0], 32, dtype=torch.float32, device=dev)
    handle().attend_once(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, mode=mode, T=b.T, S=b.S,
                         lse=lse)
    for r, rq in enumerate(b.requests):
        ref = oracle_attend(b, r)
        sl = slice(rq.q_start, rq.q_start + rq.q_len)
        compare(out[sl].cpu(), ref.out.float(), f"attend_once req {r}")
        assert (lse[sl].cpu().double() - ref.lse).abs().max().item() < 2e-3
    with pytest.raises(libape.ApeError) as e:
        handle().attend_once(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, mode=mode, T=-1.0, S=b.S)
    assert e.value.code == -4          # APE_ERR_RANGE: nothing was launched, nothing is left allocated


def test_repeated_launches_give_the_same_bits():
    """Every plan kind launched 25 times on the same workspace without a host synchronisation in between: the work split
    and the merge order are fixed by the plan, so a run that differs from the first one in a single bit means a race
    (a partial read before it was written, a stage recycled too early) -- the stand-in for a race detector here."""
    dev = torch.device("cuda:0")
    h = handle()

    def stable(make_plan, launch, out):
        plan = make_plan()
        ws = plan.alloc_workspace() if plan.workspace_bytes else None
        launch(plan, ws)
        torch.cuda.synchronize()
        first = out.clone()
        assert not torch.isnan(first.float()).any()
        for _ in range(25):
            out.fill_(0)
            launch(plan, ws)
        torch.cuda.synchronize()
        assert torch.equal(out, first)
        plan.close()
        assert h.get_status() == 0

    b = wl.make_batch(**LLAMA, l_P=64, ctx_lens=[[256] * 30, [700, 1, 300]], l_q=200, l_k=210, seed=47, T=0.9, S=0.8, name="stable",
                      with_encode_q=True)
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.zeros_like(q)
    common = dict(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests)
    for kind in (dict(), dict(per_context=True), dict(tree=([[-1] + [0] * 29, [-1, 0, 0]], None))):
        stable(lambda: h.attend_plan(mode=libape.APE_PREFILL, **common, **kind), lambda p, ws: p.attend(b.T, b.S, ws), out)
    qe = b.q_enc.to(dev)
    oe = torch.zeros_like(qe)
    rq = b.requests[0]
    stable(lambda: h.encode_plan(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=qe, out=oe, prefix=rq.prefix, ctx=rq.ctx),
           lambda p, ws: p.encode_contexts(), oe[rq.ctx[0][0]:rq.ctx[-1][0] + rq.ctx[-1][1]])
    d = wl.share_contexts(wl.make_batch(**LLAMA, l_P=16, ctx_lens=[[256] * 12] * 16, l_q=1, l_k=70, capacity=80, seed=48, T=0.9, S=0.9))
    q, k, v = d.q.to(dev), d.k_pool.to(dev), d.v_pool.to(dev)
    out = torch.zeros_like(q)
    common = dict(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=d.requests, mode=libape.APE_DECODE)
    for kind in (dict(), dict(shared=True)):
        stable(lambda: h.attend_plan(**common, **kind), lambda p, ws: p.attend(d.T, d.S, ws, kv_extra=3), out)
