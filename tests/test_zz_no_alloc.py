"""GPU test of ape_decode_noalloc, the decode step for callers that must not allocate device memory (an inference
server whose own pool owns the whole GPU, a latency-critical loop, a sandboxed plug-in).  It keeps its scratch in
a fixed device array inside the library, shared by all calls, so the test runs it twice in a row on different inputs
and compares each result with the plan-based entry point (ape_attend_plan + ape_attend), which uses caller-provided
scratch.  This file is collected last on purpose."""
import pytest
import torch

from paper_2502_05431_b200 import libape
from paper_2502_05431_b200 import workloads as wl
from tests.gpu_util import MAX_ABS, MEAN_ABS, handle

pytestmark = pytest.mark.gpu
LLAMA = dict(H_q=32, H_kv=8, d=128)
_set_up = False


def _both(b, kv_extra=0):
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out_ref = torch.full_like(q, float("nan"))
    lse_ref = torch.full((q.shape[0], b.H_q), float("nan"), dtype=torch.float32, device=dev)
    plan = handle().attend_plan(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=out_ref, requests=b.requests,
                                mode=libape.APE_DECODE, lse=lse_ref)
    ws = plan.alloc_workspace()
    plan.attend(b.T, b.S, ws, kv_extra=kv_extra)
    torch.cuda.synchronize()
    plan.close()
    out_new = torch.full_like(q, float("nan"))
    lse_new = torch.full_like(lse_ref, float("nan"))
    global _set_up
    if not _set_up:
        # The first call on a device looks up the fixed array, which is when the CUDA runtime materialises it (the
        # library image is loaded lazily); that one-time 8 MiB is not a call-time allocation, so it is kept out of
        # the measurement below.
        libape.decode_noalloc(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=out_new, requests=b.requests,
                              T=b.T, S=b.S, kv_extra=kv_extra, want_status=True)
        out_new.fill_(float("nan"))
        _set_up = True
    # everything the call needs is allocated above; from here on the library must not allocate
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]          # the driver's own count: sees cudaMalloc from any library
    st = libape.decode_noalloc(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=out_new, requests=b.requests,
                               T=b.T, S=b.S, kv_extra=kv_extra, lse=lse_new, want_status=True)
    assert st == 0
    assert torch.cuda.mem_get_info()[0] >= free_before, "device memory was allocated during the call"
    return out_ref.cpu().float(), out_new.cpu().float(), lse_ref.cpu(), lse_new.cpu()


def _close(a, b):
    assert not torch.isnan(b).any()
    err = (a - b).abs()
    assert err.max().item() <= MAX_ABS and err.mean().item() <= MEAN_ABS


def test_noalloc_decode_matches_planned_decode_twice_in_a_row():
    b1 = wl.make_batch(**LLAMA, l_P=64, ctx_lens=[[256] * 40, [512] * 11, [100, 3, 77]], l_q=1, l_k=100, capacity=170,
                       seed=21, T=0.9, S=0.9, name="noalloc_a")
    b2 = wl.make_batch(H_q=4, H_kv=1, d=64, l_P=5, ctx_lens=[[70, 1, 129]], l_q=1, l_k=3, gap=3, seed=22, T=0.6, S=1.1,
                       name="noalloc_b")
    for b, extra in ((b1, 0), (b2, 0), (b1, 33)):       # the second and third call find the first call's leftovers
        o_ref, o_new, l_ref, l_new = _both(b, kv_extra=extra)
        _close(o_ref, o_new)
        assert (l_ref - l_new).abs().max().item() < 2e-3


def test_noalloc_decode_asynchronous_form_and_limits():
    b = wl.make_batch(**LLAMA, l_P=8, ctx_lens=[[300]], l_q=1, l_k=4, capacity=6, seed=23, T=0.8, S=0.9)
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.full_like(q, float("nan"))
    assert libape.decode_noalloc(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, T=b.T, S=b.S) is None
    torch.cuda.synchronize()
    o_ref, o_new, _, _ = _both(b)
    _close(o_ref, out.cpu().float())
    # a batch whose tile list cannot fit the fixed array is refused on the host, before anything is launched:
    # 300,000 one-token contexts need 300,000 tile records (4.8 MB > 4 MiB)
    big = wl.Request(0, 1, b.requests[0].prefix, [(b.requests[0].ctx[0][0], 1)] * 300000, b.requests[0].query_kv, 6)
    with pytest.raises(libape.ApeError) as e:
        libape.decode_noalloc(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=[big], T=1.0, S=1.0)
    assert e.value.code == -6
    with pytest.raises(libape.ApeError) as e:
        libape.decode_noalloc(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, T=0.0, S=1.0)
    assert e.value.code == -4
    with pytest.raises(libape.ApeError) as e:
        libape.decode_noalloc(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, T=1.0, S=1.0, kv_extra=5)
    assert e.value.code == -4


def test_noalloc_decode_refuses_a_capturing_stream():
    """The call rebuilds its metadata from host arrays each time, so it can never be recorded into a CUDA graph: on a
    stream that is being captured it returns APE_ERR_MODE and enqueues nothing."""
    b = wl.make_batch(**LLAMA, l_P=8, ctx_lens=[[300]], l_q=1, l_k=4, capacity=6, seed=24, T=0.8, S=0.9)
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.full_like(q, float("nan"))
    kw = dict(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, T=b.T, S=b.S)
    libape.decode_noalloc(**kw)                       # the one-time set-up happens outside any capture
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        g.capture_begin()
        try:
            with pytest.raises(libape.ApeError) as e:
                libape.decode_noalloc(stream=s, **kw)
            with pytest.raises(libape.ApeError) as e2:
                handle().get_status_stream(s)
        finally:
            g.capture_end()
    assert e.value.code == -10 and e2.value.code == -10
    torch.cuda.synchronize()
    assert libape.decode_noalloc(want_status=True, **kw) == 0     # and the entry point still works afterwards


def test_noalloc_status_word_survives_asynchronous_calls():
    """A timeout raised on the fixed array stays there until a call reads it: asynchronous calls in between neither report
    nor erase it."""
    b = wl.make_batch(**LLAMA, l_P=8, ctx_lens=[[300]], l_q=1, l_k=4, capacity=6, seed=25, T=0.8, S=0.9)
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.full_like(q, float("nan"))
    kw = dict(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, T=b.T, S=b.S)
    assert libape.decode_noalloc(want_status=True, **kw) == 0
    libape.selftest_timeout_noalloc(0)                # one warp whose bounded wait runs out (about a second)
    assert libape.decode_noalloc(**kw) is None        # asynchronous: does not look at the word
    assert libape.decode_noalloc(**kw) is None
    assert libape.decode_noalloc(want_status=True, **kw) == -8
    assert libape.decode_noalloc(want_status=True, **kw) == 0
    o_ref, o_new, _, _ = _both(b)
    _close(o_ref, o_new)


def test_noalloc_size_gate_counts_fused_spans():
    """300,000 one-token contexts that touch each other are ONE span of 300,000 tokens (4,688 tiles): accepted, although
    300,000 separate tile records would not fit the fixed array."""
    n = 300000
    b = wl.make_batch(H_q=4, H_kv=1, d=64, l_P=8, ctx_lens=[[n]], l_q=1, l_k=4, capacity=6, seed=26, T=0.9, S=0.9)
    rq = b.requests[0]
    s0 = rq.ctx[0][0]
    many = wl.Request(rq.q_start, 1, rq.prefix, [(s0 + i, 1) for i in range(n)], rq.query_kv, rq.query_kv_capacity)
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out_a, out_b = torch.full_like(q, float("nan")), torch.full_like(q, float("nan"))
    kw = dict(H_q=4, H_kv=1, d=64, k_pool=k, v_pool=v, q=q, T=b.T, S=b.S)
    assert libape.decode_noalloc(out=out_a, requests=[many], want_status=True, **kw) == 0
    assert libape.decode_noalloc(out=out_b, requests=b.requests, want_status=True, **kw) == 0
    assert torch.equal(out_a, out_b) and not torch.isnan(out_a.float()).any()
