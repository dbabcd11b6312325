"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle, element by element on the same
seeded inputs.  Tolerance (bf16 output, fp32 accumulation): max-abs 2e-2, mean-abs 2e-3; relative L2 reported."""
import numpy as np
import pytest
import torch

from oracle import ape_oracle as orc
from paper_2502_05431_b200 import libape
from paper_2502_05431_b200 import workloads as wl
from tests.gpu_util import compare, gpu_attend, handle, oracle_attend

pytestmark = pytest.mark.gpu
LLAMA = dict(H_q=32, H_kv=8, d=128)


def _check_batch(b, mode, rows=None, lse_tol=2e-3, **kw):
    out, lse, n = gpu_attend(b, mode, **kw)
    assert n == 2
    for r, rq in enumerate(b.requests):
        ref = oracle_attend(b, r, rows=rows, l_k=(rq.query_kv[1] + kw.get("kv_extra", 0)) if kw.get("kv_extra") else None,
                            q_override=None if kw.get("q_override") is None else kw["q_override"][rq.q_start:rq.q_start + rq.q_len])
        compare(out[rq.q_start:rq.q_start + rq.q_len], ref.out.float(), f"{b.name} req {r} O")
        sel = ~torch.isnan(ref.lse)
        d = (lse[rq.q_start:rq.q_start + rq.q_len].double()[sel] - ref.lse[sel]).abs().max().item()
        assert d < lse_tol, f"{b.name} req {r}: LSE error {d}"


# ---- decode -------------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("kw", [
    dict(H_q=4, H_kv=1, d=64, l_P=16, ctx_lens=[[64] * 4], l_k=17, T=0.8, S=0.9),                  # tiny, d = 64
    dict(**LLAMA, l_P=5, ctx_lens=[[70, 1, 129], [200]], l_k=3, gap=3, T=0.7, S=0.8),               # ragged, gaps, 2 requests
    dict(**LLAMA, l_P=0, ctx_lens=[[]], l_k=1),                                                      # only its own key
    dict(**LLAMA, l_P=0, ctx_lens=[[333]], l_k=1, T=0.5, S=1.2, shuffle_ctx=True),
    dict(H_q=16, H_kv=1, d=128, l_P=64, ctx_lens=[[256] * 3], l_k=65, T=0.9, S=0.9),                # G = 16
    dict(H_q=8, H_kv=8, d=64, l_P=3, ctx_lens=[[100, 100]], l_k=9, T=0.9, S=0.5),                   # G = 1
    dict(H_q=16, H_kv=8, d=128, l_P=9, ctx_lens=[[65, 190]], l_k=2, T=0.9, S=0.9),                  # G = 2
    dict(H_q=8, H_kv=1, d=64, l_P=70, ctx_lens=[[64] * 5], l_k=130, T=1.3, S=0.9),                  # G = 8, d = 64
])
def test_decode_small(kw):
    b = wl.make_batch(l_q=1, seed=1, name="decode_small", **kw)
    _check_batch(b, libape.APE_DECODE)


def test_decode_many_tiles_and_growing_query_segment():
    """Enough tokens that every CTA holds several items; kv_extra grows the query segment step by step."""
    b = wl.make_batch(**LLAMA, l_P=64, ctx_lens=[[256] * 40, [512] * 11], l_q=1, l_k=100, capacity=100 + 70, seed=2,
                      T=0.9, S=0.9, name="decode_grow")
    for t in (0, 1, 27, 70):
        _check_batch(b, libape.APE_DECODE, kv_extra=t)


def test_decode_rejects_bad_arguments():
    b = wl.make_batch(**LLAMA, l_P=8, ctx_lens=[[64]], l_q=1, l_k=4, capacity=6, seed=3)
    dev = torch.device("cuda:0")
    q, k, v = b.q.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.empty_like(q)
    plan = handle().attend_plan(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, mode=libape.APE_DECODE)
    ws = plan.alloc_workspace()
    for T, S in [(0.0, 1.0), (1.0, -1.0), (float("nan"), 1.0), (1.0, float("inf"))]:
        with pytest.raises(libape.ApeError) as e:
            plan.attend(T, S, ws)
        assert e.value.code == -4
    with pytest.raises(libape.ApeError) as e:
        plan.attend(1.0, 1.0, ws, kv_extra=3)          # beyond the reserved capacity
    assert e.value.code == -4
    with pytest.raises(libape.ApeError) as e:
        plan.attend(1.0, 1.0, ws[:256])                # workspace too small
    assert e.value.code == -6
    with pytest.raises(libape.ApeError) as e:
        plan.encode_contexts()
    assert e.value.code == -10
    with pytest.raises(libape.ApeError) as e:          # head_dim 96 unsupported
        handle().attend_plan(H_q=32, H_kv=8, d=96, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests, mode=libape.APE_DECODE)
    assert e.value.code == -2
    bad = wl.Request(0, 1, (0, 8), [(10, 10 ** 9)], b.requests[0].query_kv, 6)
    with pytest.raises(libape.ApeError) as e:
        handle().attend_plan(H_q=32, H_kv=8, d=128, k_pool=k, v_pool=v, q=q, out=out, requests=[bad], mode=libape.APE_DECODE)
    assert e.value.code == -1


# ---- query prefill ----------------------------------------------------------------------------------------------------

def test_prefill_config1_tiny():
    _check_batch(wl.config1(), libape.APE_PREFILL)


@pytest.mark.parametrize("kw", [
    dict(**LLAMA, l_P=32, ctx_lens=[[256] * 10], l_q=64, T=0.9, S=0.9),                     # config 2
    dict(**LLAMA, l_P=7, ctx_lens=[[130, 1, 255], [77]], l_q=33, l_k=50, gap=5, T=0.6, S=0.7),    # ragged, l_k > l_q
    dict(**LLAMA, l_P=0, ctx_lens=[[]], l_q=200, T=1.0, S=1.0),                             # plain causal attention
    dict(H_q=8, H_kv=8, d=64, l_P=10, ctx_lens=[[300]], l_q=300, T=0.8, S=1.1),             # G = 1, d = 64, 2 row blocks
    dict(H_q=16, H_kv=1, d=128, l_P=64, ctx_lens=[[256] * 4], l_q=40, T=0.9, S=0.9),        # G = 16
    dict(**LLAMA, l_P=64, ctx_lens=[[512] * 9], l_q=320, T=0.9, S=0.9),                     # 5 row blocks > 4 siblings
    dict(H_q=16, H_kv=8, d=128, l_P=40, ctx_lens=[[300], [10, 500]], l_q=130, T=0.9, S=0.9),   # G = 2, 2 requests
    dict(H_q=8, H_kv=1, d=64, l_P=1, ctx_lens=[[129]], l_q=33, l_k=40, T=0.7, S=1.0),            # G = 8, d = 64
    dict(**LLAMA, l_P=0, ctx_lens=[[4096]], l_q=1, l_k=1, T=0.9, S=0.9),                         # a single query row
])
def test_prefill_shapes(kw):
    b = wl.make_batch(seed=4, name="prefill", **kw)
    _check_batch(b, libape.APE_PREFILL)


def test_prefill_ignores_garbage_outside_spans():
    """Pool tokens that belong to no span (gaps, reserved capacity) may hold NaN without affecting the result."""
    b = wl.make_batch(**LLAMA, l_P=20, ctx_lens=[[100, 60]], l_q=16, l_k=16, capacity=40, gap=7, seed=5, T=0.8, S=0.9, name="garbage")
    used = torch.zeros(b.k_pool.shape[0], dtype=torch.bool)
    rq = b.requests[0]
    for s, n in [rq.prefix, rq.query_kv] + rq.ctx:
        used[s:s + n] = True
    b.k_pool[~used] = float("nan")
    b.v_pool[~used] = float("nan")
    _check_batch(b, libape.APE_PREFILL)
    b1 = wl.make_batch(**LLAMA, l_P=20, ctx_lens=[[100, 60]], l_q=1, l_k=16, capacity=40, gap=7, seed=5, T=0.8, S=0.9, name="garbage_dec")
    b1.k_pool[~used] = float("nan")
    b1.v_pool[~used] = float("nan")
    _check_batch(b1, libape.APE_DECODE)


@pytest.mark.parametrize("T,S", [(0.5, 0.8), (0.5, 1.0), (0.9, 0.8), (0.9, 1.0)])
def test_prefill_config3_rag(T, S):
    b = wl.config3(T=T, S=S)
    out, lse, _ = gpu_attend(b, libape.APE_PREFILL)
    for r, rq in enumerate(b.requests):
        for rows in [(0, 4), (62, 66), (124, 128)]:
            ref = oracle_attend(b, r, rows=rows)
            compare(out[rq.q_start:rq.q_start + rq.q_len], ref.out.float(), f"cfg3 T={T} S={S} req {r} rows {rows}")


def test_prefill_config4_manyshot_128k_all_rows():
    """The 128K many-shot prefill in the launch configuration the benchmark times, every one of its 256 query rows and
    32 heads against the oracle (output and the log of Eq. 5's denominator)."""
    b = wl.config4()
    out, lse, _ = gpu_attend(b, libape.APE_PREFILL)
    assert not torch.isnan(out.float()).any()
    ref = oracle_attend(b, 0)
    compare(out, ref.out.float(), "cfg4 all rows")
    for rows in [(0, 64), (64, 128), (128, 192), (192, 256)]:            # no quarter of the row block hides behind the others
        compare(out[rows[0]:rows[1]], ref.out[rows[0]:rows[1]].float(), f"cfg4 rows {rows}")
    assert (lse.double() - ref.lse).abs().max().item() < 2e-3


def test_decode_config5_128k_all_requests():
    """Decode at 128K, batch 16, at the first, a middle and the last of the 256 steps: all 16 requests against the oracle."""
    b = wl.config5(n_req=16)
    q_steps = b.extra["q_steps"]
    for t in (0, 128, 255):
        out, lse, _ = gpu_attend(b, libape.APE_DECODE, kv_extra=t, q_override=q_steps[t].contiguous())
        for r in range(16):
            ref = oracle_attend(b, r, l_k=257 + t, q_override=q_steps[t, r:r + 1].contiguous())
            compare(out[r:r + 1], ref.out.float(), f"cfg5 step {t} req {r}")
            assert (lse[r:r + 1].double() - ref.lse).abs().max().item() < 2e-3


# ---- encode -----------------------------------------------------------------------------------------------------------

def _check_encode(b):
    dev = torch.device("cuda:0")
    q, k, v = b.q_enc.to(dev), b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], b.H_q), float("nan"), dtype=torch.float32, device=dev)
    rq = b.requests[0]
    plan = handle().encode_plan(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=out, prefix=rq.prefix, ctx=rq.ctx, lse=lse)
    plan.encode_contexts()
    torch.cuda.synchronize()
    assert handle().get_status() == 0
    out, lse = out.cpu(), lse.cpu()
    _, p, c, _ = b.views(0)
    qs = [b.q_enc[s:s + n] for s, n in rq.ctx]
    refs, lses = orc.encode(qs, p, c)
    touched = torch.zeros(out.shape[0], dtype=torch.bool)
    for (s, n), ref, l in zip(rq.ctx, refs, lses):
        if n == 0:
            continue
        compare(out[s:s + n], ref.float(), f"{b.name} ctx@{s}")
        assert (lse[s:s + n].double() - l).abs().max().item() < 2e-3
        touched[s:s + n] = True
    assert torch.isnan(out[~touched].float()).all(), "rows outside the context spans were written"


@pytest.mark.parametrize("kw", [
    dict(H_q=4, H_kv=1, d=64, l_P=16, ctx_lens=[[64] * 4]),                        # config 1 shape
    dict(**LLAMA, l_P=32, ctx_lens=[[256] * 10]),                                  # config 2
    dict(**LLAMA, l_P=0, ctx_lens=[[1, 129, 0, 300]], gap=3),                      # ragged, no prefix, an empty context
    dict(**LLAMA, l_P=200, ctx_lens=[[70, 700]]),                                  # prefix longer than a tile; 11 row blocks
    dict(H_q=8, H_kv=8, d=64, l_P=5, ctx_lens=[[300, 17]]),                        # G = 1, d = 64
    dict(H_q=8, H_kv=1, d=128, l_P=130, ctx_lens=[[33, 64, 65]]),                  # G = 8
    dict(**LLAMA, l_P=64, ctx_lens=[[10, 64, 65, 300, 1]]),                        # prefix tail shares a tile with contexts shorter / longer than the rest of it
    dict(**LLAMA, l_P=120, ctx_lens=[[7, 8, 9, 200]], gap=2),                      # 8 rows of the shared tile left for the context
    dict(H_q=8, H_kv=8, d=64, l_P=136, ctx_lens=[[250]]),                          # one whole prefix tile + a tail of 8
])
def test_encode(kw):
    b = wl.make_batch(l_q=1, seed=6, with_encode_q=True, name="encode", **kw)
    _check_encode(b)


def test_encode_bench_size_500x256():
    """The encode launch the benchmark times: 500 contexts x 256 tokens behind a 64-token prefix (16,000 work items, more
    than 100 per CTA, every context through the tile shared with the prefix tail and the bulk-store epilogue).  Every row
    of every context against the oracle; rows outside the spans must stay untouched."""
    b = wl.config4(with_encode_q=True)
    _check_encode(b)


def test_encode_many_short_items_per_cta():
    """600 contexts x 64 tokens behind a 72-token prefix: 4,800 one-row-block items, about 32 per CTA, so every CTA
    walks both Q buffers many times; the prefix tail (72 rows) shares a tile with 56 of each context's 64 tokens."""
    b = wl.make_batch(**LLAMA, l_P=72, ctx_lens=[[64] * 600], l_q=1, seed=8, with_encode_q=True, name="encode_many_items")
    _check_encode(b)


def test_encode_many_ragged_items_per_cta():
    """The same with ragged lengths (row blocks that are not full leave through per-thread stores, full ones through the
    bulk store, interleaved on the same Q buffers) and a prefix that is no multiple of 8 (no shared tile)."""
    g = torch.Generator().manual_seed(9)
    lens = torch.randint(1, 200, (400,), generator=g).tolist()
    b = wl.make_batch(**LLAMA, l_P=67, ctx_lens=[lens], l_q=1, seed=9, with_encode_q=True, gap=1, name="encode_ragged_items")
    _check_encode(b)


def test_attend_host_matches_attend():
    """The host-buffer entry point (pinned host tensors in and out) gives the same result as the device-pointer one."""
    b = wl.make_batch(**LLAMA, l_P=32, ctx_lens=[[256] * 6], l_q=64, seed=9, T=0.9, S=0.9, name="host")
    ref, _, _ = gpu_attend(b, libape.APE_PREFILL, want_lse=False)
    dev = torch.device("cuda:0")
    q, k, v = torch.zeros_like(b.q, device=dev), torch.zeros_like(b.k_pool, device=dev), torch.zeros_like(b.v_pool, device=dev)
    out = torch.zeros_like(q)
    plan = handle().attend_plan(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests,
                                mode=libape.APE_PREFILL)
    ws = plan.alloc_workspace()
    hq, hk, hv = b.q.pin_memory(), b.k_pool.pin_memory(), b.v_pool.pin_memory()
    hout = torch.empty_like(hq).pin_memory()
    h2d, d2h = plan.attend_host(b.T, b.S, ws, hq, hk, hv, hout)
    assert h2d == hq.numel() * 2 + 2 * hk.numel() * 2 and d2h == hq.numel() * 2
    assert torch.equal(hout, ref)
    plan.close()


def test_decode_step_host_appends_and_attends():
    """The host-buffer decode step: the new token's Q, K, V come from (pinned) host tensors, K and V are appended to the
    cache rows the query segment has reached, O comes back to the host.  The device pool starts with NaN in the reserved
    tail, so a missing or misplaced append cannot go unnoticed.  Three consecutive steps against the oracle."""
    b = wl.make_batch(**LLAMA, l_P=16, ctx_lens=[[256, 70], [130]], l_q=1, l_k=9, capacity=12, gap=2, seed=14, T=0.9, S=0.8,
                      name="decode_step_host")
    dev = torch.device("cuda:0")
    k, v = b.k_pool.to(dev), b.v_pool.to(dev)
    for rq in b.requests:                                   # nothing beyond the planned length is on the device yet
        s0 = rq.query_kv[0] + rq.query_kv[1]
        k[s0:rq.query_kv[0] + rq.query_kv_capacity] = float("nan")
        v[s0:rq.query_kv[0] + rq.query_kv_capacity] = float("nan")
    q = torch.zeros_like(b.q, device=dev)
    out = torch.full_like(q, float("nan"))
    plan = handle().attend_plan(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=out, requests=b.requests,
                                mode=libape.APE_DECODE)
    ws = plan.alloc_workspace()
    g = torch.Generator().manual_seed(15)
    for t in (0, 1, 2):
        hq = torch.randn(len(b.requests), b.H_q, b.d, generator=g).to(torch.bfloat16).pin_memory()
        hout = torch.empty_like(hq).pin_memory()
        if t == 0:
            up, down = plan.decode_step_host(b.T, b.S, ws, hq, hout, kv_extra=0)          # the planned tokens are all cached
            assert up == hq.numel() * 2
        else:
            rows = [rq.query_kv[0] + rq.query_kv[1] - 1 + t for rq in b.requests]
            hk = torch.stack([b.k_pool[r] for r in rows]).contiguous().pin_memory()
            hv = torch.stack([b.v_pool[r] for r in rows]).contiguous().pin_memory()
            up, down = plan.decode_step_host(b.T, b.S, ws, hq, hout, h_k_new=hk, h_v_new=hv, kv_extra=t)
            assert up == hq.numel() * 2 + 2 * hk.numel() * 2
        assert down == hq.numel() * 2
        for r, rq in enumerate(b.requests):
            ref = oracle_attend(b, r, l_k=rq.query_kv[1] + t, q_override=hq[r:r + 1].contiguous())
            compare(hout[r:r + 1], ref.out.float(), f"decode_step_host step {t} req {r}")
    assert handle().get_status() == 0
    plan.close()


# ---- per-context form (Eq. 11-12) -------------------------------------------------------------------------------------

@pytest.mark.parametrize("mode,kw", [
    (libape.APE_PREFILL, dict(**LLAMA, l_P=32, ctx_lens=[[256] * 10], l_q=64, T=0.9, S=0.7)),
    (libape.APE_PREFILL, dict(**LLAMA, l_P=7, ctx_lens=[[130, 1, 255, 0, 40], [77]], l_q=33, l_k=50, gap=5, T=0.6, S=0.5, shuffle_ctx=True)),
    (libape.APE_PREFILL, dict(H_q=4, H_kv=1, d=64, l_P=16, ctx_lens=[[64] * 4], l_q=16, T=0.8, S=0.9)),
    (libape.APE_DECODE, dict(**LLAMA, l_P=5, ctx_lens=[[70, 1, 129], [200, 300, 64, 64]], l_q=1, l_k=3, gap=3, T=0.7, S=0.6)),
    (libape.APE_DECODE, dict(**LLAMA, l_P=64, ctx_lens=[[256] * 40], l_q=1, l_k=100, T=0.9, S=0.8)),
])
def test_per_context_form(mode, kw):
    """S on every context's own log-sum-exp: checked against the oracle's per-context switch; differs from Eq. 5."""
    b = wl.make_batch(seed=11, name="per_context", **kw)
    out, lse, _ = gpu_attend(b, mode, per_context=True)
    flat, _, _ = gpu_attend(b, mode)
    differs = False
    for r, rq in enumerate(b.requests):
        q, p, c, k = b.views(r)
        ref = orc.attend(q, p, c, k, b.T, b.S, per_context=True)
        sl = slice(rq.q_start, rq.q_start + rq.q_len)
        compare(out[sl], ref.out.float(), f"per-context req {r}")
        assert (lse[sl].double() - ref.lse).abs().max().item() < 2e-3
        differs |= (out[sl].float() - flat[sl].float()).abs().max().item() > 1e-3
    assert differs, "the per-context form should not coincide with Eq. 5 here (several contexts, S != 1)"


def test_per_context_form_with_one_context_equals_flat():
    b = wl.make_batch(**LLAMA, l_P=20, ctx_lens=[[700]], l_q=40, seed=12, T=0.8, S=0.6, name="one_ctx")
    a, _, _ = gpu_attend(b, libape.APE_PREFILL, per_context=True)
    f, _, _ = gpu_attend(b, libape.APE_PREFILL)
    assert (a.float() - f.float()).abs().max().item() <= 2e-2


def test_prefill_long_query_many_row_blocks():
    """1,500 causal query rows (24 row blocks, six sibling groups) over a modest context: sampled rows against the oracle."""
    b = wl.make_batch(**LLAMA, l_P=64, ctx_lens=[[700, 300]], l_q=1500, l_k=1600, seed=13, T=0.9, S=0.9, name="long_q")
    out, lse, _ = gpu_attend(b, libape.APE_PREFILL)
    assert not torch.isnan(out.float()).any()
    for rows in [(0, 3), (63, 66), (700, 703), (1497, 1500)]:
        ref = oracle_attend(b, 0, rows=rows)
        compare(out, ref.out.float(), f"long_q rows {rows}")
        sel = ~torch.isnan(ref.lse)
        assert (lse.double()[sel] - ref.lse[sel]).abs().max().item() < 2e-3


# ---- the error path of the bounded waits -------------------------------------------------------------------------------

def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    h = handle()
    assert h.get_status() == 0
    h.selftest_timeout()                       # one warp waits (bounded, about a second) on a barrier nothing completes
    assert h.get_status() == -8                # APE_ERR_TIMEOUT, read once ...
    assert h.get_status() == 0                 # ... and cleared
    assert libape.status_string(-8)
    b = wl.make_batch(**LLAMA, l_P=16, ctx_lens=[[64, 64]], l_q=1, l_k=5, seed=77, T=0.9, S=0.9, name="after_timeout")
    _check_batch(b, libape.APE_DECODE)         # the same context still computes correctly
