"""GPU parity of the fused rotary embedding + cache write against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ape_oracle, rope_oracle as ro
from paper_2502_05431_b200 import libape, workloads as wl
from tests.gpu_util import handle, compare

pytestmark = pytest.mark.gpu


def _check_rot(got: torch.Tensor, want: np.ndarray, x_absmax: float):
    """Tolerance: the kernel rotates in fp32 from bf16 inputs and rounds once to bf16 (relative 2^-9); the fp32 sine and
    cosine of the double-reduced angle and the two fp32 products add an absolute error of a few 1e-7 times the larger
    input component, which only shows where the two terms of a component cancel."""
    g = got.detach().cpu().to(torch.float64).numpy()
    err = np.abs(g - want)
    tol = 2.0 ** -8 * np.abs(want) + 4e-6 * x_absmax
    bad = err > tol
    assert not bad.any(), (int(bad.sum()), float(err.max()))


@pytest.mark.parametrize("H,d,theta", [(8, 128, 500000.0), (32, 128, 500000.0), (8, 64, 10000.0), (1, 64, 10000.0)])
def test_rope_runs_against_oracle(H, d, theta):
    dev = "cuda:0"
    g = torch.Generator().manual_seed(11)
    n_src, n_dst = 700, 1200
    x = torch.randn(n_src, H, d, generator=g).to(torch.bfloat16)
    # ragged runs: lengths that are no multiple of the work-item size, large start positions, an empty run, a gap in dst
    runs = [(0, 5, 37, 0), (37, 100, 1, 123456), (38, 300, 0, 9), (38, 301, 300, 131000), (338, 700, 362, 17)]
    xs = x.to(dev)
    sentinel = torch.full((n_dst, H, d), 7.0, dtype=torch.bfloat16, device=dev)
    dst = sentinel.clone()
    plan = libape.RopePlan(handle(), d, theta, runs)
    plan.write(xs, dst, rotate=True)
    torch.cuda.synchronize()
    out = dst.cpu()
    touched = torch.zeros(n_dst, dtype=torch.bool)
    for s0, d0, ln, p0 in runs:
        if ln == 0:
            continue
        want = ro.rope(x[s0:s0 + ln], np.arange(p0, p0 + ln), theta)
        _check_rot(out[d0:d0 + ln], want, float(x.abs().max()))
        touched[d0:d0 + ln] = True
    assert torch.equal(out[~touched], sentinel.cpu()[~touched])          # rows outside the runs are not written
    # the copy form (V) is bit exact
    dst2 = sentinel.clone()
    plan.write(xs, dst2, rotate=False)
    torch.cuda.synchronize()
    for s0, d0, ln, p0 in runs:
        assert torch.equal(dst2[d0:d0 + ln].cpu(), x[s0:s0 + ln])
    assert handle().get_status() == 0


def test_runs_for_request_follow_position_reuse():
    b = wl.make_batch(H_q=8, H_kv=2, d=64, l_P=16, ctx_lens=[[64, 10, 33]], l_q=4, seed=3)
    rq = b.requests[0]
    runs = libape.rope_runs_for_request(rq, src_start=100)
    want_pos = ro.positions(16, [64, 10, 33], 4)
    assert [r[3] for r in runs] == [0, 16, 16, 16, int(want_pos["query"][0])]
    assert [r[2] for r in runs] == [16, 64, 10, 33, rq.query_kv[1]]
    assert [r[1] for r in runs] == [rq.prefix[0]] + [s for s, _ in rq.ctx] + [rq.query_kv[0]]
    src = [r[0] for r in runs]
    assert src[0] == 100 and all(src[i + 1] == src[i] + runs[i][2] for i in range(len(runs) - 1))


def test_rope_rejects_bad_arguments():
    h = handle()
    with pytest.raises(libape.ApeError) as e:
        libape.RopePlan(h, 96, 10000.0, [(0, 0, 4, 0)])
    assert e.value.code == -2
    with pytest.raises(libape.ApeError) as e:
        libape.RopePlan(h, 64, 0.5, [(0, 0, 4, 0)])
    assert e.value.code == -4
    with pytest.raises(libape.ApeError) as e:
        libape.RopePlan(h, 64, 10000.0, [(0, 0, -1, 0)])
    assert e.value.code == -1
    plan = libape.RopePlan(h, 64, 10000.0, [(0, 90, 20, 0)])
    x = torch.zeros(20, 2, 64, dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(libape.ApeError) as e:                            # run reaches past the destination
        plan.write(x, torch.zeros(100, 2, 64, dtype=torch.bfloat16, device="cuda:0"), rotate=True)
    assert e.value.code == -1


def test_rope_then_encode_matches_the_oracle_pipeline():
    """The step in front of the pre-caching attention: raw K, V, Q of the prefix and the contexts are rotated (position
    re-use) and written to the pool, then ape_encode_contexts runs on them.  Oracle: rope in fp64, rounded to bf16 where
    the cache is bf16, then the oracle's encode."""
    dev = "cuda:0"
    H_q, H_kv, d, theta = 8, 2, 64, 10000.0
    b = wl.make_batch(H_q=H_q, H_kv=H_kv, d=d, l_P=20, ctx_lens=[[150, 64, 7]], l_q=3, seed=5, with_encode_q=True)
    rq = b.requests[0]
    runs = libape.rope_runs_for_request(rq, src_start=0)[:-1]            # prefix and contexts (encode has no query rows)
    n_src = sum(r[2] for r in runs)
    g = torch.Generator().manual_seed(77)
    k_raw = torch.randn(n_src, H_kv, d, generator=g).to(torch.bfloat16)
    v_raw = torch.randn(n_src, H_kv, d, generator=g).to(torch.bfloat16)
    q_raw = torch.randn(n_src, H_q, d, generator=g).to(torch.bfloat16)
    n_pool = b.k_pool.shape[0]
    k_pool = torch.zeros(n_pool, H_kv, d, dtype=torch.bfloat16, device=dev)
    v_pool = torch.zeros_like(k_pool)
    q_enc = torch.zeros(n_pool, H_q, d, dtype=torch.bfloat16, device=dev)
    h = handle()
    plan = libape.RopePlan(h, d, theta, runs)
    plan.write(k_raw.to(dev), k_pool, rotate=True)
    plan.write(v_raw.to(dev), v_pool, rotate=False)
    plan.write(q_raw.to(dev), q_enc, rotate=True)
    out = torch.zeros_like(q_enc)
    ep = h.encode_plan(H_q=H_q, H_kv=H_kv, d=d, k_pool=k_pool, v_pool=v_pool, q=q_enc, out=out, prefix=rq.prefix, ctx=rq.ctx)
    ep.encode_contexts()
    torch.cuda.synchronize()
    assert h.get_status() == 0
    # oracle pipeline on the CPU
    def rot(x, run):
        s0, d0, ln, p0 = run
        return torch.from_numpy(ro.rope(x[s0:s0 + ln], np.arange(p0, p0 + ln), theta)).to(torch.bfloat16)
    pre = (rot(k_raw, runs[0]), v_raw[runs[0][0]:runs[0][0] + runs[0][2]])
    ctx_kv = [(rot(k_raw, r), v_raw[r[0]:r[0] + r[2]]) for r in runs[1:]]
    ctx_q = [rot(q_raw, r) for r in runs[1:]]
    want, _ = ape_oracle.encode([t.contiguous() for t in ctx_q], (pre[0].contiguous(), pre[1].contiguous()),
                                [(k.contiguous(), v.contiguous()) for k, v in ctx_kv])
    for n, ((s, l), w) in enumerate(zip(rq.ctx, want)):
        if l:
            compare(out[s:s + l].cpu(), w, f"rope+encode ctx {n}")


def test_rope_at_the_benchmark_size_sampled_rows():
    """K (rotated) and V (copied) of 64 + 500 x 256 tokens under position re-use, the shape bench.py times; the oracle
    checks sampled rows of every kind of run (prefix, first / middle / last context)."""
    dev = "cuda:0"
    H, d, theta, n_ctx = 8, 128, 500000.0, 500
    runs = [(0, 0, 64, 0)] + [(64 + i * 256, 64 + i * 256, 256, 64) for i in range(n_ctx)]
    n_tok = 64 + n_ctx * 256
    g = torch.Generator().manual_seed(41)
    x = torch.randn(n_tok, H, d, generator=g).to(torch.bfloat16)
    dst = torch.zeros(n_tok, H, d, dtype=torch.bfloat16, device=dev)
    plan = libape.RopePlan(handle(), d, theta, runs)
    plan.write(x.to(dev), dst, rotate=True)
    torch.cuda.synchronize()
    out = dst.cpu()
    pos = np.concatenate([np.arange(64)] + [64 + np.arange(256)] * n_ctx)
    rows = np.unique(np.concatenate([np.arange(0, 80), np.arange(64 + 255, 64 + 258), np.arange(64000, 64300),
                                     np.arange(n_tok - 300, n_tok)]))
    _check_rot(out[rows], ro.rope(x[rows], pos[rows], theta), float(x.abs().max()))
    assert handle().get_status() == 0
