"""Small single-kernel cases for profiler captures: a few launches of one path on inputs larger than L2 but small
enough that a multi-pass capture ends by itself.

    python -m paper_2502_05431_b200.profile_case prefill|decode|encode [--iters 3]

prefill: 256 query rows over prefix 64 + 250 x 256 context tokens (KV 262 MB), Llama-3-8B head shape.
rag    : 4 requests x 20 contexts of 512..1536 tokens, 128 query rows each (KV 339 MB).
decode : 4 requests x (64 + 250 x 256 + 257) cached tokens (KV 1.05 GB), one new token each.
encode : 250 contexts x 256 tokens against a 64-token prefix.
Prints the CUDA-event time per launch pair and the algorithmic work, so that a capture can be scaled.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import libape, workloads as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["prefill", "decode", "encode", "rag", "rope", "shared"])
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--n-ctx", type=int, default=250)
    args = ap.parse_args()
    dev = "cuda:0"
    h = libape.Handle(0)
    H_q, H_kv, d = 32, 8, 128
    if args.case == "rag":
        # RAG shape: 4 independent requests, 20 contexts of 512..1536 tokens each, 128 query rows (config 3)
        lens = wl.config3_lens(0)
        b = wl.make_batch(H_q=H_q, H_kv=H_kv, d=d, l_P=64, ctx_lens=lens, l_q=128, seed=0, T=0.9, S=0.8, device=dev)
        out = torch.zeros_like(b.q)
        plan = h.attend_plan(H_q=H_q, H_kv=H_kv, d=d, k_pool=b.k_pool, v_pool=b.v_pool, q=b.q, out=out, requests=b.requests,
                             mode=libape.APE_PREFILL)
        ws = plan.alloc_workspace()
        run = lambda: plan.attend(b.T, b.S, ws)
        work = {"flops": sum(4.0 * d * H_q * (128 * (64 + sum(l)) + 128 * 129 / 2) for l in lens)}
    elif args.case == "decode":
        b = wl.config5(n_req=4, n_ctx=args.n_ctx, steps=8, device=dev)
        q = b.extra["q_steps"][0].contiguous()
        out = torch.zeros_like(q)
        plan = h.attend_plan(H_q=H_q, H_kv=H_kv, d=d, k_pool=b.k_pool, v_pool=b.v_pool, q=q, out=out, requests=b.requests,
                             mode=libape.APE_DECODE)
        ws = plan.alloc_workspace()
        run = lambda: plan.attend(b.T, b.S, ws)
        work = {"bytes": 4 * (64 + args.n_ctx * 256 + 257) * 4.0 * H_kv * d}
    elif args.case == "shared":
        # 16 requests decoding over ONE set of n_ctx cached contexts (many-shot prompts shared by a batch of queries)
        b = wl.share_contexts(wl.config5(n_req=16, steps=4, n_ctx=args.n_ctx, device=dev))
        q = b.extra["q_steps"][0].contiguous()
        out = torch.zeros_like(q)
        plan = h.attend_plan(H_q=H_q, H_kv=H_kv, d=d, k_pool=b.k_pool, v_pool=b.v_pool, q=q, out=out, requests=b.requests,
                             mode=libape.APE_DECODE, shared=True)
        ws = plan.alloc_workspace()
        run = lambda: plan.attend(b.T, b.S, ws)
        # bytes an unshared decode of the same batch would read (its algorithmic bytes); the shared plan reads the
        # contexts once
        work = {"bytes": 16 * (64 + args.n_ctx * 256 + 257) * 4.0 * H_kv * d,
                "bytes_read_once": (16 * (64 + 257) + args.n_ctx * 256) * 4.0 * H_kv * d}
    elif args.case == "rope":
        # the step in front of the pre-caching attention: n_ctx contexts of 256 tokens behind a 64-token prefix;
        # K rotated (H_kv heads), V copied, Q rotated (H_q heads), all written at their cache rows
        n_tok = 64 + args.n_ctx * 256
        runs = [(0, 0, 64, 0)] + [(64 + i * 256, 64 + i * 256, 256, 64) for i in range(args.n_ctx)]
        g = torch.Generator(device=dev).manual_seed(1)
        k_raw = torch.randn(n_tok, H_kv, d, generator=g, device=dev).to(torch.bfloat16)
        v_raw = torch.randn(n_tok, H_kv, d, generator=g, device=dev).to(torch.bfloat16)
        q_raw = torch.randn(n_tok, H_q, d, generator=g, device=dev).to(torch.bfloat16)
        k_pool, v_pool, q_enc = torch.empty_like(k_raw), torch.empty_like(v_raw), torch.empty_like(q_raw)
        plan = libape.RopePlan(h, d, 500000.0, runs)
        def run():
            plan.write(k_raw, k_pool, True)
            plan.write(v_raw, v_pool, False)
            plan.write(q_raw, q_enc, True)
        work = {"bytes": 2.0 * 2 * n_tok * d * (2 * H_kv + H_q)}
    else:
        b = wl.config4(n_ctx=args.n_ctx, with_encode_q=(args.case == "encode"), device=dev)
        if args.case == "prefill":
            out = torch.zeros_like(b.q)
            plan = h.attend_plan(H_q=H_q, H_kv=H_kv, d=d, k_pool=b.k_pool, v_pool=b.v_pool, q=b.q, out=out, requests=b.requests,
                                 mode=libape.APE_PREFILL)
            ws = plan.alloc_workspace()
            run = lambda: plan.attend(b.T, b.S, ws)
            work = {"flops": 4.0 * d * H_q * (256 * (64 + args.n_ctx * 256) + 256 * 257 / 2)}
        else:
            out = torch.zeros_like(b.q_enc)
            rq = b.requests[0]
            plan = h.encode_plan(H_q=H_q, H_kv=H_kv, d=d, k_pool=b.k_pool, v_pool=b.v_pool, q=b.q_enc, out=out,
                                 prefix=rq.prefix, ctx=rq.ctx)
            run = lambda: plan.encode_contexts()
            work = {"flops": 4.0 * d * H_q * args.n_ctx * (256 * 64 + 256 * 257 / 2)}
    run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    assert h.get_status() == 0
    ms = e0.elapsed_time(e1) / args.iters
    print(json.dumps({"case": args.case, "n_ctx": args.n_ctx, "ms_per_call": ms, **work,
                      "rate": (work.get("flops", 0) / ms / 1e9) if "flops" in work else (work["bytes"] / ms / 1e6),
                      "rate_unit": "TFLOP/s" if "flops" in work else "GB/s"}))


if __name__ == "__main__":
    main()
