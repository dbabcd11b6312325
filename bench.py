#!/usr/bin/env python
"""Benchmark of the APE attention hot path at 128K context on B200.

One step = one pass of the whole path over one batch of synthetic input, every leg launched `--reps` times back to back
(so that the timed region lasts about a second and the clock record means something):
  rope     rotary embedding with position re-use of the raw K, Q (rotated) and V (copied) of the prefix and the 500
           contexts, written to their cache rows (HBM bound),
  encode   500 contexts x 256 tokens against a 64-token shared prefix (block-diagonal attention),
  prefill  256 query rows over prefix 64 + 128,000 cached context tokens + causal self (many-shot 128K case),
  decode   one new token for each of 16 requests over prefix 64 + 128,000 + (257 + t) cached tokens; t walks the 256
           decode steps of the workload as the repetitions go on,
  shared   the same decode step when all 16 requests attend to one set of contexts (read once for the batch),
  rag      query prefill of 4 requests x 20 contexts of 512..1536 tokens, 128 query rows each (the RAG shape),
  cfg2     encode + query prefill of 10 contexts x 256 tokens (fits L2: L2 is flushed before every repetition),
  forms    the 128K prefill in the per-context form (Eq. 11-12) and as a two-level context tree.
The headline metric has two halves: `value` is the prefill half (TFLOP/s, tensor-core bound) and `decode` carries the
decode half (GB/s, HBM bound).  Inputs are resident in HBM before the timed region and, except for cfg2, larger than L2
(KV 0.53 GB for prefill, 8.4 GB for decode, 0.34 GB for rag), so no L2 flush is needed between repetitions.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--reps R] [--impl reference]
    python bench.py --case prefill-small|decode-small|encode-small|rope-small|rag|shared      one small case for a profiler
    python bench.py --shard context [--gpus N]       the 128K prefill with the contexts sharded over the ranks
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

METRIC = "ape_attention_128k_prefill_tflops"
UNIT = "TFLOP/s"
H_Q, H_KV, D = 32, 8, 128
L_P, N_CTX, L_CTX, L_Q = 64, 500, 256, 256
DEC_REQ, DEC_LK, DEC_STEPS = 16, 257, 256


def attend_flops(l_q: int, l_p: int, l_c: int, l_k: int) -> float:
    """Algorithmic FLOPs: 4*d per unmasked (row, key) pair per query head."""
    pairs = l_q * (l_p + l_c) + l_q * (l_q + 1) / 2 + l_q * (l_k - l_q)
    return 4.0 * D * H_Q * pairs


def encode_flops(l_p: int, lens) -> float:
    return 4.0 * D * H_Q * sum(L * l_p + L * (L + 1) / 2 for L in lens)


def decode_bytes(n_req: int, tokens_per_req: int) -> float:
    """Algorithmic bytes of one decode step: every cached K and V row read once (+ Q and O, negligible)."""
    return n_req * (tokens_per_req * 4.0 * H_KV * D + 2 * 2.0 * H_Q * D)


# DRAM traffic per full-size launch (dram__bytes_read.sum + dram__bytes_write.sum), taken from the ncu captures
# summarised under profiles/ on smaller cases and scaled by the units processed (traffic grows in proportion to the
# cached tokens).  Valid only for the kernel sources the counters were taken with: the figure is dropped (null) as
# soon as the hash of those sources changes.
NCU_TRAFFIC = {
    "prefill": {"bytes": 2 * (267.04e6 + 11.59e6), "sources": ["ape_attn.cu", "ape_tcgen05.cuh", "ape_common.cuh"], "sha": "3ec78f118ba6054c"},
    "encode": {"bytes": 2 * (792.07e6 + 485.03e6), "sources": ["ape_attn.cu", "ape_tcgen05.cuh", "ape_common.cuh"], "sha": "3ec78f118ba6054c"},
    "decode": {"bytes": (1.05511e9 + 4.18e6) * (8409907200.0 / 1053835264.0), "sources": ["ape_decode.cu", "ape_common.cuh"], "sha": "350774570d2381af"},
    "rope": {"bytes": 2 * ((131.30e6 + 86.35e6) + (131.30e6 + 82.34e6) + (524.94e6 + 479.29e6)), "sources": ["ape_rope.cu"], "sha": "eb5f0c0e67beef74"},
}


def source_hash(files):
    import hashlib
    h = hashlib.sha256()
    for f in files:
        h.update(open(os.path.join(ROOT, "paper_2502_05431_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def ncu_traffic(which: str):
    t = NCU_TRAFFIC[which]
    try:
        return t["bytes"] if source_hash(t["sources"]) == t["sha"] else None
    except OSError:
        return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        j = json.load(open(path))
        return dict(hbm_gbs=float(j["hbm_gbs"]), tf_burst=float(j["bf16_tflops"]),
                    tf_sustained=float(j.get("bf16_tflops_sustained", j["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "25"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        import datetime
        for line in self.proc.stdout:
            f = [x.strip() for x in line.split(",")]
            try:                                     # the tool's own time stamp: immune to pipe buffering
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
            except Exception:
                ts = time.time()
            self.rows.append((ts, f[1:]))

    def stop(self, t_begin: float, t_end: float):
        """Summary of the samples taken inside [t_begin, t_end] (the timed region, under load)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        time.sleep(0.1)
        self.proc.terminate()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, r in self.rows:
            if ts < t_begin or ts > t_end:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "power_w_median": statistics.median(pw) if pw else None,
                "reasons": sorted(reasons), "samples": len(sm), "period_ms": 25}


def cpu_oracle_sample(target_s: float = 15.0):
    """The fp64 oracle, as it stands, on a bounded sample of the prefill workload (some query rows, all heads)."""
    from oracle import ape_oracle as orc
    from paper_2502_05431_b200 import workloads as wl
    b = wl.config4()
    q, p, c, k = b.views(0)
    t0 = time.time()
    orc.attend(q, p, c, k, b.T, b.S, rows=(0, 1))
    per_row = max(time.time() - t0, 1e-3)
    n = max(1, min(L_Q - 1, int(target_s / per_row)))
    t0 = time.time()
    orc.attend(q, p, c, k, b.T, b.S, rows=(L_Q - n, L_Q))
    dt = time.time() - t0
    pairs = sum((L_P + N_CTX * L_CTX) + (i + 1) for i in range(L_Q - n, L_Q))
    flops = 4.0 * D * H_Q * pairs
    return dict(value=flops / dt / 1e12, unit=UNIT, cores=orc.num_threads(), kind="oracle",
                sample=f"last {n} of {L_Q} query rows x {H_Q} heads of the 128K prefill workload, {dt:.1f} s", seconds=dt)


def run_reference(args):
    """--impl reference: the CPU oracle timed on the same metric and workload, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ape_oracle as orc
    from paper_2502_05431_b200 import workloads as wl
    b = wl.config4()
    q, p, c, k = b.views(0)
    rows_per_step = 2
    per = []
    for s in range(args.warmup + args.steps):
        r0 = (s * rows_per_step) % (L_Q - rows_per_step)
        t0 = time.time()
        orc.attend(q, p, c, k, b.T, b.S, rows=(r0, r0 + rows_per_step))
        dt = time.time() - t0
        if s >= args.warmup:
            pairs = sum((L_P + N_CTX * L_CTX) + (i + 1) for i in range(r0, r0 + rows_per_step))
            per.append((4.0 * D * H_Q * pairs, dt))
    flops = sum(f for f, _ in per); secs = sum(t for _, t in per)
    val = flops / secs / 1e12
    sample = f"{rows_per_step} of {L_Q} query rows x {H_Q} heads per step of the 128K prefill workload"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(len(per), 1), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "cfg4_manyshot_128k prefill (oracle sample)", "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ---- small single-kernel cases for profiler captures ---------------------------------------------------------------

def run_case(args):
    """A few launches of one path on inputs larger than L2 but small enough that a multi-pass capture ends by itself.
    prefill-small: 256 query rows over prefix 64 + n_ctx x 256 context tokens (KV 262 MB at n_ctx 250); rag: 4 requests x
    20 contexts of 512..1536 tokens, 128 query rows each (KV 339 MB); decode-small: 4 requests x (64 + n_ctx x 256 + 257)
    cached tokens (KV 1.05 GB); encode-small: n_ctx contexts x 256 tokens against a 64-token prefix; rope-small: K, V, Q of
    the same tokens; shared: 16 requests decoding over one set of n_ctx contexts.  Prints the CUDA-event time per call and
    the algorithmic work, so that a capture can be scaled."""
    from paper_2502_05431_b200 import libape, workloads as wl
    dev = "cuda:0"
    torch.cuda.set_device(0)
    h = libape.Handle(0)
    case, n_ctx = args.case, args.n_ctx
    if case == "rag":
        lens = wl.config3_lens(0)
        b = wl.make_batch(H_q=H_Q, H_kv=H_KV, d=D, l_P=64, ctx_lens=lens, l_q=128, seed=0, T=0.9, S=0.8, device=dev)
        out = torch.zeros_like(b.q)
        plan = h.attend_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=b.k_pool, v_pool=b.v_pool, q=b.q, out=out, requests=b.requests,
                             mode=libape.APE_PREFILL)
        ws = plan.alloc_workspace()
        run = lambda: plan.attend(b.T, b.S, ws)
        work = {"flops": sum(attend_flops(128, 64, sum(l), 128) for l in lens)}
    elif case == "decode-small":
        b = wl.config5(n_req=4, n_ctx=n_ctx, steps=8, device=dev)
        q = b.extra["q_steps"][0].contiguous()
        out = torch.zeros_like(q)
        plan = h.attend_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=b.k_pool, v_pool=b.v_pool, q=q, out=out, requests=b.requests,
                             mode=libape.APE_DECODE)
        ws = plan.alloc_workspace()
        run = lambda: plan.attend(b.T, b.S, ws)
        work = {"bytes": 4 * (64 + n_ctx * 256 + 257) * 4.0 * H_KV * D}
    elif case == "shared":
        b = wl.share_contexts(wl.config5(n_req=16, steps=4, n_ctx=n_ctx, device=dev))
        q = b.extra["q_steps"][0].contiguous()
        out = torch.zeros_like(q)
        plan = h.attend_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=b.k_pool, v_pool=b.v_pool, q=q, out=out, requests=b.requests,
                             mode=libape.APE_DECODE, shared=True)
        ws = plan.alloc_workspace()
        run = lambda: plan.attend(b.T, b.S, ws)
        work = {"bytes": 16 * (64 + n_ctx * 256 + 257) * 4.0 * H_KV * D,
                "bytes_read_once": (16 * (64 + 257) + n_ctx * 256) * 4.0 * H_KV * D}
    elif case == "rope-small":
        n_tok = 64 + n_ctx * 256
        runs = [(0, 0, 64, 0)] + [(64 + i * 256, 64 + i * 256, 256, 64) for i in range(n_ctx)]
        g = torch.Generator(device=dev).manual_seed(1)
        k_raw = torch.randn(n_tok, H_KV, D, generator=g, device=dev).to(torch.bfloat16)
        v_raw = torch.randn(n_tok, H_KV, D, generator=g, device=dev).to(torch.bfloat16)
        q_raw = torch.randn(n_tok, H_Q, D, generator=g, device=dev).to(torch.bfloat16)
        k_pool, v_pool, q_enc = torch.empty_like(k_raw), torch.empty_like(v_raw), torch.empty_like(q_raw)
        plan = libape.RopePlan(h, D, 500000.0, runs)

        def run():
            plan.write(k_raw, k_pool, True)
            plan.write(v_raw, v_pool, False)
            plan.write(q_raw, q_enc, True)
        work = {"bytes": 2.0 * 2 * n_tok * D * (2 * H_KV + H_Q)}
    else:
        b = wl.config4(n_ctx=n_ctx, with_encode_q=(case == "encode-small"), device=dev)
        if case == "prefill-small":
            out = torch.zeros_like(b.q)
            plan = h.attend_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=b.k_pool, v_pool=b.v_pool, q=b.q, out=out, requests=b.requests,
                                 mode=libape.APE_PREFILL)
            ws = plan.alloc_workspace()
            run = lambda: plan.attend(b.T, b.S, ws)
            work = {"flops": attend_flops(256, 64, n_ctx * 256, 256)}
        else:
            out = torch.zeros_like(b.q_enc)
            rq = b.requests[0]
            plan = h.encode_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=b.k_pool, v_pool=b.v_pool, q=b.q_enc, out=out,
                                 prefix=rq.prefix, ctx=rq.ctx)
            run = lambda: plan.encode_contexts()
            work = {"flops": encode_flops(64, [256] * n_ctx)}
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
    print(json.dumps({"case": case, "n_ctx": n_ctx, "ms_per_call": ms, **work,
                      "rate": (work["flops"] / ms / 1e9) if "flops" in work else (work["bytes"] / ms / 1e6),
                      "rate_unit": "TFLOP/s" if "flops" in work else "GB/s"}))


# ---- the 128K prefill with its contexts sharded over the ranks ------------------------------------------------------

def run_shard_context(args):
    """Every rank holds 1/N of the 500 contexts (plus the prefix and the query segment): ape_attend_partial over its own
    contexts, one NCCL all-gather of the fp32 context partials (O_c, LSE_c) into local memory, ape_merge_shards.  The
    only path of the library with an exchange; strong scaling (the total work is fixed)."""
    from paper_2502_05431_b200 import dist_util, libape, workloads as wl
    rank = int(os.environ.get("RANK", "0")); local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dev = torch.device(f"cuda:{local_rank}")
    if world > 1:
        import torch.distributed as td
        td.init_process_group("nccl", device_id=dev)
    h = libape.Handle(local_rank)
    b = wl.config4(seed=0, device=str(dev))           # the same seed on every rank: one request, its contexts spread out
    rq = b.requests[0]
    mine = dist_util.shard_contexts([l for _, l in rq.ctx], world)[rank]
    req = wl.Request(rq.q_start, rq.q_len, rq.prefix, [rq.ctx[i] for i in mine], rq.query_kv, rq.query_kv_capacity)
    out = torch.zeros_like(b.q)
    plan = h.attend_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=b.k_pool, v_pool=b.v_pool, q=b.q, out=out, requests=[req], mode=libape.APE_PREFILL)
    ws = plan.alloc_workspace()
    rows = b.q.shape[0]
    o_c = torch.empty((rows, H_Q, D), dtype=torch.float32, device=dev); l_c = torch.empty((rows, H_Q), dtype=torch.float32, device=dev)
    o_o, l_o = torch.empty_like(o_c), torch.empty_like(l_c)

    def step(ev=None):
        if ev: ev[0].record()
        plan.attend_partial(b.T, ws, o_c, l_c, o_o, l_o)
        if ev: ev[1].record()
        o_all, l_all = dist_util.gather_context_partials(o_c, l_c)
        if ev: ev[2].record()
        libape.merge_shards(h, H_q=H_Q, H_kv=H_KV, d=D, o_ctx_all=o_all, lse_ctx_all=l_all, o_oth=o_o, lse_oth=l_o, S=b.S, out=out)
        if ev: ev[3].record()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    if world > 1:
        td.barrier()
    torch.cuda.synchronize()
    for s in range(args.steps):
        step(events[s])
    torch.cuda.synchronize()
    if world > 1:
        td.barrier()
    assert h.get_status() == 0
    med = lambda i, j: statistics.median(e[i].elapsed_time(e[j]) for e in events)
    t_att, t_gat, t_mrg, t_all = dist_util.max_over_ranks([med(0, 1), med(1, 2), med(2, 3), med(0, 3)], dev)
    if rank == 0:
        fl = attend_flops(L_Q, L_P, N_CTX * L_CTX, L_Q)
        print(json.dumps({
            "metric": METRIC, "value": fl / (t_all * 1e-3) / 1e12, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": t_all, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "cfg4_manyshot_128k prefill, contexts sharded over the ranks", "parallelism": f"context shards x{world}",
                       "contexts_per_rank": len(mine), "exchange_bytes_per_rank": rows * H_Q * (D + 1) * 4},
            "phases_ms": {"attend_partial": t_att, "all_gather": t_gat, "merge_shards": t_mrg}, "gpu_launches": args.steps * 3}))
    if world > 1:
        td.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--reps", type=int, default=10, help="launches of every leg inside one step")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--case", default=None, choices=["prefill-small", "decode-small", "encode-small", "rope-small", "rag", "shared"])
    ap.add_argument("--iters", type=int, default=3, help="--case: timed calls")
    ap.add_argument("--n-ctx", type=int, default=250, help="--case: contexts of 256 tokens")
    ap.add_argument("--shard", default=None, choices=["context"])
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.case:
        return run_case(args)
    if args.shard:
        return run_shard_context(args)

    from paper_2502_05431_b200 import dist_util, libape, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = world > 1
    torch.cuda.set_device(local_rank)
    dev = torch.device(f"cuda:{local_rank}")
    if dist:
        import torch.distributed as td
        td.init_process_group("nccl", device_id=dev)

    libape.load()                                  # fails loudly if the CUDA library is missing
    h = libape.Handle(local_rank)
    seed = dist_util.replica_seed(0, rank)         # every rank works on its own replica (weak scaling, no exchange)
    R = max(1, args.reps)
    kw = dict(H_q=H_Q, H_kv=H_KV, d=D)

    # ---- inputs, resident in HBM ------------------------------------------------------------------------------------
    pb = wl.config4(seed=seed, with_encode_q=True, device=str(dev))          # prefill + encode share this pool
    db = wl.config5(seed=seed + 1, n_req=DEC_REQ, steps=DEC_STEPS, device=str(dev))  # decode
    rq = pb.requests[0]
    p_out = torch.zeros_like(pb.q)
    plan_p = h.attend_plan(**kw, k_pool=pb.k_pool, v_pool=pb.v_pool, q=pb.q, out=p_out, requests=pb.requests, mode=libape.APE_PREFILL)
    ws_p = plan_p.alloc_workspace()
    plan_pc = h.attend_plan(**kw, k_pool=pb.k_pool, v_pool=pb.v_pool, q=pb.q, out=p_out, requests=pb.requests, mode=libape.APE_PREFILL,
                            per_context=True)
    ws_pc = plan_pc.alloc_workspace()
    # the same prefill over a two-level context tree: 50 top-level documents (grouping nodes) of 10 chunks each, S per document
    t_nodes, t_par = [], []
    for doc in range(N_CTX // 10):
        t_nodes.append((rq.ctx[0][0], 0)); t_par.append(-1)
        root = len(t_nodes) - 1
        for ch in range(10):
            t_nodes.append(rq.ctx[doc * 10 + ch]); t_par.append(root)
    t_req = wl.Request(rq.q_start, rq.q_len, rq.prefix, t_nodes, rq.query_kv, rq.query_kv_capacity)
    plan_t = h.attend_plan(**kw, k_pool=pb.k_pool, v_pool=pb.v_pool, q=pb.q, out=p_out, requests=[t_req], mode=libape.APE_PREFILL,
                           tree=([t_par], None))
    ws_t = plan_t.alloc_workspace()
    e_out = torch.zeros_like(pb.q_enc)
    plan_e = h.encode_plan(**kw, k_pool=pb.k_pool, v_pool=pb.v_pool, q=pb.q_enc, out=e_out, prefix=rq.prefix, ctx=rq.ctx)
    # raw (un-rotated) K, V, Q of the prefix and the contexts, packed in request order; the rope leg writes them into the
    # pool rows that the encode leg reads (a rotation keeps the N(0,1) statistics of the synthetic data)
    runs = libape.rope_runs_for_request(rq, 0)[:-1]
    n_raw = sum(r[2] for r in runs)
    k_raw, v_raw, q_raw = pb.k_pool[:n_raw].clone(), pb.v_pool[:n_raw].clone(), pb.q_enc[:n_raw].clone()
    plan_r = libape.RopePlan(h, D, 500000.0, runs)
    by_rope = 2.0 * 2 * n_raw * D * (2 * H_KV + H_Q)
    q_steps = db.extra["q_steps"]                                             # [256, 16, H_q, d]: the new token's query per step
    d_q = q_steps[0].contiguous().clone()
    d_out = torch.zeros_like(d_q)
    plan_d = h.attend_plan(**kw, k_pool=db.k_pool, v_pool=db.v_pool, q=d_q, out=d_out, requests=db.requests, mode=libape.APE_DECODE)
    ws_d = plan_d.alloc_workspace()
    # the same decode batch with all 16 requests attending to request 0's contexts: the contexts are read once
    sb = wl.share_contexts(db)
    s_out = torch.zeros_like(d_q)
    plan_s = h.attend_plan(**kw, k_pool=db.k_pool, v_pool=db.v_pool, q=d_q, out=s_out, requests=sb.requests, mode=libape.APE_DECODE, shared=True)
    ws_s = plan_s.alloc_workspace()
    # RAG shape (4 requests, 20 contexts of 512..1536 tokens, 128 query rows each)
    rag_lens = wl.config3_lens(0)
    rb = wl.make_batch(**kw, l_P=64, ctx_lens=rag_lens, l_q=128, seed=seed + 2, T=0.9, S=0.8, device=str(dev))
    r_out = torch.zeros_like(rb.q)
    plan_g = h.attend_plan(**kw, k_pool=rb.k_pool, v_pool=rb.v_pool, q=rb.q, out=r_out, requests=rb.requests, mode=libape.APE_PREFILL)
    ws_g = plan_g.alloc_workspace()
    fl_rag = sum(attend_flops(128, 64, sum(l), 128) for l in rag_lens)
    # config 2: 10 contexts x 256 behind a 32-token prefix, 64 query rows (fits L2: flushed before every repetition)
    cb = wl.make_batch(**kw, l_P=32, ctx_lens=[[256] * 10], l_q=64, seed=seed + 3, T=0.9, S=0.9, with_encode_q=True, device=str(dev))
    c_out, ce_out = torch.zeros_like(cb.q), torch.zeros_like(cb.q_enc)
    plan_c = h.attend_plan(**kw, k_pool=cb.k_pool, v_pool=cb.v_pool, q=cb.q, out=c_out, requests=cb.requests, mode=libape.APE_PREFILL)
    ws_c = plan_c.alloc_workspace()
    plan_ce = h.encode_plan(**kw, k_pool=cb.k_pool, v_pool=cb.v_pool, q=cb.q_enc, out=ce_out, prefix=cb.requests[0].prefix, ctx=cb.requests[0].ctx)
    fl_c2_pre, fl_c2_enc = attend_flops(64, 32, 2560, 64), encode_flops(32, [256] * 10)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)             # larger than the 126 MB L2

    fl_prefill = attend_flops(L_Q, L_P, N_CTX * L_CTX, L_Q)
    fl_encode = encode_flops(L_P, [L_CTX] * N_CTX)
    dec_tokens = lambda t: L_P + N_CTX * L_CTX + DEC_LK + t
    legs = ["rope", "encode", "prefill", "decode", "shared", "rag", "per_context", "tree"]
    dec_t = [0]                                                               # decode step counter, walks 0..255 and wraps

    def step(ev=None):
        """ev: per leg a pair of events around its R launches; cfg2 has a pair per launch (an L2 flush in between)."""
        def leg(name, fn):
            if ev: ev[name][0].record()
            for _ in range(R):
                fn()
            if ev: ev[name][1].record()
        leg("rope", lambda: (plan_r.write(k_raw, pb.k_pool, True), plan_r.write(v_raw, pb.v_pool, False), plan_r.write(q_raw, pb.q_enc, True)))
        leg("encode", plan_e.encode_contexts)
        leg("prefill", lambda: plan_p.attend(pb.T, pb.S, ws_p))
        if ev: ev["decode_t"] = []
        def dec():
            t = dec_t[0] % DEC_STEPS
            dec_t[0] += 1
            if ev: ev["decode_t"].append(t)
            plan_d.attend(db.T, db.S, ws_d, kv_extra=t)
        leg("decode", dec)
        leg("shared", lambda: plan_s.attend(db.T, db.S, ws_s))
        leg("rag", lambda: plan_g.attend(rb.T, rb.S, ws_g))
        leg("per_context", lambda: plan_pc.attend(pb.T, pb.S, ws_pc))
        leg("tree", lambda: plan_t.attend(pb.T, pb.S, ws_t))
        for i in range(R):
            flush.zero_()
            if ev: ev["cfg2"][i][0].record()
            plan_ce.encode_contexts()
            if ev: ev["cfg2"][i][1].record()
            plan_c.attend(cb.T, cb.S, ws_c)
            if ev: ev["cfg2"][i][2].record()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert h.get_status() == 0, "a kernel reported a timed-out wait"

    E = lambda: torch.cuda.Event(enable_timing=True)
    events = []
    for _ in range(args.steps):
        ev = {n: (E(), E()) for n in legs}
        ev["cfg2"] = [(E(), E(), E()) for _ in range(R)]
        ev["all"] = (E(), E())
        events.append(ev)
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.2)
    if dist:
        td.barrier()
    torch.cuda.synchronize()
    dec_t[0] = 0
    t_begin = time.time()
    for s in range(args.steps):
        events[s]["all"][0].record()
        step(events[s])
        events[s]["all"][1].record()
    torch.cuda.synchronize()
    t_end = time.time()
    t_wall = t_end - t_begin
    if dist:
        td.barrier()
    clocks = sampler.stop(t_begin, t_end)
    assert h.get_status() == 0

    med, mean = statistics.median, statistics.fmean
    per_leg = {n: [e[n][0].elapsed_time(e[n][1]) / R for e in events] for n in legs}       # ms per launch, one value per step
    c2_enc = [x[0].elapsed_time(x[1]) for e in events for x in e["cfg2"]]
    c2_pre = [x[1].elapsed_time(x[2]) for e in events for x in e["cfg2"]]
    t_step = mean(e["all"][0].elapsed_time(e["all"][1]) for e in events)
    names = legs + ["c2_enc", "c2_pre", "step"]
    t = dict(zip(names, dist_util.max_over_ranks([med(per_leg[n]) for n in legs] + [med(c2_enc), med(c2_pre), t_step], dev)))
    t_mean = {n: mean(per_leg[n]) for n in legs}

    # ---- decode over the 256 steps of the workload: kv_extra = t, the step's own query rows ---------------------------
    dec_ev = [(E(), E()) for _ in range(DEC_STEPS)]
    for tt in range(DEC_STEPS):
        d_q.copy_(q_steps[tt])
        dec_ev[tt][0].record()
        plan_d.attend(db.T, db.S, ws_d, kv_extra=tt)
        dec_ev[tt][1].record()
    torch.cuda.synchronize()
    dec_ms = [a.elapsed_time(b) for a, b in dec_ev]
    dec_gbs = [decode_bytes(DEC_REQ, dec_tokens(tt)) / (ms * 1e-3) / 1e9 for tt, ms in enumerate(dec_ms)]
    dec_total_ms, dec_mean_gbs = dist_util.max_over_ranks([sum(dec_ms), -mean(dec_gbs)], dev)
    dec_mean_gbs = -dec_mean_gbs
    by_decode_total = sum(decode_bytes(DEC_REQ, dec_tokens(tt)) for tt in range(DEC_STEPS))

    # ---- end to end through the host-buffer entry points -----------------------------------------------------------------
    e2e = None
    if rank == 0 or dist:
        hq, hk, hv = pb.q.cpu().pin_memory(), pb.k_pool.cpu().pin_memory(), pb.v_pool.cpu().pin_memory()
        hout = torch.empty_like(hq).pin_memory()
        h2d = d2h = 0
        for i in range(1 + args.e2e_steps):
            if i == 1:
                torch.cuda.synchronize(); t0 = time.time()
            h2d, d2h = plan_p.attend_host(pb.T, pb.S, ws_p, hq, hk, hv, hout)
        torch.cuda.synchronize()
        dt = (time.time() - t0) / max(args.e2e_steps, 1)
        dt = dist_util.max_over_ranks([dt], dev)[0]
        # decode half: per step the new token's Q, K, V rows host -> device (K, V appended to the cache), O device -> host
        n_e2e = 32
        hq_d = q_steps[:n_e2e].cpu().pin_memory()
        rows = [[r.query_kv[0] + 256 + tt for r in db.requests] for tt in range(n_e2e)]
        hk_d = torch.stack([db.k_pool[rr] for rr in rows]).cpu().pin_memory()           # [steps, 16, H_kv, d]
        hv_d = torch.stack([db.v_pool[rr] for rr in rows]).cpu().pin_memory()
        ho_d = torch.empty((DEC_REQ, H_Q, D), dtype=torch.bfloat16).pin_memory()
        plan_d.decode_step_host(db.T, db.S, ws_d, hq_d[0], ho_d, h_k_new=hk_d[0], h_v_new=hv_d[0], kv_extra=0)
        torch.cuda.synchronize(); t0 = time.time()
        for tt in range(n_e2e):
            up_d, down_d = plan_d.decode_step_host(db.T, db.S, ws_d, hq_d[tt], ho_d, h_k_new=hk_d[tt], h_v_new=hv_d[tt], kv_extra=tt)
        torch.cuda.synchronize()
        dt_d = dist_util.max_over_ranks([(time.time() - t0) / n_e2e], dev)[0]
        by_e2e = mean(decode_bytes(DEC_REQ, dec_tokens(tt)) for tt in range(n_e2e))
        e2e = {"value": dist_util.whole_job_rate(fl_prefill, world, dt * 1e3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": 1e3 * dt, "what": "ape_attend_host: Q + K/V pools host->device, attend, O device->host",
               "decode": {"value": dist_util.whole_job_rate(by_e2e, world, dt_d * 1e3) / 1e9, "unit": "GB/s", "ms_per_step": 1e3 * dt_d,
                          "h2d_bytes_per_step": up_d, "d2h_bytes_per_step": down_d, "steps": n_e2e,
                          "what": "ape_decode_step_host: the new token's Q, K, V rows host->device (K, V appended to the cache), "
                                  "decode step, O device->host; the cache stays resident"}}

    if rank != 0:
        if dist:
            td.destroy_process_group()
        return

    peaks = measured_peaks()
    mhz = clocks.get("sm_mhz")
    capped = bool(mhz is not None and clocks.get("sm_max_mhz") and mhz < 0.93 * clocks["sm_max_mhz"])
    # A leg runs R times back to back inside a timed region of about a second.  The clock record decides which measured
    # matmul rate is the comparable peak: the burst rate while the median SM clock under load stays within 7% of the
    # maximum, the sustained rate (taken under the power cap at about two thirds of the maximum clock) once it sits lower.
    tf_peak = peaks["tf_sustained"] if capped else peaks["tf_burst"]
    peak_src = (f"{peaks['source']} bf16 " + (f"sustained (median SM clock {mhz:.0f} MHz: power-capped)" if capped
                                             else f"burst (median SM clock {mhz if mhz is not None else float('nan'):.0f} MHz, near maximum)"))

    def tensor_leg(ms, flops):
        tf = flops / (ms * 1e-3) / 1e12
        return {"ms": ms, "tflops": tf, "flops": flops, "frac_of_burst": tf / peaks["tf_burst"], "frac_of_sustained": tf / peaks["tf_sustained"],
                "frac_of_nominal_2250": tf / 2250.0, "mcycles": (ms * 1e-3 * mhz) if mhz else None}

    pre, enc = tensor_leg(t["prefill"], fl_prefill), tensor_leg(t["encode"], fl_encode)
    pre["ms_mean"], enc["ms_mean"] = t_mean["prefill"], t_mean["encode"]
    # Encode of short contexts moves Q in and O out once per row and K/V once per context: by the roofline of the measured
    # peaks it is bound by HBM, not by the tensor cores, whenever its FLOP per algorithmic byte sit below the ridge.
    enc_bytes = 2 * 2.0 * N_CTX * L_CTX * H_Q * D + (L_P + N_CTX * L_CTX) * 4.0 * H_KV * D
    enc_gbs = enc_bytes / (t["encode"] * 1e-3) / 1e9
    ridge = peaks["tf_burst"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    enc["roofline"] = {"bound": "hbm" if fl_encode / enc_bytes < ridge else "tensor", "algorithmic_bytes": enc_bytes,
                       "flop_per_byte": fl_encode / enc_bytes, "ridge_flop_per_byte": ridge, "achieved": enc_gbs, "peak": peaks["hbm_gbs"],
                       "unit": "GB/s", "frac": enc_gbs / peaks["hbm_gbs"], "traffic": ncu_traffic("encode"),
                       "what": "Q read + O written once per row, K/V read once per context; the tensor fractions above are the other bound"}
    tf_prefill = pre["tflops"]
    gbs_decode = by_decode_total / (dec_total_ms * 1e-3) / 1e9
    roof = {"bound": "tensor", "kernel": "ape_attn_kernel<128,1> (+ merge) on the 128K prefill", "achieved": tf_prefill,
            "peak": tf_peak, "unit": "TFLOP/s", "frac": tf_prefill / tf_peak, "traffic": ncu_traffic("prefill"),
            "algorithmic_bytes": (L_P + N_CTX * L_CTX + L_Q) * 4.0 * H_KV * D + 2 * 2.0 * L_Q * H_Q * D,
            "peak_source": peak_src, "frac_of_burst": pre["frac_of_burst"], "frac_of_sustained": pre["frac_of_sustained"],
            "frac_of_nominal_2250": pre["frac_of_nominal_2250"]}
    roof_dec = {"bound": "hbm", "kernel": "ape_decode_kernel<128> (+ merge)", "achieved": gbs_decode, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": gbs_decode / peaks["hbm_gbs"], "traffic": ncu_traffic("decode"),
                "peak_source": f"{peaks['source']} copy (read + write; a read-only stream can exceed it)", "frac_of_nominal_8000": gbs_decode / 8000.0}
    gbs_rope = by_rope / (t["rope"] * 1e-3) / 1e9
    roof_rope = {"bound": "hbm", "kernel": "ape_rope_kernel<128> x3 (K, V, Q)", "achieved": gbs_rope, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                 "frac": gbs_rope / peaks["hbm_gbs"], "traffic": ncu_traffic("rope"), "peak_source": f"{peaks['source']} copy"}
    by_step0 = decode_bytes(DEC_REQ, dec_tokens(0))
    cpu = None if args.no_cpu_baseline else cpu_oracle_sample()
    n_launch = R * (3 + plan_e.last_launches() + plan_p.last_launches() + plan_d.last_launches() + plan_s.last_launches()
                    + plan_g.last_launches() + plan_pc.last_launches() + plan_t.last_launches() + plan_ce.last_launches() + plan_c.last_launches())
    line = {
        "metric": METRIC, "value": world * tf_prefill, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "reps_per_step": R, "ms_per_step": t["step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "statistic": "median over steps of (leg time / reps_per_step); ms_per_step is the mean",
        "config": {"workload": "cfg4_manyshot_128k prefill (value) + cfg5 decode x16 + rope/encode 500x256, Llama-3-8B head shape; "
                               "also timed: cfg3 RAG prefill, cfg2 encode + prefill, per-context and tree forms",
                   "H_q": H_Q, "H_kv": H_KV, "d": D, "prefix": L_P, "contexts": f"{N_CTX}x{L_CTX}", "query_rows": L_Q,
                   "decode_batch": DEC_REQ, "T": pb.T, "S": pb.S,
                   "l2": "inputs larger than L2 (0.53 GB / 8.4 GB / 0.34 GB KV per pass); cfg2 fits L2 and is flushed (256 MB write) before every repetition",
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
        "prefill": pre,
        "decode": {"ms_per_step": dec_total_ms / DEC_STEPS, "value": world * gbs_decode, "unit": "GB/s", "steps": DEC_STEPS,
                   "bytes_first_step": by_step0, "bytes_all_steps": by_decode_total,
                   "gbs_mean_of_steps": dec_mean_gbs, "gbs_first": dec_gbs[0], "gbs_last": dec_gbs[-1], "gbs_median": med(dec_gbs),
                   "ms_first": dec_ms[0], "ms_last": dec_ms[-1],
                   "in_step": {"ms": t["decode"], "gbs": by_step0 / (t["decode"] * 1e-3) / 1e9,
                               "what": "the decode leg inside the timed steps (kv_extra walks 0..255 there too; bytes of step 0 used)"},
                   "what": "256 consecutive decode steps, kv_extra = t, the step's own query rows; value = bytes of all steps / time of all steps",
                   "roofline": roof_dec},
        "decode_shared_contexts": {"ms_per_step": t["shared"], "speedup_over_decode": t["decode"] / t["shared"],
                                   "kv_bytes_served": by_step0, "kv_bytes_read": (DEC_REQ * (L_P + DEC_LK) + N_CTX * L_CTX) * 4.0 * H_KV * D,
                                   "gbs_read": (DEC_REQ * (L_P + DEC_LK) + N_CTX * L_CTX) * 4.0 * H_KV * D / (t["shared"] * 1e-3) / 1e9,
                                   "what": "the decode batch with all requests on one set of contexts (ape_attend_plan_shared): contexts read once"},
        "rope": {"ms": t["rope"], "value": world * gbs_rope, "unit": "GB/s", "bytes": by_rope, "roofline": roof_rope},
        "encode": enc,
        "rag_cfg3": tensor_leg(t["rag"], fl_rag),
        "cfg2": {"encode": tensor_leg(t["c2_enc"], fl_c2_enc), "prefill": tensor_leg(t["c2_pre"], fl_c2_pre), "l2": "flushed before every repetition"},
        "per_context_form": dict(tensor_leg(t["per_context"], fl_prefill), what="the 128K prefill planned with ape_attend_plan_per_context (Eq. 11-12)"),
        "tree_form": dict(tensor_leg(t["tree"], fl_prefill), what="the 128K prefill over a two-level context tree, 50 documents x 10 chunks, "
                          "S per document (ape_attend_plan_tree)"),
        "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
        "gpu_launches": args.steps * n_launch,
        "wall_s_timed_region": t_wall,
    }
    print(json.dumps(line))
    if dist:
        td.destroy_process_group()


if __name__ == "__main__":
    main()
