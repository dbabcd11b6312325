#!/usr/bin/env python
"""Benchmark of the APE attention hot path at 128K context on B200.

One step = one pass of the whole path over one batch of synthetic input:
  rope     rotary embedding with position re-use of the raw K, Q (rotated) and V (copied) of the prefix and the 500
           contexts, written to their cache rows (HBM bound),
  encode   500 contexts x 256 tokens against a 64-token shared prefix (block-diagonal attention),
  prefill  256 query rows over prefix 64 + 128,000 cached context tokens + causal self (many-shot 128K case),
  decode   one new token for each of 16 requests over prefix 64 + 128,000 + 257 cached tokens,
  shared   the same decode step when all 16 requests attend to one set of contexts (read once for the batch).
The headline metric has two halves: `value` is the prefill half (TFLOP/s, tensor-core bound) and `decode`
carries the decode half (GB/s, HBM bound).  Inputs are resident in HBM before the timed region and larger than
L2 (KV 0.53 GB for prefill, 8.4 GB for decode), so no L2 flush is needed between iterations.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
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
DEC_REQ, DEC_LK = 16, 257


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
    "prefill": {"bytes": 2 * (266.98e6 + 11.47e6), "sources": ["ape_attn.cu", "ape_tcgen05.cuh", "ape_common.cuh"], "sha": "9d1b4479c5180aef"},
    "decode": {"bytes": (1.05512e9 + 4.23e6) * (8409907200.0 / 1053835264.0), "sources": ["ape_decode.cu", "ape_common.cuh"], "sha": "3b704785906cb068"},
    "rope": {"bytes": 2 * ((131.30e6 + 87.13e6) + (131.30e6 + 82.04e6) + (524.91e6 + 479.47e6)), "sources": ["ape_rope.cu"], "sha": "f5898872292cd437"},
}


def ncu_traffic(which: str):
    import hashlib
    t = NCU_TRAFFIC[which]
    h = hashlib.sha256()
    try:
        for f in t["sources"]:
            h.update(open(os.path.join(ROOT, "paper_2502_05431_b200", "csrc", f), "rb").read())
    except OSError:
        return None
    return t["bytes"] if h.hexdigest()[:16] == t["sha"] else None


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
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=3)
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

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

    # ---- inputs, resident in HBM ------------------------------------------------------------------------------------
    pb = wl.config4(seed=seed, with_encode_q=True, device=str(dev))          # prefill + encode share this pool
    db = wl.config5(seed=seed + 1, n_req=DEC_REQ, steps=8, device=str(dev))  # decode
    rq = pb.requests[0]
    p_out = torch.zeros_like(pb.q)
    plan_p = h.attend_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=pb.k_pool, v_pool=pb.v_pool, q=pb.q, out=p_out,
                           requests=pb.requests, mode=libape.APE_PREFILL)
    ws_p = plan_p.alloc_workspace()
    e_out = torch.zeros_like(pb.q_enc)
    plan_e = h.encode_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=pb.k_pool, v_pool=pb.v_pool, q=pb.q_enc, out=e_out,
                           prefix=rq.prefix, ctx=rq.ctx)
    # raw (un-rotated) K, V, Q of the prefix and the contexts, packed in request order; the rope leg writes them into the
    # pool rows that the encode leg reads (a rotation keeps the N(0,1) statistics of the synthetic data)
    runs = libape.rope_runs_for_request(rq, 0)[:-1]
    n_raw = sum(r[2] for r in runs)
    k_raw, v_raw, q_raw = pb.k_pool[:n_raw].clone(), pb.v_pool[:n_raw].clone(), pb.q_enc[:n_raw].clone()
    plan_r = libape.RopePlan(h, D, 500000.0, runs)
    by_rope = 2.0 * 2 * n_raw * D * (2 * H_KV + H_Q)
    d_q = db.extra["q_steps"][0].contiguous()
    d_out = torch.zeros_like(d_q)
    plan_d = h.attend_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=db.k_pool, v_pool=db.v_pool, q=d_q, out=d_out,
                           requests=db.requests, mode=libape.APE_DECODE)
    ws_d = plan_d.alloc_workspace()
    # the same decode batch with all 16 requests attending to request 0's contexts: the contexts are read once
    sb = wl.share_contexts(db)
    s_out = torch.zeros_like(d_q)
    plan_s = h.attend_plan(H_q=H_Q, H_kv=H_KV, d=D, k_pool=db.k_pool, v_pool=db.v_pool, q=d_q, out=s_out,
                           requests=sb.requests, mode=libape.APE_DECODE, shared=True)
    ws_s = plan_s.alloc_workspace()

    fl_prefill = attend_flops(L_Q, L_P, N_CTX * L_CTX, L_Q)
    fl_encode = encode_flops(L_P, [L_CTX] * N_CTX)
    by_decode = decode_bytes(DEC_REQ, L_P + N_CTX * L_CTX + DEC_LK)
    fl_decode = 4.0 * D * H_Q * DEC_REQ * (L_P + N_CTX * L_CTX + DEC_LK)

    def step(ev=None):
        if ev: ev[4].record()
        plan_r.write(k_raw, pb.k_pool, True)
        plan_r.write(v_raw, pb.v_pool, False)
        plan_r.write(q_raw, pb.q_enc, True)
        if ev: ev[0].record()
        plan_e.encode_contexts()
        if ev: ev[1].record()
        plan_p.attend(pb.T, pb.S, ws_p)
        if ev: ev[2].record()
        plan_d.attend(db.T, db.S, ws_d)
        if ev: ev[3].record()
        plan_s.attend(db.T, db.S, ws_s)
        if ev: ev[5].record()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert h.get_status() == 0, "a kernel reported a timed-out wait"

    sampler = ClockSampler(local_rank)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(args.steps)]
    if dist:
        td.barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_wall = time.time()
    for s in range(args.steps):
        step(events[s])
    torch.cuda.synchronize()
    t_wall = time.time() - t_wall
    if dist:
        td.barrier()
    clocks = sampler.stop()
    assert h.get_status() == 0

    t_enc = sum(e[0].elapsed_time(e[1]) for e in events) / args.steps
    t_pre = sum(e[1].elapsed_time(e[2]) for e in events) / args.steps
    t_dec = sum(e[2].elapsed_time(e[3]) for e in events) / args.steps
    t_rope = sum(e[4].elapsed_time(e[0]) for e in events) / args.steps
    t_shared = sum(e[3].elapsed_time(e[5]) for e in events) / args.steps
    t_step = events[0][4].elapsed_time(events[-1][5]) / args.steps
    t_enc, t_pre, t_dec, t_step, t_rope, t_shared = dist_util.max_over_ranks([t_enc, t_pre, t_dec, t_step, t_rope, t_shared], dev)

    # ---- end to end through the host-buffer entry point (prefill half of the metric) ---------------------------------
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
        e2e = {"value": dist_util.whole_job_rate(fl_prefill, world, dt * 1e3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": 1e3 * dt, "what": "ape_attend_host: Q + K/V pools host->device, attend, O device->host"}

    if rank != 0:
        if dist:
            td.destroy_process_group()
        return

    peaks = measured_peaks()
    tf_prefill = fl_prefill / (t_pre * 1e-3) / 1e12
    tf_encode = fl_encode / (t_enc * 1e-3) / 1e12
    gbs_decode = by_decode / (t_dec * 1e-3) / 1e9
    # the prefill kernel runs alone for ~0.5 ms inside a multi-ms step: sustained peak is the fair denominator
    roof = {"bound": "tensor", "kernel": "ape_attn_kernel<128> (+ merge) on the 128K prefill", "achieved": tf_prefill,
            "peak": peaks["tf_sustained"], "unit": "TFLOP/s", "frac": tf_prefill / peaks["tf_sustained"], "traffic": ncu_traffic("prefill"),
            "algorithmic_bytes": (L_P + N_CTX * L_CTX + L_Q) * 4.0 * H_KV * D + 2 * 2.0 * L_Q * H_Q * D,
            "peak_source": f"{peaks['source']} bf16 sustained", "frac_of_nominal_2250": tf_prefill / 2250.0}
    roof_dec = {"bound": "hbm", "kernel": "ape_decode_kernel<128> (+ merge)", "achieved": gbs_decode, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": gbs_decode / peaks["hbm_gbs"], "traffic": ncu_traffic("decode"), "peak_source": f"{peaks['source']} copy",
                "frac_of_nominal_8000": gbs_decode / 8000.0}
    gbs_rope = by_rope / (t_rope * 1e-3) / 1e9
    roof_rope = {"bound": "hbm", "kernel": "ape_rope_kernel<128> x3 (K, V, Q)", "achieved": gbs_rope, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                 "frac": gbs_rope / peaks["hbm_gbs"], "traffic": ncu_traffic("rope"), "peak_source": f"{peaks['source']} copy"}
    cpu = None if args.no_cpu_baseline else cpu_oracle_sample()
    line = {
        "metric": METRIC, "value": world * tf_prefill, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": t_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "cfg4_manyshot_128k prefill (value) + cfg5 decode x16 + rope/encode 500x256, Llama-3-8B head shape",
                   "H_q": H_Q, "H_kv": H_KV, "d": D, "prefix": L_P, "contexts": f"{N_CTX}x{L_CTX}", "query_rows": L_Q,
                   "decode_batch": DEC_REQ, "T": pb.T, "S": pb.S, "l2": "inputs larger than L2 (0.53 GB / 8.4 GB KV per pass)",
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
        "prefill": {"ms": t_pre, "tflops": tf_prefill, "flops": fl_prefill},
        "decode": {"ms_per_step": t_dec, "value": world * gbs_decode, "unit": "GB/s", "bytes": by_decode, "tflops": fl_decode / (t_dec * 1e-3) / 1e12,
                   "roofline": roof_dec},
        "decode_shared_contexts": {"ms_per_step": t_shared, "speedup_over_decode": t_dec / t_shared,
                                   "kv_bytes_served": by_decode, "kv_bytes_read": (DEC_REQ * (L_P + DEC_LK) + N_CTX * L_CTX) * 4.0 * H_KV * D,
                                   "what": "the decode batch with all requests on one set of contexts (ape_attend_plan_shared): contexts read once, "
                                           "context pass on the tensor cores (64 live rows of a 256-row block)"},
        "rope": {"ms": t_rope, "value": world * gbs_rope, "unit": "GB/s", "bytes": by_rope, "roofline": roof_rope},
        "encode": {"ms": t_enc, "tflops": tf_encode, "flops": fl_encode, "frac_of_sustained_peak": tf_encode / peaks["tf_sustained"]},
        "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
        "gpu_launches": args.steps * (3 + plan_e.last_launches() + plan_p.last_launches() + plan_d.last_launches() + plan_s.last_launches()),
        "wall_s_timed_region": t_wall,
    }
    print(json.dumps(line))
    if dist:
        td.destroy_process_group()


if __name__ == "__main__":
    main()
