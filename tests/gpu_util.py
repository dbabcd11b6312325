"""Helpers shared by the GPU parity tests: run the library through its C ABI, run the oracle, compare."""
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

from oracle import ape_oracle as orc
from paper_2502_05431_b200 import libape
from paper_2502_05431_b200.workloads import Batch

MAX_ABS = 2e-2     # tolerance of the target: bf16 output, fp32 accumulation
MEAN_ABS = 2e-3

_handle = None


def handle() -> libape.Handle:
    global _handle
    if _handle is None:
        _handle = libape.Handle(0)
    return _handle


def gpu_attend(b: Batch, mode: int, *, kv_extra: int = 0, want_lse: bool = True, q_override=None, per_context: bool = False,
               shared: bool = False):
    """Copy the batch to cuda:0, plan, launch, return (out bf16 CPU, lse fp32 CPU, plan launches)."""
    dev = torch.device("cuda:0")
    q = (b.q if q_override is None else q_override).to(dev)
    k, v = b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], b.H_q), float("nan"), dtype=torch.float32, device=dev) if want_lse else None
    plan = handle().attend_plan(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=out,
                                requests=b.requests, mode=mode, lse=lse, per_context=per_context, shared=shared)
    ws = plan.alloc_workspace()
    plan.attend(b.T, b.S, ws, kv_extra=kv_extra)
    torch.cuda.synchronize()
    assert handle().get_status() == 0
    n = plan.last_launches()
    plan.close()
    return out.cpu(), (lse.cpu() if lse is not None else None), n


def oracle_attend(b: Batch, r: int, *, rows: Optional[Tuple[int, int]] = None, l_k: Optional[int] = None, q_override=None):
    q, p, c, k = b.views(r)
    if q_override is not None:
        q = q_override
    if l_k is not None:
        s = b.requests[r].query_kv[0]
        k = (b.k_pool[s:s + l_k], b.v_pool[s:s + l_k])
    return orc.attend(q, p, c, k, b.T, b.S, rows=rows)


def compare(got: torch.Tensor, ref: torch.Tensor, what: str, max_abs: float = MAX_ABS, mean_abs: float = MEAN_ABS):
    g = got.double().numpy()
    r = ref.double().numpy()
    sel = ~np.isnan(r)
    assert sel.any(), f"{what}: oracle produced nothing"
    assert not np.isnan(g[sel]).any(), f"{what}: NaN in the GPU output"
    err = np.abs(g[sel] - r[sel])
    rel = float(np.linalg.norm(g[sel] - r[sel]) / max(np.linalg.norm(r[sel]), 1e-30))
    print(f"{what}: max_abs={err.max():.3e} mean_abs={err.mean():.3e} rel_l2={rel:.3e} |ref|max={np.abs(r[sel]).max():.3e}")
    assert err.max() <= max_abs, f"{what}: max-abs {err.max():.3e} > {max_abs}"
    assert err.mean() <= mean_abs, f"{what}: mean-abs {err.mean():.3e} > {mean_abs}"
    assert rel <= 3e-2, f"{what}: relative L2 error {rel:.3e}"
    return err.max(), err.mean(), rel
