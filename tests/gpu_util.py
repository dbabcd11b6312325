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
               shared: bool = False, tree=None):
    """Copy the batch to cuda:0, plan, launch, return (out bf16 CPU, lse fp32 CPU, plan launches)."""
    dev = torch.device("cuda:0")
    q = (b.q if q_override is None else q_override).to(dev)
    k, v = b.k_pool.to(dev), b.v_pool.to(dev)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], b.H_q), float("nan"), dtype=torch.float32, device=dev) if want_lse else None
    plan = handle().attend_plan(H_q=b.H_q, H_kv=b.H_kv, d=b.d, k_pool=k, v_pool=v, q=q, out=out,
                                requests=b.requests, mode=mode, lse=lse, per_context=per_context, shared=shared, tree=tree)
    ws, check_bands = guarded_workspace(plan)
    plan.attend(b.T, b.S, ws, kv_extra=kv_extra)
    torch.cuda.synchronize()
    assert handle().get_status() == 0
    check_bands()
    n = plan.last_launches()
    plan.close()
    return out.cpu(), (lse.cpu() if lse is not None else None), n


GUARD_BYTES = 4096


def guarded_workspace(plan, device=None):
    """A workspace of exactly the size the plan asks for, with a guard band of GUARD_BYTES on either side that is filled
    with a byte pattern (0xA5) no kernel writes.  Returns (workspace view, check): check() fails if a launch wrote outside
    the workspace it was given (the stand-in for a memory checker on the scratch the library owns during a call)."""
    dev = device if device is not None else torch.device("cuda:0")
    n = plan.workspace_bytes
    buf = torch.full((GUARD_BYTES + n + GUARD_BYTES,), 0xA5, dtype=torch.uint8, device=dev)
    ws = buf[GUARD_BYTES:GUARD_BYTES + max(n, 1)] if n > 0 else buf[GUARD_BYTES:GUARD_BYTES + 256]
    assert ws.data_ptr() % 256 == 0

    def check():
        lo, hi = buf[:GUARD_BYTES], buf[GUARD_BYTES + n:] if n > 0 else buf[GUARD_BYTES + 256:]
        assert bool((lo == 0xA5).all()) and bool((hi == 0xA5).all()), "a kernel wrote outside its workspace"
    return ws, check


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
