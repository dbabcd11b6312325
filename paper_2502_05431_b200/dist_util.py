"""Host-side helpers for runs with one process per GPU.  By default the attention path shards by request (independent
replicas, no data-path collective; the only exchange is the timing reduction below).  The context-sharded attend is the
one form with an exchange: every rank holds a subset of the contexts and the per-row context partials are all-gathered
once (`shard_contexts`, `gather_context_partials`)."""
from __future__ import annotations

from typing import List, Sequence

import torch


def max_over_ranks(values: Sequence[float], device: torch.device | str = "cpu") -> List[float]:
    """Element-wise maximum of a list of per-rank numbers over all ranks (identity without a process group)."""
    import torch.distributed as td
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if td.is_available() and td.is_initialized() and td.get_world_size() > 1:
        td.all_reduce(t, op=td.ReduceOp.MAX)
    return t.tolist()


def whole_job_rate(units_per_rank: float, world_size: int, slowest_rank_ms: float) -> float:
    """Aggregate throughput of `world_size` replicas that each processed `units_per_rank` units: all units over the
    time of the slowest rank (units per second)."""
    return world_size * units_per_rank / (slowest_rank_ms * 1e-3)


def replica_seed(base_seed: int, rank: int) -> int:
    """Every rank works on its own, differently seeded replica of the workload."""
    return base_seed + 100 * rank


def shard_contexts(ctx_lens: Sequence[int], world_size: int) -> List[List[int]]:
    """Which contexts (by index) each rank holds: longest first onto the rank with the fewest tokens so far, so the
    ranks' context passes take about the same time.  Deterministic: every rank computes the same table."""
    order = sorted(range(len(ctx_lens)), key=lambda i: (-int(ctx_lens[i]), i))
    load = [0] * world_size
    table: List[List[int]] = [[] for _ in range(world_size)]
    for i in order:
        r = min(range(world_size), key=lambda k: (load[k], k))
        table[r].append(i)
        load[r] += int(ctx_lens[i])
    return [sorted(t) for t in table]


def gather_context_partials(o_ctx: torch.Tensor, lse_ctx: torch.Tensor):
    """All-gather of one rank's context partials (fp32 [rows, H_q, d] and [rows, H_q]) into shard-major tensors
    [world, rows, H_q, d] and [world, rows, H_q], the layout ape_merge_shards reads.  NCCL on GPUs, gloo on CPU tensors;
    without a process group the single shard is returned with a leading dimension of 1."""
    import torch.distributed as td
    if not (td.is_available() and td.is_initialized()) or td.get_world_size() == 1:
        return o_ctx.unsqueeze(0).contiguous(), lse_ctx.unsqueeze(0).contiguous()
    w = td.get_world_size()
    o_all = torch.empty((w,) + tuple(o_ctx.shape), dtype=o_ctx.dtype, device=o_ctx.device)
    l_all = torch.empty((w,) + tuple(lse_ctx.shape), dtype=lse_ctx.dtype, device=lse_ctx.device)
    if o_ctx.is_cuda:
        # NCCL: one collective straight into the shard-major tensor (slab r receives rank r's partials)
        td.all_gather_into_tensor(o_all, o_ctx.contiguous())
        td.all_gather_into_tensor(l_all, lse_ctx.contiguous())
    else:
        # gloo (CPU ranks) takes the list form; the views are the slabs of the same tensor
        td.all_gather(list(o_all.unbind(0)), o_ctx.contiguous())
        td.all_gather(list(l_all.unbind(0)), lse_ctx.contiguous())
    return o_all, l_all


def attend_context_sharded(handle, plan, *, H_q: int, H_kv: int, d: int, T: float, S: float, workspace: torch.Tensor,
                           out: torch.Tensor, lse=None, kv_extra: int = 0, gather=None) -> None:
    """One context-sharded attend on this rank: `plan` was made over this rank's contexts (see `shard_contexts`), with the
    prefix and the query segment present on every rank.  Runs the local shard (ape_attend_partial), all-gathers the context
    partials (NCCL over NVLink when the tensors are on GPUs; 4 * (d + 1) bytes per row and head per rank) and merges
    (ape_merge_shards).  Every rank ends up with the full result in `out`.  `gather` replaces the all-gather (same
    signature and result layout as `gather_context_partials`), for hosts that bring their own transport."""
    from . import libape
    rows = out.shape[0]
    dev = out.device
    o_c = torch.empty((rows, H_q, d), dtype=torch.float32, device=dev)
    l_c = torch.empty((rows, H_q), dtype=torch.float32, device=dev)
    o_o, l_o = torch.empty_like(o_c), torch.empty_like(l_c)
    plan.attend_partial(T, workspace, o_c, l_c, o_o, l_o, kv_extra=kv_extra)
    o_all, l_all = (gather or gather_context_partials)(o_c, l_c)
    libape.merge_shards(handle, H_q=H_q, H_kv=H_kv, d=d, o_ctx_all=o_all, lse_ctx_all=l_all, o_oth=o_o, lse_oth=l_o, S=S,
                        out=out, lse=lse)
