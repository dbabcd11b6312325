"""ctypes loader for the fp64 CPU oracle (oracle/ape_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, the smoke check and the
benchmark's CPU-baseline leg.  The product package never imports this module.

The C file is compiled with gcc on first use (or by ``build()``); it holds the
arithmetic, this file only marshals torch CPU tensors (bf16) into plain pointers.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ape_oracle.c")
_LIB = os.path.join(_HERE, "libape_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _KV(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("len", C.c_int64),
                ("token_stride", C.c_int64), ("head_stride", C.c_int64)]


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.ape_oracle_attend.restype = C.c_int
        lib.ape_oracle_attend.argtypes = [
            C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_double,
            C.POINTER(_KV), C.POINTER(_KV), C.c_int, C.POINTER(_KV),
            C.c_double, C.c_double, C.c_int,
            C.c_int64, C.c_int64, C.c_int, C.c_int,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.ape_oracle_encode.restype = C.c_int
        lib.ape_oracle_encode.argtypes = [
            C.POINTER(C.c_void_p), C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_double,
            C.POINTER(_KV), C.POINTER(_KV), C.c_int, C.c_int64, C.c_int64,
            C.POINTER(C.c_void_p), C.POINTER(C.c_void_p)]
        lib.ape_oracle_attend_tree.restype = C.c_int
        lib.ape_oracle_attend_tree.argtypes = [
            C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_double,
            C.POINTER(_KV), C.POINTER(_KV), C.POINTER(C.c_int32), C.POINTER(C.c_uint8), C.c_int, C.POINTER(_KV),
            C.c_double, C.c_double, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        lib.ape_oracle_num_threads.restype = C.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().ape_oracle_num_threads())


def _check_bf16_cpu(t: torch.Tensor, name: str) -> None:
    if t.device.type != "cpu" or t.dtype != torch.bfloat16:
        raise TypeError(f"{name}: expected a CPU bf16 tensor, got {t.dtype} on {t.device}")
    if t.dim() != 3 or t.stride(2) != 1:
        raise ValueError(f"{name}: expected [tokens, heads, d] with contiguous d")


def _kv(k: torch.Tensor, v: torch.Tensor, name: str) -> _KV:
    _check_bf16_cpu(k, name + ".k")
    _check_bf16_cpu(v, name + ".v")
    if k.shape != v.shape or k.stride() != v.stride():
        raise ValueError(f"{name}: K and V must share shape and strides")
    return _KV(k.data_ptr(), v.data_ptr(), k.shape[0], k.stride(0) if k.shape[0] > 1 else k.shape[1] * k.shape[2],
               k.stride(1) if k.shape[1] > 1 else k.shape[2])


@dataclass
class AttendResult:
    out: torch.Tensor       # fp64 [l_q, H_q, d]
    lse: torch.Tensor       # fp64 [l_q, H_q]  log of the Eq. 5 denominator
    lse_ctx: torch.Tensor   # fp64 [l_q, H_q]  LogSumExp of the tempered context logits
    wsum: torch.Tensor      # fp64 [l_q, H_q]  sum of the final weights


def attend(q: torch.Tensor,
           prefix: Tuple[torch.Tensor, torch.Tensor],
           ctx: Sequence[Tuple[torch.Tensor, torch.Tensor]],
           query_kv: Tuple[torch.Tensor, torch.Tensor],
           T: float, S: float, *, scale: Optional[float] = None, per_context: bool = False,
           rows: Optional[Tuple[int, int]] = None, heads: Optional[Tuple[int, int]] = None) -> AttendResult:
    """APE attention (Eq. 5) of one request.  Tensors: q [l_q,H_q,d]; K/V [len,H_kv,d]; all CPU bf16.

    ``rows`` / ``heads`` restrict the evaluation to a half-open range; entries outside it are NaN.
    """
    lib = _load()
    _check_bf16_cpu(q, "q")
    l_q, H_q, d = q.shape
    H_kv = query_kv[0].shape[1]
    c = float(scale) if scale is not None else d ** -0.5
    pk = _kv(prefix[0], prefix[1], "prefix")
    qk = _kv(query_kv[0], query_kv[1], "query_kv")
    arr = (_KV * max(len(ctx), 1))()
    for n, (k, v) in enumerate(ctx):
        arr[n] = _kv(k, v, f"ctx[{n}]")
    r0, r1 = rows if rows is not None else (0, l_q)
    h0, h1 = heads if heads is not None else (0, H_q)
    out = torch.full((l_q, H_q, d), float("nan"), dtype=torch.float64)
    lse = torch.full((l_q, H_q), float("nan"), dtype=torch.float64)
    lse_ctx = torch.full((l_q, H_q), float("nan"), dtype=torch.float64)
    wsum = torch.full((l_q, H_q), float("nan"), dtype=torch.float64)
    q_ts = q.stride(0) if l_q > 1 else H_q * d
    q_hs = q.stride(1) if H_q > 1 else d
    rc = lib.ape_oracle_attend(q.data_ptr(), l_q, q_ts, q_hs, H_q, H_kv, d, c,
                               C.byref(pk), arr, len(ctx), C.byref(qk),
                               float(T), float(S), int(per_context), r0, r1, h0, h1,
                               out.data_ptr(), lse.data_ptr(), lse_ctx.data_ptr(), wsum.data_ptr())
    if rc != 0:
        raise RuntimeError(f"ape_oracle_attend failed with code {rc}")
    return AttendResult(out, lse, lse_ctx, wsum)


def attend_tree(q: torch.Tensor,
                prefix: Tuple[torch.Tensor, torch.Tensor],
                ctx: Sequence[Tuple[torch.Tensor, torch.Tensor]],
                query_kv: Tuple[torch.Tensor, torch.Tensor],
                T: float, S: float, parent: Sequence[int], scaled: Optional[Sequence[int]] = None, *,
                scale: Optional[float] = None, rows: Optional[Tuple[int, int]] = None) -> AttendResult:
    """APE attention over context trees.  ctx[n] holds node n's own tokens (may be empty), parent[n] < n is its parent
    (-1: top level); scaled[n] marks the nodes that hand S * LogSumExp upward (default: the top-level nodes).
    Returns out and lse (lse_ctx and wsum are NaN: not defined for this form)."""
    lib = _load()
    _check_bf16_cpu(q, "q")
    l_q, H_q, d = q.shape
    H_kv = query_kv[0].shape[1]
    c = float(scale) if scale is not None else d ** -0.5
    n = len(ctx)
    if len(parent) != n:
        raise ValueError("one parent per node")
    if scaled is None:
        scaled = [1 if p < 0 else 0 for p in parent]
    pk = _kv(prefix[0], prefix[1], "prefix")
    qk = _kv(query_kv[0], query_kv[1], "query_kv")
    arr = (_KV * max(n, 1))()
    for i, (k, v) in enumerate(ctx):
        arr[i] = _kv(k, v, f"ctx[{i}]")
    par = (C.c_int32 * max(n, 1))(*[int(p) for p in parent])
    sc = (C.c_uint8 * max(n, 1))(*[1 if s else 0 for s in scaled])
    r0, r1 = rows if rows is not None else (0, l_q)
    out = torch.full((l_q, H_q, d), float("nan"), dtype=torch.float64)
    lse = torch.full((l_q, H_q), float("nan"), dtype=torch.float64)
    nan = torch.full((l_q, H_q), float("nan"), dtype=torch.float64)
    q_ts = q.stride(0) if l_q > 1 else H_q * d
    q_hs = q.stride(1) if H_q > 1 else d
    rc = lib.ape_oracle_attend_tree(q.data_ptr(), l_q, q_ts, q_hs, H_q, H_kv, d, c, C.byref(pk), arr, par, sc, n, C.byref(qk),
                                    float(T), float(S), r0, r1, 0, H_q, out.data_ptr(), lse.data_ptr())
    if rc != 0:
        raise RuntimeError(f"ape_oracle_attend_tree failed with code {rc}")
    return AttendResult(out, lse, nan, nan.clone())


def encode(ctx_q: Sequence[torch.Tensor],
           prefix: Tuple[torch.Tensor, torch.Tensor],
           ctx: Sequence[Tuple[torch.Tensor, torch.Tensor]],
           *, scale: Optional[float] = None, rows: Optional[Tuple[int, int]] = None
           ) -> Tuple[List[torch.Tensor], List[torch.Tensor]]:
    """Block-diagonal context encoding.  Returns (outs, lses): fp64 [len_n,H_q,d] and [len_n,H_q] per context."""
    lib = _load()
    n_ctx = len(ctx)
    if n_ctx == 0:
        return [], []
    for n, t in enumerate(ctx_q):
        _check_bf16_cpu(t, f"ctx_q[{n}]")
    H_q, d = ctx_q[0].shape[1], ctx_q[0].shape[2]
    H_kv = ctx[0][0].shape[1]
    c = float(scale) if scale is not None else d ** -0.5
    q_ts, q_hs = H_q * d, d
    for t in ctx_q:
        if t.shape[0] > 1 and t.stride(0) != ctx_q[0].stride(0):
            raise ValueError("all ctx_q must share strides")
    for t in ctx_q:
        if t.shape[0] > 1:
            q_ts = t.stride(0)
        if H_q > 1:
            q_hs = t.stride(1)
    pk = _kv(prefix[0], prefix[1], "prefix")
    arr = (_KV * n_ctx)()
    qptr = (C.c_void_p * n_ctx)()
    outs, lses = [], []
    optr = (C.c_void_p * n_ctx)()
    lptr = (C.c_void_p * n_ctx)()
    for n in range(n_ctx):
        arr[n] = _kv(ctx[n][0], ctx[n][1], f"ctx[{n}]")
        if ctx_q[n].shape[0] != ctx[n][0].shape[0]:
            raise ValueError("ctx_q and ctx lengths differ")
        qptr[n] = ctx_q[n].data_ptr()
        outs.append(torch.full((ctx[n][0].shape[0], H_q, d), float("nan"), dtype=torch.float64))
        lses.append(torch.full((ctx[n][0].shape[0], H_q), float("nan"), dtype=torch.float64))
        optr[n] = outs[-1].data_ptr()
        lptr[n] = lses[-1].data_ptr()
    r0, r1 = rows if rows is not None else (0, max(t.shape[0] for t in ctx_q))
    rc = lib.ape_oracle_encode(qptr, q_ts, q_hs, H_q, H_kv, d, c, C.byref(pk), arr, n_ctx, r0, r1, optr, lptr)
    if rc != 0:
        raise RuntimeError(f"ape_oracle_encode failed with code {rc}")
    return outs, lses
