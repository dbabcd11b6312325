"""Thin ctypes binding over libape.so (C ABI: include/ape.h).  Argument marshalling only.

Every step of the attention path runs in the library's CUDA kernels; there is no Python or CPU fallback:
if the shared library is missing or a call fails, an exception is raised.
PyTorch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libape.so")

APE_PREFILL, APE_DECODE = 0, 1

EXPORTS = ["ape_create", "ape_destroy", "ape_attend_plan", "ape_encode_plan", "ape_plan_workspace_bytes",
           "ape_plan_destroy", "ape_attend", "ape_encode_contexts", "ape_attend_host", "ape_plan_last_launches",
           "ape_get_status", "ape_status_string", "ape_decode_noalloc", "ape_attend_plan_per_context",
           "ape_rope_runs_for_request", "ape_rope_plan", "ape_rope_write", "ape_attend_plan_shared",
           "ape_attend_partial", "ape_merge_shards", "ape_selftest_timeout", "ape_selftest_timeout_noalloc",
           "ape_set_sm_budget", "ape_get_status_stream", "ape_decode_step_host", "ape_attend_plan_tree", "ape_attend_once"]


class ApeError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: libape status {code} ({status_string(code)})")
        self.code = code


class ape_shape_t(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("softmax_scale", C.c_float)]


class ape_span_t(C.Structure):
    _fields_ = [("start", C.c_int64), ("len", C.c_int64)]


class ape_kv_pool_t(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("n_tokens", C.c_int64), ("token_stride", C.c_int64), ("head_stride", C.c_int64)]


class ape_rows_t(C.Structure):
    _fields_ = [("data", C.c_void_p), ("n_rows", C.c_int64), ("token_stride", C.c_int64), ("head_stride", C.c_int64)]


class ape_request_t(C.Structure):
    _fields_ = [("q_start", C.c_int64), ("q_len", C.c_int64), ("prefix", ape_span_t), ("ctx", C.POINTER(ape_span_t)),
                ("n_ctx", C.c_int32), ("query_kv", ape_span_t), ("query_kv_capacity", C.c_int64)]


class ape_partials_t(C.Structure):
    _fields_ = [("o_ctx", C.c_void_p), ("lse_ctx", C.c_void_p), ("o_oth", C.c_void_p), ("lse_oth", C.c_void_p)]


class ape_rope_run_t(C.Structure):
    _fields_ = [("src_start", C.c_int64), ("dst_start", C.c_int64), ("len", C.c_int64), ("pos0", C.c_int64)]


_lib = None


def load() -> C.CDLL:
    """Load libape.so (built in-tree by paper_2502_05431_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2502_05431_b200.build` "
                              "(there is no fallback path)")
        lib = C.CDLL(LIB_PATH)
        vp = C.c_void_p
        lib.ape_create.argtypes = [C.POINTER(vp), C.c_int]
        lib.ape_destroy.argtypes = [vp]
        lib.ape_attend_plan.argtypes = [vp, C.POINTER(ape_shape_t), C.POINTER(ape_kv_pool_t), C.POINTER(ape_rows_t),
                                        C.POINTER(ape_rows_t), vp, C.POINTER(ape_request_t), C.c_int32, C.c_int, C.POINTER(vp)]
        lib.ape_attend_plan_per_context.argtypes = lib.ape_attend_plan.argtypes
        lib.ape_attend_plan_shared.argtypes = lib.ape_attend_plan.argtypes[:7] + lib.ape_attend_plan.argtypes[8:]
        lib.ape_attend_plan_tree.argtypes = lib.ape_attend_plan.argtypes[:8] + [C.POINTER(C.POINTER(C.c_int32)),
                                                                                C.POINTER(C.POINTER(C.c_uint8)), C.c_int, C.POINTER(vp)]
        lib.ape_encode_plan.argtypes = [vp, C.POINTER(ape_shape_t), C.POINTER(ape_kv_pool_t), C.POINTER(ape_rows_t),
                                        C.POINTER(ape_rows_t), vp, C.POINTER(ape_span_t), C.POINTER(ape_span_t), C.c_int32,
                                        C.POINTER(vp)]
        lib.ape_plan_workspace_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
        lib.ape_attend_once.argtypes = lib.ape_attend_plan.argtypes[:9] + [C.c_float, C.c_float, vp]
        lib.ape_plan_destroy.argtypes = [vp]
        lib.ape_attend.argtypes = [vp, C.c_float, C.c_float, C.c_int64, vp, C.c_size_t, vp]
        lib.ape_encode_contexts.argtypes = [vp, vp, C.c_size_t, vp]
        lib.ape_attend_host.argtypes = [vp, C.c_float, C.c_float, C.c_int64, vp, C.c_size_t, vp, vp, vp, vp,
                                        C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), vp]
        lib.ape_decode_step_host.argtypes = lib.ape_attend_host.argtypes
        lib.ape_plan_last_launches.argtypes = [vp, C.POINTER(C.c_int32)]
        lib.ape_get_status.argtypes = [vp, C.POINTER(C.c_int32)]
        lib.ape_decode_noalloc.argtypes = [C.POINTER(ape_shape_t), C.POINTER(ape_kv_pool_t), C.POINTER(ape_rows_t),
                                           C.POINTER(ape_rows_t), vp, C.POINTER(ape_request_t), C.c_int32, C.c_float, C.c_float,
                                           C.c_int64, C.c_int, vp, C.POINTER(C.c_int32)]
        lib.ape_rope_runs_for_request.argtypes = [C.POINTER(ape_request_t), C.c_int64, C.POINTER(ape_rope_run_t), C.c_int32,
                                                  C.POINTER(C.c_int32)]
        lib.ape_rope_plan.argtypes = [vp, C.c_int32, C.c_double, C.POINTER(ape_rope_run_t), C.c_int32, C.POINTER(vp)]
        lib.ape_rope_write.argtypes = [vp, C.POINTER(ape_rows_t), C.POINTER(ape_rows_t), C.c_int32, C.c_int32, vp]
        lib.ape_attend_partial.argtypes = [vp, C.c_float, C.c_int64, vp, C.c_size_t, C.POINTER(ape_partials_t), vp]
        lib.ape_merge_shards.argtypes = [vp, C.POINTER(ape_shape_t), C.c_int64, C.c_int32, vp, vp, vp, vp, C.c_float,
                                         C.POINTER(ape_rows_t), vp, vp]
        lib.ape_selftest_timeout.argtypes = [vp, vp]
        lib.ape_selftest_timeout_noalloc.argtypes = [C.c_int, vp]
        lib.ape_set_sm_budget.argtypes = [vp, C.c_int32]
        lib.ape_get_status_stream.argtypes = [vp, vp, C.POINTER(C.c_int32)]
        lib.ape_status_string.argtypes = [C.c_int]
        lib.ape_status_string.restype = C.c_char_p
        for name in EXPORTS:
            if name != "ape_status_string":
                getattr(lib, name).restype = C.c_int
        _lib = lib
    return _lib


def selftest_timeout_noalloc(device: int = 0, stream: Optional[torch.cuda.Stream] = None) -> None:
    """ape_selftest_timeout_noalloc: a bounded wait that runs out and raises the status word of ape_decode_noalloc's array."""
    _check(load().ape_selftest_timeout_noalloc(int(device), _stream_ptr(stream)), "ape_selftest_timeout_noalloc")


def status_string(code: int) -> str:
    return load().ape_status_string(int(code)).decode()


def _check(code: int, what: str) -> None:
    if code != 0:
        raise ApeError(code, what)


def _rows(t: torch.Tensor) -> ape_rows_t:
    return ape_rows_t(t.data_ptr(), t.shape[0], t.stride(0), t.stride(1))


def _pool(k: torch.Tensor, v: torch.Tensor) -> ape_kv_pool_t:
    if k.shape != v.shape or k.stride() != v.stride():
        raise ValueError("K and V pools must share shape and strides")
    return ape_kv_pool_t(k.data_ptr(), v.data_ptr(), k.shape[0], k.stride(0), k.stride(1))


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _request_array(requests: Sequence):
    n = len(requests)
    arr = (ape_request_t * max(n, 1))()
    keep = []
    for i, r in enumerate(requests):
        spans = (ape_span_t * max(len(r.ctx), 1))(*[ape_span_t(int(s), int(l)) for s, l in r.ctx])
        keep.append(spans)
        arr[i] = ape_request_t(int(r.q_start), int(r.q_len), ape_span_t(*map(int, r.prefix)), spans, len(r.ctx),
                               ape_span_t(*map(int, r.query_kv)), int(r.query_kv_capacity))
    return arr, keep


def decode_noalloc(*, H_q: int, H_kv: int, d: int, k_pool: torch.Tensor, v_pool: torch.Tensor, q: torch.Tensor,
                   out: torch.Tensor, requests: Sequence, T: float, S: float, kv_extra: int = 0,
                   lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0, device: int = 0,
                   stream: Optional[torch.cuda.Stream] = None, want_status: bool = False) -> Optional[int]:
    """ape_decode_noalloc: one decode step without a handle, a plan or a workspace; for callers that must not
    allocate device memory.  The library keeps its scratch in a fixed 8 MiB device array; batches that do not fit
    raise ApeError(APE_ERR_WORKSPACE).  With want_status the call synchronises and returns the device status word."""
    shape = ape_shape_t(H_q, H_kv, d, softmax_scale)
    pool, qr, orows = _pool(k_pool, v_pool), _rows(q), _rows(out)
    arr, _keep = _request_array(requests)
    st = C.c_int32(0)
    _check(load().ape_decode_noalloc(C.byref(shape), C.byref(pool), C.byref(qr), C.byref(orows),
                                     lse.data_ptr() if lse is not None else None, arr, len(requests), float(T), float(S),
                                     int(kv_extra), int(device), _stream_ptr(stream), C.byref(st) if want_status else None),
           "ape_decode_noalloc")
    return int(st.value) if want_status else None


class Handle:
    """ape_create / ape_destroy."""

    def __init__(self, device: int = 0):
        self._h = C.c_void_p()
        _check(load().ape_create(C.byref(self._h), int(device)), "ape_create")
        self.device = int(device)

    def close(self) -> None:
        if self._h:
            load().ape_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def selftest_timeout(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        """ape_selftest_timeout: a bounded wait that runs out; get_status() then returns APE_ERR_TIMEOUT (-8) once."""
        _check(load().ape_selftest_timeout(self._h, _stream_ptr(stream)), "ape_selftest_timeout")

    def get_status(self) -> int:
        v = C.c_int32(0)
        _check(load().ape_get_status(self._h, C.byref(v)), "ape_get_status")
        return int(v.value)

    def get_status_stream(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        """ape_get_status_stream: the status word in stream order on `stream`; waits for that stream only."""
        v = C.c_int32(0)
        _check(load().ape_get_status_stream(self._h, _stream_ptr(stream), C.byref(v)), "ape_get_status_stream")
        return int(v.value)

    def set_sm_budget(self, n_sm: int) -> None:
        """ape_set_sm_budget: later plans use at most n_sm thread blocks (0: the whole device)."""
        _check(load().ape_set_sm_budget(self._h, int(n_sm)), "ape_set_sm_budget")

    def attend_once(self, *, H_q: int, H_kv: int, d: int, k_pool: torch.Tensor, v_pool: torch.Tensor, q: torch.Tensor,
                    out: torch.Tensor, requests: Sequence, mode: int, T: float, S: float, lse: Optional[torch.Tensor] = None,
                    softmax_scale: float = 0.0, stream: Optional[torch.cuda.Stream] = None) -> None:
        """ape_attend_once: plan, launch, wait and clean up in one call (same arguments as attend_plan, plus T and S)."""
        shape = ape_shape_t(H_q, H_kv, d, softmax_scale)
        pool, qr, orows = _pool(k_pool, v_pool), _rows(q), _rows(out)
        n = len(requests)
        arr = (ape_request_t * max(n, 1))()
        keep = []
        for i, r in enumerate(requests):
            spans = (ape_span_t * max(len(r.ctx), 1))(*[ape_span_t(int(s), int(l)) for s, l in r.ctx])
            keep.append(spans)
            arr[i] = ape_request_t(int(r.q_start), int(r.q_len), ape_span_t(*map(int, r.prefix)), spans, len(r.ctx),
                                   ape_span_t(*map(int, r.query_kv)), int(r.query_kv_capacity))
        _check(load().ape_attend_once(self._h, C.byref(shape), C.byref(pool), C.byref(qr), C.byref(orows),
                                      lse.data_ptr() if lse is not None else None, arr, n, int(mode), float(T), float(S),
                                      _stream_ptr(stream)), "ape_attend_once")

    def attend_plan(self, *, H_q: int, H_kv: int, d: int, k_pool: torch.Tensor, v_pool: torch.Tensor,
                    q: torch.Tensor, out: torch.Tensor, requests: Sequence, mode: int,
                    lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0, per_context: bool = False,
                    shared: bool = False, tree=None) -> "Plan":
        """ape_attend_plan (or ape_attend_plan_per_context: S on every context's own LSE, Eq. 11-12; or, with shared=True,
        ape_attend_plan_shared: a decode batch whose requests all attend to the same contexts).  `requests`: objects with q_start, q_len, prefix, ctx, query_kv, query_kv_capacity
        (spans are (start, len) pairs), e.g. paper_2502_05431_b200.workloads.Request.
        `tree` = (parents, scaled) selects ape_attend_plan_tree: parents[r][i] is the parent of request r's node i (its
        ctx[i]), -1 at the top level; scaled (or scaled[r]) may be None (the top-level nodes carry S)."""
        shape = ape_shape_t(H_q, H_kv, d, softmax_scale)
        pool, qr, orows = _pool(k_pool, v_pool), _rows(q), _rows(out)
        n = len(requests)
        arr = (ape_request_t * max(n, 1))()
        keep = []
        for i, r in enumerate(requests):
            spans = (ape_span_t * max(len(r.ctx), 1))(*[ape_span_t(int(s), int(l)) for s, l in r.ctx])
            keep.append(spans)
            arr[i] = ape_request_t(int(r.q_start), int(r.q_len), ape_span_t(*map(int, r.prefix)), spans, len(r.ctx),
                                   ape_span_t(*map(int, r.query_kv)), int(r.query_kv_capacity))
        p = C.c_void_p()
        if tree is not None:
            parents, scaled = tree
            par_arrs = [(C.c_int32 * max(len(pp), 1))(*[int(x) for x in pp]) for pp in parents]
            par = (C.POINTER(C.c_int32) * max(n, 1))(*[C.cast(a, C.POINTER(C.c_int32)) for a in par_arrs])
            sc = None
            if scaled is not None:
                sc_arrs = [None if ss is None else (C.c_uint8 * max(len(ss), 1))(*[1 if x else 0 for x in ss]) for ss in scaled]
                sc = (C.POINTER(C.c_uint8) * max(n, 1))(*[C.cast(a, C.POINTER(C.c_uint8)) if a is not None
                                                         else C.POINTER(C.c_uint8)() for a in sc_arrs])
            _check(load().ape_attend_plan_tree(self._h, C.byref(shape), C.byref(pool), C.byref(qr), C.byref(orows),
                                               lse.data_ptr() if lse is not None else None, arr, n, par, sc, int(mode), C.byref(p)),
                   "ape_attend_plan_tree")
            return Plan(self, p, (q, out, k_pool, v_pool, lse))
        if shared:
            _check(load().ape_attend_plan_shared(self._h, C.byref(shape), C.byref(pool), C.byref(qr), C.byref(orows),
                                                 lse.data_ptr() if lse is not None else None, arr, n, C.byref(p)),
                   "ape_attend_plan_shared")
            return Plan(self, p, (q, out, k_pool, v_pool, lse))
        fn = load().ape_attend_plan_per_context if per_context else load().ape_attend_plan
        _check(fn(self._h, C.byref(shape), C.byref(pool), C.byref(qr), C.byref(orows),
                  lse.data_ptr() if lse is not None else None, arr, n, int(mode), C.byref(p)),
               "ape_attend_plan_per_context" if per_context else "ape_attend_plan")
        return Plan(self, p, (q, out, k_pool, v_pool, lse))

    def encode_plan(self, *, H_q: int, H_kv: int, d: int, k_pool: torch.Tensor, v_pool: torch.Tensor,
                    q: torch.Tensor, out: torch.Tensor, prefix, ctx: Sequence,
                    lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0) -> "Plan":
        """ape_encode_plan.  q / out rows are aligned with the pool tokens."""
        shape = ape_shape_t(H_q, H_kv, d, softmax_scale)
        pool, qr, orows = _pool(k_pool, v_pool), _rows(q), _rows(out)
        pre = ape_span_t(int(prefix[0]), int(prefix[1]))
        spans = (ape_span_t * max(len(ctx), 1))(*[ape_span_t(int(s), int(l)) for s, l in ctx])
        p = C.c_void_p()
        _check(load().ape_encode_plan(self._h, C.byref(shape), C.byref(pool), C.byref(qr), C.byref(orows),
                                      lse.data_ptr() if lse is not None else None, C.byref(pre), spans, len(ctx), C.byref(p)),
               "ape_encode_plan")
        return Plan(self, p, (q, out, k_pool, v_pool, lse))


def merge_shards(handle: "Handle", *, H_q: int, H_kv: int, d: int, o_ctx_all: torch.Tensor, lse_ctx_all: torch.Tensor,
                 o_oth: torch.Tensor, lse_oth: torch.Tensor, S: float, out: torch.Tensor, lse: Optional[torch.Tensor] = None,
                 softmax_scale: float = 0.0, stream: Optional[torch.cuda.Stream] = None) -> None:
    """ape_merge_shards: o_ctx_all fp32 [n_shards, rows, H_q, d], lse_ctx_all fp32 [n_shards, rows, H_q] (contiguous)."""
    shape = ape_shape_t(H_q, H_kv, d, softmax_scale)
    orows = _rows(out)
    _check(load().ape_merge_shards(handle._h, C.byref(shape), int(o_ctx_all.shape[1]), int(o_ctx_all.shape[0]),
                                   o_ctx_all.data_ptr(), lse_ctx_all.data_ptr(), o_oth.data_ptr(), lse_oth.data_ptr(), float(S),
                                   C.byref(orows), lse.data_ptr() if lse is not None else None, _stream_ptr(stream)),
           "ape_merge_shards")


def rope_runs_for_request(request, src_start: int = 0):
    """ape_rope_runs_for_request: [(src_start, dst_start, len, pos0), ...] of one request under position re-use."""
    spans = (ape_span_t * max(len(request.ctx), 1))(*[ape_span_t(int(s), int(l)) for s, l in request.ctx])
    rq = ape_request_t(int(request.q_start), int(request.q_len), ape_span_t(*map(int, request.prefix)), spans,
                       len(request.ctx), ape_span_t(*map(int, request.query_kv)), int(request.query_kv_capacity))
    cap = len(request.ctx) + 2
    runs = (ape_rope_run_t * cap)()
    n = C.c_int32(0)
    _check(load().ape_rope_runs_for_request(C.byref(rq), int(src_start), runs, cap, C.byref(n)), "ape_rope_runs_for_request")
    return [(r.src_start, r.dst_start, r.len, r.pos0) for r in runs[: n.value]]


class RopePlan:
    """ape_rope_plan / ape_rope_write / ape_plan_destroy."""

    def __init__(self, handle: "Handle", d: int, theta: float, runs: Sequence):
        arr = (ape_rope_run_t * max(len(runs), 1))(*[ape_rope_run_t(*map(int, r)) for r in runs])
        self._handle, self._p = handle, C.c_void_p()
        _check(load().ape_rope_plan(handle._h, int(d), float(theta), arr, len(runs), C.byref(self._p)), "ape_rope_plan")

    def write(self, src: torch.Tensor, dst: torch.Tensor, rotate: bool, stream: Optional[torch.cuda.Stream] = None) -> None:
        """ape_rope_write: src, dst bf16 [rows, heads, d] on the plan's device."""
        st = stream if stream is not None else torch.cuda.current_stream(src.device)
        sr, dr = _rows(src), _rows(dst)
        _check(load().ape_rope_write(self._p, C.byref(sr), C.byref(dr), int(src.shape[1]), 1 if rotate else 0,
                                     C.c_void_p(st.cuda_stream)), "ape_rope_write")

    def close(self) -> None:
        if self._p:
            load().ape_plan_destroy(self._p)
            self._p = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Plan:
    """An attend or encode plan: ape_plan_workspace_bytes / ape_attend / ape_encode_contexts / ape_plan_destroy."""

    def __init__(self, handle: Handle, p: C.c_void_p, keep_alive):
        self._handle, self._p, self._keep = handle, p, keep_alive
        n = C.c_size_t(0)
        _check(load().ape_plan_workspace_bytes(self._p, C.byref(n)), "ape_plan_workspace_bytes")
        self.workspace_bytes = int(n.value)

    def alloc_workspace(self, device=None) -> torch.Tensor:
        dev = device if device is not None else self._keep[0].device
        return torch.empty(max(self.workspace_bytes, 256), dtype=torch.uint8, device=dev)

    def attend(self, T: float, S: float, workspace: torch.Tensor, kv_extra: int = 0,
               stream: Optional[torch.cuda.Stream] = None) -> None:
        _check(load().ape_attend(self._p, float(T), float(S), int(kv_extra), workspace.data_ptr(), workspace.numel(),
                                 _stream_ptr(stream)), "ape_attend")

    def attend_partial(self, T: float, workspace: torch.Tensor, o_ctx: torch.Tensor, lse_ctx: torch.Tensor,
                       o_oth: torch.Tensor, lse_oth: torch.Tensor, kv_extra: int = 0,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
        """ape_attend_partial: fp32 device tensors o_* [q rows, H_q, d], lse_* [q rows, H_q] receive this shard's segments."""
        part = ape_partials_t(o_ctx.data_ptr(), lse_ctx.data_ptr(), o_oth.data_ptr(), lse_oth.data_ptr())
        _check(load().ape_attend_partial(self._p, float(T), int(kv_extra), workspace.data_ptr(), workspace.numel(),
                                         C.byref(part), _stream_ptr(stream)), "ape_attend_partial")

    def encode_contexts(self, workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> None:
        _check(load().ape_encode_contexts(self._p, workspace.data_ptr() if workspace is not None else None,
                                          workspace.numel() if workspace is not None else 0, _stream_ptr(stream)),
               "ape_encode_contexts")

    def attend_host(self, T: float, S: float, workspace: torch.Tensor, h_q: torch.Tensor, h_k: torch.Tensor,
                    h_v: torch.Tensor, h_out: torch.Tensor, kv_extra: int = 0,
                    stream: Optional[torch.cuda.Stream] = None):
        """ape_attend_host: host tensors in, host tensor out; returns (h2d_bytes, d2h_bytes)."""
        a, b = C.c_size_t(0), C.c_size_t(0)
        _check(load().ape_attend_host(self._p, float(T), float(S), int(kv_extra), workspace.data_ptr(), workspace.numel(),
                                      h_q.data_ptr(), h_k.data_ptr(), h_v.data_ptr(), h_out.data_ptr(),
                                      C.byref(a), C.byref(b), _stream_ptr(stream)), "ape_attend_host")
        return int(a.value), int(b.value)

    def decode_step_host(self, T: float, S: float, workspace: torch.Tensor, h_q: torch.Tensor, h_out: torch.Tensor,
                         h_k_new: Optional[torch.Tensor] = None, h_v_new: Optional[torch.Tensor] = None, kv_extra: int = 0,
                         stream: Optional[torch.cuda.Stream] = None):
        """ape_decode_step_host: the new token's Q (and optionally its K, V, appended to the cache) from host tensors, O back
        to a host tensor; returns (h2d_bytes, d2h_bytes)."""
        a, b = C.c_size_t(0), C.c_size_t(0)
        _check(load().ape_decode_step_host(self._p, float(T), float(S), int(kv_extra), workspace.data_ptr(), workspace.numel(),
                                           h_q.data_ptr(), h_k_new.data_ptr() if h_k_new is not None else None,
                                           h_v_new.data_ptr() if h_v_new is not None else None, h_out.data_ptr(),
                                           C.byref(a), C.byref(b), _stream_ptr(stream)), "ape_decode_step_host")
        return int(a.value), int(b.value)

    def last_launches(self) -> int:
        n = C.c_int32(0)
        _check(load().ape_plan_last_launches(self._p, C.byref(n)), "ape_plan_last_launches")
        return int(n.value)

    def close(self) -> None:
        if self._p:
            load().ape_plan_destroy(self._p)
            self._p = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
