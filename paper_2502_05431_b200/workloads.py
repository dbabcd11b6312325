"""Seeded synthetic inputs for APE attention.

This module only draws random tensors and lays them out; it holds none of the
method's arithmetic, so both the GPU library's tests and the CPU oracle's tests
may use it.

Layout (the one the C-ABI library consumes):
  * one KV pool per batch: ``k_pool`` / ``v_pool``, bf16 ``[pool_tokens, H_kv, d]``;
  * every segment of every request (shared prefix, each cached context, the
    query's own KV) is a span ``(start, len)`` of pool tokens;
  * one Q tensor ``[sum l_q, H_q, d]`` for attend; for encode a Q tensor aligned
    with the pool (``[pool_tokens, H_q, d]``): row t is the query of pool token t.

Draw order per request (fp32 N(0,1) from ``torch.Generator('cpu')`` seeded with
``seed + request index``, then rounded to bf16): optional per-KV-head scales,
q, k_P, v_P, (k_Ci, v_Ci for i = 0..N-1), k_Q, v_Q, then encode queries.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import torch

Span = Tuple[int, int]  # (start token in the pool, length)


@dataclass
class Request:
    q_start: int
    q_len: int
    prefix: Span
    ctx: List[Span]
    query_kv: Span
    query_kv_capacity: int


@dataclass
class Batch:
    H_q: int
    H_kv: int
    d: int
    q: torch.Tensor            # bf16 [sum q_len, H_q, d]
    k_pool: torch.Tensor       # bf16 [pool_tokens, H_kv, d]
    v_pool: torch.Tensor
    requests: List[Request]
    T: float = 1.0
    S: float = 1.0
    q_enc: Optional[torch.Tensor] = None   # bf16 [pool_tokens, H_q, d], encode queries (context rows only)
    name: str = ""
    extra: Dict = field(default_factory=dict)

    def views(self, r: int):
        """(q, prefix(k,v), [ctx(k,v)], query_kv(k,v)) tensor views of request r, for per-request consumers."""
        rq = self.requests[r]
        sl = lambda s: (self.k_pool[s[0]:s[0] + s[1]], self.v_pool[s[0]:s[0] + s[1]])
        return (self.q[rq.q_start:rq.q_start + rq.q_len], sl(rq.prefix), [sl(c) for c in rq.ctx], sl(rq.query_kv))

    def to(self, device) -> "Batch":
        mv = lambda t: None if t is None else t.to(device, non_blocking=False)
        return Batch(self.H_q, self.H_kv, self.d, mv(self.q), mv(self.k_pool), mv(self.v_pool),
                     self.requests, self.T, self.S, mv(self.q_enc), self.name, dict(self.extra))


def _randn_bf16(gen: torch.Generator, shape, scale: Optional[torch.Tensor] = None) -> torch.Tensor:
    x = torch.randn(shape, generator=gen, dtype=torch.float32, device=gen.device)
    if scale is not None:
        x = x * scale.view(1, -1, 1)
    return x.to(torch.bfloat16)


def share_contexts(b: Batch) -> Batch:
    """The same tensors with every request pointed at request 0's contexts (each keeps its own prefix, query rows and
    query segment): a batch of queries over one set of cached contexts.  The span tables of the requests list the shared
    contexts in different (rotated) orders."""
    ctx0 = list(b.requests[0].ctx)
    reqs = []
    for i, r in enumerate(b.requests):
        k = i % max(len(ctx0), 1)
        reqs.append(Request(r.q_start, r.q_len, r.prefix, ctx0[k:] + ctx0[:k], r.query_kv, r.query_kv_capacity))
    return Batch(b.H_q, b.H_kv, b.d, b.q, b.k_pool, b.v_pool, reqs, b.T, b.S, b.q_enc, b.name + "+shared", dict(b.extra))


def make_batch(*, H_q: int, H_kv: int, d: int, l_P: int, ctx_lens: Sequence[Sequence[int]], l_q: int,
               l_k: Optional[int] = None, capacity: Optional[int] = None, seed: int = 0,
               T: float = 1.0, S: float = 1.0, head_scale: bool = False, gap: int = 0,
               with_encode_q: bool = False, shuffle_ctx: bool = False, name: str = "",
               device: Optional[str] = None) -> Batch:
    """Build a batch of ``len(ctx_lens)`` requests with independent context sets.

    ``gap`` leaves that many unused (zero) tokens after every span so that spans are
    not adjacent; ``shuffle_ctx`` lists each request's contexts in a seeded random
    order different from their order in the pool.  ``l_k`` is the number of keys in the
    query's own segment (default ``l_q``); ``capacity`` reserves room for decode appends.
    ``device``: draw and keep the tensors there (e.g. "cuda:0", for workloads too large to draw on the host
    in reasonable time); the values then come from that device's generator, same distribution and layout.
    """
    dev = torch.device(device) if device is not None else torch.device("cpu")
    n_req = len(ctx_lens)
    l_k = l_q if l_k is None else l_k
    capacity = l_k if capacity is None else capacity
    assert capacity >= l_k >= l_q
    per_req_tokens = [l_P + sum(cl) + capacity + gap * (len(cl) + 2) for cl in ctx_lens]
    pool_tokens = sum(per_req_tokens)
    k_pool = torch.zeros((pool_tokens, H_kv, d), dtype=torch.bfloat16, device=dev)
    v_pool = torch.zeros((pool_tokens, H_kv, d), dtype=torch.bfloat16, device=dev)
    q = torch.zeros((n_req * l_q, H_q, d), dtype=torch.bfloat16, device=dev)
    q_enc = torch.zeros((pool_tokens, H_q, d), dtype=torch.bfloat16, device=dev) if with_encode_q else None
    requests: List[Request] = []
    cur = 0
    for r, lens in enumerate(ctx_lens):
        gen = torch.Generator(device=dev).manual_seed(seed + r)
        sk = sv = None
        if head_scale:
            sk = torch.rand(H_kv, generator=gen, device=dev) * 1.5 + 0.5
            sv = torch.rand(H_kv, generator=gen, device=dev) * 1.5 + 0.5
        q[r * l_q:(r + 1) * l_q] = _randn_bf16(gen, (l_q, H_q, d))
        bulk = dev.type != "cpu"     # on a device: one draw per tensor and request (same distribution, few launches)
        if bulk:
            n_tok = per_req_tokens[r]
            k_pool[cur:cur + n_tok] = _randn_bf16(gen, (n_tok, H_kv, d), sk)
            v_pool[cur:cur + n_tok] = _randn_bf16(gen, (n_tok, H_kv, d), sv)
            if with_encode_q:
                q_enc[cur:cur + n_tok] = _randn_bf16(gen, (n_tok, H_q, d))
        prefix = (cur, l_P)
        if l_P and not bulk:
            k_pool[cur:cur + l_P] = _randn_bf16(gen, (l_P, H_kv, d), sk)
            v_pool[cur:cur + l_P] = _randn_bf16(gen, (l_P, H_kv, d), sv)
        cur += l_P + gap
        spans: List[Span] = []
        for L in lens:
            if L and not bulk:
                k_pool[cur:cur + L] = _randn_bf16(gen, (L, H_kv, d), sk)
                v_pool[cur:cur + L] = _randn_bf16(gen, (L, H_kv, d), sv)
            spans.append((cur, L))
            cur += L + gap
        qkv = (cur, l_k)
        if not bulk:
            k_pool[cur:cur + capacity] = _randn_bf16(gen, (capacity, H_kv, d), sk)
            v_pool[cur:cur + capacity] = _randn_bf16(gen, (capacity, H_kv, d), sv)
        cur += capacity + gap
        if with_encode_q and not bulk:
            for (s, L) in spans:
                if L:
                    q_enc[s:s + L] = _randn_bf16(gen, (L, H_q, d))
        if shuffle_ctx and len(spans) > 1:
            perm = torch.randperm(len(spans), generator=gen, device=dev).tolist()
            spans = [spans[p] for p in perm]
        requests.append(Request(r * l_q, l_q, prefix, spans, qkv, capacity))
    assert cur == pool_tokens
    return Batch(H_q, H_kv, d, q, k_pool, v_pool, requests, T, S, q_enc, name)


# ---- the benchmark configurations (shapes follow the paper's efficiency and RAG workloads) --------------------

LLAMA3_8B = dict(H_q=32, H_kv=8, d=128)


def config1(seed: int = 0) -> Batch:
    """Tiny case: 4 q heads / 1 KV head, d 64, prefix 16, 4 contexts x 64 (positions reused), 16 causal query rows."""
    return make_batch(H_q=4, H_kv=1, d=64, l_P=16, ctx_lens=[[64] * 4], l_q=16, seed=seed, T=0.8, S=0.9,
                      with_encode_q=True, name="cfg1_tiny")


def config2(seed: int = 0) -> Batch:
    """Llama-3-8B head shape, prefix 32, 10 contexts x 256, 64 query rows: encode, then query prefill."""
    return make_batch(**LLAMA3_8B, l_P=32, ctx_lens=[[256] * 10], l_q=64, seed=seed, T=0.9, S=0.9,
                      with_encode_q=True, name="cfg2_llama_10x256")


def config3_lens(seed: int = 0, n_req: int = 4, n_ctx: int = 20) -> List[List[int]]:
    gen = torch.Generator(device="cpu").manual_seed(1000 + seed)
    return [torch.randint(512, 1537, (n_ctx,), generator=gen).tolist() for _ in range(n_req)]


def config3(seed: int = 0, T: float = 0.9, S: float = 0.8) -> Batch:
    """RAG shape: prefix 64, 20 contexts with lengths uniform in [512,1536], 128 query rows, 4 independent requests."""
    return make_batch(**LLAMA3_8B, l_P=64, ctx_lens=config3_lens(seed), l_q=128, seed=seed, T=T, S=S,
                      name="cfg3_rag")


def config4(seed: int = 0, n_ctx: int = 500, with_encode_q: bool = False, device: Optional[str] = None) -> Batch:
    """Many-shot 128K: prefix 64, 500 contexts x 256 tokens, 256 causal query rows, per-KV-head scale U[0.5,2]."""
    return make_batch(**LLAMA3_8B, l_P=64, ctx_lens=[[256] * n_ctx], l_q=256, seed=seed, T=0.9, S=0.9,
                      head_scale=True, with_encode_q=with_encode_q, name="cfg4_manyshot_128k", device=device)


def config5(seed: int = 0, n_req: int = 16, n_ctx: int = 500, steps: int = 256, device: Optional[str] = None) -> Batch:
    """Decode at 128K: per request prefix 64 + 500x256 contexts + 256 cached query tokens; one new row per step.

    The pool reserves ``256 + steps`` query-segment tokens per request, all pre-drawn, so step t reads
    ``256 + t + 1`` of them; ``extra['q_steps']`` holds the new token's query for every step,
    bf16 ``[steps, n_req, H_q, d]``.
    """
    b = make_batch(**LLAMA3_8B, l_P=64, ctx_lens=[[256] * n_ctx] * n_req, l_q=1, l_k=257, capacity=256 + steps,
                   seed=seed, T=0.9, S=0.9, name="cfg5_decode_128k", device=device)
    gen = torch.Generator(device=b.q.device).manual_seed(seed + 7919)
    b.extra["q_steps"] = torch.randn((steps, n_req, b.H_q, b.d), generator=gen, dtype=torch.float32,
                                     device=b.q.device).to(torch.bfloat16)
    b.extra["steps"] = steps
    return b
