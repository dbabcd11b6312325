"""fp64 CPU oracle for the rotary position embedding with position re-use.

TEST INFRASTRUCTURE ONLY: imported by the test-suite and the smoke check.  The product package never imports it.

What it computes
  * rotary embedding of Su et al. (the relative position embedding the paper builds on, Section 2 "Position
    Embedding"), in the half-split pairing that the paper's base models (the Llama family) use: component i of a head
    is paired with component i + d/2 and the pair is rotated by the angle pos * theta^(-2i/d);
  * the positions of an APE request (Section 1, "Re-using Positions for Long Context"; Section 4.1 for the shared
    prefix): the prefix sits at 0 .. l_P-1, EVERY context starts right after the prefix, at l_P, and the query starts
    after the longest context, at l_P + max_i l_i.

Plain numpy in float64; inputs are bf16 tensors widened exactly.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np
import torch


def inv_freq(d: int, theta: float) -> np.ndarray:
    """Angular frequency of pair i, i = 0 .. d/2-1: theta^(-2i/d)."""
    i = np.arange(d // 2, dtype=np.float64)
    return np.float64(theta) ** (-(2.0 * i) / np.float64(d))


def rope(x: torch.Tensor, pos: Sequence[int], theta: float) -> np.ndarray:
    """x: [n, H, d] (any float dtype, widened exactly), pos: n integer positions.  Returns float64 [n, H, d]."""
    xf = x.detach().cpu().to(torch.float64).numpy()
    n, _, d = xf.shape
    p = np.asarray(pos, dtype=np.float64).reshape(n, 1, 1)
    ang = p * inv_freq(d, theta).reshape(1, 1, d // 2)
    c, s = np.cos(ang), np.sin(ang)
    a, b = xf[..., : d // 2], xf[..., d // 2:]
    out = np.empty_like(xf)
    out[..., : d // 2] = a * c - b * s
    out[..., d // 2:] = b * c + a * s
    return out


def positions(l_P: int, ctx_lens: Sequence[int], l_q: int) -> Dict[str, object]:
    """Position of every token of a request under position re-use."""
    longest = max(ctx_lens) if len(ctx_lens) else 0
    return {
        "prefix": np.arange(l_P, dtype=np.int64),
        "contexts": [l_P + np.arange(l, dtype=np.int64) for l in ctx_lens],
        "query": l_P + longest + np.arange(l_q, dtype=np.int64),
    }
