"""Pins of the rotary-embedding oracle against things other than itself: complex multiplication, closed forms,
the invariants of a rotation, and the position rule of position re-use (Sections 1 and 2 of the paper)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import rope_oracle as ro

HERE = os.path.dirname(os.path.abspath(__file__))


def _rand(n, H, d, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(n, H, d, generator=g).to(torch.bfloat16)


def test_complex_multiplication_form():
    # a rotation of the pair (a, b) by phi is the complex product (a + ib) e^{i phi}: numpy's complex arithmetic
    x = _rand(9, 3, 16, 1)
    pos = [0, 1, 2, 5, 17, 100, 1000, 65535, 131071]
    theta = 500000.0
    out = ro.rope(x, pos, theta)
    xf = x.to(torch.float64).numpy()
    z = xf[..., :8] + 1j * xf[..., 8:]
    k = np.arange(8)
    w = np.exp(1j * np.asarray(pos, dtype=np.float64)[:, None, None] * (theta ** (-2.0 * k / 16.0))[None, None, :])
    zz = z * w
    np.testing.assert_allclose(out[..., :8], zz.real, rtol=0, atol=1e-12)
    np.testing.assert_allclose(out[..., 8:], zz.imag, rtol=0, atol=1e-12)


def test_position_zero_is_identity():
    x = _rand(4, 2, 64, 2)
    np.testing.assert_array_equal(ro.rope(x, [0, 0, 0, 0], 10000.0), x.to(torch.float64).numpy())


def test_golden_closed_form_d4():
    want = {}
    with open(os.path.join(HERE, "golden", "rope_d4_closed_form.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            i, v = line.split()
            want[int(i)] = float(v)
    x = torch.tensor([[[1.0, 2.0, 0.0, 0.0]]], dtype=torch.bfloat16)
    out = ro.rope(x, [3], 10000.0)[0, 0]
    for i in range(4):
        assert abs(out[i] - want[i]) < 5e-12, (i, out[i], want[i])


def test_unit_vector_d2():
    # d = 2: a single pair with frequency 1; (1, 0) at position p goes to (cos p, sin p)
    x = torch.tensor([[[1.0, 0.0]]], dtype=torch.bfloat16)
    for p in (1, 2, 10, 1000):
        out = ro.rope(x, [p], 10000.0)[0, 0]
        assert abs(out[0] - math.cos(p)) < 1e-12 and abs(out[1] - math.sin(p)) < 1e-12


def test_second_component_uses_second_frequency():
    # a mistake in the pairing (interleaved instead of half-split) or in the exponent moves this value
    x = torch.tensor([[[0.0, 1.0, 0.0, 0.0]]], dtype=torch.bfloat16)
    out = ro.rope(x, [50], 10000.0)[0, 0]
    assert abs(out[1] - math.cos(0.5)) < 1e-12 and abs(out[3] - math.sin(0.5)) < 1e-12
    assert out[0] == 0.0 and out[2] == 0.0


def test_norm_of_every_pair_is_kept():
    x = _rand(6, 4, 128, 3)
    pos = [3, 77, 1024, 4097, 99999, 131000]
    out = ro.rope(x, pos, 500000.0)
    xf = x.to(torch.float64).numpy()
    np.testing.assert_allclose(out[..., :64] ** 2 + out[..., 64:] ** 2, xf[..., :64] ** 2 + xf[..., 64:] ** 2, rtol=1e-12)


def test_scores_depend_on_the_position_difference_only():
    q, k = _rand(1, 1, 64, 4), _rand(1, 1, 64, 5)
    theta = 10000.0
    def score(m, n):
        return float((ro.rope(q, [m], theta) * ro.rope(k, [n], theta)).sum())
    base = score(7, 0)
    for shift in (1, 13, 500, 100000):
        assert abs(score(7 + shift, shift) - base) < 1e-8 * max(1.0, abs(base))
    # and q at position m against k at position n equals q rotated by m - n against the raw k
    kf = k.to(torch.float64).numpy()
    assert abs(score(40, 33) - float((ro.rope(q, [7], theta) * kf).sum())) < 1e-9


def test_rotation_by_opposite_position_undoes_it():
    x = _rand(3, 2, 32, 6)
    out = ro.rope(x, [5, 50, 500], 10000.0)
    back = ro.rope(torch.from_numpy(out), [-5, -50, -500], 10000.0)
    np.testing.assert_allclose(back, x.to(torch.float64).numpy(), atol=1e-12)


def test_position_reuse_rule():
    # every context starts right after the prefix; the query starts after the longest context
    p = ro.positions(l_P=16, ctx_lens=[64, 10, 33], l_q=4)
    assert p["prefix"].tolist() == list(range(16))
    assert [c[0] for c in p["contexts"]] == [16, 16, 16]
    assert [c[-1] for c in p["contexts"]] == [79, 25, 48]
    assert p["query"].tolist() == [80, 81, 82, 83]
    # without contexts the query follows the prefix
    assert ro.positions(5, [], 2)["query"].tolist() == [5, 6]


def test_same_tokens_in_two_contexts_get_the_same_keys():
    # position re-use: a context's keys do not depend on which slot it takes among the contexts
    k = _rand(10, 2, 16, 7)
    p = ro.positions(4, [10, 10], 1)
    a = ro.rope(k, p["contexts"][0], 10000.0)
    b = ro.rope(k, p["contexts"][1], 10000.0)
    np.testing.assert_array_equal(a, b)
