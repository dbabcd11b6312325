"""Pins for the oracle's context-tree form (ape_oracle_attend_tree), against things other than itself:

  * the dense one-softmax statement of the same reading (tests/brute_force.py::tree_bias, numpy, independent);
  * the two printed formulas the family contains: one node per context is the appendix's Eq. 11-12 (checked against the
    oracle's per-context switch AND the independent numpy form), one tree over all contexts is Eq. 5;
  * a single branch (a chain of nodes) is Eq. 5 with its tokens as one context;
  * S = 1 is ordinary attention (torch's scaled_dot_product_attention in fp64) whatever the tree;
  * hand-derived closed forms for zero queries (tests/golden/tree_closed_form_q0.txt);
  * invariants: order of siblings, regrouping below the scaled nodes.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import ape_oracle as orc
from paper_2502_05431_b200 import workloads as wl
from tests import brute_force as bf
from tests.test_oracle_pins import _sdpa_concat

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _batch(lens, seed=0, H_q=4, H_kv=2, d=16, l_P=3, l_q=5, l_k=None):
    return wl.make_batch(H_q=H_q, H_kv=H_kv, d=d, l_P=l_P, ctx_lens=[list(lens)], l_q=l_q, l_k=l_k, seed=seed)


TREES = [
    # (node lengths, parent, scaled or None)
    ((5, 7, 4), (-1, -1, -1), None),                                   # a forest of leaves
    ((0, 5, 7, 4), (-1, 0, 0, 0), None),                               # one grouping root over three leaves
    ((3, 4, 9), (-1, 0, 0), (1, 1, 1)),                                # root with own tokens, everything scaled
    ((2, 0, 6, 3, 5, 1, 4), (-1, 0, 1, 1, 0, -1, 5), None),            # depth 3, an empty inner node, two top-level trees
    ((2, 0, 6, 3, 5, 1, 4), (-1, 0, 1, 1, 0, -1, 5), (0, 1, 0, 1, 1, 1, 0)),   # S at mixed levels
    ((4, 3, 2, 1), (-1, 0, 1, 2), (1, 1, 1, 1)),                       # a chain, S at every level
    ((0, 0, 5), (-1, 0, 1), None),                                     # grouping nodes only above one leaf
    ((0, 3, 0), (-1, 0, 0), None),                                     # an empty leaf
]


@pytest.mark.parametrize("tree", range(len(TREES)))
@pytest.mark.parametrize("T,S", [(1.0, 1.0), (0.8, 0.9), (0.5, 0.4), (1.3, 1.2)])
def test_tree_oracle_equals_dense_bias_softmax(tree, T, S):
    lens, parent, scaled = TREES[tree]
    b = _batch(lens, seed=tree, l_k=7 if tree % 2 else None)
    q, p, c, k = b.views(0)
    res = orc.attend_tree(q, p, c, k, T, S, parent, scaled)
    ref, lam = bf.tree_bias(q, p, c, k, T, S, parent, scaled)
    np.testing.assert_allclose(res.out.numpy(), ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(res.lse.numpy(), lam, rtol=0, atol=1e-11)


@pytest.mark.parametrize("T,S", [(0.8, 0.9), (0.6, 0.5)])
def test_one_node_per_context_is_the_per_context_form(T, S):
    """Depth 1: every context a top-level node -> Eq. 11-12."""
    b = _batch((5, 7, 0, 4), seed=11)
    q, p, c, k = b.views(0)
    res = orc.attend_tree(q, p, c, k, T, S, [-1] * 4)
    np.testing.assert_allclose(res.out.numpy(), orc.attend(q, p, c, k, T, S, per_context=True).out.numpy(), atol=1e-12)
    np.testing.assert_allclose(res.out.numpy(), bf.per_context(q, p, c, k, T, S), atol=1e-12)
    assert np.abs(res.out.numpy() - orc.attend(q, p, c, k, T, S).out.numpy()).max() > 1e-4      # and not Eq. 5


@pytest.mark.parametrize("T,S", [(0.8, 0.9), (0.6, 0.5)])
def test_one_tree_over_all_contexts_is_eq5(T, S):
    """All contexts under one root -> the whole context mass is raised to S: Eq. 5, however the tree is shaped below."""
    b = _batch((5, 7, 4, 6), seed=12)
    q, p, c, k = b.views(0)
    flat = orc.attend(q, p, c, k, T, S)
    empty = (p[0][:0], p[1][:0])
    for nodes, parent in [
        ([empty] + list(c), [-1, 0, 0, 0, 0]),                         # a grouping root
        (list(c), [-1, 0, 0, 0]),                                      # the first context is the root
        (list(c), [-1, 0, 1, 2]),                                      # a chain
        ([empty, empty] + list(c), [-1, 0, 1, 1, 0, 0]),               # an inner grouping node
    ]:
        res = orc.attend_tree(q, p, nodes, k, T, S, parent)
        np.testing.assert_allclose(res.out.numpy(), flat.out.numpy(), atol=1e-12)
        np.testing.assert_allclose(res.lse.numpy(), flat.lse.numpy(), atol=1e-11)
        np.testing.assert_allclose(res.out.numpy(), bf.flat_bias(q, p, list(c), k, T, S)[0], atol=1e-12)


def test_a_single_branch_is_eq5_with_one_context():
    b = _batch((4, 3, 6), seed=13)
    q, p, c, k = b.views(0)
    joined = (torch.cat([x[0] for x in c]), torch.cat([x[1] for x in c]))
    res = orc.attend_tree(q, p, c, k, 0.7, 0.6, [-1, 0, 1])
    np.testing.assert_allclose(res.out.numpy(), orc.attend(q, p, [joined], k, 0.7, 0.6).out.numpy(), atol=1e-12)
    np.testing.assert_allclose(res.out.numpy(), bf.two_pass(q, p, [joined], k, 0.7, 0.6), atol=1e-12)


@pytest.mark.parametrize("tree", range(len(TREES)))
@pytest.mark.parametrize("T", [1.0, 0.6])
def test_S1_is_ordinary_attention_for_any_tree(tree, T):
    lens, parent, scaled = TREES[tree]
    b = _batch(lens, seed=20 + tree)
    q, p, c, k = b.views(0)
    res = orc.attend_tree(q, p, c, k, T, 1.0, parent, scaled)
    np.testing.assert_allclose(res.out.numpy(), _sdpa_concat(q, p, c, k, T), atol=1e-12)


def test_golden_closed_form_zero_query():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "tree_closed_form_q0.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for idx, (S, l_P, row, n0, n1, n2, w_o, w0, w1, w2, log_den) in enumerate(rows):
        S, l_P, row, lens = float(S), int(l_P), int(row), (int(n0), int(n1), int(n2))
        b = wl.make_batch(H_q=2, H_kv=1, d=8, l_P=l_P, ctx_lens=[list(lens)], l_q=row + 1, seed=3)
        b.q.zero_()
        q, p, c, k = b.views(0)
        scaled = (1, 1, 1) if idx == 0 else None
        for T in (1.0, 0.4):                          # T is irrelevant when all logits are zero
            res = orc.attend_tree(q, p, c, k, T, S, [-1, 0, 0], scaled)
            expect = float(w_o) * (p[1].double().sum(0) + k[1][:row + 1].double().sum(0))
            for (kk, vv), w in zip(c, (w0, w1, w2)):
                expect = expect + float(w) * vv.double().sum(0)
            np.testing.assert_allclose(res.out[row].numpy(), expect.repeat(2, 1).numpy(), rtol=0, atol=1e-13)
            assert abs(res.lse[row, 0].item() - float(log_den)) < 1e-13


def test_order_of_siblings_does_not_matter():
    lens, parent = (0, 5, 7, 4, 2, 3), [-1, 0, 0, -1, 3, 3]
    b = _batch(lens, seed=31)
    q, p, c, k = b.views(0)
    a = orc.attend_tree(q, p, c, k, 0.8, 0.7, parent, [1, 1, 0, 1, 0, 1])
    # the two top-level trees swapped, and the children inside each swapped
    order = [3, 5, 4, 0, 2, 1]
    new_index = {old: new for new, old in enumerate(order)}
    c2 = [c[o] for o in order]
    parent2 = [(-1 if parent[o] < 0 else new_index[parent[o]]) for o in order]
    scaled2 = [[1, 1, 0, 1, 0, 1][o] for o in order]
    r = orc.attend_tree(q, p, c2, k, 0.8, 0.7, parent2, scaled2)
    np.testing.assert_allclose(a.out.numpy(), r.out.numpy(), atol=1e-12)


def test_regrouping_below_the_scaled_nodes_does_not_matter_but_moving_S_does():
    b = _batch((0, 5, 7, 4, 6), seed=32)
    q, p, c, k = b.views(0)
    empty = (p[0][:0], p[1][:0])
    a = orc.attend_tree(q, p, c, k, 0.8, 0.6, [-1, 0, 0, 0, 0])                               # root scaled, four leaves
    g = orc.attend_tree(q, p, [c[0], empty, c[1], c[2], c[3], c[4]], k, 0.8, 0.6, [-1, 0, 1, 1, 0, 0])   # two leaves regrouped
    np.testing.assert_allclose(a.out.numpy(), g.out.numpy(), atol=1e-12)
    m = orc.attend_tree(q, p, c, k, 0.8, 0.6, [-1, 0, 0, 0, 0], [0, 1, 1, 1, 1])              # S moved to the leaves
    assert np.abs(a.out.numpy() - m.out.numpy()).max() > 1e-4
    np.testing.assert_allclose(m.out.numpy(), orc.attend(q, p, c, k, 0.8, 0.6, per_context=True).out.numpy(), atol=1e-12)


def test_bad_trees_are_refused():
    b = _batch((3, 4), seed=33)
    q, p, c, k = b.views(0)
    for parent in ([0, -1], [-1, 1], [-1, 5], [-2, 0]):
        with pytest.raises(RuntimeError):
            orc.attend_tree(q, p, c, k, 0.8, 0.9, parent)
