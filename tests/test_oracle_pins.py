"""Pins for the fp64 CPU oracle: it is checked against things other than itself.

  * dense brute force over the concatenated sequence (tests/brute_force.py, numpy, written independently);
  * a library routine: torch's scaled_dot_product_attention in fp64 for the cases that reduce to ordinary attention;
  * closed forms of Eq. 5 (hand-derived numbers in tests/golden/closed_form_q0.txt);
  * invariants the equations imply (normalisation, permutation, context splitting, N=1 equivalence).
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import ape_oracle as orc
from paper_2502_05431_b200 import workloads as wl
from tests import brute_force as bf

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _tiny(seed=0, H_q=4, H_kv=2, d=16, l_P=3, lens=(5, 7, 4), l_q=6, l_k=None, **kw):
    return wl.make_batch(H_q=H_q, H_kv=H_kv, d=d, l_P=l_P, ctx_lens=[list(lens)], l_q=l_q, l_k=l_k, seed=seed, **kw)


def _sdpa_concat(q, prefix, ctx, qkv, T):
    """Ordinary attention (library routine) over [P | C/T | Q-causal] in fp64."""
    l_q, H_q, d = q.shape
    H_kv = qkv[0].shape[1]
    G = H_q // H_kv
    ks = [prefix[0].double()] + [k.double() / T for k, _ in ctx] + [qkv[0].double()]
    vs = [prefix[1].double()] + [v.double() for _, v in ctx] + [qkv[1].double()]
    K = torch.cat(ks, 0).repeat_interleave(G, dim=1).transpose(0, 1)   # [H_q, L, d]
    V = torch.cat(vs, 0).repeat_interleave(G, dim=1).transpose(0, 1)
    Q = q.double().transpose(0, 1)
    L, l_k = K.shape[1], qkv[0].shape[0]
    mask = torch.ones(l_q, L, dtype=torch.bool)
    i = torch.arange(l_q)[:, None]
    j = torch.arange(l_k)[None, :]
    mask[:, L - l_k:] = j <= i + (l_k - l_q)
    O = torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=mask)
    return O.transpose(0, 1).numpy()


CASES = [
    dict(),                                             # GQA 4/2, three ragged contexts
    dict(H_q=4, H_kv=1, d=8, l_P=0, lens=(9,), l_q=3),  # no prefix, one context
    dict(H_q=2, H_kv=2, d=8, l_P=4, lens=(), l_q=5),    # no context at all
    dict(H_q=6, H_kv=3, d=8, l_P=2, lens=(3, 0, 6), l_q=2, l_k=7),   # an empty context; more keys than rows
    dict(H_q=4, H_kv=1, d=32, l_P=5, lens=(8, 8), l_q=1, l_k=9),     # decode-shaped row
]


@pytest.mark.parametrize("case", range(len(CASES)))
@pytest.mark.parametrize("T,S", [(1.0, 1.0), (0.7, 1.0), (1.0, 0.6), (0.8, 0.9), (0.3, 0.2), (1.4, 1.3)])
def test_oracle_equals_dense_bias_softmax(case, T, S):
    b = _tiny(seed=case, **CASES[case])
    q, p, c, k = b.views(0)
    res = orc.attend(q, p, c, k, T, S)
    ref, lam = bf.flat_bias(q, p, c, k, T, S)
    np.testing.assert_allclose(res.out.numpy(), ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(res.lse.numpy(), lam, rtol=0, atol=1e-11)
    np.testing.assert_allclose(res.wsum.numpy(), 1.0, rtol=0, atol=1e-12)


@pytest.mark.parametrize("case", range(len(CASES)))
@pytest.mark.parametrize("T,S", [(0.8, 0.9), (0.5, 0.5), (1.0, 1.0)])
def test_oracle_equals_two_pass_merge(case, T, S):
    """Eq. 5 and the 'Efficient Implementation' form (two attentions + softmax over [S*LSE_C, LSE_other]) agree."""
    b = _tiny(seed=10 + case, **CASES[case])
    q, p, c, k = b.views(0)
    res = orc.attend(q, p, c, k, T, S)
    np.testing.assert_allclose(res.out.numpy(), bf.two_pass(q, p, c, k, T, S), rtol=0, atol=1e-12)


@pytest.mark.parametrize("case", range(len(CASES)))
@pytest.mark.parametrize("T", [1.0, 0.6])
def test_S1_reduces_to_library_attention(case, T):
    """S=1: plain parallel encoding (T=1) or ordinary attention with the context keys divided by T."""
    b = _tiny(seed=20 + case, **CASES[case])
    q, p, c, k = b.views(0)
    res = orc.attend(q, p, c, k, T, 1.0)
    np.testing.assert_allclose(res.out.numpy(), _sdpa_concat(q, p, c, k, T), rtol=0, atol=1e-12)


def test_custom_scale_is_used():
    b = _tiny(seed=3)
    q, p, c, k = b.views(0)
    a = orc.attend(q, p, c, k, 0.8, 0.9, scale=0.5).out.numpy()
    ref, _ = bf.flat_bias(q, p, c, k, 0.8, 0.9, scale=0.5)
    np.testing.assert_allclose(a, ref, atol=1e-12)
    assert np.abs(a - orc.attend(q, p, c, k, 0.8, 0.9).out.numpy()).max() > 1e-3


def _const_batch(l_P, L_C, l_q, vP, vC, vQ, n_ctx=1, d=8):
    """Zero queries, constant values per segment."""
    lens = [L_C // n_ctx] * n_ctx
    lens[-1] += L_C - sum(lens)
    b = wl.make_batch(H_q=2, H_kv=1, d=d, l_P=l_P, ctx_lens=[lens], l_q=l_q, seed=0)
    b.q.zero_()
    rq = b.requests[0]
    for (s, n), val in [(rq.prefix, vP), (rq.query_kv, vQ)] + [(c, vC) for c in rq.ctx]:
        b.v_pool[s:s + n] = val
    return b


def test_golden_closed_form_zero_query():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "closed_form_q0.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    for l_P, L_C, S, i, vP, vC, vQ, expect in rows:
        l_P, L_C, i = int(l_P), int(L_C), int(i)
        for n_ctx in (1, 4):
            b = _const_batch(l_P, L_C, i + 1, float(vP), float(vC), float(vQ), n_ctx=n_ctx)
            q, p, c, k = b.views(0)
            # T is irrelevant when all logits are zero
            for T in (1.0, 0.4):
                res = orc.attend(q, p, c, k, T, float(S))
                np.testing.assert_allclose(res.out[i].numpy(), float(expect), rtol=0, atol=2e-12)
                assert abs(res.lse[i, 0].item() - math.log(l_P + L_C ** float(S) + i + 1)) < 1e-12


def test_closed_form_general_zero_query():
    """Random V, zero Q: O[i] = (sum V_P + L_C^(S-1) sum V_C + sum_{j<=i+off} V_j) / (l_P + L_C^S + i+off+1)."""
    b = _tiny(seed=5, l_k=9)
    b.q.zero_()
    q, p, c, k = b.views(0)
    S = 0.65
    res = orc.attend(q, p, c, k, 0.5, S)
    G = b.H_q // b.H_kv
    VP, VQ = p[1].double().numpy(), k[1].double().numpy()
    VC = np.concatenate([v.double().numpy() for _, v in c])
    l_P, L_C, off = VP.shape[0], VC.shape[0], k[0].shape[0] - q.shape[0]
    for i in range(q.shape[0]):
        for h in range(b.H_q):
            g = h // G
            num = VP[:, g].sum(0) + L_C ** (S - 1) * VC[:, g].sum(0) + VQ[:i + off + 1, g].sum(0)
            np.testing.assert_allclose(res.out[i, h].numpy(), num / (l_P + L_C ** S + i + off + 1), atol=1e-13)


def test_constant_context_key_mass_and_sign_of_S():
    """All context keys equal: Z_C = L_C e^{x/T}.  S<1 raises the context mass when LSE_C<0 and lowers it when LSE_C>0."""
    d, L_C, T = 8, 6, 0.5
    for sign in (+1.0, -1.0):
        b = wl.make_batch(H_q=1, H_kv=1, d=d, l_P=2, ctx_lens=[[L_C]], l_q=1, seed=1)
        rq = b.requests[0]
        b.q[:] = 1.0
        b.k_pool[rq.ctx[0][0]:rq.ctx[0][0] + L_C] = sign * 1.0      # x = c * d * sign
        b.v_pool.zero_()
        b.v_pool[rq.ctx[0][0]:rq.ctx[0][0] + L_C] = 1.0             # output = context mass
        q, p, c, k = b.views(0)
        x = sign * d ** 0.5
        lse_c = math.log(L_C) + x / T
        Zo = float(np.exp(bf._lse(d ** -0.5 * (q.double().numpy()[0, 0] @ np.concatenate(
            [p[0].double().numpy()[:, 0], k[0].double().numpy()[:, 0]]).T))))
        masses = {}
        for S in (1.0, 0.7):
            res = orc.attend(q, p, c, k, T, S)
            assert abs(res.lse_ctx.item() - lse_c) < 1e-12
            expect = math.exp(S * lse_c) / (math.exp(S * lse_c) + Zo)
            np.testing.assert_allclose(res.out.numpy(), expect, atol=1e-13)
            masses[S] = expect
        assert (masses[0.7] < masses[1.0]) == (lse_c > 0)


def test_normalisation_and_context_mass():
    b = _tiny(seed=7)
    q, p, c, k = b.views(0)
    T, S = 0.8, 0.9
    b.v_pool[:] = 1.0
    res = orc.attend(*b.views(0), T, S)
    np.testing.assert_allclose(res.out.numpy(), 1.0, atol=1e-13)          # weights sum to one
    b.v_pool.zero_()
    for s, n in b.requests[0].ctx:
        b.v_pool[s:s + n] = 1.0
    res = orc.attend(*b.views(0), T, S)
    mass = torch.exp(S * res.lse_ctx - res.lse)                           # Z_C^S / (Z_P + Z_C^S + Z_Q)
    np.testing.assert_allclose(res.out[..., 0].numpy(), mass.numpy(), atol=1e-13)
    # the same mass from dense logits
    Q, KP, VP, KC, VC, KQ, VQ = bf._gather(q, p, c, k)
    G = b.H_q // b.H_kv
    for h in range(b.H_q):
        g = h // G
        zc = np.exp(Q[:, h] @ KC[:, g].T * (16 ** -0.5) / T).sum(-1)
        zp = np.exp(Q[:, h] @ KP[:, g].T * (16 ** -0.5)).sum(-1)
        xq = np.where(bf._causal_mask(Q.shape[0], KQ.shape[0]), Q[:, h] @ KQ[:, g].T * (16 ** -0.5), -np.inf)
        zq = np.exp(xq).sum(-1)
        np.testing.assert_allclose(mass[:, h].numpy(), zc ** S / (zp + zc ** S + zq), rtol=1e-12)


def test_invariant_to_context_order_and_to_splitting_a_context():
    b = _tiny(seed=8, lens=(6, 4, 8))
    q, p, c, k = b.views(0)
    T, S = 0.7, 0.8
    base = orc.attend(q, p, c, k, T, S).out.numpy()
    perm = [c[2], c[0], c[1]]
    np.testing.assert_allclose(orc.attend(q, p, perm, k, T, S).out.numpy(), base, atol=1e-13)
    # tokens inside the context segment may be permuted too
    idx = torch.randperm(6, generator=torch.Generator().manual_seed(0))
    shuffled = [(c[0][0][idx].contiguous(), c[0][1][idx].contiguous()), c[1], c[2]]
    np.testing.assert_allclose(orc.attend(q, p, shuffled, k, T, S).out.numpy(), base, atol=1e-13)
    # Eq. 5 treats all contexts as one segment: splitting one leaves the result unchanged ...
    split = [(c[0][0][:2], c[0][1][:2]), (c[0][0][2:], c[0][1][2:]), c[1], c[2]]
    np.testing.assert_allclose(orc.attend(q, p, split, k, T, S).out.numpy(), base, atol=1e-13)
    # ... whereas the per-context form (Eq. 11-12) does depend on the boundaries when S != 1
    pc = orc.attend(q, p, c, k, T, S, per_context=True).out.numpy()
    pc_split = orc.attend(q, p, split, k, T, S, per_context=True).out.numpy()
    assert np.abs(pc - pc_split).max() > 1e-4
    assert np.abs(pc - base).max() > 1e-4


def test_per_context_form():
    b = _tiny(seed=9, lens=(6, 4, 8))
    q, p, c, k = b.views(0)
    for T, S in [(0.7, 0.8), (1.0, 1.0), (0.5, 1.2)]:
        got = orc.attend(q, p, c, k, T, S, per_context=True).out.numpy()
        np.testing.assert_allclose(got, bf.per_context(q, p, c, k, T, S), atol=1e-12)
    # one context: both forms coincide; S = 1: both coincide for any N
    one = [c[0]]
    a = orc.attend(q, p, one, k, 0.7, 0.8, per_context=True).out.numpy()
    np.testing.assert_allclose(a, orc.attend(q, p, one, k, 0.7, 0.8).out.numpy(), atol=1e-13)
    a = orc.attend(q, p, c, k, 0.7, 1.0, per_context=True).out.numpy()
    np.testing.assert_allclose(a, orc.attend(q, p, c, k, 0.7, 1.0).out.numpy(), atol=1e-13)


def test_each_parameter_matters():
    """Guards against an oracle that ignores T, S, the causal offset or the head mapping."""
    b = _tiny(seed=11, l_k=9)
    q, p, c, k = b.views(0)
    base = orc.attend(q, p, c, k, 0.8, 0.9).out.numpy()
    assert np.abs(orc.attend(q, p, c, k, 0.9, 0.9).out.numpy() - base).max() > 1e-4
    assert np.abs(orc.attend(q, p, c, k, 0.8, 0.8).out.numpy() - base).max() > 1e-4
    k_short = (k[0][:6], k[1][:6])
    assert np.abs(orc.attend(q, p, c, k_short, 0.8, 0.9).out.numpy() - base).max() > 1e-4
    # heads of one group see the same K/V: swapping two KV heads changes the result
    sw = lambda t: t[:, [1, 0]].contiguous()
    swapped = orc.attend(q, (sw(p[0]), sw(p[1])), [(sw(a), sw(bb)) for a, bb in c], (sw(k[0]), sw(k[1])), 0.8, 0.9)
    assert np.abs(swapped.out.numpy() - base).max() > 1e-4
    # ... and equals the original with the two head groups exchanged, if the queries are exchanged as well
    q_sw = q[:, [2, 3, 0, 1]].contiguous()
    both = orc.attend(q_sw, (sw(p[0]), sw(p[1])), [(sw(a), sw(bb)) for a, bb in c], (sw(k[0]), sw(k[1])), 0.8, 0.9)
    np.testing.assert_allclose(both.out.numpy()[:, [2, 3, 0, 1]], base, atol=1e-13)


def test_row_and_head_subsets():
    b = _tiny(seed=12)
    q, p, c, k = b.views(0)
    full = orc.attend(q, p, c, k, 0.8, 0.9)
    part = orc.attend(q, p, c, k, 0.8, 0.9, rows=(2, 4), heads=(1, 3))
    np.testing.assert_array_equal(part.out[2:4, 1:3].numpy(), full.out[2:4, 1:3].numpy())
    assert torch.isnan(part.out[0]).all() and torch.isnan(part.out[2, 0]).all()


def test_rejects_bad_arguments():
    b = _tiny(seed=13)
    q, p, c, k = b.views(0)
    for T, S in [(0.0, 1.0), (-1.0, 1.0), (1.0, 0.0), (float("nan"), 1.0)]:
        with pytest.raises(RuntimeError):
            orc.attend(q, p, c, k, T, S)
    with pytest.raises(RuntimeError):
        orc.attend(q, p, c, (k[0][:3], k[1][:3]), 1.0, 1.0)     # fewer keys than rows


# ---- encode ------------------------------------------------------------------------------------------------------

def _enc_views(b):
    rq = b.requests[0]
    qs = [b.q_enc[s:s + n] for s, n in rq.ctx]
    _, p, c, _ = b.views(0)
    return qs, p, c


@pytest.mark.parametrize("kw", [dict(), dict(l_P=0, lens=(5,)), dict(H_q=6, H_kv=3, d=8, lens=(1, 9, 2))])
def test_encode_equals_block_diagonal_mask(kw):
    b = _tiny(seed=14, with_encode_q=True, **kw)
    qs, p, c = _enc_views(b)
    outs, lses = orc.encode(qs, p, c)
    ref = bf.encode_blockdiag(qs, p, c)
    for o, r in zip(outs, ref):
        np.testing.assert_allclose(o.numpy(), r, atol=1e-12)


def test_encode_single_context_is_sequential_causal_attention():
    """One context, no position reuse: encode rows + attend rows (T=S=1) are the rows of one causal pass over [P;C;Q]."""
    b = _tiny(seed=15, lens=(7,), with_encode_q=True, H_q=4, H_kv=2)
    qs, p, c = _enc_views(b)
    q, _, _, k = b.views(0)
    G = b.H_q // b.H_kv
    l_P, l_C, l_q = p[0].shape[0], c[0][0].shape[0], q.shape[0]
    # a full sequence needs queries for the prefix rows too; they are not compared
    Qall = torch.cat([torch.zeros(l_P, b.H_q, b.d, dtype=torch.bfloat16), qs[0], q]).double().transpose(0, 1)
    Kall = torch.cat([p[0], c[0][0], k[0]]).double().repeat_interleave(G, 1).transpose(0, 1)
    Vall = torch.cat([p[1], c[0][1], k[1]]).double().repeat_interleave(G, 1).transpose(0, 1)
    seq = torch.nn.functional.scaled_dot_product_attention(Qall, Kall, Vall, is_causal=True).transpose(0, 1).numpy()
    outs, _ = orc.encode(qs, p, c)
    np.testing.assert_allclose(outs[0].numpy(), seq[l_P:l_P + l_C], atol=1e-12)
    att = orc.attend(q, p, c, k, 1.0, 1.0).out.numpy()
    np.testing.assert_allclose(att, seq[l_P + l_C:], atol=1e-12)


def test_encode_contexts_do_not_see_each_other():
    b = _tiny(seed=16, with_encode_q=True)
    qs, p, c = _enc_views(b)
    base, _ = orc.encode(qs, p, c)
    s, n = b.requests[0].ctx[1]
    b.k_pool[s:s + n] = 3.0
    b.v_pool[s:s + n] = -5.0
    qs, p, c = _enc_views(b)
    new, _ = orc.encode(qs, p, c)
    np.testing.assert_array_equal(new[0].numpy(), base[0].numpy())
    np.testing.assert_array_equal(new[2].numpy(), base[2].numpy())
    assert np.abs(new[1].numpy() - base[1].numpy()).max() > 1e-3


def test_oracle_on_tiny_benchmark_case():
    """The tiny benchmark case (16 + 4x64 + 16 tokens) against the dense form, and its LSE identity."""
    b = wl.config1()
    q, p, c, k = b.views(0)
    res = orc.attend(q, p, c, k, b.T, b.S)
    ref, lam = bf.flat_bias(q, p, c, k, b.T, b.S)
    np.testing.assert_allclose(res.out.numpy(), ref, atol=1e-12)
    np.testing.assert_allclose(res.lse.numpy(), lam, atol=1e-11)
