"""Brute-force statements of APE attention in numpy fp64, independent of oracle/.

Three forms, each built from a textbook routine (a row softmax over one dense logit matrix, or two
ordinary attentions merged), used to pin the C oracle:

  flat_bias      one softmax over the concatenated sequence [P | C_1..C_N | Q]; context columns carry
                 x/T + (S-1)*LSE_C(row), which is Eq. 5's (sum a')^(S-1) factor in the log domain.
  two_pass       the "Efficient Implementation" form: ordinary attention over the context keys with
                 temperature, ordinary attention over the rest, LSE of the context times S, softmax over
                 the two LSEs, weighted sum.
  per_context    the appendix's hierarchical form (Eq. 11-12): S on every context's own LSE.
"""
import numpy as np


def _f64(t):
    return t.to(dtype=__import__("torch").float64).numpy()


def _lse(x, axis=-1):
    m = np.max(x, axis=axis, keepdims=True)
    m = np.where(np.isfinite(m), m, 0.0)
    with np.errstate(divide="ignore"):
        return (m + np.log(np.sum(np.exp(x - m), axis=axis, keepdims=True))).squeeze(axis)


def _softmax(x):
    m = np.max(x, axis=-1, keepdims=True)
    e = np.exp(x - m)
    return e / e.sum(axis=-1, keepdims=True)


def _gather(q, prefix, ctx, qkv):
    """fp64 arrays: q [l_q,H_q,d]; K,V per segment [len,H_kv,d]; context segments concatenated."""
    Q = _f64(q)
    KP, VP = _f64(prefix[0]), _f64(prefix[1])
    KQ, VQ = _f64(qkv[0]), _f64(qkv[1])
    H_kv, d = KQ.shape[1], KQ.shape[2]
    if len(ctx):
        KC = np.concatenate([_f64(k) for k, _ in ctx], axis=0)
        VC = np.concatenate([_f64(v) for _, v in ctx], axis=0)
    else:
        KC = np.zeros((0, H_kv, d))
        VC = np.zeros((0, H_kv, d))
    return Q, KP, VP, KC, VC, KQ, VQ


def _causal_mask(l_q, l_k):
    i = np.arange(l_q)[:, None]
    j = np.arange(l_k)[None, :]
    return j <= i + (l_k - l_q)


def flat_bias(q, prefix, ctx, qkv, T, S, scale=None):
    Q, KP, VP, KC, VC, KQ, VQ = _gather(q, prefix, ctx, qkv)
    l_q, H_q, d = Q.shape
    H_kv = KQ.shape[1]
    G = H_q // H_kv
    c = d ** -0.5 if scale is None else scale
    l_P, L_C, l_k = KP.shape[0], KC.shape[0], KQ.shape[0]
    out = np.zeros((l_q, H_q, d))
    lam = np.zeros((l_q, H_q))
    mask = _causal_mask(l_q, l_k)
    for h in range(H_q):
        g = h // G
        K = np.concatenate([KP[:, g], KC[:, g], KQ[:, g]], axis=0)
        V = np.concatenate([VP[:, g], VC[:, g], VQ[:, g]], axis=0)
        X = c * (Q[:, h] @ K.T)                      # [l_q, l_P+L_C+l_k]
        if L_C:
            XC = X[:, l_P:l_P + L_C] / T
            X[:, l_P:l_P + L_C] = XC + (S - 1.0) * _lse(XC)[:, None]
        X[:, l_P + L_C:] = np.where(mask, X[:, l_P + L_C:], -np.inf)
        out[:, h] = _softmax(X) @ V
        lam[:, h] = _lse(X)
    return out, lam


def _plain_attention(Qh, K, V, c, mask=None):
    """Textbook softmax attention of one head; returns (out, lse).  Empty key set -> (0, -inf)."""
    if K.shape[0] == 0:
        return np.zeros((Qh.shape[0], V.shape[1])), np.full((Qh.shape[0],), -np.inf)
    X = c * (Qh @ K.T)
    if mask is not None:
        X = np.where(mask, X, -np.inf)
    return _softmax(X) @ V, _lse(X)


def two_pass(q, prefix, ctx, qkv, T, S, scale=None):
    Q, KP, VP, KC, VC, KQ, VQ = _gather(q, prefix, ctx, qkv)
    l_q, H_q, d = Q.shape
    G = H_q // KQ.shape[1]
    c = d ** -0.5 if scale is None else scale
    l_P, l_k = KP.shape[0], KQ.shape[0]
    out = np.zeros((l_q, H_q, d))
    mask_o = np.concatenate([np.ones((l_q, l_P), dtype=bool), _causal_mask(l_q, l_k)], axis=1)
    for h in range(H_q):
        g = h // G
        o_c, lse_c = _plain_attention(Q[:, h], KC[:, g], VC[:, g], c / T)
        o_o, lse_o = _plain_attention(Q[:, h], np.concatenate([KP[:, g], KQ[:, g]]),
                                      np.concatenate([VP[:, g], VQ[:, g]]), c, mask_o)
        w = _softmax(np.stack([S * lse_c, lse_o], axis=-1))
        out[:, h] = w[:, :1] * o_c + w[:, 1:] * o_o
    return out


def per_context(q, prefix, ctx, qkv, T, S, scale=None):
    Q, KP, VP, _, _, KQ, VQ = _gather(q, prefix, ctx, qkv)
    l_q, H_q, d = Q.shape
    G = H_q // KQ.shape[1]
    c = d ** -0.5 if scale is None else scale
    l_k = KQ.shape[0]
    out = np.zeros((l_q, H_q, d))
    for h in range(H_q):
        g = h // G
        parts = []
        if KP.shape[0]:
            parts.append(_plain_attention(Q[:, h], KP[:, g], VP[:, g], c))
        for k, v in ctx:
            if k.shape[0]:
                o, l = _plain_attention(Q[:, h], _f64(k)[:, g], _f64(v)[:, g], c / T)
                parts.append((o, S * l))
        parts.append(_plain_attention(Q[:, h], KQ[:, g], VQ[:, g], c, _causal_mask(l_q, l_k)))
        w = _softmax(np.stack([l for _, l in parts], axis=-1))
        out[:, h] = sum(w[:, n:n + 1] * parts[n][0] for n in range(len(parts)))
    return out


def tree_bias(q, prefix, ctx, qkv, T, S, parent, scaled=None, scale=None):
    """Context trees as ONE dense softmax over the concatenation [P | node_0 .. node_N-1 | Q]: with Z_n the mass of node n
    (its own tempered weights plus Z_c^{s_c} of every child c) and s_n = S on scaled nodes, 1 elsewhere, a token of node n
    carries its tempered logit plus (s_m - 1) * log Z_m for every node m on the path from n up to its root: each level's
    softmax weight Z_m^{s_m} / Z_parent written as a bias.  Returns (out, log of the denominator)."""
    Q, KP, VP, KC, VC, KQ, VQ = _gather(q, prefix, ctx, qkv)
    n = len(ctx)
    if scaled is None:
        scaled = [1 if p < 0 else 0 for p in parent]
    s = [S if scaled[i] else 1.0 for i in range(n)]
    lens = [k.shape[0] for k, _ in ctx]
    offs = np.concatenate([[0], np.cumsum(lens)]).astype(int)
    l_q, H_q, d = Q.shape
    G = H_q // KQ.shape[1]
    c = d ** -0.5 if scale is None else scale
    l_P, L_C, l_k = KP.shape[0], KC.shape[0], KQ.shape[0]
    children = [[j for j in range(n) if parent[j] == i] for i in range(n)]
    out = np.zeros((l_q, H_q, d))
    lam = np.zeros((l_q, H_q))
    mask = _causal_mask(l_q, l_k)
    for h in range(H_q):
        g = h // G
        K = np.concatenate([KP[:, g], KC[:, g], KQ[:, g]], axis=0)
        V = np.concatenate([VP[:, g], VC[:, g], VQ[:, g]], axis=0)
        X = c * (Q[:, h] @ K.T)
        XC = X[:, l_P:l_P + L_C] / T
        logZ = [None] * n

        def mass(i):                       # log Z_i per row, by its definition (recursion over the children)
            if logZ[i] is None:
                terms = [XC[:, offs[i]:offs[i + 1]]] + [(s[j] * mass(j))[:, None] for j in children[i]]
                logZ[i] = _lse(np.concatenate(terms, axis=1)) if sum(t.shape[1] for t in terms) else np.full(l_q, -np.inf)
            return logZ[i]
        bias = np.zeros((l_q, L_C))
        for i in range(n):
            m = i
            while m >= 0:
                z = mass(m)
                if lens[i]:
                    bias[:, offs[i]:offs[i + 1]] += ((s[m] - 1.0) * z)[:, None]
                m = parent[m]
        X[:, l_P:l_P + L_C] = XC + bias
        X[:, l_P + L_C:] = np.where(mask, X[:, l_P + L_C:], -np.inf)
        out[:, h] = _softmax(X) @ V
        lam[:, h] = _lse(X)
    return out, lam


def encode_blockdiag(ctx_q, prefix, ctx, scale=None):
    """One dense masked softmax over [P | C_1 | ... | C_N] for all context rows at once."""
    KP, VP = _f64(prefix[0]), _f64(prefix[1])
    Qs = [_f64(t) for t in ctx_q]
    lens = [t.shape[0] for t in Qs]
    Q = np.concatenate(Qs, axis=0)
    KC = np.concatenate([_f64(k) for k, _ in ctx], axis=0)
    VC = np.concatenate([_f64(v) for _, v in ctx], axis=0)
    H_q, d = Q.shape[1], Q.shape[2]
    G = H_q // KC.shape[1]
    c = d ** -0.5 if scale is None else scale
    l_P, L = KP.shape[0], sum(lens)
    owner = np.concatenate([np.full(n, i) for i, n in enumerate(lens)])
    pos = np.concatenate([np.arange(n) for n in lens])
    mask_c = (owner[:, None] == owner[None, :]) & (pos[None, :] <= pos[:, None])
    mask = np.concatenate([np.ones((L, l_P), dtype=bool), mask_c], axis=1)
    out = np.zeros((L, H_q, d))
    for h in range(H_q):
        g = h // G
        X = c * (Q[:, h] @ np.concatenate([KP[:, g], KC[:, g]]).T)
        X = np.where(mask, X, -np.inf)
        out[:, h] = _softmax(X) @ np.concatenate([VP[:, g], VC[:, g]])
    res, o = [], 0
    for n in lens:
        res.append(out[o:o + n])
        o += n
    return res
