"""Pins for the Eq. 8 oracle: closed forms, invariances and library routines, none of which
re-uses the oracle's own formulation."""

from __future__ import annotations

import numpy as np


def pin_two_feature_closed_form(agg):
    """D_v = 2: LN maps (a, b) to +-(1, -1)/sqrt(1 + eps') and Norm to +-(1, -1)/sqrt(2), so every
    cosine is +1 or -1 and the weights are e^{+-1/tau} / sum, by hand."""
    x0 = np.array([[3.0, 1.0], [0.0, 5.0], [2.0, -2.0], [-1.0, 4.0]])  # signs of (a-b): + - + -
    a = np.array([[10.0, 2.0], [1.0, 7.0]])                            # + and -
    tau = 0.5
    z, w = agg.anchor_aggregate(x0, a, tau)
    ep, em = np.exp(1 / tau), np.exp(-1 / tau)
    row_plus = np.array([ep, em, ep, em]) / (2 * ep + 2 * em)
    row_minus = np.array([em, ep, em, ep]) / (2 * ep + 2 * em)
    assert np.allclose(w, np.stack([row_plus, row_minus]), rtol=1e-12, atol=0)
    assert np.allclose(z, np.stack([row_plus @ x0, row_minus @ x0]), rtol=1e-12)
    # hand value: anchor 0 puts e^2 / (2e^2 + 2e^-2) = 1 / (2 (1 + e^-4)) on token 0, e^-4 = 0.0183156388887...
    assert abs(w[0, 0] - 0.5 / 1.01831563888873418) < 1e-12


def pin_library_routines(agg):
    """zscore (scipy), normalize (scikit-learn) and softmax (scipy) compose to the same weights."""
    from scipy.special import softmax
    from scipy.stats import zscore
    from sklearn.preprocessing import normalize

    rng = np.random.default_rng(61)
    x0 = rng.standard_normal((37, 24)) * 3 + 1.5
    a = rng.standard_normal((5, 24))
    tau = 0.2
    k0 = normalize(zscore(x0, axis=1, ddof=0))
    q = normalize(zscore(a, axis=1, ddof=0))
    want_w = softmax(q @ k0.T / tau, axis=1)
    z, w = agg.anchor_aggregate(x0, a, tau)
    assert np.allclose(w, want_w, rtol=1e-9, atol=1e-15)
    assert np.allclose(z, want_w @ x0, rtol=1e-9, atol=1e-12)


def pin_convexity_and_limits(agg):
    rng = np.random.default_rng(67)
    x0 = rng.standard_normal((50, 16)) + 0.3
    a = rng.standard_normal((7, 16))
    z, w = agg.anchor_aggregate(x0, a, 0.1)
    assert w.shape == (7, 50) and np.all(w >= 0)
    assert np.allclose(w.sum(axis=1), 1.0, rtol=0, atol=1e-12), "softmax runs over the dense tokens"
    assert np.all(z <= x0.max(axis=0) + 1e-12) and np.all(z >= x0.min(axis=0) - 1e-12)
    # tau -> infinity: uniform weights, every anchor returns the mean token
    z_inf, w_inf = agg.anchor_aggregate(x0, a, 1e12)
    assert np.allclose(w_inf, 1 / 50, rtol=1e-9) and np.allclose(z_inf, np.tile(x0.mean(axis=0), (7, 1)), atol=1e-9)
    # tau -> 0: one-hot at the token with the largest cosine to the anchor
    cent = lambda v: (v - v.mean(axis=1, keepdims=True))
    unit = lambda v: v / np.linalg.norm(v, axis=1, keepdims=True)
    cos = unit(cent(a)) @ unit(cent(x0)).T
    z_0, w_0 = agg.anchor_aggregate(x0, a, 1e-4)
    assert np.array_equal(w_0.argmax(axis=1), cos.argmax(axis=1))
    assert np.allclose(z_0, x0[cos.argmax(axis=1)], atol=1e-6)
    # identical dense tokens: every anchor returns that token, whatever tau
    same = np.tile(rng.standard_normal(16), (9, 1))
    z_same, _ = agg.anchor_aggregate(same, a, 0.05)
    assert np.allclose(z_same, same[:7], atol=1e-12)


def pin_invariances(agg):
    """LN + Norm remove a per-token positive scale and shift, so W_A does not see them; Z_0 is
    linear in the tokens it averages; permuting the tokens permutes the columns of W_A."""
    rng = np.random.default_rng(71)
    x0 = rng.standard_normal((20, 12))
    a = rng.standard_normal((4, 12))
    scale = rng.uniform(0.5, 4.0, (20, 1))
    shift = rng.standard_normal((20, 1))
    _, w = agg.anchor_aggregate(x0, a, 0.3)
    z2, w2 = agg.anchor_aggregate(scale * x0 + shift, a, 0.3)
    assert np.allclose(w, w2, rtol=1e-6, atol=1e-12)
    assert np.allclose(z2, w @ (scale * x0 + shift), rtol=1e-6, atol=1e-9)
    _, w3 = agg.anchor_aggregate(x0, 7.0 * a - 2.0, 0.3)  # the anchors are normalised as well
    assert np.allclose(w, w3, rtol=1e-6, atol=1e-12)
    perm = rng.permutation(20)
    z4, w4 = agg.anchor_aggregate(x0[perm], a, 0.3)
    assert np.allclose(w4, w[:, perm], rtol=1e-12) and np.allclose(z4, w @ x0, rtol=1e-10, atol=1e-12)
    # a constant token has no direction: logit 0 for every anchor
    x1 = x0.copy()
    x1[3] = 2.5
    _, w5 = agg.anchor_aggregate(x1, a, 0.3)
    others = np.delete(np.arange(20), 3)
    ratio = w5[:, 3] / w5[:, others].sum(axis=1)
    k = agg.l2_normalize(agg.layer_norm(x1[others]))
    q = agg.l2_normalize(agg.layer_norm(a))
    assert np.allclose(ratio, 1.0 / np.exp(q @ k.T / 0.3).sum(axis=1), rtol=1e-9)


def pin_layer_norm_and_norm(agg):
    """The two normalisations on rows worked by hand: (1,-1,1,-1) has mean 0 and biased variance 1,
    so LN divides by sqrt(1 + 1e-5); (3,4) has l2 norm 5; the zero row stays zero."""
    ln = agg.layer_norm(np.array([[1.0, -1.0, 1.0, -1.0], [2.0, 4.0, 6.0, 8.0]]))
    assert np.allclose(ln[0], np.array([1, -1, 1, -1]) / np.sqrt(1 + 1e-5), rtol=1e-14)
    assert np.allclose(ln[1], np.array([-3, -1, 1, 3]) / np.sqrt(5 + 1e-5), rtol=1e-14)  # mean 5, variance 5
    nm = agg.l2_normalize(np.array([[3.0, 4.0], [0.0, 0.0], [0.0, -2.0]]))
    assert np.allclose(nm, [[0.6, 0.8], [0.0, 0.0], [0.0, -1.0]], rtol=1e-15)


def pin_batch_and_mass(agg):
    rng = np.random.default_rng(73)
    x0 = rng.standard_normal((3, 11, 8))
    a = rng.standard_normal((4, 8))
    z, mass = agg.anchor_aggregate_batch(x0, a, 0.25)
    for i in range(3):
        z_i, w_i = agg.anchor_aggregate(x0[i], a, 0.25)
        assert np.array_equal(z[i], z_i) and np.allclose(mass[i], w_i.sum(axis=0))
    assert np.allclose(mass.sum(axis=1), 4.0)  # every anchor hands out exactly one unit


ALL_AGGREGATE_PINS = [pin_two_feature_closed_form, pin_library_routines, pin_convexity_and_limits,
                      pin_invariances, pin_layer_norm_and_norm, pin_batch_and_mass]


# ---------------------------------------------------------------- KV-compressed attention (Eq. 9)

def _dense_attention(q, k, v, n_heads):
    """Ordinary multi-head attention from library routines (scipy softmax)."""
    from scipy.special import softmax

    d = q.shape[1] // n_heads
    out = np.empty_like(q)
    for h in range(n_heads):
        c = slice(h * d, (h + 1) * d)
        out[:, c] = softmax(q[:, c] @ k[:, c].T / np.sqrt(d), axis=1) @ v[:, c]
    return out


def pin_identity_assignment_is_dense_attention(agg):
    """S = M_e and R = identity (or any permutation of it, or a positive diagonal): nothing is
    compressed, Eq. 9 is ordinary attention over the compact tokens themselves."""
    rng = np.random.default_rng(81)
    m_e, dim, heads = 12, 8, 2
    q, k, v = (rng.standard_normal((m_e, dim)) for _ in range(3))
    want = _dense_attention(q, k, v, heads)
    out, k_c, v_c = agg.kv_compressed_attention(q, k, v, np.eye(m_e), heads)
    assert np.allclose(out, want, rtol=1e-12, atol=1e-14) and np.allclose(k_c, k) and np.allclose(v_c, v)
    perm = rng.permutation(m_e)
    out_p, k_p, _ = agg.kv_compressed_attention(q, k, v, np.eye(m_e)[:, perm], heads)
    assert np.allclose(out_p, want, rtol=1e-12, atol=1e-14) and np.allclose(k_p, k[perm])
    out_d, _, _ = agg.kv_compressed_attention(q, k, v, np.diag(rng.uniform(0.5, 3.0, m_e)), heads)
    assert np.allclose(out_d, want, rtol=1e-12, atol=1e-14), "column normalisation removes a column's scale"


def pin_compression_closed_forms(agg):
    rng = np.random.default_rng(83)
    m_e, dim, heads, s = 10, 6, 3, 4
    q, k, v = (rng.standard_normal((m_e, dim)) for _ in range(3))
    # one memory anchor that every token feeds equally: K_c, V_c are the means, every query returns mean(V)
    out, k_c, v_c = agg.kv_compressed_attention(q, k, v, np.ones((m_e, 1)), heads)
    assert np.allclose(k_c[0], k.mean(axis=0)) and np.allclose(v_c[0], v.mean(axis=0))
    assert np.allclose(out, np.tile(v.mean(axis=0), (m_e, 1)))
    # hard assignment: anchor j averages exactly the tokens assigned to it
    assign = rng.integers(0, s, m_e)
    assign[:s] = np.arange(s)  # no empty anchor
    r = np.zeros((m_e, s))
    r[np.arange(m_e), assign] = 1.0
    out, k_c, v_c = agg.kv_compressed_attention(q, k, v, r, heads)
    for j in range(s):
        assert np.allclose(k_c[j], k[assign == j].mean(axis=0)) and np.allclose(v_c[j], v[assign == j].mean(axis=0))
    assert np.allclose(out, _dense_attention(q, k_c, v_c, heads), rtol=1e-12, atol=1e-14)
    # the columns of the normalised assignment sum to one; outputs are convex combinations of V_c rows
    rbar = agg.column_normalize(rng.uniform(0.1, 1.0, (m_e, s)))
    assert np.allclose(rbar.sum(axis=0), 1.0)
    assert np.all(out <= v_c.max(axis=0) + 1e-12) and np.all(out >= v_c.min(axis=0) - 1e-12)
    # hand-worked: two tokens, one head of size 1, two anchors with R = [[1, 1], [0, 1]]
    q1, k1, v1 = np.array([[1.0], [0.0]]), np.array([[2.0], [4.0]]), np.array([[10.0], [20.0]])
    out1, kc1, vc1 = agg.kv_compressed_attention(q1, k1, v1, np.array([[1.0, 1.0], [0.0, 1.0]]), 1)
    assert np.allclose(kc1[:, 0], [2.0, 3.0]) and np.allclose(vc1[:, 0], [10.0, 15.0])
    w = np.exp([2.0, 3.0]) / np.exp([2.0, 3.0]).sum()  # query 1 . K_c / sqrt(1)
    assert np.allclose(out1[:, 0], [w @ [10.0, 15.0], 12.5])  # the zero query weighs both anchors equally


def pin_layer_composition(agg):
    """Eq. 9 from the hidden states is the attention of the three projections; heads do not mix."""
    rng = np.random.default_rng(87)
    m_e, dim, heads, s = 9, 8, 4, 3
    h = rng.standard_normal((m_e, dim))
    w_q, w_k, w_v = (rng.standard_normal((dim, dim)) for _ in range(3))
    r = rng.uniform(0.1, 1.0, (m_e, s))
    full = agg.compact_visual_layer(h, w_q, w_k, w_v, r, heads)
    want, _, _ = agg.kv_compressed_attention(h @ w_q, h @ w_k, h @ w_v, r, heads)
    assert np.allclose(full, want)
    d = dim // heads
    q, k, v = h @ w_q, h @ w_k, h @ w_v
    k2 = k.copy()
    k2[:, d:2 * d] *= -2.0  # changing head 1's keys leaves the other heads' outputs untouched
    out2, _, _ = agg.kv_compressed_attention(q, k2, v, r, heads)
    assert np.allclose(out2[:, :d], want[:, :d]) and np.allclose(out2[:, 2 * d:], want[:, 2 * d:])
    assert not np.allclose(out2[:, d:2 * d], want[:, d:2 * d])


ALL_ATTENTION_PINS = [pin_identity_assignment_is_dense_attention, pin_compression_closed_forms, pin_layer_composition]
