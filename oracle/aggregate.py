"""CPU oracle of CIVIC's compact visual aggregation (Eq. 8)  --  TEST INFRASTRUCTURE.

Plain numpy in fp64, the paper's steps in the paper's order and notation.  Used only by the
tests, the smoke check and the benchmark's CPU-baseline leg; the CUDA library neither imports it
nor shares anything with it.

    K_0 = Norm(LN(X_0)),  Q_A = Norm(LN(A))
    W_A = softmax(Q_A K_0^T / tau)      softmax over the dense-token dimension
    Z_0 = W_A X_0

X_0 [T_e, D_v] are the dense patch embeddings, A [M_e, D_v] the compact anchors, LN is layer
normalisation over the feature dimension, Norm is l2 normalisation of every row.

What the paper leaves open, and the reading taken here: LN has no learned scale or shift (the
paper names none) and uses eps = 1e-5 inside the square root; Norm divides by max(||v||, 1e-12)
(both are the defaults of the framework the paper says it used).  A row of X_0 whose features
are all equal therefore maps to the zero vector, logit 0.
"""

from __future__ import annotations

import numpy as np

LN_EPS = 1e-5
NORM_EPS = 1e-12


def layer_norm(v: np.ndarray) -> np.ndarray:
    """LN over the last axis: (v - mean) / sqrt(var + eps), biased variance."""
    v = np.asarray(v, dtype=np.float64)
    mean = v.mean(axis=-1, keepdims=True)
    var = ((v - mean) ** 2).mean(axis=-1, keepdims=True)
    return (v - mean) / np.sqrt(var + LN_EPS)


def l2_normalize(v: np.ndarray) -> np.ndarray:
    """Norm over the last axis: v / max(||v||_2, eps)."""
    v = np.asarray(v, dtype=np.float64)
    norm = np.sqrt((v * v).sum(axis=-1, keepdims=True))
    return v / np.maximum(norm, NORM_EPS)


def aggregation_weights(x0: np.ndarray, anchors: np.ndarray, tau: float) -> np.ndarray:
    """W_A [M_e, T_e] of Eq. 8."""
    k0 = l2_normalize(layer_norm(x0))
    q_a = l2_normalize(layer_norm(anchors))
    logits = q_a @ k0.T / float(tau)
    logits = logits - logits.max(axis=1, keepdims=True)  # softmax over the dense tokens (axis 1)
    e = np.exp(logits)
    return e / e.sum(axis=1, keepdims=True)


def anchor_aggregate(x0: np.ndarray, anchors: np.ndarray, tau: float):
    """Eq. 8 for one image: returns (Z_0 [M_e, D_v], W_A [M_e, T_e]) in fp64."""
    x0 = np.asarray(x0, dtype=np.float64)
    w_a = aggregation_weights(x0, anchors, tau)
    return w_a @ x0, w_a


def anchor_aggregate_batch(x0: np.ndarray, anchors: np.ndarray, tau: float):
    """x0 [n_img, T_e, D_v] with shared anchors: (Z_0 [n_img, M_e, D_v], token mass [n_img, T_e]).

    The token mass is the column sum of W_A: how much of all anchors' attention a dense token
    receives (a natural per-token importance score)."""
    z, mass = [], []
    for img in np.asarray(x0):
        z_i, w_i = anchor_aggregate(img, anchors, tau)
        z.append(z_i)
        mass.append(w_i.sum(axis=0))
    return np.stack(z), np.stack(mass)


# ---------------------------------------------------------------------------------------------
# Compact visual encoding layer: KV-compressed attention (Eq. 9)
#
#     Q = H W_Q,  K = H W_K,  V = H W_V
#     K_c = Rbar^T K,  V_c = Rbar^T V           Rbar = R with every column normalised
#     Attn_c = softmax(Q K_c^T / sqrt(d)) V_c   per head, d the per-head dimension
#
# H [M_e, D_v] are the compact hidden states, R [M_e, S] the KV assignment matrix onto S memory
# anchors.  Readings where the paper is silent: R is non-negative and "column-normalised" means
# every column is divided by its sum, so a row of K_c is a weighted average of the rows of K;
# heads split the feature dimension into n_heads contiguous blocks of d = D_v / n_heads, K_c and
# V_c are compressed over the whole feature dimension at once (R does not depend on the head);
# the softmax runs over the S memory anchors; no output projection (Eq. 9 has none).

def column_normalize(r: np.ndarray) -> np.ndarray:
    r = np.asarray(r, dtype=np.float64)
    return r / r.sum(axis=0, keepdims=True)


def kv_compressed_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, r: np.ndarray, n_heads: int):
    """q, k, v [M_e, D] (already projected), r [M_e, S] -> (Attn_c [M_e, D], K_c [S, D], V_c [S, D])."""
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    m_e, dim = q.shape
    d = dim // n_heads
    rbar = column_normalize(r)
    k_c = rbar.T @ k
    v_c = rbar.T @ v
    out = np.empty_like(q)
    for h in range(n_heads):
        cols = slice(h * d, (h + 1) * d)
        logits = q[:, cols] @ k_c[:, cols].T / np.sqrt(d)
        logits = logits - logits.max(axis=1, keepdims=True)  # softmax over the S memory anchors
        e = np.exp(logits)
        out[:, cols] = (e / e.sum(axis=1, keepdims=True)) @ v_c[:, cols]
    return out, k_c, v_c


def compact_visual_layer(h: np.ndarray, w_q: np.ndarray, w_k: np.ndarray, w_v: np.ndarray, r: np.ndarray,
                         n_heads: int) -> np.ndarray:
    """Eq. 9 from the hidden states: projections, then the KV-compressed attention."""
    h = np.asarray(h, dtype=np.float64)
    return kv_compressed_attention(h @ w_q, h @ w_k, h @ w_v, r, n_heads)[0]
