"""Reference for the draft model's target-feature aggregation (TEST INFRASTRUCTURE ONLY).

Sec. 3.1.1 of the paper: a few learnable meta queries f_q [Q, D], shared by all tokens, attend over
the L target-layer features of each token i, f_i [L, D], and the attention outputs are flattened:
f_c^i = Flatten(CrossAttention(f_q, f_i, f_i)) in R^(Q*D).  The paper does not give the module's
head count or projections; the reading taken here is the attention core of a multi-head module:

    for token i, head h (D = H * d):   s[q, l] = scale * <qp[q, h], k_i[l, h]>
                                       p = softmax_l(s);   out[i, q, h] = sum_l p[q, l] * v_i[l, h]

with qp the (already projected, token-independent) meta queries and k_i, v_i the token's projected
layer features (the un-projected reading passes f_i for both).  Projections are plain GEMMs outside.
Plain numpy fp64 on the exact bf16 values; nothing shared with the GPU library.
"""
from __future__ import annotations

import numpy as np


def feature_attention(qp: np.ndarray, k: np.ndarray, v: np.ndarray, H: int, scale: float) -> np.ndarray:
    """qp [Q, D], k and v [S, L, D] (float64) -> out [S, Q, D]."""
    Q, D = qp.shape
    S, L, _ = k.shape
    d = D // H
    out = np.zeros((S, Q, D))
    for i in range(S):
        for h in range(H):
            sl = slice(h * d, (h + 1) * d)
            s = scale * (qp[:, sl] @ k[i, :, sl].T)              # [Q, L]
            s = s - s.max(axis=1, keepdims=True)
            p = np.exp(s)
            p = p / p.sum(axis=1, keepdims=True)
            out[i, :, sl] = p @ v[i, :, sl]
    return out
