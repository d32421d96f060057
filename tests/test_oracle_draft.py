"""Pins of the feature-aggregation reference (oracle/draft_attention.py)."""
import numpy as np
import torch

from oracle.draft_attention import feature_attention


def rnd(g, *shape):
    return g.standard_normal(shape)


def test_against_torch_sdpa():
    """Each token is an ordinary non-causal attention problem with Q queries and L keys per head."""
    g = np.random.default_rng(0)
    S, L, Q, H, d = 5, 7, 3, 4, 8
    qp, k, v = rnd(g, Q, H * d), rnd(g, S, L, H * d), rnd(g, S, L, H * d)
    got = feature_attention(qp, k, v, H, 0.3)
    tq = torch.from_numpy(qp).view(1, Q, H, d).permute(0, 2, 1, 3).expand(S, H, Q, d)
    tk = torch.from_numpy(k).view(S, L, H, d).permute(0, 2, 1, 3)
    tv = torch.from_numpy(v).view(S, L, H, d).permute(0, 2, 1, 3)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=0.3)
    ref = ref.permute(0, 2, 1, 3).reshape(S, Q, H * d).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_closed_forms():
    g = np.random.default_rng(1)
    S, L, Q, H, d = 3, 6, 2, 2, 4
    qp, k, v = rnd(g, Q, H * d), rnd(g, S, L, H * d), rnd(g, S, L, H * d)
    # one layer only: the output is that layer's value row, whatever the queries are
    out = feature_attention(qp, k[:, :1], v[:, :1], H, 1.0)
    np.testing.assert_allclose(out, np.repeat(v[:, :1], Q, axis=1), atol=1e-14)
    # equal keys: plain mean over the layers
    out = feature_attention(qp, np.repeat(k[:, :1], L, axis=1), v, H, 1.0)
    np.testing.assert_allclose(out, np.repeat(v.mean(axis=1, keepdims=True), Q, axis=1), atol=1e-14)
    # a dominant key in one head moves only that head's slice
    k2 = k.copy()
    k2[1, 4, :d] = qp[0, :d] * 50.0
    out = feature_attention(qp, k2, v, H, 1.0)
    np.testing.assert_allclose(out[1, 0, :d], v[1, 4, :d], atol=1e-8)
    base = feature_attention(qp, k, v, H, 1.0)
    np.testing.assert_allclose(out[1, :, d:], base[1, :, d:], atol=1e-14)      # other head untouched
    np.testing.assert_allclose(out[0], base[0], atol=1e-14)                    # other tokens untouched
    # heads do not mix: permuting the heads of all operands permutes the output slices
    perm = feature_attention(np.roll(qp, d, 1), np.roll(k, d, 2), np.roll(v, d, 2), H, 1.0)
    np.testing.assert_allclose(perm, np.roll(base, d, 2), atol=1e-14)
