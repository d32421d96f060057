"""Pins for the checker's tree attention: brute force, library routine, closed forms."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_18824_b200 import workloads as wl
from helpers import Tiny, root_path


def brute_force_row(p: Tiny, b, i, h):
    """Ordinary causal attention of the LAST position of the explicit linear
    sequence [prefix tokens..., tokens on the root path of node i]."""
    kvh = h // (p.Hq // p.Hkv)
    path = root_path(p.parents[b], i)
    K = np.concatenate([p.prefix(p.k_cache, b, kvh), wl.bf16_bits_to_f64(p.k_tree[b, path, kvh])])
    V = np.concatenate([p.prefix(p.v_cache, b, kvh), wl.bf16_bits_to_f64(p.v_tree[b, path, kvh])])
    q = wl.bf16_bits_to_f64(p.q[b, i, h])
    s = (K @ q) * p.scale
    w = np.exp(s - s.max())
    return (w[:, None] * V).sum(0) / w.sum(), s.max() + np.log(w.sum())


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_tree_attention_equals_per_path_causal_attention(seed):
    p = Tiny(seed, lens=(5, 70) if seed else (0, 64))
    out, lse = oracle.attention(oracle.Geometry.of(p), p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    for b in range(p.B):
        for i in range(p.T_max):
            for h in range(p.Hq):
                o, l = brute_force_row(p, b, i, h)
                np.testing.assert_allclose(out[b, i, h], o, rtol=1e-12, atol=1e-14)
                np.testing.assert_allclose(lse[b, i, h], l, rtol=1e-12)


def test_sampled_rows_match_full():
    p = Tiny(3)
    g = oracle.Geometry.of(p)
    out, lse = oracle.attention(g, p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    rows = np.array([[0, 0, 0], [1, 7, 3], [1, 4, 2], [0, 5, 1]], dtype=np.int32)
    o, l = oracle.attention_rows(g, p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale, rows)
    for n, (b, i, h) in enumerate(rows):
        np.testing.assert_array_equal(o[n], out[b, i, h])
        assert l[n] == lse[b, i, h]


def test_chain_reduces_to_library_causal_attention():
    """parent[i] = i-1 is chain decoding: plain causal attention of the new
    tokens over prefix + themselves, here computed by torch's SDPA in fp64."""
    B, T, Hq, Hkv, D = 2, 6, 4, 2, 16
    p = Tiny(5, B=B, T=T, Hq=Hq, Hkv=Hkv, D=D, lens=(9, 66),
             parents=np.stack([wl.chain_tree(T)] * B))
    out, _ = oracle.attention(oracle.Geometry.of(p), p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    G = Hq // Hkv
    for b in range(B):
        P = int(p.len[b])
        for h in range(Hq):
            kvh = h // G
            K = np.concatenate([p.prefix(p.k_cache, b, kvh), wl.bf16_bits_to_f64(p.k_tree[b, :, kvh])])
            V = np.concatenate([p.prefix(p.v_cache, b, kvh), wl.bf16_bits_to_f64(p.v_tree[b, :, kvh])])
            Q = np.zeros((P + T, D))
            Q[P:] = wl.bf16_bits_to_f64(p.q[b, :, h])
            o = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(Q)[None, None], torch.from_numpy(K)[None, None],
                torch.from_numpy(V)[None, None], is_causal=True, scale=p.scale)[0, 0, P:].numpy()
            np.testing.assert_allclose(out[b, :, h], o, rtol=1e-10, atol=1e-13)


def test_constant_v_and_equal_k_closed_forms():
    p = Tiny(7)
    g = oracle.Geometry.of(p)
    # V constant => output is that constant whatever the mask and scores
    c = wl.f32_to_bf16_bits(np.array([0.375], dtype=np.float32))[0]
    vc = np.full_like(p.v_cache, c)
    vt = np.full_like(p.v_tree, c)
    out, _ = oracle.attention(g, p.k_cache, vc, p.q, p.k_tree, vt, p.scale)
    np.testing.assert_allclose(out, 0.375, rtol=1e-13)
    # all keys equal => uniform weights => mean of the visible V rows,
    # whose count is len + depth + 1; lse = score + log(count)
    kc = np.broadcast_to(p.k_tree[0, 0, 0], p.k_cache.shape).copy()
    kt = np.broadcast_to(p.k_tree[0, 0, 0], p.k_tree.shape).copy()
    out, lse = oracle.attention(g, kc, p.v_cache, p.q, kt, p.v_tree, p.scale)
    G = p.Hq // p.Hkv
    for b in range(p.B):
        for i in range(p.T_max):
            path = root_path(p.parents[b], i)
            for h in range(p.Hq):
                kvh = h // G
                Vv = np.concatenate([p.prefix(p.v_cache, b, kvh), wl.bf16_bits_to_f64(p.v_tree[b, path, kvh])])
                assert Vv.shape[0] == p.len[b] + len(path)
                np.testing.assert_allclose(out[b, i, h], Vv.mean(0), rtol=1e-11, atol=1e-14)
                s = p.scale * wl.bf16_bits_to_f64(p.q[b, i, h]) @ wl.bf16_bits_to_f64(p.k_tree[0, 0, 0])
                np.testing.assert_allclose(lse[b, i, h], s + np.log(len(Vv)), rtol=1e-11)


def test_planted_dominant_key():
    p = Tiny(8, B=1, T=8, Hq=2, Hkv=1, D=16, lens=(100,), gain=0.01)
    # one prefix key aligned with the query at a large magnitude dominates the softmax
    t_star = 77
    blk = p.block_table[0, t_star // 64]
    qv = np.zeros(p.D, dtype=np.float32); qv[3] = 8.0
    p.q[:] = wl.f32_to_bf16_bits(qv)
    kv = np.zeros(p.D, dtype=np.float32); kv[3] = 32.0
    p.k_cache[blk, 0, t_star % 64] = wl.f32_to_bf16_bits(kv)
    out, lse = oracle.attention(oracle.Geometry.of(p), p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    want = wl.bf16_bits_to_f64(p.v_cache[blk, 0, t_star % 64])
    np.testing.assert_allclose(out[0, :, :], np.broadcast_to(want, out[0].shape), atol=1e-12)
    np.testing.assert_allclose(lse, 8.0 * 32.0 * p.scale, rtol=1e-12)


def test_invariants_gqa_paging_relabel_scale_and_garbage():
    p = Tiny(9, B=1, T=8, Hq=4, Hkv=2, D=16, lens=(70,))
    g = oracle.Geometry.of(p)
    base, _ = oracle.attention(g, p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    # heads of one group given the same q give the same output; a head of the
    # other group (different K/V) does not
    q2 = p.q.copy(); q2[:, :, 1] = q2[:, :, 0]; q2[:, :, 2] = q2[:, :, 0]
    o2, _ = oracle.attention(g, p.k_cache, p.v_cache, q2, p.k_tree, p.v_tree, p.scale)
    np.testing.assert_array_equal(o2[:, :, 0], o2[:, :, 1])
    assert np.abs(o2[:, :, 0] - o2[:, :, 2]).max() > 1e-3
    # same logical content under another block permutation
    perm = np.random.default_rng(1).permutation(p.num_blocks)
    kc2 = np.empty_like(p.k_cache); vc2 = np.empty_like(p.v_cache)
    kc2[perm] = p.k_cache; vc2[perm] = p.v_cache
    p2 = Tiny(9, B=1, T=8, Hq=4, Hkv=2, D=16, lens=(70,))
    p2.block_table = perm[p.block_table].astype(np.int32)
    o3, _ = oracle.attention(oracle.Geometry.of(p2), kc2, vc2, p.q, p.k_tree, p.v_tree, p.scale)
    np.testing.assert_array_equal(o3, base)
    # slots at and beyond len hold garbage that must not matter
    kc4, vc4 = p.k_cache.copy(), p.v_cache.copy()
    blk = p.block_table[0, 1]
    kc4[blk, :, 6:] = 0x7F7F; vc4[blk, :, 6:] = 0xFF7F      # +/- max finite bf16
    o4, _ = oracle.attention(g, kc4, vc4, p.q, p.k_tree, p.v_tree, p.scale)
    np.testing.assert_array_equal(o4, base)
    # a visible key must matter: changing prefix slot len-1 changes the result
    kc5 = p.k_cache.copy(); kc5[blk, :, 5] ^= 0x8000
    o5, _ = oracle.attention(g, kc5, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    assert np.abs(o5 - base).max() > 1e-6
    # doubling the scale equals doubling q (exact in bf16)
    qd = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(p.q) * 2)
    o6, _ = oracle.attention(g, p.k_cache, p.v_cache, qd, p.k_tree, p.v_tree, p.scale)
    o7, _ = oracle.attention(g, p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, 2 * p.scale)
    np.testing.assert_allclose(o6, o7, rtol=1e-12)
    assert np.abs(o6 - base).max() > 1e-3
    # relabelling nodes (keeping parent < child) permutes the outputs
    par = p.parents[0]
    # swap two siblings-or-unrelated adjacent nodes i, i+1 where parent[i+1] != i
    i = next(i for i in range(1, 7) if par[i + 1] != i)
    newid = np.arange(8); newid[i], newid[i + 1] = i + 1, i
    par_r = np.empty(8, dtype=np.int32)
    for old in range(8):
        par_r[newid[old]] = -1 if par[old] < 0 else newid[par[old]]
    inv = np.argsort(newid)
    pr = Tiny(9, B=1, T=8, Hq=4, Hkv=2, D=16, lens=(70,), parents=par_r[None])
    pr.block_table = p.block_table
    o8, _ = oracle.attention(oracle.Geometry.of(pr), p.k_cache, p.v_cache, p.q[:, inv], p.k_tree[:, inv],
                             p.v_tree[:, inv], p.scale)
    np.testing.assert_array_equal(o8[:, newid], base)


def test_sibling_is_invisible_and_ancestor_is_visible():
    # tree 0 -> {1, 2}; node 2 must not see node 1; node 1 must see node 0
    par = np.array([[-1, 0, 0]], dtype=np.int32)
    p = Tiny(11, B=1, T=3, Hq=1, Hkv=1, D=16, lens=(0,), parents=par)
    g = oracle.Geometry.of(p)
    base, _ = oracle.attention(g, p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    vt = p.v_tree.copy(); vt[0, 1] ^= 0x8000
    o, _ = oracle.attention(g, p.k_cache, p.v_cache, p.q, p.k_tree, vt, p.scale)
    np.testing.assert_array_equal(o[0, 2], base[0, 2])
    np.testing.assert_array_equal(o[0, 0], base[0, 0])
    assert np.abs(o[0, 1] - base[0, 1]).max() > 1e-6
    vt = p.v_tree.copy(); vt[0, 0] ^= 0x8000
    o, _ = oracle.attention(g, p.k_cache, p.v_cache, p.q, p.k_tree, vt, p.scale)
    assert np.abs(o[0, 1] - base[0, 1]).max() > 1e-6
    # root with empty prefix sees only itself: output is its own V row
    np.testing.assert_allclose(base[0, 0, 0], wl.bf16_bits_to_f64(p.v_tree[0, 0, 0]), rtol=1e-15)
