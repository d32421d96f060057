"""The seeded input recipes: shapes, determinism, tree validity."""
import numpy as np

from paper_2509_18824_b200 import workloads as wl


def test_bf16_round_trip_and_rounding():
    x = np.array([1.0, 1.00390625, 1.005859375, -2.5, 0.0, 3.0e38], dtype=np.float32)
    b = wl.f32_to_bf16_bits(x)
    y = wl.bf16_bits_to_f32(b)
    assert y[0] == 1.0 and y[3] == -2.5 and y[4] == 0.0
    assert y[1] == 1.0            # tie rounds to even mantissa
    assert y[2] == 1.0078125      # above the tie rounds up
    np.testing.assert_array_equal(wl.f32_to_bf16_bits(y), b)


def test_trees_are_valid_and_reach_their_depth():
    for cfg in ("c2", "c3", "c4", "c5"):
        w = wl.make_geometry(wl.spec(cfg))
        assert w.parents.shape == (w.B, 60)
        depths = []
        for b in range(w.B):
            par = w.parents[b]
            assert par[0] == -1 and all(0 <= par[i] < i for i in range(1, 60))
            d = wl.node_depths(par)
            assert all(np.diff(d) >= 0)                   # numbered by depth
            assert np.bincount(par[1:]).max() <= 10       # top-k 10 expansion
            depths.append(int(d.max()))
        if cfg == "c4":
            assert set(depths) <= {4, 5, 6, 7} and len(set(depths)) > 1
            assert w.len.min() >= 512 and w.len.max() <= 16384
            assert len(np.unique(w.block_table[0, :(w.len[0] + 60 + 63) // 64])) == (w.len[0] + 60 + 63) // 64
        else:
            assert depths == [6] * w.B
    w = wl.make_geometry(wl.spec("c1"))
    np.testing.assert_array_equal(w.parents[0], [-1, 0, 0, 1, 1, 2, 3, 3])
    w = wl.make_geometry(wl.spec("chain11"))
    np.testing.assert_array_equal(w.parents[0], np.arange(-1, 10))
    w = wl.make_geometry(wl.spec("tree28"))
    assert w.T_max == 28 and (w.n_nodes == 28).all()
    assert [int(wl.node_depths(w.parents[b]).max()) for b in range(w.B)] == [5] * w.B


def test_generation_is_deterministic_and_scaled():
    a = wl.make("c1")
    b = wl.make("c1")
    for x, y in ((a.q[0], b.q[0]), (a.k_cache[0], b.k_cache[0]), (a.W, b.W), (a.hidden, b.hidden),
                 (a.draft_tok, b.draft_tok)):
        np.testing.assert_array_equal(x, y)
    q = wl.bf16_bits_to_f32(a.q[0])
    assert abs(q.std() * np.sqrt(128) - 1) < 0.1
    Wf = wl.bf16_bits_to_f32(a.W)
    assert abs(Wf.std() * np.sqrt(256) - 1) < 0.05
    assert a.k_cache[0].shape == (a.num_blocks, 1, 64, 128)
    # slots beyond the prefix are poisoned with large finite values
    blk = a.block_table[0, 2]
    assert np.abs(wl.bf16_bits_to_f32(a.k_cache[0][blk])).min() > 5e4


def test_image_prefix_has_double_variance():
    w = wl.make_geometry(wl.spec("c3"))
    w.spec.prefix = 8192
    wl.fill_attention(w, layers=[0])
    k = wl.bf16_bits_to_f32(w.k_cache[0])
    first = k[w.block_table[0, :64]].var()
    second = k[w.block_table[0, 64:128]].var()
    assert abs(first / second - 2.0) < 0.05
