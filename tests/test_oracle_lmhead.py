"""Pins for the checker's LM-head argmax."""
import numpy as np

import oracle
from paper_2509_18824_b200 import workloads as wl


def bf(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_matches_numpy_matmul_and_full_logits():
    g = np.random.default_rng(0)
    M, Hd, V = 7, 96, 1000
    h = bf(g.standard_normal((M, Hd)))
    W = bf(g.standard_normal((V, Hd)))
    ref = wl.bf16_bits_to_f64(h) @ wl.bf16_bits_to_f64(W).T
    lg = oracle.logits(h, W)
    np.testing.assert_allclose(lg, ref, rtol=1e-12, atol=1e-12)
    am, t1, t2 = oracle.lmhead(h, W)
    np.testing.assert_array_equal(am, ref.argmax(1))
    np.testing.assert_allclose(t1, ref.max(1), rtol=1e-12)
    np.testing.assert_allclose(t2, np.sort(ref, 1)[:, -2], rtol=1e-12)
    am2, t12, t22 = oracle.lmhead(h, W, rows=[5, 0, 3])
    np.testing.assert_array_equal(am2, am[[5, 0, 3]])
    np.testing.assert_array_equal(t12, t1[[5, 0, 3]])
    np.testing.assert_array_equal(t22, t2[[5, 0, 3]])


def test_identity_weights_give_argmax_of_hidden():
    g = np.random.default_rng(1)
    n = 64
    h = bf(g.standard_normal((9, n)))
    W = bf(np.eye(n))
    am, t1, _ = oracle.lmhead(h, W)
    hf = wl.bf16_bits_to_f64(h)
    np.testing.assert_array_equal(am, hf.argmax(1))
    np.testing.assert_array_equal(t1, hf.max(1))


def test_transposed_operand_would_fail():
    # W[v][k] with V != Hd and a planted row: row v* = 4*hidden[r] wins for row r only
    g = np.random.default_rng(2)
    M, Hd, V = 5, 32, 77
    h = bf(g.standard_normal((M, Hd)))
    W = bf(0.05 * g.standard_normal((V, Hd)))
    stars = [70, 3, 41, 76, 0]
    for r, v in enumerate(stars):
        W[v] = bf(4.0 * wl.bf16_bits_to_f32(h[r]))
    am, _, _ = oracle.lmhead(h, W)
    np.testing.assert_array_equal(am, stars)


def test_exact_ties_take_lowest_index_and_report_zero_gap():
    g = np.random.default_rng(3)
    M, Hd, V = 3, 16, 300
    h = bf(g.standard_normal((M, Hd)))
    W = bf(0.01 * g.standard_normal((V, Hd)))
    row = bf(8.0 * wl.bf16_bits_to_f32(h[1]))
    for v in (290, 17, 150):      # three identical winning rows, far apart (different thread slabs)
        W[v] = row
    am, t1, t2 = oracle.lmhead(h, W)
    assert am[1] == 17
    assert t1[1] == t2[1]
    ref = wl.bf16_bits_to_f64(h) @ wl.bf16_bits_to_f64(W).T
    np.testing.assert_array_equal(am, ref.argmax(1))
