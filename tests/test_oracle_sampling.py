"""Pins of the sampling-temperature reference (oracle/sampling.py): what the rule must do is fixed
here by statistics, limits and library routines, not by re-typing its formula."""
import numpy as np

import oracle
from oracle import sampling as smp
from helpers import Tiny


def test_emitted_token_follows_the_target_distribution():
    """Monte Carlo: whatever the drafted children are, the FIRST emitted token must be distributed
    as p (that is what "lossless" means); a wrong residual update, a missing renormalisation or an
    off-by-one in the inverse CDF shifts the frequencies by far more than the 5-sigma band."""
    g = np.random.default_rng(0)
    V, n_draw = 7, 120000
    for kids in ([], [3], [5, 0, 2], [1, 2, 3, 4, 5, 6]):
        T = 1 + len(kids)
        parents = np.array([-1] + [0] * len(kids))
        tok = np.array([0] + kids)
        logits = g.standard_normal((T, V)) * 2.0
        p, _ = smp.softmax_rows(logits, 1.3)
        counts = np.zeros(V)
        for _ in range(n_draw):
            path, out = smp.verify_sequence(parents, T, tok, logits, 1.3, g.random(T), g.random())
            counts[out[0]] += 1
        sigma = np.sqrt(n_draw * p[0] * (1 - p[0]))
        assert (np.abs(counts - n_draw * p[0]) <= 5 * sigma + 1).all(), (kids, counts / n_draw, p[0])


def test_second_token_follows_the_child_distribution():
    """Given that child c was accepted, the next emitted token is distributed as p_c."""
    g = np.random.default_rng(1)
    V = 5
    parents = np.array([-1, 0, 0, 1, 1, 2])
    tok = np.array([0, 2, 4, 1, 3, 0])
    logits = g.standard_normal((6, V)) * 1.5
    p, _ = smp.softmax_rows(logits, 1.0)
    counts = {1: np.zeros(V), 2: np.zeros(V)}
    for _ in range(150000):
        path, out = smp.verify_sequence(parents, 6, tok, logits, 1.0, g.random(6), g.random())
        if len(path) >= 2:
            counts[path[1]][out[1]] += 1
    for c in (1, 2):
        n = counts[c].sum()
        sigma = np.sqrt(n * p[c] * (1 - p[c]))
        assert (np.abs(counts[c] - n * p[c]) <= 5 * sigma + 1).all()


def test_zero_temperature_limit_is_the_greedy_rule():
    """With a very large inverse temperature p is one-hot on the arg-max, so the walk must follow
    exactly the nodes whose token equals the target arg-max: the greedy checker's path."""
    g = np.random.default_rng(2)
    for seed in range(40):
        t = Tiny(seed, B=1, T=8, lens=(5,))
        V = 6
        logits = g.standard_normal((8, V))
        am = logits.argmax(1).astype(np.int32)
        tok = np.zeros(8, dtype=np.int32)
        for i in range(8):                               # distinct tokens among siblings
            kids = smp.children_of(t.parents[0], 8, i)
            tok[kids] = g.permutation(V)[:len(kids)]
        ref = oracle.accept(oracle.Geometry.of(t), tok[None], am[None])
        path, out = smp.verify_sequence(t.parents[0], 8, tok, logits, 1e4, g.random(8) * 0.999 + 5e-4, g.random())
        assert path == list(ref[1][0][:ref[0][0]])
        assert out == list(ref[2][0][:ref[0][0]])


def test_single_child_is_the_textbook_accept_test():
    """One drafted token: accepted exactly when u < p(x); otherwise the replacement never is x."""
    g = np.random.default_rng(3)
    V = 9
    for _ in range(300):
        logits = g.standard_normal((2, V)) * 2
        p, _ = smp.softmax_rows(logits, 0.7)
        x = int(g.integers(V))
        u, w = g.random(2), g.random()
        path, out = smp.verify_sequence(np.array([-1, 0]), 2, np.array([0, x]), logits, 0.7, u, w)
        if u[1] < p[0, x]:
            assert path == [0, 1] and out[0] == x
        else:
            assert path == [0] and out[0] != x


def test_inverse_cdf_against_cumsum_searchsorted():
    g = np.random.default_rng(4)
    for _ in range(200):
        V = int(g.integers(3, 40))
        p = g.random(V); p /= p.sum()
        excl = list(g.choice(V, size=int(g.integers(0, V - 1)), replace=False))
        R = 1.0 - p[excl].sum()
        w = g.random()
        t, margin = smp.residual_sample(p, excl, R, w)
        q = p.copy(); q[excl] = 0.0
        want = int(np.searchsorted(np.cumsum(q), w * R, side="left"))
        while q[want] == 0.0:                            # searchsorted may land on a zero-mass token
            want += 1
        assert t == want and t not in excl and margin >= 0.0
    # ends of the interval
    p = np.array([0.2, 0.0, 0.5, 0.3])
    assert smp.residual_sample(p, [], 1.0, 0.0)[0] == 0
    assert smp.residual_sample(p, [], 1.0, 1.0)[0] == 3
    assert smp.residual_sample(p, [0], 0.8, 1e-9)[0] == 2


def test_walk_margin_is_the_closest_comparison():
    """The margin the walk reports bounds how far an input may move before the path changes: shifting
    every probability by less than the margin leaves the path as it is."""
    g = np.random.default_rng(5)
    for seed in range(200):
        t = Tiny(seed, B=1, T=12, lens=(3,))
        pc = g.random(12) * 0.6
        u = g.random(12)
        a, Ra, margin = smp.accept_walk(t.parents[0], 12, np.arange(12), pc, u)
        if not np.isfinite(margin):
            continue
        eps = 0.1 * margin          # residuals accumulate at most a handful of shifted probabilities
        for sign in (-1.0, 1.0):
            b, _, _ = smp.accept_walk(t.parents[0], 12, np.arange(12), np.clip(pc + sign * eps, 0, 1), u)
            assert a == b


# ---------------------------------------------------------------- the probabilities themselves
def check_softmax_against_libraries(softmax_rows):
    """softmax_rows(logits, inv_temp) -> (p, lse) against routines that share nothing with it:
    torch.log_softmax / torch.logsumexp in fp64, scipy.special.softmax, and a case worked by hand."""
    import torch
    from scipy import special
    g = np.random.default_rng(6)
    for shape, inv_temp, gain in (((3, 7), 1.0, 1.0), ((5, 129), 0.37, 4.0), ((2, 1000), 6.0, 2.0), ((4, 1), 2.0, 1.0),
                                  ((2, 33), 40.0, 30.0)):
        lg = g.standard_normal(shape) * gain
        p, lse = softmax_rows(lg, inv_temp)
        z = torch.from_numpy(lg).double() * inv_temp
        np.testing.assert_allclose(p, torch.log_softmax(z, dim=-1).exp().numpy(), rtol=1e-12, atol=1e-300)
        np.testing.assert_allclose(lse, torch.logsumexp(z, dim=-1).numpy(), rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(p, special.softmax(lg * inv_temp, axis=-1), rtol=1e-12, atol=1e-300)
        np.testing.assert_allclose(p.sum(-1), 1.0, rtol=1e-13)
    # by hand: logits (0, 1) at inverse temperature ln 2 are exponents (0, ln 2): weights 1 and 2
    p, lse = softmax_rows(np.array([[0.0, 1.0]]), np.log(2.0))
    np.testing.assert_allclose(p, [[1 / 3, 2 / 3]], rtol=1e-15)
    np.testing.assert_allclose(lse, [np.log(3.0)], rtol=1e-15)
    # three equal logits: uniform, lse = c * inv_temp + ln 3 (no overflow at a large offset)
    p, lse = softmax_rows(np.full((1, 3), 800.0), 1.5)
    np.testing.assert_allclose(p, np.full((1, 3), 1 / 3), rtol=1e-15)
    np.testing.assert_allclose(lse, [1200.0 + np.log(3.0)], rtol=1e-15)


def test_softmax_rows_against_torch_scipy_and_a_hand_case():
    check_softmax_against_libraries(smp.softmax_rows)


def test_softmax_pins_catch_planted_mistakes():
    """The same checks must reject plausible wrong versions of softmax_rows (planted here, on the CPU)."""
    import pytest

    def squared_temperature(lg, it):
        return smp.softmax_rows(lg, it * it)

    def base_two(lg, it):
        z = np.asarray(lg, dtype=np.float64) * it
        m = z.max(-1, keepdims=True)
        e = np.exp2(z - m)
        s = e.sum(-1, keepdims=True)
        return e / s, (m + np.log2(s))[..., 0]

    def lse_without_the_maximum(lg, it):
        p, lse = smp.softmax_rows(lg, it)
        return p, lse - (np.asarray(lg) * it).max(-1)

    def temperature_divides(lg, it):
        return smp.softmax_rows(lg, 1.0 / it)

    for wrong in (squared_temperature, base_two, lse_without_the_maximum, temperature_divides):
        with pytest.raises(AssertionError):
            check_softmax_against_libraries(wrong)
