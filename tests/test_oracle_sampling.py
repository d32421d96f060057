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


def test_walk_in_float32_differs_only_on_close_calls():
    """The float32 variant (the kernel's arithmetic) takes the same decisions as the fp64 definition
    except where u * R is within rounding of p."""
    g = np.random.default_rng(5)
    diff = 0
    for seed in range(200):
        t = Tiny(seed, B=1, T=12, lens=(3,))
        pc = g.random(12) * 0.6
        u = g.random(12)
        a, Ra = smp.accept_walk(t.parents[0], 12, np.arange(12), pc, u)
        b, Rb = smp.accept_walk(t.parents[0], 12, np.arange(12), pc.astype(np.float32), u.astype(np.float32), dtype=np.float32)
        diff += (a != b)
    assert diff <= 1
