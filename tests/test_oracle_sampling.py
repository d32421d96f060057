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


# ---------------------------------------------------------------------------------------------------
# chains drafted by sampling from a draft distribution q (the rule in its general form)
# ---------------------------------------------------------------------------------------------------
def chain_q_pins(verify_chain_q):
    """Everything that fixes the general-q chain rule; raises AssertionError on the first pin that fails."""
    g = np.random.default_rng(5)
    V, T = 6, 3
    # (1) Monte Carlo: drafts really drawn from q; the first emitted token must follow p_0 and, given that
    # the first draft was accepted, the second must follow p_1 - for a draft far from and one close to p
    for spread in (2.0, 0.3):
        logits = g.standard_normal((T, V)) * 1.5
        p, _ = smp.softmax_rows(logits, 1.1)
        q, _ = smp.softmax_rows(logits + g.standard_normal((T, V)) * spread, 0.9)
        n_draw = 60000
        first, second = np.zeros(V), np.zeros(V)
        cdf = np.cumsum(q, axis=1)
        for _ in range(n_draw):
            tok = np.zeros(T, dtype=np.int64)
            for j in range(1, T):
                tok[j] = min(int(np.searchsorted(cdf[j - 1], g.random(), side="right")), V - 1)
            n_acc, out = verify_chain_q(T, tok, logits, 1.1, q, g.random(T), g.random())
            assert len(out) == n_acc
            first[out[0]] += 1
            if n_acc >= 2:
                second[out[1]] += 1
        for counts, target in ((first, p[0]), (second, p[1])):
            n = counts.sum()
            sigma = np.sqrt(n * target * (1 - target))
            assert (np.abs(counts - n * target) <= 5 * sigma + 1).all(), (spread, counts / n, target)
    # (2) point-mass drafts: the tree rule on a chain, already pinned, must come out
    for seed in range(30):
        g2 = np.random.default_rng(100 + seed)
        T2 = 5
        logits = g2.standard_normal((T2, V)) * 2.0
        tok = g2.integers(0, V, size=T2)
        q = np.zeros((T2, V))
        for j in range(1, T2):
            q[j - 1, tok[j]] = 1.0
        u, w = g2.random(T2), g2.random()
        parents = np.arange(-1, T2 - 1)
        path, out_ref = smp.verify_sequence(parents, T2, tok, logits, 1.4, u, w)
        n_acc, out = verify_chain_q(T2, tok, logits, 1.4, q, u, w)
        assert n_acc == len(path) and out == out_ref, (seed, out, out_ref)
    # (3) q = p: every draft is accepted whatever u < 1 is, and the last token comes from p_leaf by the
    # library's inverse CDF
    logits = g.standard_normal((4, V))
    p, _ = smp.softmax_rows(logits, 1.0)
    tok = np.array([0, 2, 5, 1])
    for w in (0.0, 0.31, 0.77, 0.999):
        n_acc, out = verify_chain_q(4, tok, logits, 1.0, p, np.full(4, 0.999999), w)
        assert n_acc == 4 and out[:3] == [2, 5, 1]
        assert out[3] == int(np.searchsorted(np.cumsum(p[3]), w * p[3].sum(), side="left"))
    # (4) by hand: p = (0.5, 0.3, 0.2), q = (0.2, 0.7, 0.1), draft token 1: kept iff u < 3/7; otherwise the
    # residual is (0.3, 0, 0.1) / 0.4 = (0.75, 0, 0.25)
    logits = np.log(np.array([[0.5, 0.3, 0.2], [0.2, 0.2, 0.6]]))
    q = np.array([[0.2, 0.7, 0.1], [1 / 3, 1 / 3, 1 / 3]])
    tok = np.array([0, 1])
    assert verify_chain_q(2, tok, logits, 1.0, q, [0.0, 0.42], 0.7)[0] == 2          # 0.42 < 3/7: accepted
    assert verify_chain_q(2, tok, logits, 1.0, q, [0.0, 0.42], 0.5)[1] == [1, 2]     # then from p_1 = (.2, .2, .6): 0.5 -> token 2
    assert verify_chain_q(2, tok, logits, 1.0, q, [0.0, 0.43], 0.7) == (1, [0])      # 0.43 > 3/7: rejected; 0.7 < 0.75 -> token 0
    assert verify_chain_q(2, tok, logits, 1.0, q, [0.0, 0.43], 0.8) == (1, [2])      # 0.8 > 0.75 -> token 2


def test_chain_rule_with_a_general_draft_distribution():
    chain_q_pins(smp.verify_chain_q)


def test_chain_q_pins_catch_planted_mistakes():
    """Each plausible mistake in the general-q rule must trip at least one pin."""
    import pytest

    def mutant(accept=None, residual=None, use_q_after_full_accept=False):
        def f(n_nodes, draft_tok, logits, inv_temp, q_rows, u, w):
            p, _ = smp.softmax_rows(logits, inv_temp)
            n = int(n_nodes)
            q_rows = np.asarray(q_rows, dtype=np.float64)
            n_acc = 1
            for j in range(1, n):
                pt, qt = p[j - 1, draft_tok[j]], q_rows[j - 1, draft_tok[j]]
                ok = accept(u[j], pt, qt) if accept else (u[j] * qt < pt)
                if not ok:
                    break
                n_acc += 1
            stop = n_acc - 1
            if n_acc < n or use_q_after_full_accept:
                r = residual(p[stop], q_rows[stop]) if residual else np.maximum(p[stop] - q_rows[stop], 0)
            else:
                r = p[stop]
            t, _ = smp.residual_sample(r, [], float(r.sum()), w)
            return n_acc, [int(draft_tok[j]) for j in range(1, n_acc)] + [t]
        return f

    chain_q_pins(mutant())                                            # the harness itself is sound
    for bad in (mutant(accept=lambda u, p, q: u * p < q),             # ratio upside down
                mutant(accept=lambda u, p, q: u < p),                 # q forgotten in the test
                mutant(residual=lambda p, q: np.maximum(q - p, 0)),   # sign of the residual
                mutant(residual=lambda p, q: p),                      # no residual correction at all
                mutant(residual=lambda p, q: np.abs(p - q)),          # not clipped
                mutant(use_q_after_full_accept=True)):                # residual applied although nothing was rejected
        with pytest.raises(AssertionError):
            chain_q_pins(bad)


# ---------------------------------------------------------------------------------------------------
# trees whose children were sampled independently from the draft distribution of their parent
# ---------------------------------------------------------------------------------------------------
def tree_q_pins(verify_tree_q):
    g = np.random.default_rng(6)
    V = 6
    # (1) Monte Carlo on a fixed shape (root with three children, the first two with two children each);
    # every child's token is drawn from its parent's q.  First emitted token ~ p_root; given that child c
    # of the root was accepted, the second ~ p_c.
    parents = np.array([-1, 0, 0, 0, 1, 1, 2, 2])
    T = len(parents)
    for spread in (1.5, 0.3):
        logits = g.standard_normal((T, V)) * 1.5
        p, _ = smp.softmax_rows(logits, 1.2)
        q, _ = smp.softmax_rows(logits + g.standard_normal((T, V)) * spread, 1.0)
        cdf = np.cumsum(q, axis=1)
        first = np.zeros(V)
        second = {1: np.zeros(V), 2: np.zeros(V), 3: np.zeros(V)}
        for _ in range(60000):
            tok = np.zeros(T, dtype=np.int64)
            for j in range(1, T):
                tok[j] = min(int(np.searchsorted(cdf[parents[j]], g.random(), side="right")), V - 1)
            path, out, *_ = verify_tree_q(parents, T, tok, logits, 1.2, q, g.random(T), g.random())
            first[out[0]] += 1
            if len(path) >= 2:
                second[path[1]][out[1]] += 1
        checks = [(first, p[0])] + [(second[c], p[c]) for c in (1, 2, 3)]
        for counts, target in checks:
            n = counts.sum()
            assert n > 500
            sigma = np.sqrt(n * target * (1 - target))
            assert (np.abs(counts - n * target) <= 5 * sigma + 1).all(), (spread, counts / n, target)
    # (2) a chain is a tree: the chain rule, already pinned, must come out
    for seed in range(30):
        g2 = np.random.default_rng(200 + seed)
        T2 = 5
        logits = g2.standard_normal((T2, V)) * 2.0
        q, _ = smp.softmax_rows(g2.standard_normal((T2, V)), 1.0)
        tok = g2.integers(0, V, size=T2)
        u, w = g2.random(T2), g2.random()
        n_acc, out_ref = smp.verify_chain_q(T2, tok, logits, 1.3, q, u, w)
        path, out, *_ = verify_tree_q(np.arange(-1, T2 - 1), T2, tok, logits, 1.3, q, u, w)
        assert path == list(range(n_acc)) and out == out_ref, (seed, out, out_ref)
    # (3) by hand: p = (0.5, 0.3, 0.2), q = (0.2, 0.7, 0.1), children of the root carry tokens 1 and 0.
    #   child 1 (token 1): kept iff u < 3/7.  Rejected: r = (0.3, 0, 0.1) / 0.4 = (0.75, 0, 0.25).
    #   child 2 (token 0): kept iff u * 0.2 < 0.75, i.e. always.  With tokens 1 and 1 instead: r(1) = 0, never.
    #   Both rejected (tokens 1, 1): r <- max(r - q, 0) = (0.55, 0, 0.15) / 0.7: w = 0.78 -> token 0, 0.79 -> token 2.
    logits = np.log(np.array([[0.5, 0.3, 0.2], [0.2, 0.2, 0.6], [0.1, 0.8, 0.1]]))
    q = np.array([[0.2, 0.7, 0.1], [1 / 3, 1 / 3, 1 / 3], [1 / 3, 1 / 3, 1 / 3]])
    par = np.array([-1, 0, 0])
    assert verify_tree_q(par, 3, np.array([0, 1, 0]), logits, 1.0, q, [0, 0.43, 0.999], 0.05)[:2] == ([0, 2], [0, 0])
    assert verify_tree_q(par, 3, np.array([0, 1, 0]), logits, 1.0, q, [0, 0.42, 0.999], 0.5)[:2] == ([0, 1], [1, 2])
    assert verify_tree_q(par, 3, np.array([0, 1, 1]), logits, 1.0, q, [0, 0.43, 0.0001], 0.78)[:2] == ([0], [0])
    assert verify_tree_q(par, 3, np.array([0, 1, 1]), logits, 1.0, q, [0, 0.43, 0.0001], 0.79)[:2] == ([0], [2])


def test_tree_rule_with_sampled_children():
    tree_q_pins(smp.verify_tree_q)


def test_tree_q_pins_catch_planted_mistakes():
    import pytest

    def mutant(renormalise=True, subtract=lambda r, q: np.maximum(r - q, 0.0), reset=True,
               accept=lambda u, qx, rx: u * qx < rx):
        def f(parents, n_nodes, draft_tok, logits, inv_temp, q_rows, u, w):
            p, _ = smp.softmax_rows(logits, inv_temp)
            q_rows = np.asarray(q_rows, dtype=np.float64)
            n = int(n_nodes)
            cur, path = 0, [0]
            r = p[0].copy()
            while True:
                if reset:
                    r = p[cur].copy()
                q = q_rows[cur]
                nxt = -1
                for c in smp.children_of(parents, n, cur):
                    x = int(draft_tok[c])
                    if accept(u[c], q[x], r[x]):
                        nxt = c
                        break
                    r = subtract(r, q)
                    if renormalise and r.sum() > 0:
                        r = r / r.sum()
                if nxt < 0:
                    t, _ = smp.residual_sample(r, [], float(r.sum()), w)
                    return path, [int(draft_tok[j]) for j in path[1:]] + [t], 0, 0, 0
                cur = nxt
                path.append(cur)
                if not reset:
                    r = p[cur].copy() * 0 + r       # (keeps the parent's residual: the planted mistake)
        return f

    tree_q_pins(mutant())                                                   # the harness itself is sound
    for bad in (mutant(renormalise=False),                                  # residual not renormalised between siblings
                mutant(subtract=lambda r, q: np.maximum(q - r, 0.0)),       # sign
                mutant(subtract=lambda r, q: r),                            # no residual update
                mutant(reset=False),                                        # the child starts from its parent's residual
                mutant(accept=lambda u, qx, rx: u * rx < qx)):              # ratio upside down
        with pytest.raises(AssertionError):
            tree_q_pins(bad)
