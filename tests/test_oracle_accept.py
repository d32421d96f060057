"""Pins for the checker's greedy acceptance: exhaustive enumeration, a
sequential greedy walker, planted paths and hand-worked cases."""
import os

import numpy as np
import pytest

import oracle
from paper_2509_18824_b200 import workloads as wl
from helpers import root_path


class G:
    pass


def geom(parents, lens=None):
    parents = np.asarray(parents, dtype=np.int32)
    if parents.ndim == 1:
        parents = parents[None]
    g = G()
    g.B, g.T_max = parents.shape
    g.Hq, g.Hkv, g.D = 1, 1, 8
    g.parents = parents
    g.n_nodes = np.full(g.B, g.T_max, dtype=np.int32)
    g.len = np.zeros(g.B, dtype=np.int32) if lens is None else np.asarray(lens, dtype=np.int32)
    g.block_table = np.zeros((g.B, 4), dtype=np.int32)
    return oracle.Geometry.of(g)


def enumerate_paths(parents, draft, target):
    """Every root-to-node path, validity straight from the tokens."""
    best, best_len = 0, 1
    for i in range(len(parents)):
        path = root_path(parents, i)
        if all(draft[path[k]] == target[path[k - 1]] for k in range(1, len(path))):
            if len(path) > best_len:
                best, best_len = i, len(path)
    return root_path(parents, best)


def greedy_walk(parents, draft, target):
    """Simulates greedy decoding token by token: from the current node the
    target emits target[node]; we may step to a child that drafted exactly
    that token.  With duplicate children every choice is explored."""
    T = len(parents)
    kids = [[j for j in range(T) if parents[j] == i] for i in range(T)]

    def longest(node):
        best = [node]
        for c in kids[node]:
            if draft[c] == target[node]:
                cand = [node] + longest(c)
                if len(cand) > len(best):          # children visited in index order
                    best = cand
        return best
    return longest(0)


def test_hand_worked_cases():
    fn = os.path.join(os.path.dirname(__file__), "golden", "accept_tiny_tree.txt")
    n = 0
    for line in open(fn):
        if line.startswith("#") or not line.strip():
            continue
        d, t, na, path, out = [np.array(x.split(), dtype=np.int32) for x in line.split("|")]
        n_acc, p, o, nl = oracle.accept(geom(wl.TINY_PARENTS, [100]), d, t)
        assert n_acc[0] == na[0]
        np.testing.assert_array_equal(p[0, :na[0]], path)
        np.testing.assert_array_equal(o[0, :na[0]], out)
        assert (p[0, na[0]:] == -1).all() and (o[0, na[0]:] == -1).all()
        assert nl[0] == 100 + na[0]
        n += 1
    assert n == 5


@pytest.mark.parametrize("seed", range(6))
def test_random_tiny_trees_against_enumeration_and_walker(seed):
    g = np.random.default_rng(seed)
    for _ in range(300):
        T = int(g.integers(1, 9))
        vocab = int(g.integers(2, 5))
        par = np.array([-1] + [int(g.integers(0, i)) for i in range(1, T)], dtype=np.int32)
        d = g.integers(0, vocab, size=T).astype(np.int32)
        t = g.integers(0, vocab, size=T).astype(np.int32)
        n_acc, p, o, nl = oracle.accept(geom(par, [7]), d, t)
        want = enumerate_paths(par, d, t)
        assert n_acc[0] == len(want)
        np.testing.assert_array_equal(p[0, :len(want)], want)
        walk = greedy_walk(par, d, t)
        assert len(walk) == len(want)
        # emitted tokens are what sequential greedy decoding emits along the walk
        emitted = [t[x] for x in want]
        np.testing.assert_array_equal(o[0, :len(want)], emitted)
        assert nl[0] == 7 + len(want)


def test_full_size_tree_exhaustive_and_planted():
    sp = wl.spec("c5")
    w = wl.make_geometry(sp)
    g = np.random.default_rng(0)
    target = g.integers(0, w.V, size=(w.B, w.T_max)).astype(np.int32)
    w.draft_tok = None
    for lengths in (None, np.arange(w.B) % 7):
        wl.plant(w, target, lengths)
        n_acc, p, o, nl = oracle.accept(oracle.Geometry.of(w), w.draft_tok, target)
        for b in range(w.B):
            want = root_path(w.parents[b], int(w.planted_node[b]))
            assert n_acc[b] == w.planted_len[b] + 1 == len(want)
            np.testing.assert_array_equal(p[b, :len(want)], want)
            np.testing.assert_array_equal(p[b, :n_acc[b]], enumerate_paths(w.parents[b], w.draft_tok[b], target[b]))
            assert o[b, n_acc[b] - 1] == target[b, want[-1]]
        if lengths is not None:
            np.testing.assert_array_equal(w.planted_len, lengths)


def test_bad_trees_are_rejected():
    for par in ([0, 0, 1], [-1, 1, 0], [-1, 0, 3, 1], [-1, -1]):
        with pytest.raises(ValueError):
            oracle.accept(geom(par), np.zeros(len(par), np.int32), np.zeros(len(par), np.int32))
