"""Reference for verification at a sampling temperature (TEST INFRASTRUCTURE ONLY).

The paper validates the draft's tokens with the target model and keeps the
target's output distribution unchanged (Sec. 1: "batch-validated by the target
model", lossless; the speculative-sampling lineage it cites in Sec. 1 gives the
rule for sampling: accept a drafted token x with probability min(1, p(x)/q(x)),
otherwise resample from the normalised positive part of p - q).  The drafts of
an EAGLE-style tree are chosen deterministically (top-k), i.e. q is a point
mass on each child's token, and the rule becomes sequential rejection without
replacement:

    at node i with target distribution p_i = softmax(logits_i / tau), residual mass R = 1:
      for every child c of i, in node order:
          accept c  iff  u[c] * R < p_i(token[c]);     then continue at c with R = 1
          otherwise R -= p_i(token[c])
      if no child was accepted (or i is a leaf): emit one token from p_i restricted to the
      tokens that are not children of i, by inverse CDF in vocabulary order with the
      uniform w:  the first token t whose cumulative remaining mass reaches w * R.

Every random number is an input (u per node, w per sequence).  Plain numpy,
fp64 throughout; no code shared with the GPU library.  Siblings must carry
distinct tokens.

For a CHAIN whose tokens were sampled from draft distributions (node j's token x_j drawn from q_{j-1},
the draft model's distribution behind node j-1) the rule keeps its general form (accept_chain_q,
residual_sample_q, verify_chain_q below):

    walking down the chain from the root, accept x_j  iff  u[j] * q_{j-1}(x_j) < p_{j-1}(x_j),
    i.e. with probability min(1, p/q); at the first rejection, behind node i = j - 1, emit one token
    from the normalised positive part of p_i - q_i; if every draft was accepted emit one token from
    p_leaf.  Inverse CDF in vocabulary order with the uniform w, as above.

For a TREE whose children were sampled (every child of node i drawn independently from the same draft
distribution q_i; tokens may repeat) the rule is applied child after child, each rejection replacing
the target distribution by its residual (verify_tree_q below):

    at node i: r = p_i; for every child c of i in node order with token x:
        accept c  iff  u[c] * q_i(x) < r(x)            (probability min(1, r/q)); continue at c
        otherwise r <- normalised positive part of r - q_i
    where no child is accepted: emit one token from r by inverse CDF with w.
    Every r met this way has the form max(p_i - a q_i, 0) / b with scalars a, b (a = 0, b = 1 at the
    start; a rejection makes a <- a + b and b <- sum_v max(p_i - a q_i, 0)), which the function below
    does NOT use: it carries the vector r itself.

Parity with the paper's own acceptance statistics is unpinned (they need the
trained models).  The functions are pinned in tests/test_oracle_sampling.py:
softmax_rows against torch's log_softmax / logsumexp in fp64, scipy's softmax
and a hand-computed case; the rule by Monte-Carlo frequencies against p, by the
zero-temperature limit (the greedy rule), by the single-child case (the
textbook accept test) and by numpy's cumsum/searchsorted for the inverse CDF;
the general-q chain rule by Monte-Carlo frequencies against p, by the point-mass
case (where it must reproduce verify_sequence), by q = p (everything accepted)
and by a hand-computed case; the sampled-tree rule by Monte-Carlo frequencies
with children drawn independently from q, by chains (where it must reproduce
verify_chain_q) and by a hand-computed case.
"""
from __future__ import annotations

import numpy as np


def softmax_rows(logits: np.ndarray, inv_temp: float):
    """p = softmax(logits * inv_temp) per row and lse = log sum exp(logits * inv_temp), fp64."""
    z = np.asarray(logits, dtype=np.float64) * float(inv_temp)
    m = z.max(axis=-1, keepdims=True)
    e = np.exp(z - m)
    s = e.sum(axis=-1, keepdims=True)
    return e / s, (m + np.log(s))[..., 0]


def children_of(parents: np.ndarray, n: int, i: int):
    return [j for j in range(i + 1, n) if parents[j] == i]


def accept_walk(parents, n_nodes, draft_tok, p_child, u):
    """The acceptance walk of ONE sequence, fp64.

    p_child[j] = probability of draft_tok[j] under the target distribution at parent(j) (j >= 1),
    u[j] = the uniform drawn for node j.
    Returns (path, R, margin): the accepted root path, the residual mass left at its last node, and
    the smallest |u * R - p| over the comparisons the walk made (how close its closest decision was;
    infinity when it made none).
    """
    parents = np.asarray(parents)
    p_child = np.asarray(p_child, dtype=np.float64)
    u = np.asarray(u, dtype=np.float64)
    n = int(n_nodes)
    cur, path = 0, [0]
    margin = np.inf
    while True:
        nxt = -1
        R = 1.0
        kids = children_of(parents, n, cur)
        toks = [int(draft_tok[c]) for c in kids]
        assert len(set(toks)) == len(toks), "siblings must carry distinct tokens"
        for c in kids:
            margin = min(margin, abs(u[c] * R - p_child[c]))
            if u[c] * R < p_child[c]:
                nxt = c
                break
            R = R - p_child[c]
        if nxt < 0:
            return path, R, margin
        cur = nxt
        path.append(cur)


def residual_sample(p_row, excluded, R, w):
    """First token t (vocabulary order, tokens in `excluded` carry no mass) whose cumulative mass
    reaches w * R; the last token with mass if rounding leaves the sum short.  Returns (t, margin):
    margin = distance of the target from the nearer end of t's CDF interval (how close the decision
    was)."""
    p = np.array(p_row, dtype=np.float64)
    if len(excluded):
        p[np.asarray(excluded, dtype=np.int64)] = 0.0
    target = float(w) * float(R)
    acc = 0.0
    last = -1
    for t in range(len(p)):
        if p[t] <= 0.0:
            continue
        last = t
        if acc + p[t] >= target:
            return t, min(target - acc, acc + p[t] - target)
        acc += p[t]
    return last, 0.0


def verify_sequence(parents, n_nodes, draft_tok, logits, inv_temp, u, w):
    """Whole rule for one sequence from the target's logits [T, V] (fp64 definition).
    Returns (path, out_tok): accepted nodes and the emitted tokens (accepted drafts, then the
    residual sample at the last accepted node)."""
    p, _ = softmax_rows(logits, inv_temp)
    n = int(n_nodes)
    p_child = np.zeros(len(parents))
    for j in range(1, n):
        p_child[j] = p[parents[j], draft_tok[j]]
    path, R, _ = accept_walk(parents, n, draft_tok, p_child, u)
    last = path[-1]
    excl = [int(draft_tok[c]) for c in children_of(parents, n, last)]
    t, _ = residual_sample(p[last], excl, R, w)
    return path, [int(draft_tok[j]) for j in path[1:]] + [t]


def accept_chain_q(n_nodes, p_tok, q_tok, u):
    """Acceptance along a chain drafted by sampling, fp64.

    p_tok[j], q_tok[j] = probability of node j's token under the target's and under the draft's
    distribution behind node j - 1 (j >= 1); u[j] the uniform drawn for node j.
    Returns (n_acc, margin): accepted nodes including the root, and the smallest |u * q - p| compared."""
    p_tok = np.asarray(p_tok, dtype=np.float64)
    q_tok = np.asarray(q_tok, dtype=np.float64)
    u = np.asarray(u, dtype=np.float64)
    n_acc, margin = 1, np.inf
    for j in range(1, int(n_nodes)):
        margin = min(margin, abs(u[j] * q_tok[j] - p_tok[j]))
        if not (u[j] * q_tok[j] < p_tok[j]):
            break
        n_acc += 1
    return n_acc, margin


def residual_sample_q(p_row, q_row, w):
    """One token from the normalised positive part of p - q (from p itself when q_row is None): the
    first token, in vocabulary order, at which the cumulative mass reaches w times the total mass; the
    last token with mass if rounding leaves the sum short.  Returns (t, margin, total): margin as in
    residual_sample, total = the mass that was normalised by."""
    r = np.array(p_row, dtype=np.float64)
    if q_row is not None:
        r = np.maximum(r - np.asarray(q_row, dtype=np.float64), 0.0)
    total = float(r.sum())
    t, margin = residual_sample(r, [], total, w)
    return t, margin, total


def verify_chain_q(n_nodes, draft_tok, logits, inv_temp, q_rows, u, w):
    """Whole rule for one chain (node j's parent is node j - 1) from the target's logits [T, V] and the
    draft's distributions q_rows [T, V] (row i = the distribution node i + 1's token was drawn from).
    Returns (n_acc, out_tok): out_tok = the accepted drafts, then the token drawn where the walk stopped."""
    p, _ = softmax_rows(logits, inv_temp)
    n = int(n_nodes)
    q_rows = np.asarray(q_rows, dtype=np.float64)
    p_tok = np.zeros(n)
    q_tok = np.zeros(n)
    for j in range(1, n):
        p_tok[j] = p[j - 1, draft_tok[j]]
        q_tok[j] = q_rows[j - 1, draft_tok[j]]
    n_acc, _ = accept_chain_q(n, p_tok, q_tok, u)
    stop = n_acc - 1
    rejected = n_acc < n
    t, _, _ = residual_sample_q(p[stop], q_rows[stop] if rejected else None, w)
    return n_acc, [int(draft_tok[j]) for j in range(1, n_acc)] + [t]


def verify_tree_q(parents, n_nodes, draft_tok, logits, inv_temp, q_rows, u, w):
    """Whole rule for one tree whose children were sampled from q_rows[i] (the draft's distribution
    behind node i), from the target's logits [T, V], fp64.  Returns (path, out_tok, walk_margin,
    draw_margin, mass): the accepted root path, the emitted tokens, the smallest relative distance
    |u q - r| / r over the accept tests made (infinity if none or r = 0 cases only), the distance of
    the last draw's target from the nearer end of its CDF interval, and the mass it was normalised by
    (before normalisation: the sum of the positive part carried so far, relative to p_i)."""
    p, _ = softmax_rows(logits, inv_temp)
    q_rows = np.asarray(q_rows, dtype=np.float64)
    u = np.asarray(u, dtype=np.float64)
    n = int(n_nodes)
    cur, path = 0, [0]
    walk_margin = np.inf
    while True:
        r = p[cur].copy()
        q = q_rows[cur]
        nxt = -1
        for c in children_of(parents, n, cur):
            x = int(draft_tok[c])
            if r[x] > 0.0:
                walk_margin = min(walk_margin, abs(u[c] * q[x] - r[x]) / r[x])
            if u[c] * q[x] < r[x]:
                nxt = c
                break
            r = np.maximum(r - q, 0.0)
            tot = r.sum()
            if tot > 0.0:
                r = r / tot
        if nxt < 0:
            total = float(r.sum())
            t, draw_margin = residual_sample(r, [], total, w)
            return path, [int(draft_tok[j]) for j in path[1:]] + [t], walk_margin, draw_margin, total
        cur = nxt
        path.append(cur)
