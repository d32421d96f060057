"""Pins for compaction, and the end-to-end losslessness invariant: draft ->
verify -> accept -> compact must emit exactly what sequential greedy decoding
emits and leave exactly its KV cache behind (Hyper-Bagel Sec. 4.1)."""
import numpy as np

import oracle
from paper_2509_18824_b200 import workloads as wl
from helpers import Tiny, root_path


def test_compaction_moves_exactly_the_accepted_rows():
    p = Tiny(21, B=3, T=8, Hq=2, Hkv=2, D=16, lens=(60, 1, 127))   # 60+: crosses a block boundary
    g = oracle.Geometry.of(p)
    rng = np.random.default_rng(0)
    n_acc = np.array([5, 1, 3], dtype=np.int32)
    path = np.full((3, 8), -1, dtype=np.int32)
    for b in range(3):
        leaf = int(rng.integers(0, 8))
        while len(root_path(p.parents[b], leaf)) != n_acc[b]:
            leaf = int(rng.integers(0, 8))
            if all(len(root_path(p.parents[b], x)) != n_acc[b] for x in range(8)):
                n_acc[b] = 1
        path[b, :n_acc[b]] = root_path(p.parents[b], leaf)
    kc0, vc0 = p.k_cache.copy(), p.v_cache.copy()
    oracle.compact(g, p.k_cache, p.v_cache, p.k_tree, p.v_tree, n_acc, path)
    touched = np.zeros(p.k_cache.shape[:3], dtype=bool)
    for b in range(3):
        for k in range(n_acc[b]):
            t = int(p.len[b]) + k
            blk = p.block_table[b, t // 64]
            for kvh in range(p.Hkv):
                np.testing.assert_array_equal(p.k_cache[blk, kvh, t % 64], p.k_tree[b, path[b, k], kvh])
                np.testing.assert_array_equal(p.v_cache[blk, kvh, t % 64], p.v_tree[b, path[b, k], kvh])
                touched[blk, kvh, t % 64] = True
    assert touched.sum() == n_acc.sum() * p.Hkv
    np.testing.assert_array_equal(p.k_cache[~touched], kc0[~touched])
    np.testing.assert_array_equal(p.v_cache[~touched], vc0[~touched])


class ToyTarget:
    """One attention layer + LM head with fixed random bf16 weights.  Token x
    at any position has q/k/v rows E_q[x], E_k[x], E_v[x] (no positional term,
    so a token's KV does not depend on where it sits); the hidden state is the
    attention output rounded to bf16; next token = argmax(hidden . W^T)."""

    def __init__(self, seed, vocab=12, D=16):
        g = np.random.default_rng(seed)
        self.V, self.D = vocab, D
        mk = lambda k: wl.f32_to_bf16_bits((k * g.standard_normal((vocab, D))).astype(np.float32))
        self.Eq, self.Ek, self.Ev, self.W = mk(1.5), mk(1.0), mk(1.0), mk(1.0)

    def greedy(self, prompt, n_new):
        """Plain sequential decoding with a dense, growing KV list."""
        toks = list(prompt)
        for _ in range(n_new):
            K = wl.bf16_bits_to_f64(self.Ek[toks]); Vv = wl.bf16_bits_to_f64(self.Ev[toks])
            q = wl.bf16_bits_to_f64(self.Eq[toks[-1]])
            s = K @ q / np.sqrt(self.D)
            w = np.exp(s - s.max())
            hid = wl.f32_to_bf16_bits(((w[:, None] * Vv).sum(0) / w.sum()).astype(np.float32))
            logits = wl.bf16_bits_to_f64(self.W) @ wl.bf16_bits_to_f64(hid)
            toks.append(int(np.argmax(logits)))
        return toks


def test_toy_speculative_loop_is_lossless():
    tgt = ToyTarget(4)
    prompt = [3, 1, 4, 1, 5, 9, 2, 6]
    steps, T = 12, 8
    want = tgt.greedy(prompt, 6 * steps)
    rng = np.random.default_rng(7)

    # paged cache for one sequence, blocks deliberately out of order
    nblk = 4
    table = np.array([[2, 0, 3, 1]], dtype=np.int32)
    kc = np.zeros((nblk, 1, 64, tgt.D), dtype=np.uint16); vc = np.zeros_like(kc)
    committed = list(prompt)               # tokens emitted so far; the last one is not cached yet
    for t, x in enumerate(committed[:-1]):
        kc[table[0, t // 64], 0, t % 64] = tgt.Ek[x]; vc[table[0, t // 64], 0, t % 64] = tgt.Ev[x]
    emitted_per_step = []
    for step in range(steps):
        P = len(committed) - 1
        par = np.array([-1] + [int(rng.integers(0, i)) for i in range(1, T)], dtype=np.int32)
        # an arbitrary draft: half the nodes guess the true continuation, the rest are noise
        truth = tgt.greedy(committed, 6)[len(committed):]
        tok = np.zeros(T, dtype=np.int32); tok[0] = committed[-1]
        depth = np.zeros(T, dtype=int)
        for i in range(1, T):
            depth[i] = depth[par[i]] + 1
            tok[i] = truth[depth[i] - 1] if rng.random() < 0.6 else int(rng.integers(0, tgt.V))

        class W_: pass
        g = W_(); g.B, g.T_max, g.Hq, g.Hkv, g.D = 1, T, 1, 1, tgt.D
        g.block_table, g.len = table, np.array([P], np.int32)
        g.n_nodes, g.parents = np.array([T], np.int32), par[None]
        G = oracle.Geometry.of(g)
        q = tgt.Eq[tok][None, :, None, :]; kt = tgt.Ek[tok][None, :, None, :]; vt = tgt.Ev[tok][None, :, None, :]
        out, _ = oracle.attention(G, kc, vc, q, kt, vt, 1.0 / np.sqrt(tgt.D))
        hidden = wl.f32_to_bf16_bits(out[0, :, 0, :].astype(np.float32))
        am, _, _ = oracle.lmhead(hidden, tgt.W)
        n_acc, path, out_tok, new_len = oracle.accept(G, tok[None], am[None])
        oracle.compact(G, kc, vc, kt, vt, n_acc, path)
        committed += [int(x) for x in out_tok[0, :n_acc[0]]]
        emitted_per_step.append(int(n_acc[0]))
        assert new_len[0] == len(committed) - 1
    assert committed == want[:len(committed)]
    assert max(emitted_per_step) > 1            # speculation actually accepted something
    # cache content equals the dense cache of sequential decoding
    for t, x in enumerate(committed[:-1]):
        np.testing.assert_array_equal(kc[table[0, t // 64], 0, t % 64], tgt.Ek[x])
        np.testing.assert_array_equal(vc[table[0, t // 64], 0, t % 64], tgt.Ev[x])
