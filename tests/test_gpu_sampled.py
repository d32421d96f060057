"""GPU parity of verification at a sampling temperature: sd_lmhead_stats, sd_accept_tree_sampled and
the fused sd_lmhead_accept_sampled_compact against oracle/sampling.py on the same seeded inputs
(uniform numbers are inputs on both sides)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import sampling as smp
from paper_2509_18824_b200 import binding as sd
from paper_2509_18824_b200 import workloads as wl
from paper_2509_18824_b200.step import VerifyStep, to_device

pytestmark = pytest.mark.gpu

CLOSE = 2e-5          # a CDF crossing nearer than this may fall either way in fp32
WALK_CLOSE = 2e-4     # a comparison u * R < p nearer than this may fall either way: the kernel's p (fp32 dot product
                      # of 3584 terms, ex2.approx) is within 1e-4 relative of the fp64 value


def run_stats(hidden, W, inv_temp):
    h, Wd = to_device(hidden), to_device(W)
    M, V = hidden.shape[0], W.shape[0]
    am = torch.full((M,), -5, dtype=torch.int32, device="cuda")
    mx = torch.zeros(M, dtype=torch.float32, device="cuda")
    lse = torch.zeros(M, dtype=torch.float32, device="cuda")
    ws = torch.empty(sd.sd_workspace_bytes(None, M, V), dtype=torch.uint8, device="cuda")
    st = sd.new_status()
    sd.sd_lmhead_stats(h, Wd, inv_temp, am, mx, lse, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return am.cpu().numpy(), mx.cpu().numpy(), lse.cpu().numpy()


@pytest.mark.parametrize("M,Hd,V,inv_temp", [(5, 128, 1000, 1.0), (61, 192, 129, 0.5), (130, 64, 4099, 2.0),
                                             (600, 128, 2500, 1.0), (3, 64, 100, 1.0), (2, 64, 1, 1.0)])
def test_lmhead_stats_small_shapes(M, Hd, V, inv_temp):
    g = np.random.default_rng(M + V)
    h = wl.f32_to_bf16_bits((g.standard_normal((M, Hd)) * 2).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, Hd)) / np.sqrt(Hd)).astype(np.float32))
    am, mx, lse = run_stats(h, W, inv_temp)
    lg = oracle.logits(h, W)
    _, rlse = smp.softmax_rows(lg, inv_temp)
    np.testing.assert_allclose(lse, rlse, rtol=0, atol=3e-4)
    ram, t1, t2 = oracle.lmhead(h, W)
    ok = (t1 - t2) > 1e-3
    np.testing.assert_array_equal(am[ok], ram[ok])


def test_lmhead_stats_full_vocabulary():
    for gain, inv_temp in ((1.0, 1.0), (30.0, 1.0), (30.0, 0.25)):
        w = wl.make("c2", attention=False, hidden_gain=gain)
        am, mx, lse = run_stats(w.hidden, w.W, inv_temp)
        lg = oracle.logits(w.hidden, w.W)
        _, rlse = smp.softmax_rows(lg, inv_temp)
        np.testing.assert_allclose(lse, rlse, rtol=0, atol=5e-4)


def good_drafts(w, lg, seed):
    """Children of every node get the target's most likely tokens at that node (a good drafter),
    in shuffled order, so that some are accepted; siblings are distinct by construction."""
    g = np.random.default_rng(seed)
    tok = np.zeros((w.B, w.T_max), dtype=np.int32)
    for b in range(w.B):
        n = int(w.n_nodes[b])
        for i in range(n):
            kids = smp.children_of(w.parents[b], n, i)
            if kids:
                top = np.argsort(-lg[b * w.T_max + i])[:len(kids)]
                tok[b, kids] = g.permutation(top)
    return tok


def run_sampled(w, tok, inv_temp, u, wv, groups=True):
    """groups=True: the LM-head pass also leaves its per-group statistics and the last token is drawn
    from them; False: the stop rows go through the LM head a second time."""
    bt = sd.Batch.of(w)
    st = sd.new_status()
    h, Wd = to_device(w.hidden), to_device(w.W)
    M, V = w.hidden.shape[0], w.W.shape[0]
    B, T = w.B, w.T_max
    ws = torch.zeros(sd.sd_workspace_bytes(bt, M, V), dtype=torch.uint8, device="cuda")
    lse = torch.zeros(M, dtype=torch.float32, device="cuda")
    gs = torch.zeros(sd.group_stats_shape(M, V), dtype=torch.float32, device="cuda") if groups else None
    sd.sd_lmhead_stats(h, Wd, inv_temp, None, None, lse, ws, st, group_stats=gs)
    n_acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    path = torch.full((B, T), -9, dtype=torch.int32, device="cuda")
    out_tok = torch.full((B, T), -9, dtype=torch.int32, device="cuda")
    new_len = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    sd.sd_accept_tree_sampled(bt, h, Wd, inv_temp, lse, to_device(tok), to_device(u), to_device(wv),
                              n_acc, path, out_tok, new_len, ws, st, group_stats=gs)
    torch.cuda.synchronize()
    return (n_acc.cpu().numpy(), path.cpu().numpy(), out_tok.cpu().numpy(), new_len.cpu().numpy(), int(st.item()))


@pytest.mark.parametrize("cfg,over,inv_temp", [
    ("c1", dict(), 1.0), ("c1", dict(), 3.0),
    ("c5", dict(L=1, V=8192, Hd=512, prefix=100), 5.0),
    ("c4", dict(L=1, V=4096, Hd=256, prefix_range=(40, 300)), 3.0),          # 16 sequences: two residual passes
    ("chain11", dict(L=1, V=3000, Hd=128, prefix=70), 2.5),
    ("c1", dict(V=96, Hd=64), 1.5),                                          # vocabulary below one 128-row tile
])
@pytest.mark.parametrize("groups", [True, False])
def test_sampled_acceptance_against_the_reference(cfg, over, inv_temp, groups):
    w = wl.make(cfg, attention=False, hidden_gain=24.0, **over)
    B, T, V = w.B, w.T_max, w.W.shape[0]
    lg = oracle.logits(w.hidden, w.W)
    tok = good_drafts(w, lg, 1)
    g = np.random.default_rng(7)
    p64, _ = smp.softmax_rows(lg, inv_temp)
    accepted_total = 0
    for rep in range(3 if B > 1 else 25):
        u = g.random((B, T)).astype(np.float32)
        wv = g.random(B).astype(np.float32)
        n_acc, path, out_tok, new_len, status = run_sampled(w, tok, inv_temp, u, wv, groups)
        assert status == 0
        close_calls = 0
        for b in range(B):
            n = int(w.n_nodes[b])
            par = w.parents[b]
            # the walk against the fp64 definition: same path unless one of its comparisons was a close call
            pc64 = np.zeros(T)
            for j in range(1, n):
                pc64[j] = p64[b * T + par[j], tok[b, j]]
            pth64, R64, walk_margin = smp.accept_walk(par, n, tok[b], pc64, u[b].astype(np.float64))
            assert (path[b, n_acc[b]:] == -1).all()
            assert new_len[b] == w.len[b] + n_acc[b]
            got_path = [int(x) for x in path[b, :n_acc[b]]]
            assert list(out_tok[b, :n_acc[b] - 1]) == [int(tok[b, j]) for j in got_path[1:]]
            if got_path != pth64:
                assert walk_margin <= WALK_CLOSE, (b, got_path, pth64, walk_margin)
                close_calls += 1
                continue
            # the drawn token: inverse CDF over the stop row without its drafted children
            last = pth64[-1]
            excl = [int(tok[b, c]) for c in smp.children_of(par, n, last)]
            t_ref, margin = smp.residual_sample(p64[b * T + last], excl, R64, float(wv[b]))
            got = int(out_tok[b, n_acc[b] - 1])
            assert got not in excl and 0 <= got < V
            if got != t_ref:
                assert margin <= CLOSE * max(R64, 1e-3), (b, got, t_ref, margin)
                close_calls += 1
            accepted_total += n_acc[b] - 1
        assert close_calls <= max(1, B // 8), close_calls
    assert accepted_total > 0          # the drafts were good enough for the walk to move at all


def test_sampled_zero_temperature_equals_greedy_acceptance():
    """Large inverse temperature: the sampled rule must reproduce sd_accept_tree's outputs exactly
    (path, accepted drafts, and the bonus token = arg-max at the last accepted node)."""
    w = wl.make("c5", attention=False, hidden_gain=40.0, L=1, V=8192, Hd=512, prefix=100)
    ram, t1, t2 = oracle.lmhead(w.hidden, w.W)
    assert (t1 - t2).min() > 2e-3
    wl.plant(w, ram.reshape(w.B, w.T_max))
    ref = oracle.accept(oracle.Geometry.of(w), w.draft_tok, ram.reshape(w.B, w.T_max))
    g = np.random.default_rng(3)
    u = (g.random((w.B, w.T_max)) * 0.98 + 0.01).astype(np.float32)
    wv = (g.random(w.B) * 0.98 + 0.01).astype(np.float32)
    n_acc, path, out_tok, new_len, status = run_sampled(w, w.draft_tok, 4000.0, u, wv)
    assert status == 0
    for got, want in zip((n_acc, path, out_tok, new_len), ref):
        np.testing.assert_array_equal(got, want)


def test_sampled_bad_inputs_are_reported():
    w = wl.make("c1", attention=False, hidden_gain=16.0)
    tok = np.zeros((1, 8), dtype=np.int32); tok[0, 3] = 5000                 # outside the vocabulary
    u = np.full((1, 8), 0.5, np.float32); wv = np.full(1, 0.5, np.float32)
    *_, status = run_sampled(w, tok, 1.0, u, wv)
    assert status == sd.SD_ERR_BOUNDS
    dup = np.array([[0, 7, 7, 1, 2, 3, 4, 5]], dtype=np.int32)              # nodes 1 and 2 are siblings with one token
    *_, status = run_sampled(w, dup, 1.0, np.full((1, 8), 0.999, np.float32), wv)
    assert status == sd.SD_ERR_INVALID_ARG
    w.parents = w.parents.copy(); w.parents[0, 3] = 6
    *_, status = run_sampled(w, np.arange(8, dtype=np.int32)[None], 1.0, u, wv)
    assert status == sd.SD_ERR_INVALID_TREE


@pytest.mark.parametrize("groups", [True, False])
def test_sampled_full_size_c5(groups):
    """Vocabulary 152064, 8 x 60-node trees: the walk and the drawn tokens against the fp64 rule on
    fp64 logits; a differing decision must be a close call of the fp64 walk, and at most one may occur."""
    w = wl.make("c5", attention=False, hidden_gain=40.0)
    B, T, V = w.B, w.T_max, w.V
    ram, t1, t2 = oracle.lmhead(w.hidden, w.W)                   # good drafts: children get the arg-max first
    g = np.random.default_rng(11)
    tok = g.integers(0, V, size=(B, T)).astype(np.int32)
    for b in range(B):
        for i in range(int(w.n_nodes[b])):
            kids = smp.children_of(w.parents[b], int(w.n_nodes[b]), i)
            if kids:
                tok[b, kids[0]] = ram[b * T + i]
                for k, c in enumerate(kids[1:]):
                    tok[b, c] = (ram[b * T + i] + 1 + k) % V
    inv_temp = 6.0
    u = g.random((B, T)).astype(np.float32)
    wv = g.random(B).astype(np.float32)
    n_acc, path, out_tok, new_len, status = run_sampled(w, tok, inv_temp, u, wv, groups)
    assert status == 0
    # fp64 probabilities of the rows the rule may look at: every parent (child probabilities) and every
    # node a walk stopped at (the residual draw)
    rows = sorted({b * T + int(w.parents[b][j]) for b in range(B) for j in range(1, int(w.n_nodes[b]))}
                  | {b * T + int(path[b, k]) for b in range(B) for k in range(n_acc[b])})
    p64, _ = smp.softmax_rows(oracle.logits(w.hidden[rows], w.W), inv_temp)
    row_of = {r: i for i, r in enumerate(rows)}
    moved = 0
    close_calls = 0
    for b in range(B):
        n, par = int(w.n_nodes[b]), w.parents[b]
        pc64 = np.zeros(T)
        for j in range(1, n):
            pc64[j] = p64[row_of[b * T + int(par[j])], tok[b, j]]
        pth64, R64, walk_margin = smp.accept_walk(par, n, tok[b], pc64, u[b].astype(np.float64))
        got_path = [int(x) for x in path[b, :n_acc[b]]]
        if got_path != pth64:
            assert walk_margin <= WALK_CLOSE, (b, got_path, pth64, walk_margin)
            close_calls += 1
            continue
        last = pth64[-1]
        excl = [int(tok[b, c]) for c in smp.children_of(par, n, last)]
        t_ref, margin = smp.residual_sample(p64[row_of[b * T + last]], excl, float(R64), float(wv[b]))
        got = int(out_tok[b, n_acc[b] - 1])
        assert got not in excl
        assert got == t_ref or margin <= CLOSE, (b, got, t_ref, margin)
        moved += n_acc[b] - 1
    assert moved > 0 and close_calls <= 1


def test_sampled_gpu_output_frequencies_follow_the_target_distribution():
    """Losslessness measured on the GPU path itself: 16 identical sequences (root + 3 drafted children)
    verified with fresh uniforms 300 times; the FIRST emitted token of every sequence must be
    distributed as the target's p at the root (5 sigma), whichever route produced it (an accepted
    child or the residual draw)."""
    B, T, Hd, V, inv_temp, reps = 16, 4, 64, 16, 1.2, 300
    g = np.random.default_rng(21)
    bf = lambda a: wl.f32_to_bf16_bits(a.astype(np.float32))
    hid_one = bf(g.standard_normal((T, Hd)))
    W = bf(g.standard_normal((V, Hd)) * 0.25)

    class Geo:
        pass
    w = Geo()
    w.B, w.T_max, w.Hq, w.Hkv, w.D = B, T, 4, 1, 128
    w.block_table = np.arange(B, dtype=np.int32).reshape(B, 1)
    w.len = np.full(B, 5, np.int32)
    w.n_nodes = np.full(B, T, np.int32)
    w.parents = np.tile(np.array([-1, 0, 0, 0], np.int32), (B, 1))
    w.hidden = np.tile(hid_one, (B, 1))
    w.W = W
    lg = oracle.logits(hid_one, W)
    p, _ = smp.softmax_rows(lg, inv_temp)
    order = np.argsort(-p[0])
    tok = np.tile(np.array([0, order[1], order[0], order[3]], np.int32), (B, 1))   # children: 2nd, 1st and 4th most likely
    counts = np.zeros(V)
    for rep in range(reps):
        u = g.random((B, T)).astype(np.float32)
        wv = g.random(B).astype(np.float32)
        n_acc, path, out_tok, new_len, status = run_sampled(w, tok, inv_temp, u, wv)
        assert status == 0
        np.add.at(counts, out_tok[:, 0], 1)
    n = B * reps
    sigma = np.sqrt(n * p[0] * (1 - p[0]))
    assert (np.abs(counts - n * p[0]) <= 5 * sigma + 1).all(), (counts / n, p[0])


def decisive_uniforms(w, tok, p64_of_row, g, floor=20 * WALK_CLOSE):
    """Uniform numbers under which no comparison of the fp64 walk is a close call (redrawn per
    sequence until the smallest |u * R - p| on its walk exceeds `floor`), with the fp64 walk's results."""
    B, T = w.B, w.T_max
    u = np.zeros((B, T), np.float32)
    n_acc = np.zeros(B, np.int32)
    path = np.full((B, T), -1, np.int32)
    stop_R = np.zeros(B)
    for b in range(B):
        n, par = int(w.n_nodes[b]), w.parents[b]
        pc64 = np.zeros(T)
        for j in range(1, n):
            pc64[j] = p64_of_row(b * T + int(par[j]))[tok[b, j]]
        for _ in range(200):
            u[b] = g.random(T).astype(np.float32)
            pth, R, margin = smp.accept_walk(par, n, tok[b], pc64, u[b].astype(np.float64))
            if margin > floor:
                break
        else:
            raise AssertionError("no decisive uniforms found")
        n_acc[b] = len(pth)
        path[b, :len(pth)] = pth
        stop_R[b] = R
    return u, n_acc, path, stop_R


def step_outputs(vs):
    return dict(lse=vs.lse_rows.cpu().numpy(), n_acc=vs.n_acc.cpu().numpy(), path=vs.path.cpu().numpy(),
                out_tok=vs.out_tok.cpu().numpy(), new_len=vs.new_len.cpu().numpy(),
                k=[x.cpu().numpy() for x in vs.k_cache], v=[x.cpu().numpy() for x in vs.v_cache])


@pytest.mark.parametrize("cfg,over,inv_temp", [
    ("c1", dict(L=1), 2.0),
    ("c2", dict(L=3, V=5000, Hd=256), 3.0),
    ("c5", dict(L=9, V=8192, Hd=512, prefix=200), 5.0),                      # nine layers over eight CTAs
    ("c4", dict(L=2, V=4096, Hd=256, prefix_range=(40, 300)), 3.0),          # 960 rows: the internal fall-back
    ("chain11", dict(L=4, V=3000, Hd=128, prefix=70), 2.5),
])
def test_fused_sampled_tail_equals_the_separate_calls_and_the_reference(cfg, over, inv_temp):
    """sd_lmhead_accept_sampled_compact against sd_lmhead_stats + sd_accept_tree_sampled +
    sd_compact_kv: every output and every cache byte identical.  Against the checker: with uniforms
    under which the fp64 walk has no close call the path must be the fp64 path, the drawn token the
    fp64 token (or a close call of the CDF), and the caches those the checker's compaction leaves."""
    w = wl.make(cfg, hidden_gain=24.0, **over)
    B, T, V, L = w.B, w.T_max, w.W.shape[0], w.L
    lg = oracle.logits(w.hidden, w.W)
    p64, lse64 = smp.softmax_rows(lg, inv_temp)
    tok = good_drafts(w, lg, 5)
    w.draft_tok = tok
    g = np.random.default_rng(17)
    u, ref_n_acc, ref_path, stop_R = decisive_uniforms(w, tok, lambda r: p64[r], g)
    wv = g.random(B).astype(np.float32)
    res = []
    for fused in (False, True):
        vs = VerifyStep(w)
        vs.tail_sampled(inv_temp, to_device(u), to_device(wv), fused=fused)
        torch.cuda.synchronize()
        vs.check_status()
        res.append(step_outputs(vs))
    for key in ("lse", "n_acc", "path", "out_tok", "new_len"):
        np.testing.assert_array_equal(res[0][key], res[1][key], err_msg=key)
    for l in range(L):
        np.testing.assert_array_equal(res[0]["k"][l], res[1]["k"][l])
        np.testing.assert_array_equal(res[0]["v"][l], res[1]["v"][l])
    got = res[1]
    np.testing.assert_allclose(got["lse"], lse64, rtol=0, atol=5e-4)
    np.testing.assert_array_equal(got["n_acc"], ref_n_acc)
    np.testing.assert_array_equal(got["path"], ref_path)
    np.testing.assert_array_equal(got["new_len"], w.len + ref_n_acc)
    close_calls = 0
    for b in range(B):
        n, par, na = int(w.n_nodes[b]), w.parents[b], int(ref_n_acc[b])
        assert list(got["out_tok"][b, :na - 1]) == [int(tok[b, j]) for j in ref_path[b, 1:na]]
        assert (got["out_tok"][b, na:] == -1).all()
        last = int(ref_path[b, na - 1])
        excl = [int(tok[b, c]) for c in smp.children_of(par, n, last)]
        t_ref, margin = smp.residual_sample(p64[b * T + last], excl, float(stop_R[b]), float(wv[b]))
        t_got = int(got["out_tok"][b, na - 1])
        assert t_got not in excl and 0 <= t_got < V
        if t_got != t_ref:
            assert margin <= CLOSE * max(float(stop_R[b]), 1e-3), (b, t_got, t_ref, margin)
            close_calls += 1
    assert close_calls <= max(1, B // 8)
    assert B == 1 or (ref_n_acc > 1).any()                                   # some walk moved
    G = oracle.Geometry.of(w)
    for l in range(L):
        rk, rv = w.k_cache[l].copy(), w.v_cache[l].copy()
        oracle.compact(G, rk, rv, w.k_tree[l], w.v_tree[l], ref_n_acc, ref_path)
        np.testing.assert_array_equal(got["k"][l].view(np.uint16), rk)
        np.testing.assert_array_equal(got["v"][l].view(np.uint16), rv)


def test_fused_sampled_tail_bad_tree_touches_no_cache():
    w = wl.make("c1", hidden_gain=16.0)
    w.parents = w.parents.copy(); w.parents[0, 3] = 5
    vs = VerifyStep(w)
    before_k, before_v = vs.k_cache[0].clone(), vs.v_cache[0].clone()
    vs.status.zero_()
    vs.tail_sampled(1.0, to_device(np.full((1, 8), 0.5, np.float32)), to_device(np.full(1, 0.5, np.float32)))
    torch.cuda.synchronize()
    assert int(vs.status.item()) == sd.SD_ERR_INVALID_TREE
    assert int(vs.n_acc[0].item()) == 0
    assert torch.equal(before_k, vs.k_cache[0]) and torch.equal(before_v, vs.v_cache[0])


def test_fused_sampled_tail_full_vocabulary():
    """Batch 8, 60-node trees, vocabulary 152064, four layers: the fused call against the fp64 rule on
    the rows the rule looks at, and against the checker's compaction."""
    w = wl.make("c5", hidden_gain=40.0, L=4, prefix=300)
    B, T, V, L = w.B, w.T_max, w.V, w.L
    ram, t1, t2 = oracle.lmhead(w.hidden, w.W)
    g = np.random.default_rng(12)
    tok = g.integers(0, V, size=(B, T)).astype(np.int32)
    for b in range(B):
        for i in range(int(w.n_nodes[b])):
            kids = smp.children_of(w.parents[b], int(w.n_nodes[b]), i)
            if kids:
                tok[b, kids[0]] = ram[b * T + i]
                for k, c in enumerate(kids[1:]):
                    tok[b, c] = (ram[b * T + i] + 1 + k) % V
    w.draft_tok = tok
    inv_temp = 6.0
    rows = sorted({b * T + int(w.parents[b][j]) for b in range(B) for j in range(1, int(w.n_nodes[b]))}
                  | {b * T + j for b in range(B) for j in range(int(w.n_nodes[b]))})
    p64, lse64 = smp.softmax_rows(oracle.logits(w.hidden[rows], w.W), inv_temp)
    row_of = {r: i for i, r in enumerate(rows)}
    u, ref_n_acc, ref_path, stop_R = decisive_uniforms(w, tok, lambda r: p64[row_of[r]], g)
    wv = g.random(B).astype(np.float32)
    vs = VerifyStep(w)
    vs.tail_sampled(inv_temp, to_device(u), to_device(wv))
    torch.cuda.synchronize()
    vs.check_status()
    got = step_outputs(vs)
    np.testing.assert_allclose(got["lse"][rows], lse64, rtol=0, atol=5e-4)
    np.testing.assert_array_equal(got["n_acc"], ref_n_acc)
    np.testing.assert_array_equal(got["path"], ref_path)
    for b in range(B):
        n, par, na = int(w.n_nodes[b]), w.parents[b], int(ref_n_acc[b])
        last = int(ref_path[b, na - 1])
        excl = [int(tok[b, c]) for c in smp.children_of(par, n, last)]
        t_ref, margin = smp.residual_sample(p64[row_of[b * T + last]], excl, float(stop_R[b]), float(wv[b]))
        t_got = int(got["out_tok"][b, na - 1])
        assert t_got not in excl
        assert t_got == t_ref or margin <= CLOSE, (b, t_got, t_ref, margin)
    assert (ref_n_acc > 1).any()
    G = oracle.Geometry.of(w)
    for l in range(L):
        rk, rv = w.k_cache[l].copy(), w.v_cache[l].copy()
        oracle.compact(G, rk, rv, w.k_tree[l], w.v_tree[l], ref_n_acc, ref_path)
        np.testing.assert_array_equal(got["k"][l].view(np.uint16), rk)
        np.testing.assert_array_equal(got["v"][l].view(np.uint16), rv)


# ---------------------------------------------------------------------------------------------------
# chains drafted by sampling from the draft model's own distributions: sd_accept_chain_sampled
# ---------------------------------------------------------------------------------------------------
def drafted_chain(w, lg, inv_temp, spread, seed):
    """A drafter close to, but not, the target: q[b][i] = softmax of the target's logits behind node i
    plus noise (float32, the array both sides read); node i + 1's token is drawn from it."""
    g = np.random.default_rng(seed)
    B, T, V = w.B, w.T_max, lg.shape[1]
    q64, _ = smp.softmax_rows(lg + g.standard_normal(lg.shape) * spread, inv_temp * 0.8)
    q = np.ascontiguousarray(q64.astype(np.float32).reshape(B, T, V))
    tok = np.zeros((B, T), dtype=np.int32)
    for b in range(B):
        for j in range(1, int(w.n_nodes[b])):
            cdf = np.cumsum(q[b, j - 1].astype(np.float64))
            tok[b, j] = min(int(np.searchsorted(cdf, g.random() * cdf[-1], side="right")), V - 1)
    q_tok = np.zeros((B, T), dtype=np.float32)
    for b in range(B):
        for j in range(1, int(w.n_nodes[b])):
            q_tok[b, j] = q[b, j - 1, tok[b, j]]
    return q, tok, q_tok


def run_chain_q(w, tok, q, q_tok, inv_temp, u, wv, keep_logits=False):
    """keep_logits: the LM-head pass keeps its raw logits and the draw uses them; otherwise the stop rows
    go through the LM head a second time."""
    bt = sd.Batch.of(w)
    st = sd.new_status()
    h, Wd = to_device(w.hidden), to_device(w.W)
    M, V = w.hidden.shape[0], w.W.shape[0]
    B, T = w.B, w.T_max
    ws = torch.zeros(sd.sd_workspace_bytes(bt, M, V), dtype=torch.uint8, device="cuda")
    lse = torch.zeros(M, dtype=torch.float32, device="cuda")
    logits = None
    if keep_logits:
        logits = torch.full((M, V), float("nan"), dtype=torch.float32, device="cuda")
        sd.sd_lmhead_stats_logits(h, Wd, inv_temp, None, None, lse, logits, ws, st)
    else:
        sd.sd_lmhead_stats(h, Wd, inv_temp, None, None, lse, ws, st)
    n_acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    path = torch.full((B, T), -9, dtype=torch.int32, device="cuda")
    out_tok = torch.full((B, T), -9, dtype=torch.int32, device="cuda")
    new_len = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    sd.sd_accept_chain_sampled(bt, h, Wd, inv_temp, lse, to_device(tok), to_device(q_tok), to_device(q),
                               to_device(u), to_device(wv), n_acc, path, out_tok, new_len, ws, st, logits=logits)
    torch.cuda.synchronize()
    return (n_acc.cpu().numpy(), path.cpu().numpy(), out_tok.cpu().numpy(), new_len.cpu().numpy(), int(st.item()))


def decisive_chain_inputs(w, tok, q, p64_of_row, g, floor=20 * WALK_CLOSE, floor_w=2e-3):
    """Uniforms under which neither an accept test (u * q against p, the two further apart than `floor`
    times p: the kernel's p is within 1e-4 relative of the fp64 value) nor the last token's CDF crossing
    of the fp64 rule is a close call, with the fp64 rule's results (n_acc and the emitted tokens)."""
    B, T = w.B, w.T_max
    u = np.zeros((B, T), np.float32)
    wv = np.zeros(B, np.float32)
    ref_n, ref_out = np.zeros(B, np.int32), np.full((B, T), -1, np.int32)
    for b in range(B):
        n = int(w.n_nodes[b])
        p_tok, q_tok = np.zeros(n), np.zeros(n)
        for j in range(1, n):
            p_tok[j] = p64_of_row(b * T + j - 1)[tok[b, j]]
            q_tok[j] = q[b, j - 1, tok[b, j]]
        for _ in range(400):
            u[b] = g.random(T).astype(np.float32)
            na, _ = smp.accept_chain_q(n, p_tok, q_tok, u[b].astype(np.float64))
            looked_at = range(1, min(na + 1, n))             # the accepted nodes and the rejected one
            if all(abs(u[b, j] * q_tok[j] - p_tok[j]) > floor * p_tok[j] for j in looked_at):
                break
        else:
            raise AssertionError("no decisive uniforms found")
        stop = na - 1
        for _ in range(400):
            wv[b] = np.float32(g.random())
            t, margin, total = smp.residual_sample_q(p64_of_row(b * T + stop), q[b, stop] if na < n else None, float(wv[b]))
            if margin > floor_w * total:
                break
        else:
            raise AssertionError("no decisive w found")
        ref_n[b] = na
        ref_out[b, :na - 1] = tok[b, 1:na]
        ref_out[b, na - 1] = t
    return u, wv, ref_n, ref_out


@pytest.mark.parametrize("cfg,over,inv_temp,spread", [
    ("chain11", dict(L=1, V=3000, Hd=128, prefix=70), 2.5, 0.6),
    ("chain11", dict(L=1, V=3000, Hd=128, prefix=70), 2.5, 0.05),            # a drafter very close to the target
    ("chain11", dict(L=1, V=96, Hd=64, prefix=70), 1.5, 1.0),                # vocabulary below one 128-row tile
    ("chain11", dict(L=1, V=8192, Hd=512, prefix=100, B=16), 4.0, 0.4),      # 16 sequences
])
@pytest.mark.parametrize("keep_logits", [False, True])
def test_chain_acceptance_with_a_draft_distribution_against_the_reference(cfg, over, inv_temp, spread, keep_logits):
    w = wl.make(cfg, attention=False, hidden_gain=24.0, **over)
    B, T, V = w.B, w.T_max, w.W.shape[0]
    lg = oracle.logits(w.hidden, w.W)
    p64, _ = smp.softmax_rows(lg, inv_temp)
    q, tok, q_tok = drafted_chain(w, lg, inv_temp, spread, 3)
    g = np.random.default_rng(8)
    moved = rejected = 0
    for rep in range(3):
        u, wv, ref_n, ref_out = decisive_chain_inputs(w, tok, q, lambda r: p64[r], g)
        n_acc, path, out_tok, new_len, status = run_chain_q(w, tok, q, q_tok, inv_temp, u, wv, keep_logits)
        assert status == 0
        np.testing.assert_array_equal(n_acc, ref_n)
        np.testing.assert_array_equal(out_tok, ref_out)
        np.testing.assert_array_equal(new_len, w.len + ref_n)
        for b in range(B):
            assert list(path[b, :ref_n[b]]) == list(range(ref_n[b])) and (path[b, ref_n[b]:] == -1).all()
        moved += int((ref_n > 1).sum())
        rejected += int((ref_n < w.n_nodes).sum())
    assert moved > 0 and rejected > 0                       # both branches of the rule were exercised


def test_chain_acceptance_draft_equal_to_the_target_accepts_everything():
    w = wl.make("chain11", attention=False, hidden_gain=24.0, L=1, V=3000, Hd=128, prefix=70)
    B, T, V = w.B, w.T_max, w.W.shape[0]
    inv_temp = 2.0
    lg = oracle.logits(w.hidden, w.W)
    p64, _ = smp.softmax_rows(lg, inv_temp)
    q = np.ascontiguousarray(p64.astype(np.float32).reshape(B, T, V))
    g = np.random.default_rng(4)
    tok = np.zeros((B, T), np.int32)
    for b in range(B):
        for j in range(1, T):
            tok[b, j] = np.argsort(-p64[b * T + j - 1])[g.integers(0, 3)]       # a likely token (any token works)
    q_tok = np.zeros((B, T), np.float32)
    for b in range(B):
        q_tok[b, 1:] = q[b, np.arange(T - 1), tok[b, 1:]]
    u = (g.random((B, T)) * 0.98).astype(np.float32)
    wv = g.random(B).astype(np.float32)
    n_acc, path, out_tok, new_len, status = run_chain_q(w, tok, q, q_tok, inv_temp, u, wv, keep_logits=True)
    assert status == 0
    np.testing.assert_array_equal(n_acc, w.n_nodes)
    for b in range(B):
        n = int(w.n_nodes[b])
        assert list(out_tok[b, :n - 1]) == list(tok[b, 1:n])
        t_ref, margin, total = smp.residual_sample_q(p64[b * T + n - 1], None, float(wv[b]))
        assert out_tok[b, n - 1] == t_ref or margin <= CLOSE


def test_chain_acceptance_refuses_trees_that_branch():
    w = wl.make("c1", attention=False, hidden_gain=16.0)                    # an 8-node tree with branches
    V = w.W.shape[0]
    q = np.full((1, 8, V), 1.0 / V, np.float32)
    tok = np.arange(8, dtype=np.int32)[None]
    half = np.full((1, 8), 0.5, np.float32)
    n_acc, *_, status = run_chain_q(w, tok, q, np.full((1, 8), 1.0 / V, np.float32), 1.0, half, np.full(1, 0.5, np.float32))
    assert status == sd.SD_ERR_UNSUPPORTED and n_acc[0] == 0


def test_kept_logits_are_the_logits():
    """sd_lmhead_stats_logits: every stored logit against the fp64 product (rows beyond one 32-column
    chunk, a vocabulary with a ragged last tile), lse as without the logits."""
    g = np.random.default_rng(31)
    M, Hd, V = 45, 192, 1000
    h = wl.f32_to_bf16_bits((g.standard_normal((M, Hd)) * 2).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, Hd)) / np.sqrt(Hd)).astype(np.float32))
    hd, Wd = to_device(h), to_device(W)
    lse = torch.zeros(M, dtype=torch.float32, device="cuda")
    logits = torch.full((M, V), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(sd.sd_workspace_bytes(None, M, V), dtype=torch.uint8, device="cuda")
    st = sd.new_status()
    sd.sd_lmhead_stats_logits(hd, Wd, 1.3, None, None, lse, logits, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    lg = oracle.logits(h, W)
    np.testing.assert_allclose(logits.cpu().numpy(), lg, rtol=0, atol=2e-5 * np.abs(lg).max())
    np.testing.assert_allclose(lse.cpu().numpy(), smp.softmax_rows(lg, 1.3)[1], rtol=0, atol=3e-4)


@pytest.mark.parametrize("keep_logits", [False, True])
def test_chain_acceptance_full_vocabulary(keep_logits):
    """Root + 10 drafts, 8 sequences, vocabulary 152064, draft distributions of the full width."""
    w = wl.make("chain11", attention=False, hidden_gain=40.0)
    B, T, V = w.B, w.T_max, w.V
    inv_temp = 6.0
    lg = oracle.logits(w.hidden, w.W)
    p64, _ = smp.softmax_rows(lg, inv_temp)
    q, tok, q_tok = drafted_chain(w, lg, inv_temp, 0.15, 9)
    g = np.random.default_rng(10)
    u, wv, ref_n, ref_out = decisive_chain_inputs(w, tok, q, lambda r: p64[r], g)
    n_acc, path, out_tok, new_len, status = run_chain_q(w, tok, q, q_tok, inv_temp, u, wv, keep_logits)
    assert status == 0
    np.testing.assert_array_equal(n_acc, ref_n)
    np.testing.assert_array_equal(out_tok, ref_out)
    assert (ref_n > 1).any() and (ref_n < w.n_nodes).any()


def test_chain_acceptance_gpu_output_frequencies_follow_the_target_distribution():
    """Losslessness of the general rule measured on the GPU path: 16 identical chains (root + 2 drafts)
    whose drafts are drawn afresh from q 300 times; the first emitted token of every sequence must be
    distributed as the target's p at the root (5 sigma), whether it was an accepted draft or a redraw."""
    B, T, Hd, V, inv_temp, reps = 16, 3, 64, 16, 1.2, 300
    g = np.random.default_rng(22)
    bf = lambda a: wl.f32_to_bf16_bits(a.astype(np.float32))
    hid_one = bf(g.standard_normal((T, Hd)))
    W = bf(g.standard_normal((V, Hd)) * 0.25)

    class Geo:
        pass
    w = Geo()
    w.B, w.T_max, w.Hq, w.Hkv, w.D = B, T, 4, 1, 128
    w.block_table = np.arange(B, dtype=np.int32).reshape(B, 1)
    w.len = np.full(B, 5, np.int32)
    w.n_nodes = np.full(B, T, np.int32)
    w.parents = np.tile(np.array([-1, 0, 1], np.int32), (B, 1))
    w.hidden = np.tile(hid_one, (B, 1))
    w.W = W
    lg = oracle.logits(hid_one, W)
    p, _ = smp.softmax_rows(lg, inv_temp)
    q_one, _ = smp.softmax_rows(lg + g.standard_normal(lg.shape) * 0.8, 1.0)
    q = np.ascontiguousarray(np.tile(q_one.astype(np.float32)[None], (B, 1, 1)))
    cdf = np.cumsum(q_one.astype(np.float32).astype(np.float64), axis=1)
    counts = np.zeros(V)
    for rep in range(reps):
        tok = np.zeros((B, T), np.int32)
        q_tok = np.zeros((B, T), np.float32)
        for b in range(B):
            for j in range(1, T):
                tok[b, j] = min(int(np.searchsorted(cdf[j - 1], g.random() * cdf[j - 1, -1], side="right")), V - 1)
                q_tok[b, j] = q[b, j - 1, tok[b, j]]
        u = g.random((B, T)).astype(np.float32)
        wv = g.random(B).astype(np.float32)
        n_acc, path, out_tok, new_len, status = run_chain_q(w, tok, q, q_tok, inv_temp, u, wv)
        assert status == 0
        np.add.at(counts, out_tok[:, 0], 1)
    n = B * reps
    sigma = np.sqrt(n * p[0] * (1 - p[0]))
    assert (np.abs(counts - n * p[0]) <= 5 * sigma + 1).all(), (counts / n, p[0])


# ---------------------------------------------------------------------------------------------------
# trees whose children were sampled from their parent's draft distribution: sd_accept_tree_sampled_q
# ---------------------------------------------------------------------------------------------------
def drafted_tree(w, lg, inv_temp, spread, seed):
    """q[b][i] = softmax of the target's logits behind node i plus noise (float32, read by both sides);
    every child of node i carries a token drawn from q[b][i], independently of its siblings."""
    g = np.random.default_rng(seed)
    B, T, V = w.B, w.T_max, lg.shape[1]
    q64, _ = smp.softmax_rows(lg + g.standard_normal(lg.shape) * spread, inv_temp * 0.8)
    q = np.ascontiguousarray(q64.astype(np.float32).reshape(B, T, V))
    tok = np.zeros((B, T), dtype=np.int32)
    for b in range(B):
        cdfs = {}
        for j in range(1, int(w.n_nodes[b])):
            i = int(w.parents[b][j])
            if i not in cdfs:
                cdfs[i] = np.cumsum(q[b, i].astype(np.float64))
            tok[b, j] = min(int(np.searchsorted(cdfs[i], g.random() * cdfs[i][-1], side="right")), V - 1)
    return q, tok


def run_tree_q(w, tok, q, inv_temp, u, wv):
    bt = sd.Batch.of(w)
    st = sd.new_status()
    h, Wd = to_device(w.hidden), to_device(w.W)
    M, V = w.hidden.shape[0], w.W.shape[0]
    B, T = w.B, w.T_max
    ws = torch.zeros(sd.sd_workspace_bytes(bt, M, V), dtype=torch.uint8, device="cuda")
    lse = torch.zeros(M, dtype=torch.float32, device="cuda")
    logits = torch.full((M, V), float("nan"), dtype=torch.float32, device="cuda")
    sd.sd_lmhead_stats_logits(h, Wd, inv_temp, None, None, lse, logits, ws, st)
    n_acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    path = torch.full((B, T), -9, dtype=torch.int32, device="cuda")
    out_tok = torch.full((B, T), -9, dtype=torch.int32, device="cuda")
    new_len = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    sd.sd_accept_tree_sampled_q(bt, inv_temp, lse, logits, to_device(tok), to_device(q), to_device(u), to_device(wv),
                                n_acc, path, out_tok, new_len, st)
    torch.cuda.synchronize()
    return (n_acc.cpu().numpy(), path.cpu().numpy(), out_tok.cpu().numpy(), new_len.cpu().numpy(), int(st.item()))


def decisive_tree_inputs(w, tok, q, lg, inv_temp, g, floor=20 * WALK_CLOSE, floor_w=2e-3):
    """Uniforms under which the fp64 rule makes no close call (accept tests further than `floor`, relative,
    from equality; the last draw further than floor_w of the mass from a CDF step), and its results."""
    B, T = w.B, w.T_max
    u = np.zeros((B, T), np.float32)
    wv = np.zeros(B, np.float32)
    ref_n, ref_path, ref_out = np.zeros(B, np.int32), np.full((B, T), -1, np.int32), np.full((B, T), -1, np.int32)
    rejections = 0
    for b in range(B):
        n = int(w.n_nodes[b])
        rows = slice(b * T, b * T + T)
        for _ in range(400):
            u[b] = g.random(T).astype(np.float32)
            wv[b] = np.float32(g.random())
            path, out, walk_margin, draw_margin, total = smp.verify_tree_q(
                w.parents[b], n, tok[b], lg[rows], inv_temp, q[b], u[b].astype(np.float64), float(wv[b]))
            if walk_margin > floor and draw_margin > floor_w * total:
                break
        else:
            raise AssertionError("no decisive uniforms found")
        ref_n[b] = len(path)
        ref_path[b, :len(path)] = path
        ref_out[b, :len(out)] = out
        rejections += sum(1 for c in range(1, n) if int(w.parents[b][c]) in path and c not in path)
    return u, wv, ref_n, ref_path, ref_out, rejections


@pytest.mark.parametrize("cfg,over,inv_temp,spread", [
    ("c1", dict(), 2.0, 0.8),
    ("c1", dict(V=96, Hd=64), 1.5, 1.0),                                     # slices of 12 vocabulary entries
    ("c5", dict(L=1, V=8192, Hd=512, prefix=100), 4.0, 0.5),                 # 60-node trees: up to ten siblings
    ("c5", dict(L=1, V=8192, Hd=512, prefix=100), 4.0, 0.05),                # a drafter very close to the target
    ("c4", dict(L=1, V=4099, Hd=256, prefix_range=(40, 300)), 3.0, 0.6),     # 16 ragged trees, odd vocabulary
    ("chain11", dict(L=1, V=3000, Hd=128, prefix=70), 2.5, 0.6),
])
def test_tree_acceptance_with_sampled_children_against_the_reference(cfg, over, inv_temp, spread):
    w = wl.make(cfg, attention=False, hidden_gain=24.0, **over)
    B, T, V = w.B, w.T_max, w.W.shape[0]
    lg = oracle.logits(w.hidden, w.W)
    q, tok = drafted_tree(w, lg, inv_temp, spread, 13)
    g = np.random.default_rng(14)
    moved = rejected = 0
    for rep in range(3 if B > 1 else 12):
        u, wv, ref_n, ref_path, ref_out, rej = decisive_tree_inputs(w, tok, q, lg, inv_temp, g)
        n_acc, path, out_tok, new_len, status = run_tree_q(w, tok, q, inv_temp, u, wv)
        assert status == 0
        np.testing.assert_array_equal(n_acc, ref_n)
        np.testing.assert_array_equal(path, ref_path)
        np.testing.assert_array_equal(out_tok, ref_out)
        np.testing.assert_array_equal(new_len, w.len + ref_n)
        moved += int((ref_n > 1).sum())
        rejected += rej
    assert moved > 0 and rejected > 0


def test_tree_acceptance_with_sampled_children_full_vocabulary():
    """One 60-node tree over the vocabulary of 152064 (slices of 19008 entries per CTA)."""
    w = wl.make("c2", attention=False, hidden_gain=40.0)
    lg = oracle.logits(w.hidden, w.W)
    inv_temp = 6.0
    q, tok = drafted_tree(w, lg, inv_temp, 0.15, 15)
    g = np.random.default_rng(16)
    total_rej = 0
    for rep in range(4):
        u, wv, ref_n, ref_path, ref_out, rej = decisive_tree_inputs(w, tok, q, lg, inv_temp, g)
        n_acc, path, out_tok, new_len, status = run_tree_q(w, tok, q, inv_temp, u, wv)
        assert status == 0
        np.testing.assert_array_equal(n_acc, ref_n)
        np.testing.assert_array_equal(path, ref_path)
        np.testing.assert_array_equal(out_tok, ref_out)
        total_rej += rej
    assert total_rej > 0


def test_tree_acceptance_with_sampled_children_reports_bad_inputs():
    w = wl.make("c1", attention=False, hidden_gain=16.0)
    V = w.W.shape[0]
    q = np.full((1, 8, V), 1.0 / V, np.float32)
    half, wv = np.full((1, 8), 0.5, np.float32), np.full(1, 0.5, np.float32)
    tok = np.arange(8, dtype=np.int32)[None].copy(); tok[0, 3] = V + 5
    n_acc, *_, status = run_tree_q(w, tok, q, 1.0, half, wv)
    assert status == sd.SD_ERR_BOUNDS and n_acc[0] == 0
    w.parents = w.parents.copy(); w.parents[0, 3] = 6
    n_acc, *_, status = run_tree_q(w, np.arange(8, dtype=np.int32)[None], q, 1.0, half, wv)
    assert status == sd.SD_ERR_INVALID_TREE and n_acc[0] == 0


def test_tree_acceptance_with_sampled_children_gpu_frequencies():
    """Losslessness on the GPU path: 16 identical trees (root with three children, the first with two),
    children redrawn from q 300 times; the first emitted token must be distributed as p at the root."""
    B, T, Hd, V, inv_temp, reps = 16, 6, 64, 16, 1.2, 300
    g = np.random.default_rng(23)
    bf = lambda a: wl.f32_to_bf16_bits(a.astype(np.float32))
    hid_one = bf(g.standard_normal((T, Hd)))
    W = bf(g.standard_normal((V, Hd)) * 0.25)

    class Geo:
        pass
    w = Geo()
    w.B, w.T_max, w.Hq, w.Hkv, w.D = B, T, 4, 1, 128
    w.block_table = np.arange(B, dtype=np.int32).reshape(B, 1)
    w.len = np.full(B, 5, np.int32)
    w.n_nodes = np.full(B, T, np.int32)
    par = np.array([-1, 0, 0, 0, 1, 1], np.int32)
    w.parents = np.tile(par, (B, 1))
    w.hidden = np.tile(hid_one, (B, 1))
    w.W = W
    lg = oracle.logits(hid_one, W)
    p, _ = smp.softmax_rows(lg, inv_temp)
    q_one, _ = smp.softmax_rows(lg + g.standard_normal(lg.shape) * 0.8, 1.0)
    q = np.ascontiguousarray(np.tile(q_one.astype(np.float32)[None], (B, 1, 1)))
    cdf = np.cumsum(q_one.astype(np.float32).astype(np.float64), axis=1)
    counts = np.zeros(V)
    for rep in range(reps):
        tok = np.zeros((B, T), np.int32)
        for b in range(B):
            for j in range(1, T):
                i = par[j]
                tok[b, j] = min(int(np.searchsorted(cdf[i], g.random() * cdf[i, -1], side="right")), V - 1)
        u = g.random((B, T)).astype(np.float32)
        wv = g.random(B).astype(np.float32)
        n_acc, path, out_tok, new_len, status = run_tree_q(w, tok, q, inv_temp, u, wv)
        assert status == 0
        np.add.at(counts, out_tok[:, 0], 1)
    n = B * reps
    sigma = np.sqrt(n * p[0] * (1 - p[0]))
    assert (np.abs(counts - n * p[0]) <= 5 * sigma + 1).all(), (counts / n, p[0])
