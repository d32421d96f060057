"""GPU parity: every library call against the fp64 checker on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_18824_b200 import binding as sd
from paper_2509_18824_b200 import workloads as wl
from paper_2509_18824_b200.step import VerifyStep, to_device
from helpers import Tiny, root_path
from gpu_util import (gpu_attention, check_attention, gpu_lmhead, check_argmax)

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ trees / accept
def run_accept(w, draft, target):
    bt = sd.Batch.of(w)
    st = sd.new_status()
    B, T = w.B, w.T_max
    n_acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    path = torch.full((B, T), -9, dtype=torch.int32, device="cuda")
    out_tok = torch.full((B, T), -9, dtype=torch.int32, device="cuda")
    new_len = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    sd.sd_accept_tree(bt, to_device(draft), to_device(target), n_acc, path, out_tok, new_len, st)
    torch.cuda.synchronize()
    return [x.cpu().numpy() for x in (n_acc, path, out_tok, new_len)], int(st.item())


@pytest.mark.parametrize("cfg", ["c1", "c2", "c4", "c5", "chain11"])
def test_accept_bit_exact_random_small_vocab(cfg):
    w = wl.make_geometry(wl.spec(cfg))
    g = np.random.default_rng(1)
    for vocab in (2, 3, 50):
        draft = g.integers(0, vocab, size=(w.B, w.T_max)).astype(np.int32)
        target = g.integers(0, vocab, size=(w.B, w.T_max)).astype(np.int32)
        ref = oracle.accept(oracle.Geometry.of(w), draft, target)
        got, status = run_accept(w, draft, target)
        assert status == 0
        for a, b in zip(got, ref):
            np.testing.assert_array_equal(a, b)


def test_accept_planted_and_ragged_node_counts():
    w = wl.make_geometry(wl.spec("c5"))
    g = np.random.default_rng(2)
    target = g.integers(0, w.V, size=(w.B, w.T_max)).astype(np.int32)
    wl.plant(w, target, np.arange(w.B) % 7)
    ref = oracle.accept(oracle.Geometry.of(w), w.draft_tok, target)
    got, status = run_accept(w, w.draft_tok, target)
    assert status == 0
    for a, b in zip(got, ref):
        np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(got[0], w.planted_len + 1)
    # fewer nodes than T_max in some sequences
    w.n_nodes = np.array([60, 1, 33, 2, 59, 17, 60, 5], dtype=np.int32)
    draft = g.integers(0, 2, size=(w.B, w.T_max)).astype(np.int32)
    target = g.integers(0, 2, size=(w.B, w.T_max)).astype(np.int32)
    ref = oracle.accept(oracle.Geometry.of(w), draft, target)
    got, status = run_accept(w, draft, target)
    assert status == 0
    for a, b in zip(got, ref):
        np.testing.assert_array_equal(a, b)


def test_tree_prepare_masks_and_bad_tree_status():
    w = wl.make_geometry(wl.spec("c4"))
    bt = sd.Batch.of(w)
    st = sd.new_status()
    sd.sd_tree_prepare(bt, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    am = bt.anc_mask.cpu().numpy().view(np.uint64)
    for b in range(w.B):
        for i in range(w.T_max):
            want = sum(1 << j for j in root_path(w.parents[b], i))
            assert int(am[b, i]) == want
    bad = wl.make_geometry(wl.spec("c1"))
    bad.parents = bad.parents.copy(); bad.parents[0, 3] = 5      # parent > child
    bt = sd.Batch.of(bad)
    st = sd.new_status()
    sd.sd_tree_prepare(bt, st)
    torch.cuda.synchronize()
    assert int(st.item()) == sd.SD_ERR_INVALID_TREE
    _, status = run_accept(bad, np.zeros((1, 8), np.int32), np.zeros((1, 8), np.int32))
    assert status == sd.SD_ERR_INVALID_TREE


# ------------------------------------------------------------------ attention
def tiny128(seed, **kw):
    kw.setdefault("D", 128)
    return Tiny(seed, **kw)


@pytest.mark.parametrize("lens", [(0, 1), (63, 64), (65, 127), (128, 129), (700, 5), (1023, 1025)])
def test_attention_edge_lengths_peaked_scores(lens):
    p = tiny128(sum(lens), B=2, T=8, Hq=8, Hkv=2, lens=lens, gain=4.0)
    out, lse, status = gpu_attention(p)
    assert status == 0
    ref, rlse = oracle.attention(oracle.Geometry.of(p), p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    check_attention(out, ref, f"lens={lens}")
    np.testing.assert_allclose(lse, rlse, rtol=2e-3, atol=2e-3)


def test_attention_gqa7_wide_trees_and_unused_nodes():
    g = np.random.default_rng(0)
    T = 64
    par = np.stack([np.array([-1] + [int(g.integers(max(0, i - 9), i)) for i in range(1, T)]) for _ in range(3)])
    p = tiny128(5, B=3, T=T, Hq=14, Hkv=2, lens=(300, 64, 1500), parents=par, gain=3.0)
    p.n_nodes = np.array([64, 7, 33], dtype=np.int32)
    out, lse, status = gpu_attention(p)
    assert status == 0
    ref, rlse = oracle.attention(oracle.Geometry.of(p), p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    check_attention(out, ref)
    for b in range(3):          # rows of unused nodes are zeroed
        assert (out[b, p.n_nodes[b]:] == 0).all()
    ok = np.isfinite(rlse)
    np.testing.assert_allclose(lse[ok], rlse[ok], rtol=2e-3, atol=2e-3)


@pytest.mark.parametrize("Hq,Hkv,T", [(8, 1, 64), (3, 3, 5), (16, 2, 33), (4, 4, 1), (8, 1, 8), (5, 1, 13), (6, 1, 32)])
def test_attention_group_sizes_and_tree_sizes(Hq, Hkv, T):
    """Largest supported shape (64 nodes x 8 grouped heads = 512 rows per KV head), no grouping at
    all, a single-node tree (plain decoding), odd sizes; 64 rows exactly (one half-height row tile),
    65 rows (one full-height tile), 192 rows (a full tile and a half-height one that is full)."""
    g = np.random.default_rng(Hq * 100 + T)
    par = np.stack([np.array([-1] + [int(g.integers(0, i)) for i in range(1, T)]) for _ in range(2)])
    p = tiny128(40 + T, B=2, T=T, Hq=Hq, Hkv=Hkv, lens=(257, 64), parents=par, gain=3.0)
    out, lse, status = gpu_attention(p)
    assert status == 0
    ref, rlse = oracle.attention(oracle.Geometry.of(p), p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    check_attention(out, ref, f"Hq={Hq} Hkv={Hkv} T={T}")
    np.testing.assert_allclose(lse, rlse, rtol=2e-3, atol=2e-3)


def test_attention_planted_key_large_v_and_bad_block_table():
    p = tiny128(6, B=1, T=8, Hq=4, Hkv=1, lens=(900,), gain=1.0)
    # one key with score ~ +30, V rows scaled by 64
    qv = wl.bf16_bits_to_f32(p.q[0, 5, 2])
    t_star = 517
    blk = p.block_table[0, t_star // 64]
    p.k_cache[blk, 0, t_star % 64] = wl.f32_to_bf16_bits(qv * (30.0 / (p.scale * float(qv @ qv))))
    p.v_cache[:] = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(p.v_cache) * 64)
    p.v_tree[:] = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(p.v_tree) * 64)
    out, lse, status = gpu_attention(p)
    assert status == 0
    ref, rlse = oracle.attention(oracle.Geometry.of(p), p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    d = np.abs(out - ref)
    assert np.sqrt((d ** 2).sum() / (ref ** 2).sum()) <= 2e-2
    assert abs(rlse[0, 5, 2] - 30.0) < 0.1 and abs(lse[0, 5, 2] - rlse[0, 5, 2]) < 0.05
    # a block-table entry outside the cache is reported, not dereferenced
    p.block_table = p.block_table.copy(); p.block_table[0, 3] = p.num_blocks + 100
    _, _, status = gpu_attention(p)
    assert status == sd.SD_ERR_BOUNDS


def test_attention_length_beyond_the_block_table_is_reported():
    """A cached length that needs more blocks than max_blocks_per_seq is an error (SD_ERR_BOUNDS in the
    status word), not a silently shortened sequence."""
    p = tiny128(7, B=2, T=8, Hq=4, Hkv=2, lens=(100, 40), gain=2.0)
    _, _, status = gpu_attention(p)
    assert status == 0
    p.len = p.len.copy(); p.len[1] = 64 * p.block_table.shape[1] + 1
    _, _, status = gpu_attention(p)
    assert status == sd.SD_ERR_BOUNDS


def test_compaction_reports_a_corrupt_block_table_entry():
    """Block-table entries of -2 (and any other value outside [0, num_blocks)) under an accepted node are
    reported as SD_ERR_BOUNDS and nothing is written through them."""
    sp = wl.spec("c5"); sp.L = 2; sp.prefix = 100; sp.B = 3
    w = wl.make_geometry(sp)
    wl.fill_attention(w)
    g = np.random.default_rng(6)
    target = g.integers(0, 5, size=(w.B, w.T_max)).astype(np.int32)
    wl.plant(w, target, np.array([3, 2, 4]))
    n_acc, path, _, _ = oracle.accept(oracle.Geometry.of(w), w.draft_tok, target)
    for bad in (-2, -1, 10 ** 6):
        w2_table = w.block_table.copy()
        w2_table[1, int(w.len[1]) // 64] = bad            # the block that sequence 1's accepted rows go to
        geo = type("G", (), dict(B=w.B, T_max=w.T_max, Hq=w.Hq, Hkv=w.Hkv, D=w.D, block_table=w2_table,
                                 len=w.len, n_nodes=w.n_nodes, parents=w.parents))
        bt = sd.Batch.of(geo)
        st = sd.new_status()
        kc = [to_device(x) for x in w.k_cache]; vc = [to_device(x) for x in w.v_cache]
        kt = [to_device(x) for x in w.k_tree]; vt = [to_device(x) for x in w.v_tree]
        sd.sd_compact_kv(bt, sd.LayerSet(kc, vc, kt, vt), to_device(n_acc), to_device(path), st)
        torch.cuda.synchronize()
        assert int(st.item()) == sd.SD_ERR_BOUNDS, bad
        # sequences 0 and 2 were compacted as usual, sequence 1 wrote nothing
        G2 = oracle.Geometry(w.B, w.T_max, w.Hq, w.Hkv, w.D, w.block_table, w.len, w.n_nodes, w.parents)
        na2 = n_acc.copy(); na2[1] = 0
        for l in range(w.L):
            rk, rv = w.k_cache[l].copy(), w.v_cache[l].copy()
            oracle.compact(G2, rk, rv, w.k_tree[l], w.v_tree[l], na2, path)
            np.testing.assert_array_equal(kc[l].cpu().numpy().view(np.uint16), rk)
            np.testing.assert_array_equal(vc[l].cpu().numpy().view(np.uint16), rv)


def test_attention_any_bit_pattern_in_invisible_slots():
    """Cache slots at and beyond len, and the K/V rows of unused tree nodes, may hold NaN and
    infinity bit patterns (memory that was never written): no key there is visible to any row, so
    the output must equal the checker's, which never reads them."""
    p = tiny128(77, B=4, T=16, Hq=14, Hkv=2, lens=(5, 70, 64, 0), gain=3.0)
    p.n_nodes = np.array([16, 3, 9, 1], dtype=np.int32)
    junk = np.array([0x7FC0, 0x7F80, 0xFF80, 0xFFFF, 0x7FFF], dtype=np.uint16)
    for b in range(p.B):
        P = int(p.len[b])
        for j in range(P // 64, (P + p.T_max + 63) // 64):      # the sequence's own blocks from slot len on
            blk = int(p.block_table[b, j])
            lo = max(0, P - j * 64)
            for arr in (p.k_cache, p.v_cache):
                shape = arr[blk, :, lo:].shape
                arr[blk, :, lo:] = junk[np.arange(int(np.prod(shape))) % len(junk)].reshape(shape)
        for arr in (p.k_tree, p.v_tree):
            shape = arr[b, p.n_nodes[b]:].shape
            arr[b, p.n_nodes[b]:] = junk[np.arange(int(np.prod(shape))) % len(junk)].reshape(shape)
    out, lse, status = gpu_attention(p)
    assert status == 0
    ref, rlse = oracle.attention(oracle.Geometry.of(p), p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    for b in range(p.B):
        nb = int(p.n_nodes[b])
        assert np.isfinite(out[b, :nb]).all() and np.isfinite(ref[b, :nb]).all()
        check_attention(out[b, :nb], ref[b, :nb], f"sequence {b}")
        np.testing.assert_allclose(lse[b, :nb], rlse[b, :nb], rtol=2e-3, atol=2e-3)
        assert (out[b, nb:] == 0).all()


@pytest.mark.parametrize("cfg,gain", [("c1", 1.0), ("c1", 45.0), ("c2", 1.0), ("c2", 45.0)])
def test_attention_configs_full_compare(cfg, gain):
    w = wl.make(cfg, lmhead=False, q_gain=gain)
    out, lse, status = gpu_attention(w, layer=0)
    assert status == 0
    ref, rlse = oracle.attention(oracle.Geometry.of(w), w.k_cache[0], w.v_cache[0], w.q[0], w.k_tree[0],
                                 w.v_tree[0], w.scale)
    mx, mean, rel = check_attention(out, ref, f"{cfg} gain {gain}")
    np.testing.assert_allclose(lse, rlse, rtol=2e-3, atol=2e-3)


def test_attention_is_deterministic_run_to_run():
    """Many short CTAs (17 key chunks of two tiles): repeated runs must give identical bits,
    which a lost synchronisation between the MMA, softmax and epilogue roles would not."""
    w = wl.make("c2", lmhead=False, q_gain=45.0)
    ref, _ = oracle.attention(oracle.Geometry.of(w), w.k_cache[0], w.v_cache[0], w.q[0], w.k_tree[0],
                              w.v_tree[0], w.scale)
    first = None
    for rep in range(6):
        out, lse, status = gpu_attention(w, layer=0)
        assert status == 0
        check_attention(out, ref, f"run {rep}")
        if first is None:
            first = (out.copy(), lse.copy())
        else:
            np.testing.assert_array_equal(out, first[0])
            np.testing.assert_array_equal(lse, first[1])


def sample_rows(w, n, seed):
    g = np.random.default_rng(seed)
    rows = np.stack([g.integers(0, w.B, n), g.integers(0, w.T_max, n), g.integers(0, w.Hq, n)], 1).astype(np.int32)
    rows[0] = (0, 0, 0)
    rows[1] = (w.B - 1, w.T_max - 1, w.Hq - 1)
    return rows


def check_every_row(got, ref, what):
    """Row by row, so that one wrong (sequence, KV head) group cannot hide in an average: the error of
    a row against its own norm.  bf16 output rounding alone is 2^-9 relative per element."""
    ok = np.isfinite(ref).all(axis=-1)
    d = np.linalg.norm(got[ok].astype(np.float64) - ref[ok], axis=-1)
    nr = np.linalg.norm(ref[ok], axis=-1)
    worst = (d / (nr + 1e-30)).max()
    assert (d <= 1.5e-2 * nr + 1e-7).all(), f"{what}: a row is off by {worst:.3e} of its norm"


@pytest.mark.parametrize("cfg,gain", [("c3", 1.0), ("c3", 45.0), ("c4", 1.0), ("c4", 45.0),
                                      ("chain11", 1.0), ("chain11", 45.0), ("tree28", 1.0), ("tree28", 45.0)])
def test_attention_full_size_every_row(cfg, gain):
    """The configured shapes in full (c3: 4 x 8192 prefix; c4: 16 ragged sequences through the shuffled
    block table; chain11: the paper's chain setting; tree28: a short tree, one full and one partly
    filled row tile), at unit scale and with peaked scores: every row of the one-layer call against the
    checker."""
    w = wl.make(cfg, lmhead=False, q_gain=gain)
    out, lse, status = gpu_attention(w, layer=0)
    assert status == 0
    ref, rlse = oracle.attention(oracle.Geometry.of(w), w.k_cache[0], w.v_cache[0], w.q[0], w.k_tree[0],
                                 w.v_tree[0], w.scale)
    live = np.isfinite(rlse)
    assert live.sum() == int(w.n_nodes.sum()) * w.Hq
    mx, mean, rel = check_attention(out[live], ref[live], f"{cfg} gain {gain}")
    check_every_row(out, ref, f"{cfg} gain {gain}")
    np.testing.assert_allclose(lse[live], rlse[live], rtol=2e-3, atol=2e-3)
    assert np.isfinite(out).all() and (out[~live] == 0).all()          # rows of unused nodes are zeroed
    print(f"{cfg} gain {gain}: {int(live.sum())} rows, max abs {mx:.2e}, mean abs {mean:.2e}, rel L2 {rel:.2e}")


def test_attention_result_does_not_depend_on_the_split_count(monkeypatch):
    """One shape with the keys of a sequence split into 1, 2, 4 and 8 chunks (test hook
    SDV_TEST_CHUNKS): every split against the checker, and the splits against each other within the
    rounding of the fp32 merge and the bf16 output (two bf16 steps)."""
    w = wl.make("c2", lmhead=False, q_gain=45.0)
    ref, rlse = oracle.attention(oracle.Geometry.of(w), w.k_cache[0], w.v_cache[0], w.q[0], w.k_tree[0],
                                 w.v_tree[0], w.scale)
    outs = {}
    for c in (1, 2, 4, 8):
        monkeypatch.setenv("SDV_TEST_CHUNKS", str(c))
        out, lse, status = gpu_attention(w, layer=0)
        assert status == 0
        check_attention(out, ref, f"{c} chunks")
        check_every_row(out, ref, f"{c} chunks")
        np.testing.assert_allclose(lse, rlse, rtol=2e-3, atol=2e-3)
        outs[c] = out
    monkeypatch.delenv("SDV_TEST_CHUNKS")
    # Chunks keep their own reference maxima, so P is rounded to bf16 at different scales and the partial
    # sums are merged in fp32: per row the results agree to a few bf16 steps of the row's size.
    differ = 0
    for c in (2, 4, 8):
        d = np.linalg.norm((outs[c] - outs[1]).astype(np.float64), axis=-1)
        nr = np.linalg.norm(outs[1].astype(np.float64), axis=-1)
        assert (d <= 6e-3 * nr + 1e-7).all(), f"{c} chunks against 1: {(d / (nr + 1e-30)).max():.3e}"
        differ += int((d > 0).sum())
    assert differ > 0          # the hook did change the plan (different merge orders round differently somewhere)


def gpu_attention_layers(w, layers):
    """sd_verify_attention_layers over the listed layers of a workload; returns per-layer (out, lse)."""
    bt = sd.Batch.of(w)
    st = sd.new_status()
    sd.sd_tree_prepare(bt, st)
    dev = lambda xs: [to_device(xs[l]) for l in layers]
    kc, vc, q, kt, vt = dev(w.k_cache), dev(w.v_cache), dev(w.q), dev(w.k_tree), dev(w.v_tree)
    out = [torch.full((w.B, w.T_max, w.Hq, w.D), 7.0, dtype=torch.bfloat16, device="cuda") for _ in layers]
    lse = [torch.full((w.B, w.T_max, w.Hq), 7.0, dtype=torch.float32, device="cuda") for _ in layers]
    ws = torch.empty(sd.sd_workspace_bytes(bt), dtype=torch.uint8, device="cuda")
    ls = sd.AttentionLayerSet(kc, vc, q, kt, vt, out, lse)
    sd.sd_verify_attention_layers(bt, ls, float(w.scale), ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return [(o.float().cpu().numpy(), l.cpu().numpy()) for o, l in zip(out, lse)]


@pytest.mark.parametrize("cfg,L,gain", [("c1", 3, 45.0), ("c2", 2, 45.0), ("c2", 5, 1.0)])
def test_attention_layers_call_full_compare(cfg, L, gain):
    """Several layers in one call (few enough that the keys are still split into chunks): every
    layer against the checker, element by element."""
    w = wl.make(cfg, lmhead=False, q_gain=gain, L=L)
    got = gpu_attention_layers(w, list(range(L)))
    G = oracle.Geometry.of(w)
    for l in range(L):
        ref, rlse = oracle.attention(G, w.k_cache[l], w.v_cache[l], w.q[l], w.k_tree[l], w.v_tree[l], w.scale)
        check_attention(got[l][0], ref, f"{cfg} layer {l}")
        np.testing.assert_allclose(got[l][1], rlse, rtol=2e-3, atol=2e-3)


@pytest.mark.parametrize("cfg,L", [("c5", 7), ("chain11", 28)])
def test_attention_layers_call_full_size_with_remainder_launch(cfg, L):
    """Full-size calls of a few rounds of CTAs (896 CTAs = 3.03 rounds in both cases), which the library
    issues as whole-sequence CTAs plus a chunked remainder: sampled rows of every layer against the
    checker, among them the last sequence's last rows, which the remainder launch computes."""
    w = wl.make(cfg, lmhead=False, q_gain=45.0, L=L)
    rows = sample_rows(w, 24, 11)
    G = oracle.Geometry.of(w)
    first = None
    for attempt in range(2):                           # twice: a race would not hit the same rows again
        got = gpu_attention_layers(w, list(range(L)))
        if first is None:
            first = got
        else:                                          # same inputs, bit-identical outputs
            assert all(np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) for a, b in zip(first, got))
        for l in range(L):
            if attempt == 0:
                ref, rlse = oracle.attention_rows(G, w.k_cache[l], w.v_cache[l], w.q[l], w.k_tree[l], w.v_tree[l],
                                                  w.scale, rows)
                check_attention(got[l][0][rows[:, 0], rows[:, 1], rows[:, 2]], ref, f"{cfg} layer {l}")
                np.testing.assert_allclose(got[l][1][rows[:, 0], rows[:, 1], rows[:, 2]], rlse, rtol=2e-3, atol=2e-3)
            # every row of the layer against the one-layer call (itself checked against the checker above
            # and elsewhere): per row, so that one wrong (sequence, KV head) group cannot hide in an average
            single, _, status = gpu_attention(w, layer=l)
            assert status == 0
            d = np.linalg.norm(got[l][0].astype(np.float64) - single, axis=-1)
            ref_norm = np.linalg.norm(single.astype(np.float64), axis=-1)
            assert (d <= 1e-2 * ref_norm + 1e-6).all(), f"{cfg} layer {l}: rows differ from the one-layer call"


@pytest.mark.parametrize("L,lens,n_nodes", [(33, (130, 61), (24, 9)), (30, (300, 61, 190), (24, 9, 17))])
def test_attention_layers_call_many_layers_ragged(L, lens, n_nodes):
    """Ragged lengths, unused nodes, shuffled blocks, every layer against the checker.  First case:
    more layers than one launch holds (33 > 32).  Second case: 30 layers x 3 sequences x 2 KV heads x
    2 row tiles = 360 CTAs, more than one round of the 296 resident ones, so the call is issued as a
    launch of whole-sequence CTAs plus the remainder (the shortest sequence's last layers) in key chunks."""
    B = len(lens)
    g = np.random.default_rng(21)
    T = 24
    par = np.stack([np.array([-1] + [int(g.integers(max(0, i - 5), i)) for i in range(1, T)]) for _ in range(B)])
    w = tiny128(100, B=B, T=T, Hq=14, Hkv=2, lens=lens, parents=par, gain=3.0)
    w.n_nodes = np.array(n_nodes, dtype=np.int32)

    class Layer:
        pass
    ps = []
    for l in range(L):                                 # same geometry for all layers, own tensors each
        p = Layer()
        gl = np.random.default_rng(500 + l)
        for name, k in (("q", 3.0), ("k_tree", 1.0), ("v_tree", 0.3), ("k_cache", 1.0), ("v_cache", 0.3)):
            shape = getattr(w, name).shape
            setattr(p, name, wl.f32_to_bf16_bits((gl.standard_normal(shape) * k).astype(np.float32)))
        ps.append(p)

    class Stack:
        pass
    sw = Stack()
    for name in ("B", "T_max", "Hq", "Hkv", "D", "block_table", "len", "n_nodes", "parents", "scale"):
        setattr(sw, name, getattr(w, name))
    for name in ("k_cache", "v_cache", "q", "k_tree", "v_tree"):
        setattr(sw, name, [getattr(p, name) for p in ps])
    got = gpu_attention_layers(sw, list(range(L)))
    G = oracle.Geometry.of(w)
    for l in range(L):
        ref, rlse = oracle.attention(G, ps[l].k_cache, ps[l].v_cache, ps[l].q, ps[l].k_tree, ps[l].v_tree, w.scale)
        check_attention(got[l][0], ref, f"layer {l}")
        ok = np.isfinite(rlse)
        np.testing.assert_allclose(got[l][1][ok], rlse[ok], rtol=2e-3, atol=2e-3)
        assert (got[l][0][1, 9:] == 0).all()                     # rows of unused nodes are zeroed


# ------------------------------------------------------------------ LM head
@pytest.mark.parametrize("M,Hd,V", [(1, 64, 1), (5, 128, 1000), (8, 256, 1024), (61, 192, 129), (130, 64, 4099)])
def test_lmhead_small_shapes_crisp(M, Hd, V):
    g = np.random.default_rng(M + V)
    h = wl.f32_to_bf16_bits(g.standard_normal((M, Hd)).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, Hd)) / np.sqrt(Hd)).astype(np.float32))
    am, mx = gpu_lmhead(h, W)
    ram, t1, t2 = oracle.lmhead(h, W)
    check_argmax(am, mx, ram, t1, t2)


def test_lmhead_more_rows_than_one_pass():
    """More than 512 rows are processed in several passes over the vocabulary."""
    g = np.random.default_rng(11)
    M, Hd, V = 1100, 128, 2500
    h = wl.f32_to_bf16_bits(g.standard_normal((M, Hd)).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, Hd)) / np.sqrt(Hd)).astype(np.float32))
    am, mx = gpu_lmhead(h, W)
    ram, t1, t2 = oracle.lmhead(h, W)
    check_argmax(am, mx, ram, t1, t2)


def test_lmhead_exact_ties_lowest_index():
    g = np.random.default_rng(4)
    M, Hd, V = 6, 128, 3000
    h = wl.f32_to_bf16_bits(g.standard_normal((M, Hd)).astype(np.float32))
    W = wl.f32_to_bf16_bits((0.01 * g.standard_normal((V, Hd))).astype(np.float32))
    W[[2999, 130, 1500, 131]] = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(h[2]) * 4)
    am, mx = gpu_lmhead(h, W)
    ram, t1, t2 = oracle.lmhead(h, W)
    assert am[2] == 130 == ram[2]
    np.testing.assert_array_equal(am, ram)


def test_lmhead_c1_and_c2_full():
    for cfg, gain in (("c1", 1.0), ("c1", 16.0), ("c2", 1.0), ("c2", 60.0)):
        w = wl.make(cfg, attention=False, hidden_gain=gain)
        am, mx = gpu_lmhead(w.hidden, w.W)
        ram, t1, t2 = oracle.lmhead(w.hidden, w.W)
        in_band, mis_in, mis_out = check_argmax(am, mx, ram, t1, t2, require_all=(gain > 1))
        print(f"{cfg} gain {gain}: rows {len(am)}, in band {in_band}, mismatches in band {mis_in}, outside {mis_out}")


# ------------------------------------------------------------------ compaction
def test_compact_bit_exact_and_touches_nothing_else():
    sp = wl.spec("c5"); sp.L = 3; sp.prefix = 250; sp.B = 5
    w = wl.make_geometry(sp)
    w.len = np.array([250, 58, 63, 64, 0], dtype=np.int32)     # 58+: crossing a block boundary
    wl.fill_attention(w)
    g = np.random.default_rng(5)
    target = g.integers(0, 5, size=(w.B, w.T_max)).astype(np.int32)
    wl.plant(w, target, np.array([6, 5, 0, 3, 6]))
    G = oracle.Geometry.of(w)
    n_acc, path, _, _ = oracle.accept(G, w.draft_tok, target)
    bt = sd.Batch.of(w)
    st = sd.new_status()
    kc = [to_device(x) for x in w.k_cache]; vc = [to_device(x) for x in w.v_cache]
    kt = [to_device(x) for x in w.k_tree]; vt = [to_device(x) for x in w.v_tree]
    ls = sd.LayerSet(kc, vc, kt, vt)
    sd.sd_compact_kv(bt, ls, to_device(n_acc), to_device(path), st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    for l in range(w.L):
        rk, rv = w.k_cache[l].copy(), w.v_cache[l].copy()
        oracle.compact(G, rk, rv, w.k_tree[l], w.v_tree[l], n_acc, path)
        assert not np.array_equal(rk, w.k_cache[l])
        np.testing.assert_array_equal(kc[l].cpu().numpy().view(np.uint16), rk)
        np.testing.assert_array_equal(vc[l].cpu().numpy().view(np.uint16), rv)


# ------------------------------------------------------------------ nothing is written outside the outputs
class Guarded:
    """Tensors carved out of one device buffer with 4 KiB guard bands of a fixed byte pattern around
    each; intact() tells whether every guard byte is still there."""

    GUARD, FILL = 4096, 0x5A

    def __init__(self):
        self.specs, self.total = [], self.GUARD

    def reserve(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        self.specs.append((self.total, n, shape, dtype))
        self.total += (n + 255) // 256 * 256 + self.GUARD
        return len(self.specs) - 1

    def build(self):
        self.buf = torch.full((self.total,), self.FILL, dtype=torch.uint8, device="cuda")
        return [self.buf[o:o + n].view(dt).view(shape) for o, n, shape, dt in self.specs]

    def intact(self):
        keep = torch.ones(self.total, dtype=torch.bool, device="cuda")
        for o, n, _, _ in self.specs:
            keep[o:o + n] = False
        return bool((self.buf[keep] == self.FILL).all())


def test_calls_write_only_their_outputs():
    """Attention, LM head and acceptance outputs (and the workspace) sit between guard bands; after
    the calls every guard byte is unchanged, and the results are still the checker's."""
    g = np.random.default_rng(8)
    T = 60
    par = np.stack([np.array([-1] + [int(g.integers(max(0, i - 9), i)) for i in range(1, T)]) for _ in range(2)])
    p = tiny128(31, B=2, T=T, Hq=28, Hkv=4, lens=(700, 63), parents=par, gain=3.0)
    p.n_nodes = np.array([60, 41], dtype=np.int32)
    M, Hd, V = p.B * T, 256, 3000
    hidden = wl.f32_to_bf16_bits((g.standard_normal((M, Hd)) / 4).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, Hd)) / 4).astype(np.float32))
    draft = g.integers(0, V, size=(p.B, T)).astype(np.int32)
    bt = sd.Batch.of(p)
    st = sd.new_status()
    sd.sd_tree_prepare(bt, st)
    gd = Guarded()
    ws_bytes = sd.sd_workspace_bytes(bt, M, V)
    for shape, dt in (((p.B, T, p.Hq, p.D), torch.bfloat16), ((p.B, T, p.Hq), torch.float32),
                      ((M,), torch.int32), ((M,), torch.float32), ((p.B,), torch.int32), ((p.B, T), torch.int32),
                      ((p.B, T), torch.int32), ((p.B,), torch.int32), ((ws_bytes,), torch.uint8)):
        gd.reserve(shape, dt)
    out, lse, am, mx, n_acc, path, out_tok, new_len, ws = gd.build()
    kc, vc, q, kt, vt = (to_device(x) for x in (p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree))   # kept alive:
    hd, Wd, dd = to_device(hidden), to_device(W), to_device(draft)                # the calls only take pointers
    sd.sd_verify_attention(bt, sd.kv_layer(kc, vc), q, kt, vt, float(p.scale), out, lse, ws, st)
    sd.sd_lmhead_argmax(hd, Wd, am, mx, ws, st)
    sd.sd_accept_tree(bt, dd, am.view(p.B, T), n_acc, path, out_tok, new_len, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert gd.intact()
    G = oracle.Geometry.of(p)
    ref, _ = oracle.attention(G, p.k_cache, p.v_cache, p.q, p.k_tree, p.v_tree, p.scale)
    for b in range(p.B):
        check_attention(out.float().cpu().numpy()[b, :p.n_nodes[b]], ref[b, :p.n_nodes[b]], f"sequence {b}")
    ram, t1, t2 = oracle.lmhead(hidden, W)
    check_argmax(am.cpu().numpy(), mx.cpu().numpy(), ram, t1, t2)
    ref_acc = oracle.accept(G, draft, am.cpu().numpy().reshape(p.B, T))
    for got, want in zip((n_acc, path, out_tok, new_len), ref_acc):
        np.testing.assert_array_equal(got.cpu().numpy(), want)


# ------------------------------------------------------------------ the whole step
def test_chained_step_tiny():
    """run(): attention -> LM head -> accept -> compact chained on the device, crisp logits."""
    w = wl.make("c1", hidden_gain=16.0)
    ram, t1, t2 = oracle.lmhead(w.hidden, w.W)
    assert (t1 - t2).min() > 1e-3
    wl.plant(w, ram.reshape(w.B, w.T_max), np.array([3]))
    G = oracle.Geometry.of(w)
    ref_acc = oracle.accept(G, w.draft_tok, ram.reshape(w.B, w.T_max))
    vs = VerifyStep(w, keep_host_inputs=True)
    for mode in ("device", "host", "host", "host"):        # the host path alternates between two input sets
        vs.run() if mode == "device" else vs.run_from_host()
        torch.cuda.synchronize()
        vs.check_status()
        np.testing.assert_array_equal(vs.argmax.cpu().numpy(), ram)
        for got, ref in zip((vs.n_acc, vs.path, vs.out_tok, vs.new_len), ref_acc):
            np.testing.assert_array_equal(got.cpu().numpy(), ref)
    assert vs.host_out["n_acc"][0] == 4
    # each host-path step uses the inputs that are in pinned memory when it is issued: drafts planted
    # for another accepted length, two steps (one per device-side input set), then the first again
    first = w.draft_tok.copy()
    wl.plant(w, ram.reshape(w.B, w.T_max), np.array([1]))
    other = w.draft_tok.copy()
    for drafts, want in ((other, 2), (other, 2), (first, 4)):
        torch.cuda.synchronize()                  # the previous step has read the pinned buffer
        vs.host["draft_tok"].copy_(torch.from_numpy(drafts))
        vs.run_from_host()
        torch.cuda.synchronize()
        vs.check_status()
        assert vs.host_out["n_acc"][0] == want
    w.draft_tok = first
    rk, rv = w.k_cache[0].copy(), w.v_cache[0].copy()
    oracle.compact(G, rk, rv, w.k_tree[0], w.v_tree[0], ref_acc[0], ref_acc[1])
    np.testing.assert_array_equal(vs.k_cache[0].cpu().numpy().view(np.uint16), rk)
    np.testing.assert_array_equal(vs.v_cache[0].cpu().numpy().view(np.uint16), rv)


@pytest.mark.parametrize("per_layer", [True, False])
def test_step_replayed_from_a_cuda_graph(per_layer):
    """The step's library calls (one attention call per layer, or all three layers in one call) recorded
    into a CUDA graph and replayed: same outputs and the same cache bytes as the directly issued step
    (the checker's, via test_chained_step_tiny's route)."""
    w = wl.make("c1", hidden_gain=16.0, L=3)
    ram, _, _ = oracle.lmhead(w.hidden, w.W)
    wl.plant(w, ram.reshape(w.B, w.T_max), np.array([2]))
    ref_acc = oracle.accept(oracle.Geometry.of(w), w.draft_tok, ram.reshape(w.B, w.T_max))
    vs = VerifyStep(w)
    graph = vs.capture(per_layer=per_layer)
    outs = (vs.n_acc, vs.path, vs.out_tok, vs.new_len, vs.argmax)
    state = list(vs.out) + list(vs.k_cache) + list(vs.v_cache)
    direct = [t.clone() for t in outs] + [t.clone() for t in state]
    for t in outs:
        t.fill_(-3)
    for l in range(vs.L):
        vs.out[l].fill_(7.0)
        vs.k_cache[l].copy_(to_device(w.k_cache[l])); vs.v_cache[l].copy_(to_device(w.v_cache[l]))   # undo the compaction
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    vs.check_status()
    for got, ref in zip(list(outs) + state, direct):
        assert torch.equal(got, ref)
    for got, ref in zip((vs.n_acc, vs.path, vs.out_tok, vs.new_len), ref_acc):
        np.testing.assert_array_equal(got.cpu().numpy(), ref)


@pytest.mark.parametrize("cfg,over", [("c1", dict(L=1)), ("c2", dict(L=3)),
                                      ("c5", dict(L=2, V=8192, Hd=512, prefix=200)),
                                      ("c4", dict(L=2, V=4096, Hd=256, prefix_range=(40, 300)))])
def test_fused_tail_equals_separate_calls(cfg, over):
    """sd_lmhead_accept_compact against sd_lmhead_argmax + sd_accept_tree + sd_compact_kv on the same
    inputs: every output and every cache byte identical; acceptance also against the checker."""
    w = wl.make(cfg, hidden_gain=16.0, **over)        # c4: 960 rows, more than one LM-head pass
    L = w.L
    ram, t1, t2 = oracle.lmhead(w.hidden, w.W)
    g = np.random.default_rng(3)
    wl.plant(w, ram.reshape(w.B, w.T_max), g.integers(0, 4, size=w.B))
    res = []
    for fused in (False, True):
        vs = VerifyStep(w)
        if fused:
            vs.tail()
        else:
            vs.lmhead(); vs.accept(); vs.compact()
        torch.cuda.synchronize()
        vs.check_status()
        res.append(dict(argmax=vs.argmax.cpu().numpy(), maxlogit=vs.maxlogit.cpu().numpy(),
                        n_acc=vs.n_acc.cpu().numpy(), path=vs.path.cpu().numpy(), out_tok=vs.out_tok.cpu().numpy(),
                        new_len=vs.new_len.cpu().numpy(),
                        k=[x.cpu().numpy() for x in vs.k_cache], v=[x.cpu().numpy() for x in vs.v_cache]))
    for key in ("argmax", "maxlogit", "n_acc", "path", "out_tok", "new_len"):
        np.testing.assert_array_equal(res[0][key], res[1][key], err_msg=key)
    for l in range(L):
        np.testing.assert_array_equal(res[0]["k"][l], res[1]["k"][l])
        np.testing.assert_array_equal(res[0]["v"][l], res[1]["v"][l])
    np.testing.assert_array_equal(res[1]["argmax"], ram)             # crisp logits: every row must match
    G = oracle.Geometry.of(w)
    ref_acc = oracle.accept(G, w.draft_tok, ram.reshape(w.B, w.T_max))
    for got, ref in zip((res[1]["n_acc"], res[1]["path"], res[1]["out_tok"], res[1]["new_len"]), ref_acc):
        np.testing.assert_array_equal(got, ref)
    for l in range(L):
        rk, rv = w.k_cache[l].copy(), w.v_cache[l].copy()
        oracle.compact(G, rk, rv, w.k_tree[l], w.v_tree[l], ref_acc[0], ref_acc[1])
        np.testing.assert_array_equal(res[1]["k"][l].view(np.uint16), rk)
        np.testing.assert_array_equal(res[1]["v"][l].view(np.uint16), rv)


def test_fused_tail_bad_tree_touches_no_cache():
    w = wl.make("c1", hidden_gain=16.0)
    w.parents = w.parents.copy(); w.parents[0, 3] = 5
    vs = VerifyStep(w)
    before_k = vs.k_cache[0].clone()
    vs.status.zero_()
    vs.tail()
    torch.cuda.synchronize()
    assert int(vs.status.item()) == sd.SD_ERR_INVALID_TREE
    assert torch.equal(before_k, vs.k_cache[0])


def test_full_step_c5_shapes():
    """28 layers, batch 8, prefix 4096: planted paths are recovered bit-exactly,
    attention agrees on sampled rows in every layer, caches match after compaction."""
    w = wl.make("c5")
    ram, t1, t2 = oracle.lmhead(w.hidden, w.W)
    wl.plant(w, ram.reshape(w.B, w.T_max))
    G = oracle.Geometry.of(w)
    ref_acc = oracle.accept(G, w.draft_tok, ram.reshape(w.B, w.T_max))
    np.testing.assert_array_equal(ref_acc[0], w.planted_len + 1)

    vs = VerifyStep(w)
    for l in range(vs.L):                              # one call per layer ...
        vs.attention(l)
    torch.cuda.synchronize()
    single = [o.clone() for o in vs.out]
    for o in vs.out:
        o.fill_(7.0)
    vs.attention_layers()                              # ... and all layers in one call, as run() does
    vs.lmhead()
    torch.cuda.synchronize()
    vs.check_status()
    for l in range(vs.L):                              # the two ways differ only by fp32 merge rounding
        a, s1 = vs.out[l].float(), single[l].float()
        d = (a - s1).abs().max().item()
        assert d <= 2e-3, f"layer {l}: all-layers call differs from the single-layer call by {d}"
        rel = (a - s1).norm(dim=-1) / (s1.norm(dim=-1) + 1e-6)        # per row: a wrong group cannot hide
        assert rel.max().item() <= 1e-2, f"layer {l}: a row differs from the single-layer call by {rel.max().item():.3f}"
    am = vs.argmax.cpu().numpy()
    in_band, mis_in, mis_out = check_argmax(am, vs.maxlogit.cpu().numpy(), ram, t1, t2)
    print(f"c5 LM head: rows {len(am)}, in band {in_band}, mismatches in band {mis_in}, outside {mis_out}")
    # acceptance on the checker's argmax is bit exact
    vs.accept(target=to_device(ram))
    vs.compact()
    torch.cuda.synchronize()
    vs.check_status()
    for got, ref in zip((vs.n_acc, vs.path, vs.out_tok, vs.new_len), ref_acc):
        np.testing.assert_array_equal(got.cpu().numpy(), ref)
    rows = sample_rows(w, 24, 9)
    for l in range(w.L):
        if l in (0, w.L // 2, w.L - 1):              # three layers in full, row by row
            ref, _ = oracle.attention(G, w.k_cache[l], w.v_cache[l], w.q[l], w.k_tree[l], w.v_tree[l], w.scale)
            got = vs.out[l].float().cpu().numpy()
            check_attention(got, ref, f"layer {l}")
            check_every_row(got, ref, f"layer {l}")
        else:                                        # the others on sampled rows (and, above, every row against the one-layer call)
            ref, _ = oracle.attention_rows(G, w.k_cache[l], w.v_cache[l], w.q[l], w.k_tree[l], w.v_tree[l], w.scale, rows)
            got = vs.out[l].float().cpu().numpy()[rows[:, 0], rows[:, 1], rows[:, 2]]
            check_attention(got, ref, f"layer {l}")
        rk, rv = w.k_cache[l], w.v_cache[l]          # compact the host copy in place
        oracle.compact(G, rk, rv, w.k_tree[l], w.v_tree[l], ref_acc[0], ref_acc[1])
        assert np.array_equal(vs.k_cache[l].cpu().numpy().view(np.uint16), rk)
        assert np.array_equal(vs.v_cache[l].cpu().numpy().view(np.uint16), rv)


@pytest.mark.parametrize("cfg", ["c3", "c4"])
def test_whole_chain_at_the_configured_shape(cfg):
    """c3 (240 rows) and c4 (960 rows, 16 ragged sequences, shuffled paged table, tree depths 4-7) at the
    configured sizes: LM head over vocabulary 152064 against the checker (band rule, three counts), greedy
    acceptance on the checker's arg-max with planted paths (bit exact), compaction through the block
    table at the real lengths (caches byte-equal), then the same three steps through the fused call."""
    w = wl.make(cfg)
    ram, t1, t2 = oracle.lmhead(w.hidden, w.W)
    wl.plant(w, ram.reshape(w.B, w.T_max))
    G = oracle.Geometry.of(w)
    ref_acc = oracle.accept(G, w.draft_tok, ram.reshape(w.B, w.T_max))
    np.testing.assert_array_equal(ref_acc[0], w.planted_len + 1)
    vs = VerifyStep(w)
    vs.lmhead()
    torch.cuda.synchronize()
    vs.check_status()
    am = vs.argmax.cpu().numpy()
    in_band, mis_in, mis_out = check_argmax(am, vs.maxlogit.cpu().numpy(), ram, t1, t2)
    print(f"{cfg} LM head: rows {len(am)}, in band {in_band}, mismatches in band {mis_in}, outside {mis_out}")
    vs.accept(target=to_device(ram))
    vs.compact()
    torch.cuda.synchronize()
    vs.check_status()
    for got, ref in zip((vs.n_acc, vs.path, vs.out_tok, vs.new_len), ref_acc):
        np.testing.assert_array_equal(got.cpu().numpy(), ref)
    rk, rv = w.k_cache[0].copy(), w.v_cache[0].copy()
    oracle.compact(G, rk, rv, w.k_tree[0], w.v_tree[0], ref_acc[0], ref_acc[1])
    assert not np.array_equal(rk, w.k_cache[0])
    assert np.array_equal(vs.k_cache[0].cpu().numpy().view(np.uint16), rk)
    assert np.array_equal(vs.v_cache[0].cpu().numpy().view(np.uint16), rv)
    # the fused call on fresh caches: its own arg-max decides, so rows inside the band may move a path;
    # where its arg-max equals the checker's on every row of a sequence, that sequence must agree exactly
    vs2 = VerifyStep(w)
    vs2.tail()
    torch.cuda.synchronize()
    vs2.check_status()
    am2 = vs2.argmax.cpu().numpy().reshape(w.B, w.T_max)
    same = (am2 == ram.reshape(w.B, w.T_max)).all(axis=1)
    assert same.sum() >= w.B // 2
    for got, ref in zip((vs2.n_acc, vs2.path, vs2.out_tok, vs2.new_len), ref_acc):
        np.testing.assert_array_equal(got.cpu().numpy()[same], ref[same])
    if same.all():
        assert np.array_equal(vs2.k_cache[0].cpu().numpy().view(np.uint16), rk)
        assert np.array_equal(vs2.v_cache[0].cpu().numpy().view(np.uint16), rv)


# ------------------------------------------------------------------ several steps in a row: lossless decoding
def test_speculative_loop_on_gpu_is_lossless():
    """Twelve verify steps of a toy target (one attention layer + LM head; a token's q/k/v rows depend
    on the token only) through the library: arbitrary draft trees, attention, fused LM head +
    acceptance + compaction, lengths advanced from new_len.  The emitted tokens must equal plain
    sequential greedy decoding computed in fp64 on the host, and the caches must hold exactly the
    committed tokens' K/V rows (Sec. 4.1 of the paper: verification leaves the target's output
    unchanged).  Logit gaps of the toy are checked to be far above bf16 rounding first."""
    D, V, T, B, steps = 128, 40, 8, 2, 12
    g = np.random.default_rng(10)
    mk = lambda s: wl.f32_to_bf16_bits((s * g.standard_normal((V, D))).astype(np.float32))
    Eq, Ek, Ev, W = mk(2.0), mk(1.0), mk(1.0), mk(1.0)
    f64 = wl.bf16_bits_to_f64

    def greedy(prompt, n_new):
        toks, min_gap = list(prompt), np.inf
        for _ in range(n_new):
            s = f64(Ek[toks]) @ f64(Eq[toks[-1]]) / np.sqrt(D)
            w = np.exp(s - s.max())
            hid = wl.f32_to_bf16_bits(((w[:, None] * f64(Ev[toks])).sum(0) / w.sum()).astype(np.float32))
            lg = f64(W) @ f64(hid)
            top = np.sort(lg)[-2:]
            min_gap = min(min_gap, top[1] - top[0])
            toks.append(int(np.argmax(lg)))
        return toks, min_gap

    prompts = [[3, 1, 4, 1, 5, 9, 2, 6], [7, 7, 2, 30, 11] + [(5 * i + 3) % V for i in range(60)]]   # the second starts past a block
    want, gaps = zip(*(greedy(p, 7 * steps) for p in prompts))
    assert min(gaps) > 0.04, gaps        # bf16 rounding of the hidden state moves a logit by about 0.002

    nblk_per = 4
    table = np.array([[2, 0, 3, 1], [5, 7, 4, 6]], dtype=np.int32)
    kc = np.zeros((B * nblk_per, 1, 64, D), dtype=np.uint16); vc = np.zeros_like(kc)
    committed = [list(p) for p in prompts]
    for b in range(B):
        for t, x in enumerate(committed[b][:-1]):
            kc[table[b, t // 64], 0, t % 64] = Ek[x]; vc[table[b, t // 64], 0, t % 64] = Ev[x]
    kcd, vcd = to_device(kc), to_device(vc)
    Wd = to_device(W)
    st = sd.new_status()
    emitted = []
    for step in range(steps):
        par = np.stack([np.array([-1] + [int(g.integers(0, i)) for i in range(1, T)], dtype=np.int32) for _ in range(B)])
        tok = np.zeros((B, T), dtype=np.int32)
        for b in range(B):
            truth = greedy(committed[b], 7)[0][len(committed[b]):]
            tok[b, 0] = committed[b][-1]
            depth = np.zeros(T, dtype=int)
            for i in range(1, T):
                depth[i] = depth[par[b, i]] + 1
                sib = {int(tok[b, j]) for j in range(1, i) if par[b, j] == par[b, i]}
                cand = truth[depth[i] - 1] if g.random() < 0.6 else int(g.integers(0, V))
                while cand in sib:                                  # siblings carry distinct tokens
                    cand = int(g.integers(0, V))
                tok[b, i] = cand
        lens = np.array([len(c) - 1 for c in committed], dtype=np.int32)
        bt = sd.Batch(B, T, 1, 1, D, table, lens, np.full(B, T, np.int32), par)
        sd.sd_tree_prepare(bt, st)
        q, kt, vt = to_device(Eq[tok][:, :, None, :]), to_device(Ek[tok][:, :, None, :]), to_device(Ev[tok][:, :, None, :])
        out = torch.zeros((B, T, 1, D), dtype=torch.bfloat16, device="cuda")
        ws = torch.empty(sd.sd_workspace_bytes(bt, B * T, V), dtype=torch.uint8, device="cuda")
        sd.sd_verify_attention(bt, sd.kv_layer(kcd, vcd), q, kt, vt, 1.0 / np.sqrt(D), out, None, ws, st)
        hidden = out.view(torch.int16).reshape(B * T, D)             # the attention output IS the hidden state
        am = torch.zeros(B * T, dtype=torch.int32, device="cuda")
        n_acc = torch.zeros(B, dtype=torch.int32, device="cuda"); new_len = torch.zeros(B, dtype=torch.int32, device="cuda")
        path = torch.zeros((B, T), dtype=torch.int32, device="cuda"); out_tok = torch.zeros((B, T), dtype=torch.int32, device="cuda")
        ls = sd.LayerSet([kcd], [vcd], [kt], [vt])
        sd.sd_lmhead_accept_compact(bt, hidden, Wd, to_device(tok), ls, am, None, n_acc, path, out_tok, new_len, ws, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        na, ot, nl = n_acc.cpu().numpy(), out_tok.cpu().numpy(), new_len.cpu().numpy()
        for b in range(B):
            committed[b] += [int(x) for x in ot[b, :na[b]]]
            assert nl[b] == len(committed[b]) - 1
        emitted.append(int(na.sum()))
    for b in range(B):
        assert committed[b] == want[b][:len(committed[b])]
    assert max(emitted) > B                                           # speculation accepted drafts
    kc_after, vc_after = kcd.cpu().numpy().view(np.uint16), vcd.cpu().numpy().view(np.uint16)
    for b in range(B):
        for t, x in enumerate(committed[b][:-1]):
            np.testing.assert_array_equal(kc_after[table[b, t // 64], 0, t % 64], Ek[x])
            np.testing.assert_array_equal(vc_after[table[b, t // 64], 0, t % 64], Ev[x])
