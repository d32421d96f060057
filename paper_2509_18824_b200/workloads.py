"""Seeded synthetic inputs for draft-tree verification.

This module only *makes inputs*: random bf16 tensors, tree shapes, block
tables, prefix lengths and planted draft tokens.  It holds none of the
arithmetic of the verification step itself (no attention, no projection, no
acceptance rule, no ancestor-mask construction), so both the GPU library and
the independent CPU checker can be fed the very same bits from here without
sharing any of their own code.

All tensors are numpy arrays.  bf16 values are carried as ``uint16`` bit
patterns.  Random numbers come from numpy's counter-based Philox generator,
keyed by ``(seed, crc32(tensor name), chunk index)``, so every tensor is
reproducible on any machine and independent of the order of generation.

The shapes stand in for a 7B-class GQA decoder (28 query heads, 4 KV heads,
head_dim 128, hidden 3584, vocabulary 152064) serving long interleaved
multimodal contexts; the paper evaluates on real multimodal data with trained
weights, which these synthetic tensors replace.
"""
from __future__ import annotations

import zlib
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

BLOCK = 64          # tokens per KV-cache block
GENERATOR_VERSION = 1


# --------------------------------------------------------------------------
# bf16 bit helpers (representation only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even), returned as uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# --------------------------------------------------------------------------
# keyed random streams
# --------------------------------------------------------------------------
def stream(seed: int, name: str, chunk: int = 0) -> np.random.Generator:
    """Independent generator for (seed, tensor name, chunk)."""
    h = zlib.crc32(name.encode())
    return np.random.Generator(np.random.Philox(key=[(int(seed) << 32) | h, int(chunk)]))


_CHUNK = 1 << 22


def normal_bf16(seed: int, name: str, shape, scale: float, threads: int = 8) -> np.ndarray:
    """bf16 bits of ``scale * N(0,1)`` with the given shape."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    nchunks = (n + _CHUNK - 1) // _CHUNK

    def work(c):
        lo = c * _CHUNK
        hi = min(n, lo + _CHUNK)
        g = stream(seed, name, c)
        x = g.standard_normal(hi - lo, dtype=np.float32)
        x *= np.float32(scale)
        out[lo:hi] = f32_to_bf16_bits(x)

    if nchunks <= 1 or threads <= 1:
        for c in range(nchunks):
            work(c)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(nchunks)))
    return out.reshape(shape)


# --------------------------------------------------------------------------
# tree shapes
# --------------------------------------------------------------------------
TINY_PARENTS = np.array([-1, 0, 0, 1, 1, 2, 3, 3], dtype=np.int32)   # 8 nodes, depth 3


def chain_tree(n_nodes: int) -> np.ndarray:
    """Chain decoding: node i hangs off node i-1."""
    return np.arange(-1, n_nodes - 1, dtype=np.int32)


def eagle_style_tree(g: np.random.Generator, n_nodes: int, depth: int, topk: int = 10) -> np.ndarray:
    """Parent array of a synthetic draft tree grown level by level.

    Each level expands at most ``topk`` frontier nodes into ``topk`` candidate
    children whose scores are the parent's cumulative score plus a negative,
    rank-decaying random increment; the ``topk`` best candidates of a level form
    the next frontier.  After ``depth`` levels the ``n_nodes - 1`` candidates
    with the best cumulative score are kept (the set is ancestor-closed because
    scores fall along every path).  If that set does not reach ``depth``, its
    worst leaves are exchanged for the best chain that does.  Nodes are
    numbered by (depth, score) so that ``parent[i] < i``; node 0 is the root.
    """
    assert n_nodes >= depth + 1 and depth >= 1
    # candidate records: cum score, parent candidate index (-1 = root), level
    cum: List[float] = []
    par: List[int] = []
    lvl: List[int] = []
    frontier = [(-1, 0.0)]
    for level in range(1, depth + 1):
        level_ids = []
        for (pid, pcum) in frontier:
            inc = np.cumsum(g.exponential(0.7, size=topk)) + 0.05
            for k in range(topk):
                cum.append(pcum - float(inc[k]))
                par.append(pid)
                lvl.append(level)
                level_ids.append(len(cum) - 1)
        level_ids.sort(key=lambda c: -cum[c])
        frontier = [(c, cum[c]) for c in level_ids[:topk]]
    order = sorted(range(len(cum)), key=lambda c: -cum[c])
    keep = set(order[: n_nodes - 1])
    if max(lvl[c] for c in keep) < depth:
        best_deep = max((c for c in range(len(cum)) if lvl[c] == depth), key=lambda c: cum[c])
        chain = []
        c = best_deep
        while c != -1:
            chain.append(c)
            c = par[c]
        chain_set = set(chain)
        keep |= chain_set
        while len(keep) > n_nodes - 1:
            has_child = {par[c] for c in keep}
            leaves = [c for c in keep if c not in has_child and c not in chain_set]
            worst = min(leaves, key=lambda c: cum[c])
            keep.remove(worst)
    kept = sorted(keep, key=lambda c: (lvl[c], -cum[c]))
    new_id = {c: i + 1 for i, c in enumerate(kept)}
    new_id[-1] = 0
    parents = np.full(n_nodes, -1, dtype=np.int32)
    for c in kept:
        parents[new_id[c]] = new_id[par[c]]
    assert all(0 <= parents[i] < i for i in range(1, n_nodes))
    return parents


def node_depths(parents: np.ndarray) -> np.ndarray:
    """Depth of every node (root = 0) of one parent array; shape bookkeeping
    for the generators only."""
    d = np.zeros(len(parents), dtype=np.int32)
    for i in range(1, len(parents)):
        d[i] = d[parents[i]] + 1
    return d


# --------------------------------------------------------------------------
# workload description
# --------------------------------------------------------------------------
@dataclass
class Spec:
    name: str
    seed: int
    B: int
    Hq: int
    Hkv: int
    D: int
    T: int                      # tree nodes per sequence, root included
    tree: str                   # "tiny" | "eagle" | "chain"
    depth: int                  # tree depth (edges below the root); for "eagle"
    depth_range: Optional[tuple] = None   # per-sequence depth drawn from this range
    prefix: int = 0             # fixed prefix length, or
    prefix_range: Optional[tuple] = None  # per-sequence uniform range
    paged_shuffle: bool = False
    image_prefix: int = 0       # first this many positions get 2x variance K/V
    Hd: int = 3584
    V: int = 152064
    L: int = 1
    plant: bool = False
    q_gain: float = 1.0         # stress: multiply q by this
    hidden_gain: float = 1.0    # stress: multiply hidden by this
    v_gain: float = 1.0
    spare_blocks: int = 3


def spec(config: str) -> Spec:
    """The five benchmark configurations plus supplements, by name."""
    c = config
    if c == "c1":
        return Spec("c1", 0, 1, 4, 1, 128, 8, "tiny", 3, prefix=128, Hd=256, V=1024)
    if c == "c2":
        return Spec("c2", 1, 1, 28, 4, 128, 60, "eagle", 6, prefix=2048)
    if c == "c3":
        return Spec("c3", 2, 4, 28, 4, 128, 60, "eagle", 6, prefix=8192, image_prefix=4096)
    if c == "c4":
        return Spec("c4", 3, 16, 28, 4, 128, 60, "eagle", 6, depth_range=(4, 7),
                    prefix_range=(512, 16384), paged_shuffle=True)
    if c == "c5":
        return Spec("c5", 4, 8, 28, 4, 128, 60, "eagle", 6, prefix=4096, L=28, plant=True)
    if c == "chain11":   # the paper's own setting: 10 drafted tokens in a chain
        return Spec("chain11", 5, 8, 28, 4, 128, 11, "chain", 10, prefix=4096, L=1)
    if c == "tree28":    # a short tree (root + 27 drafts, depth 5): 196 query rows per KV head, near the ridge point
        return Spec("tree28", 6, 8, 28, 4, 128, 28, "eagle", 5, prefix=4096, L=1)
    raise KeyError(config)


@dataclass
class Workload:
    spec: Spec
    B: int
    T_max: int
    Hq: int
    Hkv: int
    D: int
    Hd: int
    V: int
    L: int
    num_blocks: int
    max_blocks: int
    len: np.ndarray             # [B] i32
    n_nodes: np.ndarray         # [B] i32
    parents: np.ndarray         # [B,T_max] i32
    block_table: np.ndarray     # [B,max_blocks] i32
    q: List[np.ndarray] = field(default_factory=list)        # L x [B,T,Hq,D] u16
    k_tree: List[np.ndarray] = field(default_factory=list)   # L x [B,T,Hkv,D] u16
    v_tree: List[np.ndarray] = field(default_factory=list)
    k_cache: List[np.ndarray] = field(default_factory=list)  # L x [num_blocks,Hkv,64,D] u16
    v_cache: List[np.ndarray] = field(default_factory=list)
    hidden: Optional[np.ndarray] = None                       # [B*T,Hd] u16
    W: Optional[np.ndarray] = None                            # [V,Hd] u16
    draft_tok: Optional[np.ndarray] = None                    # [B,T] i32
    planted_len: Optional[np.ndarray] = None                  # [B] i32 (after plant())
    planted_node: Optional[np.ndarray] = None

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.D))

    @property
    def M(self) -> int:
        return self.B * self.T_max


def make_geometry(sp: Spec) -> Workload:
    """Lengths, trees and block table (no big tensors)."""
    g = stream(sp.seed, "geometry")
    B, T = sp.B, sp.T
    if sp.prefix_range is not None:
        lo, hi = sp.prefix_range
        lens = g.integers(lo, hi + 1, size=B).astype(np.int32)
    else:
        lens = np.full(B, sp.prefix, dtype=np.int32)
    parents = np.zeros((B, T), dtype=np.int32)
    for b in range(B):
        gt = stream(sp.seed, "tree", b)
        if sp.tree == "tiny":
            assert T == 8
            parents[b] = TINY_PARENTS
        elif sp.tree == "chain":
            parents[b] = chain_tree(T)
        else:
            d = sp.depth
            if sp.depth_range is not None:
                d = int(gt.integers(sp.depth_range[0], sp.depth_range[1] + 1))
            parents[b] = eagle_style_tree(gt, T, d)
    n_nodes = np.full(B, T, dtype=np.int32)
    need = (lens.astype(np.int64) + T + BLOCK - 1) // BLOCK          # blocks per sequence
    max_blocks = int(need.max())
    num_blocks = int(need.sum()) + sp.spare_blocks
    if sp.paged_shuffle:
        pool = g.permutation(num_blocks).astype(np.int32)
    else:
        pool = np.arange(num_blocks, dtype=np.int32)
    table = np.zeros((B, max_blocks), dtype=np.int32)
    at = 0
    for b in range(B):
        nb = int(need[b])
        table[b, :nb] = pool[at:at + nb]
        table[b, nb:] = pool[at]          # unused entries stay valid block ids
        at += nb
    return Workload(sp, B, T, sp.Hq, sp.Hkv, sp.D, sp.Hd, sp.V, sp.L, num_blocks, max_blocks,
                    lens, n_nodes, parents, table)


def fill_attention(w: Workload, layers: Optional[List[int]] = None, poison_tail: bool = True,
                   threads: int = 8) -> Workload:
    """q / tree K,V / paged cache K,V for the given layers (default all)."""
    sp = w.spec
    s = 1.0 / np.sqrt(sp.D)
    layers = list(range(w.L)) if layers is None else layers
    w.q, w.k_tree, w.v_tree, w.k_cache, w.v_cache = [], [], [], [], []
    for l in layers:
        q = normal_bf16(sp.seed, f"q{l}", (w.B, w.T_max, w.Hq, w.D), s * sp.q_gain, threads)
        kt = normal_bf16(sp.seed, f"kt{l}", (w.B, w.T_max, w.Hkv, w.D), s, threads)
        vt = normal_bf16(sp.seed, f"vt{l}", (w.B, w.T_max, w.Hkv, w.D), s * sp.v_gain, threads)
        kc = normal_bf16(sp.seed, f"kc{l}", (w.num_blocks, w.Hkv, BLOCK, w.D), s, threads)
        vc = normal_bf16(sp.seed, f"vc{l}", (w.num_blocks, w.Hkv, BLOCK, w.D), s * sp.v_gain, threads)
        if sp.image_prefix > 0:
            # first `image_prefix` positions of every sequence: variance doubled
            nb_img = sp.image_prefix // BLOCK
            for b in range(w.B):
                blk = w.block_table[b, :nb_img]
                for arr in (kc, vc):
                    x = bf16_bits_to_f32(arr[blk]) * np.float32(np.sqrt(2.0))
                    arr[blk] = f32_to_bf16_bits(x)
        if poison_tail:
            # slots at and beyond len[b] hold large finite garbage that must not matter
            big = f32_to_bf16_bits(np.array([6.0e4, -6.0e4], dtype=np.float32))
            for b in range(w.B):
                P = int(w.len[b])
                nb = (P + w.T_max + BLOCK - 1) // BLOCK
                for j in range(P // BLOCK, nb):
                    lo = max(0, P - j * BLOCK)
                    blk = int(w.block_table[b, j])
                    for arr in (kc, vc):
                        arr[blk, :, lo:, 0::2] = big[0]
                        arr[blk, :, lo:, 1::2] = big[1]
        w.q.append(q); w.k_tree.append(kt); w.v_tree.append(vt)
        w.k_cache.append(kc); w.v_cache.append(vc)
    return w


def fill_lmhead(w: Workload, threads: int = 8) -> Workload:
    sp = w.spec
    s = 1.0 / np.sqrt(w.Hd)
    w.hidden = normal_bf16(sp.seed, "hidden", (w.B * w.T_max, w.Hd), s * sp.hidden_gain, threads)
    w.W = normal_bf16(sp.seed, "W", (w.V, w.Hd), s, threads)
    w.draft_tok = stream(sp.seed, "draft").integers(0, w.V, size=(w.B, w.T_max)).astype(np.int32)
    return w


def plant(w: Workload, target_argmax: np.ndarray, lengths: Optional[np.ndarray] = None) -> Workload:
    """Rewrite ``draft_tok`` so that exactly one path of a drawn length matches.

    ``target_argmax`` ([B,T] int) is supplied by the caller.  Per sequence a
    length l in 0..depth and a node at depth l are drawn; draft tokens along
    its root path are set to the target token of their parent; every other
    node gets a token that differs from its parent's target token and from its
    already-assigned siblings.
    """
    sp = w.spec
    g = stream(sp.seed, "plant")
    a = np.asarray(target_argmax).reshape(w.B, w.T_max)
    tok = np.zeros((w.B, w.T_max), dtype=np.int32)
    w.planted_len = np.zeros(w.B, dtype=np.int32)
    w.planted_node = np.zeros(w.B, dtype=np.int32)
    for b in range(w.B):
        par = w.parents[b]
        n = int(w.n_nodes[b])
        dep = node_depths(par[:n])
        maxd = int(dep.max())
        l = int(g.integers(0, maxd + 1)) if lengths is None else int(lengths[b])
        cands = np.nonzero(dep == l)[0]
        node = int(cands[int(g.integers(0, len(cands)))])
        on_path = set()
        c = node
        while c > 0:
            on_path.add(c)
            c = int(par[c])
        used: Dict[int, set] = {}
        tok[b, 0] = int(g.integers(0, w.V))
        for j in sorted(on_path):
            tok[b, j] = a[b, par[j]]
            used.setdefault(int(par[j]), set()).add(int(tok[b, j]))
        for j in range(1, n):
            if j in on_path:
                continue
            p = int(par[j])
            s = used.setdefault(p, set())
            while True:
                t = int(g.integers(0, w.V))
                if t != int(a[b, p]) and t not in s:
                    break
            tok[b, j] = t
            s.add(t)
        w.planted_len[b] = l
        w.planted_node[b] = node
    w.draft_tok = tok
    return w


def make(config: str, attention: bool = True, lmhead: bool = True,
         layers: Optional[List[int]] = None, threads: int = 8, **overrides) -> Workload:
    sp = spec(config)
    for k, v in overrides.items():
        setattr(sp, k, v)
    w = make_geometry(sp)
    if attention:
        fill_attention(w, layers, threads=threads)
    if lmhead:
        fill_lmhead(w, threads=threads)
    return w
