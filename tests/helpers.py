"""Small shared helpers for the tests: tiny random problems in numpy."""
import numpy as np

from paper_2509_18824_b200 import workloads as wl


class Tiny:
    """A small attention/accept problem with the attribute names the checker's
    Geometry.of() expects."""

    def __init__(self, seed, B=2, T=8, Hq=4, Hkv=2, D=16, lens=(5, 70), parents=None,
                 shuffle=True, gain=4.0, spare=2, block=64):
        g = np.random.default_rng(seed)
        self.B, self.T_max, self.Hq, self.Hkv, self.D = B, T, Hq, Hkv, D
        self.len = np.array(lens, dtype=np.int32)
        assert len(lens) == B
        if parents is None:
            parents = np.zeros((B, T), dtype=np.int32)
            for b in range(B):
                parents[b, 0] = -1
                for i in range(1, T):
                    parents[b, i] = g.integers(0, i)
        self.parents = np.asarray(parents, dtype=np.int32).reshape(B, T)
        self.n_nodes = np.full(B, T, dtype=np.int32)
        need = (self.len.astype(np.int64) + T + block - 1) // block
        self.max_blocks = int(need.max())
        self.num_blocks = int(need.sum()) + spare
        pool = g.permutation(self.num_blocks) if shuffle else np.arange(self.num_blocks)
        self.block_table = np.zeros((B, self.max_blocks), dtype=np.int32)
        at = 0
        for b in range(B):
            self.block_table[b, :need[b]] = pool[at:at + need[b]]
            self.block_table[b, need[b]:] = pool[at]
            at += need[b]
        s = 1.0 / np.sqrt(D)

        def rnd(shape, k=1.0):
            return wl.f32_to_bf16_bits((g.standard_normal(shape) * s * k).astype(np.float32))

        self.q = rnd((B, T, Hq, D), gain * np.sqrt(D))
        self.k_tree = rnd((B, T, Hkv, D))
        self.v_tree = rnd((B, T, Hkv, D), 3.0)
        self.k_cache = rnd((self.num_blocks, Hkv, block, D))
        self.v_cache = rnd((self.num_blocks, Hkv, block, D), 3.0)
        self.scale = float(s)

    # logical (unpaged) view of the prefix of sequence b, head kvh: [P, D] float64
    def prefix(self, cache, b, kvh):
        P = int(self.len[b])
        rows = []
        for t in range(P):
            blk = self.block_table[b, t // 64]
            rows.append(cache[blk, kvh, t % 64])
        if not rows:
            return np.zeros((0, self.D))
        return wl.bf16_bits_to_f64(np.stack(rows))


def root_path(parents, i):
    """Nodes from the root down to i (inclusive)."""
    p = []
    while i >= 0:
        p.append(int(i))
        i = int(parents[i])
    return p[::-1]
