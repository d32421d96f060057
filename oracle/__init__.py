"""ctypes front end of the fp64 CPU reference checker (TEST INFRASTRUCTURE ONLY).

The arithmetic lives in ``sd_oracle.c`` (plain C, fp64); this file only
compiles it with gcc when needed and marshals numpy arrays.  It shares nothing
with the GPU library and must never be imported by it: callers are the tests,
the smoke check and the CPU-baseline leg of the benchmark.

Parity with the paper's reported acceptance statistics is unpinned (they need
trained models); every function is pinned by the CPU test-suite against closed
forms, brute force and library routines.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sd_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile sd_oracle.c into liboracle.so next to it (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Geom(C.Structure):
    _fields_ = [("B", C.c_int32), ("T_max", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32),
                ("D", C.c_int32), ("block", C.c_int32), ("max_blocks", C.c_int32),
                ("block_table", C.c_void_p), ("len", C.c_void_p),
                ("n_nodes", C.c_void_p), ("parents", C.c_void_p)]


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_num_threads.restype = C.c_int
        for f in ("orc_attention", "orc_attention_rows", "orc_lmhead", "orc_logits", "orc_compact"):
            getattr(_lib, f).restype = None
        _lib.orc_accept.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(_L().orc_num_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


class Geometry:
    """Host-side description of a batch: lengths, trees, block table."""

    def __init__(self, B, T_max, Hq, Hkv, D, block_table, lens, n_nodes, parents, block=64):
        self.B, self.T_max, self.Hq, self.Hkv, self.D, self.block = B, T_max, Hq, Hkv, D, block
        self.block_table = _c(block_table, np.int32).reshape(B, -1)
        self.len = _c(lens, np.int32)
        self.n_nodes = _c(n_nodes, np.int32)
        self.parents = _c(parents, np.int32).reshape(B, T_max)
        self.max_blocks = self.block_table.shape[1]
        self._g = _Geom(B, T_max, Hq, Hkv, D, block, self.max_blocks,
                        _p(self.block_table), _p(self.len), _p(self.n_nodes), _p(self.parents))

    @classmethod
    def of(cls, w) -> "Geometry":
        """From any object with the attribute names used by the workload generator."""
        return cls(w.B, w.T_max, w.Hq, w.Hkv, w.D, w.block_table, w.len, w.n_nodes, w.parents)

    def ref(self):
        return C.byref(self._g)


def attention(g: Geometry, k_cache, v_cache, q, k_tree, v_tree, scale: float):
    """All rows.  Returns (out [B,T,Hq,D] f64, lse [B,T,Hq] f64); rows of nodes
    beyond n_nodes[b] are NaN."""
    kc, vc, q, kt, vt = (_c(x, np.uint16) for x in (k_cache, v_cache, q, k_tree, v_tree))
    out = np.full((g.B, g.T_max, g.Hq, g.D), np.nan, dtype=np.float64)
    lse = np.full((g.B, g.T_max, g.Hq), np.nan, dtype=np.float64)
    _L().orc_attention(g.ref(), _p(kc), _p(vc), _p(q), _p(kt), _p(vt), C.c_double(scale), _p(out), _p(lse))
    return out, lse


def attention_rows(g: Geometry, k_cache, v_cache, q, k_tree, v_tree, scale: float, rows):
    """Sampled rows: ``rows`` is [n,3] of (b, node, head).  Returns (out [n,D], lse [n])."""
    kc, vc, q, kt, vt = (_c(x, np.uint16) for x in (k_cache, v_cache, q, k_tree, v_tree))
    rows = _c(rows, np.int32).reshape(-1, 3)
    n = rows.shape[0]
    out = np.zeros((n, g.D), dtype=np.float64)
    lse = np.zeros(n, dtype=np.float64)
    _L().orc_attention_rows(g.ref(), _p(kc), _p(vc), _p(q), _p(kt), _p(vt), C.c_double(scale),
                            _p(rows), C.c_int(n), _p(out), _p(lse))
    return out, lse


def lmhead(hidden, W, rows: Optional[Sequence[int]] = None):
    """Returns (argmax i32, top1 f64, top2 f64) for all rows or the listed rows."""
    hidden, W = _c(hidden, np.uint16), _c(W, np.uint16)
    M, Hd = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == Hd
    r = None if rows is None else _c(rows, np.int32)
    n = M if r is None else len(r)
    am = np.zeros(n, dtype=np.int32)
    t1 = np.zeros(n, dtype=np.float64)
    t2 = np.zeros(n, dtype=np.float64)
    _L().orc_lmhead(_p(hidden), _p(W), C.c_int(M), C.c_int(Hd), C.c_int(V), _p(r), C.c_int(n),
                    _p(am), _p(t1), _p(t2))
    return am, t1, t2


def logits(hidden, W):
    hidden, W = _c(hidden, np.uint16), _c(W, np.uint16)
    M, Hd = hidden.shape
    V = W.shape[0]
    out = np.zeros((M, V), dtype=np.float64)
    _L().orc_logits(_p(hidden), _p(W), C.c_int(M), C.c_int(Hd), C.c_int(V), _p(out))
    return out


def accept(g: Geometry, draft_tok, target_argmax):
    """Returns (n_acc [B], path [B,T], out_tok [B,T], new_len [B]); raises on a bad tree."""
    dt = _c(draft_tok, np.int32).reshape(g.B, g.T_max)
    tg = _c(target_argmax, np.int32).reshape(g.B, g.T_max)
    n_acc = np.zeros(g.B, dtype=np.int32)
    path = np.zeros((g.B, g.T_max), dtype=np.int32)
    out_tok = np.zeros((g.B, g.T_max), dtype=np.int32)
    new_len = np.zeros(g.B, dtype=np.int32)
    rc = _L().orc_accept(g.ref(), _p(dt), _p(tg), _p(n_acc), _p(path), _p(out_tok), _p(new_len))
    if rc != 0:
        raise ValueError("parent array is not a tree with parent < child")
    return n_acc, path, out_tok, new_len


def compact(g: Geometry, k_cache, v_cache, k_tree, v_tree, n_acc, path):
    """One layer, in place on ``k_cache``/``v_cache`` (uint16, C-contiguous)."""
    for a in (k_cache, v_cache):
        assert a.dtype == np.uint16 and a.flags["C_CONTIGUOUS"] and a.flags["WRITEABLE"]
    kt, vt = _c(k_tree, np.uint16), _c(v_tree, np.uint16)
    na, pa = _c(n_acc, np.int32), _c(path, np.int32)
    _L().orc_compact(g.ref(), _p(k_cache), _p(v_cache), _p(kt), _p(vt), _p(na), _p(pa))
