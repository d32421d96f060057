"""ctypes binding of libsdverify.so: same names as the C header, argument
marshalling only.  Tensors are torch CUDA tensors (device memory and streams
are all torch is used for); every step of the computation runs in the
library's kernels.  There is no CPU fallback: if the shared library cannot be
loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsdverify.so")

SD_OK = 0
SD_ERR_INVALID_ARG = -1
SD_ERR_INVALID_TREE = -2
SD_ERR_UNSUPPORTED = -3
SD_ERR_WORKSPACE = -4
SD_ERR_CUDA = -5
SD_ERR_TIMEOUT = -6
SD_ERR_BOUNDS = -7

# kernel launches behind one call (kept in step with the kernels; used for launch accounting)
KERNELS_PER_ATTENTION = 1      # split-KV chunks merge inside the kernel (thread-block cluster)
ATTENTION_LAYERS_PER_LAUNCH = 32   # sd_verify_attention_layers: layers sharing one launch
KERNELS_PER_TAIL = 2               # sd_lmhead_accept_compact: LM-head tiles + fused tail kernel
KERNELS_PER_LMHEAD = 2         # tiles + cross-slab reduce
KERNELS_PER_SAMPLED_TAIL = 2       # sd_lmhead_accept_sampled_compact: LM-head tiles + one cluster kernel

EXPORTS = ["sd_version", "sd_status_string", "sd_workspace_bytes", "sd_tree_prepare",
           "sd_verify_attention", "sd_verify_attention_layers", "sd_lmhead_argmax", "sd_lmhead_argmax_static", "sd_accept_tree",
           "sd_compact_kv", "sd_lmhead_accept_compact", "sd_lmhead_stats", "sd_accept_tree_sampled", "sd_lmhead_accept_sampled_compact", "sd_accept_chain_sampled", "sd_lmhead_stats_logits", "sd_accept_tree_sampled_q",
           "sd_draft_feature_attention"]


class sd_kv_layer(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("num_blocks", C.c_int32)]


class sd_batch(C.Structure):
    _fields_ = [("B", C.c_int32), ("T_max", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32),
                ("D", C.c_int32), ("block_size", C.c_int32), ("max_blocks_per_seq", C.c_int32),
                ("block_table", C.c_void_p), ("len", C.c_void_p), ("n_nodes", C.c_void_p),
                ("parents", C.c_void_p), ("anc_mask", C.c_void_p)]


def _load(path: str = LIB_PATH) -> C.CDLL:
    if path == LIB_PATH and not os.path.exists(LIB_PATH):
        from . import build as _build          # needs nvcc; raises if it fails
        _build.build()
    lib = C.CDLL(path)
    lib.sd_version.restype = C.c_int
    lib.sd_status_string.restype = C.c_char_p
    lib.sd_status_string.argtypes = [C.c_int]
    lib.sd_workspace_bytes.restype = C.c_size_t
    lib.sd_workspace_bytes.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
    lib.sd_tree_prepare.restype = C.c_int
    lib.sd_tree_prepare.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    lib.sd_verify_attention.restype = C.c_int
    lib.sd_verify_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                        C.c_void_p, C.c_void_p]
    lib.sd_verify_attention_layers.restype = C.c_int
    lib.sd_verify_attention_layers.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_size_t, C.c_void_p, C.c_void_p]
    lib.sd_lmhead_argmax.restype = C.c_int
    lib.sd_lmhead_argmax.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    lib.sd_lmhead_argmax_static.restype = C.c_int
    lib.sd_lmhead_argmax_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.sd_accept_tree.restype = C.c_int
    lib.sd_accept_tree.argtypes = [C.c_void_p] * 9
    lib.sd_compact_kv.restype = C.c_int
    lib.sd_compact_kv.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.sd_lmhead_accept_compact.restype = C.c_int
    lib.sd_lmhead_accept_compact.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p,
                                             C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    lib.sd_lmhead_stats.restype = C.c_int
    lib.sd_lmhead_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float,
                                    C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                    C.c_void_p, C.c_void_p]
    lib.sd_accept_tree_sampled.restype = C.c_int
    lib.sd_accept_tree_sampled.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    lib.sd_accept_chain_sampled.restype = C.c_int
    lib.sd_accept_tree_sampled_q.restype = C.c_int
    lib.sd_accept_tree_sampled_q.argtypes = [C.c_void_p, C.c_int32, C.c_float] + [C.c_void_p] * 12
    lib.sd_lmhead_stats_logits.restype = C.c_int
    lib.sd_lmhead_stats_logits.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                           C.c_void_p, C.c_void_p]
    lib.sd_accept_chain_sampled.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float,
                                            C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    lib.sd_lmhead_accept_sampled_compact.restype = C.c_int
    lib.sd_lmhead_accept_sampled_compact.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float,
                                                     C.c_void_p, C.c_void_p, C.c_void_p,
                                                     C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                                     C.c_void_p, C.c_void_p,
                                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                                     C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    lib.sd_draft_feature_attention.restype = C.c_int
    lib.sd_draft_feature_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                               C.c_int32, C.c_int32, C.c_float, C.c_void_p, C.c_void_p]
    return lib


lib = _load()


class SdError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(sd_status_string(code))


def sd_version() -> int:
    return int(lib.sd_version())


def sd_status_string(code: int) -> str:
    return lib.sd_status_string(int(code)).decode()


def _check(code: int) -> None:
    if code != SD_OK:
        raise SdError(code)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Batch:
    """Owns the device arrays named by the C struct ``sd_batch``."""

    def __init__(self, B, T_max, Hq, Hkv, D, block_table, lens, n_nodes, parents,
                 block_size=64, device="cuda"):
        dev = torch.device(device)
        to = lambda a: torch.as_tensor(a, dtype=torch.int32).contiguous().to(dev)
        self.B, self.T_max, self.Hq, self.Hkv, self.D = int(B), int(T_max), int(Hq), int(Hkv), int(D)
        self.block_table = to(block_table).reshape(self.B, -1).contiguous()
        self.len = to(lens)
        self.n_nodes = to(n_nodes)
        self.parents = to(parents).reshape(self.B, self.T_max).contiguous()
        self.anc_mask = torch.zeros((self.B, self.T_max), dtype=torch.int64, device=dev)
        self.max_blocks = int(self.block_table.shape[1])
        self.c = sd_batch(self.B, self.T_max, self.Hq, self.Hkv, self.D, int(block_size), self.max_blocks,
                          self.block_table.data_ptr(), self.len.data_ptr(), self.n_nodes.data_ptr(),
                          self.parents.data_ptr(), self.anc_mask.data_ptr())

    @classmethod
    def of(cls, w, device="cuda") -> "Batch":
        """From any object carrying B, T_max, Hq, Hkv, D, block_table, len, n_nodes, parents."""
        return cls(w.B, w.T_max, w.Hq, w.Hkv, w.D, w.block_table, w.len, w.n_nodes, w.parents, device=device)

    def ref(self):
        return C.byref(self.c)


def kv_layer(k_cache: torch.Tensor, v_cache: torch.Tensor) -> sd_kv_layer:
    """Descriptor of one layer's paged cache.  The struct only carries addresses, so the returned
    object also holds on to the two tensors: a descriptor built from temporaries stays valid."""
    layer = sd_kv_layer(_ptr(k_cache), _ptr(v_cache), int(k_cache.shape[0]))
    layer._keep = (k_cache, v_cache)
    return layer


def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=device)


def sd_workspace_bytes(batch: Optional[Batch], M: int = 0, V: int = 0) -> int:
    return int(lib.sd_workspace_bytes(batch.ref() if batch is not None else None, int(M), int(V)))


def sd_tree_prepare(batch: Batch, status: torch.Tensor, stream=None) -> None:
    _check(lib.sd_tree_prepare(batch.ref(), _ptr(status), _stream(stream)))


def sd_verify_attention(batch: Batch, cache: sd_kv_layer, q, k_tree, v_tree, scale: float,
                        out, lse, workspace, status, stream=None) -> None:
    _check(lib.sd_verify_attention(batch.ref(), C.byref(cache), _ptr(q), _ptr(k_tree), _ptr(v_tree),
                                   C.c_float(scale), _ptr(out), _ptr(lse), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _ptr(status),
                                   _stream(stream)))


class AttentionLayerSet:
    """Host arrays of per-layer pointers for ``sd_verify_attention_layers`` (built once, reused)."""

    def __init__(self, k_caches, v_caches, qs, k_trees, v_trees, outs, lses=None):
        L = len(k_caches)
        self.L = L
        self.caches = (sd_kv_layer * L)(*[kv_layer(k, v) for k, v in zip(k_caches, v_caches)])
        self.q = (C.c_void_p * L)(*[_ptr(t) for t in qs])
        self.kt = (C.c_void_p * L)(*[_ptr(t) for t in k_trees])
        self.vt = (C.c_void_p * L)(*[_ptr(t) for t in v_trees])
        self.out = (C.c_void_p * L)(*[_ptr(t) for t in outs])
        self.lse = (C.c_void_p * L)(*[_ptr(t) for t in lses]) if lses is not None else None
        self._keep = (list(k_caches), list(v_caches), list(qs), list(k_trees), list(v_trees), list(outs),
                      list(lses) if lses is not None else None)


def sd_verify_attention_layers(batch: Batch, layers: AttentionLayerSet, scale: float, workspace, status,
                               stream=None) -> None:
    _check(lib.sd_verify_attention_layers(batch.ref(), layers.caches, layers.L, layers.q, layers.kt, layers.vt,
                                          C.c_float(scale), layers.out, layers.lse, _ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _ptr(status),
                                          _stream(stream)))


def sd_lmhead_argmax(hidden, W, argmax, maxlogit, workspace, status, stream=None) -> None:
    M, Hd = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == Hd
    _check(lib.sd_lmhead_argmax(_ptr(hidden), _ptr(W), int(M), int(Hd), int(V), _ptr(argmax),
                                _ptr(maxlogit), _ptr(workspace),
                                workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))


def sd_lmhead_argmax_static(hidden, W, argmax, maxlogit, status, stream=None) -> None:
    """LM-head arg-max using the scratch table built into the library: for callers
    that may not allocate device memory.  At most 512 rows per call."""
    M, Hd = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == Hd
    _check(lib.sd_lmhead_argmax_static(_ptr(hidden), _ptr(W), int(M), int(Hd), int(V), _ptr(argmax),
                                       _ptr(maxlogit), _ptr(status), _stream(stream)))


def sd_accept_tree(batch: Batch, draft_tok, target_argmax, n_acc, path, out_tok, new_len,
                   status, stream=None) -> None:
    _check(lib.sd_accept_tree(batch.ref(), _ptr(draft_tok), _ptr(target_argmax), _ptr(n_acc), _ptr(path),
                              _ptr(out_tok), _ptr(new_len), _ptr(status), _stream(stream)))


class LayerSet:
    """Host arrays of per-layer descriptors for ``sd_compact_kv`` (built once, reused)."""

    def __init__(self, k_caches: Sequence[torch.Tensor], v_caches: Sequence[torch.Tensor],
                 k_trees: Sequence[torch.Tensor], v_trees: Sequence[torch.Tensor]):
        L = len(k_caches)
        self.L = L
        self.layers = (sd_kv_layer * L)(*[kv_layer(k, v) for k, v in zip(k_caches, v_caches)])
        self.kt = (C.c_void_p * L)(*[_ptr(t) for t in k_trees])
        self.vt = (C.c_void_p * L)(*[_ptr(t) for t in v_trees])
        self._keep = (list(k_caches), list(v_caches), list(k_trees), list(v_trees))


def sd_compact_kv(batch: Batch, layers: LayerSet, n_acc, path, status, stream=None) -> None:
    _check(lib.sd_compact_kv(batch.ref(), layers.layers, layers.L, layers.kt, layers.vt,
                             _ptr(n_acc), _ptr(path), _ptr(status), _stream(stream)))


def sd_lmhead_accept_compact(batch: Batch, hidden, W, draft_tok, layers: LayerSet, argmax, maxlogit,
                             n_acc, path, out_tok, new_len, workspace, status, stream=None) -> None:
    """LM-head arg-max over the B * T_max rows of `hidden`, greedy acceptance and KV compaction in all
    layers; the three steps share one tail kernel."""
    M, Hd = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == Hd and M == batch.B * batch.T_max
    _check(lib.sd_lmhead_accept_compact(batch.ref(), _ptr(hidden), _ptr(W), int(Hd), int(V), _ptr(draft_tok),
                                        layers.layers, layers.L, layers.kt, layers.vt, _ptr(argmax), _ptr(maxlogit),
                                        _ptr(n_acc), _ptr(path), _ptr(out_tok), _ptr(new_len), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))


def group_stats_shape(M: int, V: int):
    """Shape (float32) of the optional per-group statistics table of sd_lmhead_stats."""
    return ((V + 31) // 32, M, 2)


def sd_lmhead_stats(hidden, W, inv_temp: float, argmax, maxlogit, lse, workspace, status, stream=None,
                    group_stats=None) -> None:
    """LM-head arg-max plus lse[r] = log sum_v exp(logit[r][v] * inv_temp); optionally the per-group
    (maximum, sum) table that lets sd_accept_tree_sampled skip its second pass over W."""
    M, Hd = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == Hd
    _check(lib.sd_lmhead_stats(_ptr(hidden), _ptr(W), int(M), int(Hd), int(V), C.c_float(inv_temp), _ptr(argmax),
                               _ptr(maxlogit), _ptr(lse), _ptr(group_stats), _ptr(workspace),
                               workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))


def sd_accept_tree_sampled(batch: Batch, hidden, W, inv_temp: float, lse, draft_tok, u, w,
                           n_acc, path, out_tok, new_len, workspace, status, stream=None, group_stats=None) -> None:
    """Acceptance at a sampling temperature (uniforms u [B,T] and w [B] are inputs)."""
    M, Hd = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == Hd and M == batch.B * batch.T_max
    _check(lib.sd_accept_tree_sampled(batch.ref(), _ptr(hidden), _ptr(W), int(Hd), int(V), C.c_float(inv_temp),
                                      _ptr(lse), _ptr(group_stats), _ptr(draft_tok), _ptr(u), _ptr(w), _ptr(n_acc), _ptr(path),
                                      _ptr(out_tok), _ptr(new_len), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))


def sd_lmhead_stats_logits(hidden, W, inv_temp: float, argmax, maxlogit, lse, logits, workspace, status,
                           stream=None) -> None:
    """sd_lmhead_stats that also keeps the raw logits [M,V] (device f32)."""
    M, Hd = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == Hd and tuple(logits.shape) == (M, V) and logits.dtype == torch.float32 and logits.is_contiguous()
    _check(lib.sd_lmhead_stats_logits(_ptr(hidden), _ptr(W), int(M), int(Hd), int(V), C.c_float(inv_temp), _ptr(argmax),
                                      _ptr(maxlogit), _ptr(lse), _ptr(logits), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))


def sd_accept_tree_sampled_q(batch: Batch, inv_temp: float, lse, logits, draft_tok, q_rows, u, w,
                             n_acc, path, out_tok, new_len, status, stream=None) -> None:
    """Acceptance at a sampling temperature for trees whose children were sampled from q_rows [B,T,V];
    lse [M] and logits [M,V] from sd_lmhead_stats_logits (device f32)."""
    M, V = logits.shape
    assert M == batch.B * batch.T_max and tuple(q_rows.shape) == (batch.B, batch.T_max, V)
    assert logits.dtype == torch.float32 and q_rows.dtype == torch.float32 and logits.is_contiguous() and q_rows.is_contiguous()
    _check(lib.sd_accept_tree_sampled_q(batch.ref(), int(V), C.c_float(inv_temp), _ptr(lse), _ptr(logits), _ptr(draft_tok),
                                        _ptr(q_rows), _ptr(u), _ptr(w), _ptr(n_acc), _ptr(path), _ptr(out_tok),
                                        _ptr(new_len), _ptr(status), _stream(stream)))


def sd_accept_chain_sampled(batch: Batch, hidden, W, inv_temp: float, lse, draft_tok, q_tok, q_rows, u, w,
                            n_acc, path, out_tok, new_len, workspace, status, stream=None, logits=None) -> None:
    """Acceptance at a sampling temperature for chains drafted by sampling: q_tok [B,T] the draft's
    probability of every drafted token, q_rows [B,T,V] its distributions (device f32); logits: what
    sd_lmhead_stats_logits kept, or None (the stop rows then go through the LM head once more)."""
    M, Hd = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == Hd and M == batch.B * batch.T_max
    assert tuple(q_rows.shape) == (batch.B, batch.T_max, V) and q_rows.dtype == torch.float32 and q_rows.is_contiguous()
    _check(lib.sd_accept_chain_sampled(batch.ref(), _ptr(hidden), _ptr(W), int(Hd), int(V), C.c_float(inv_temp),
                                       _ptr(lse), _ptr(logits), _ptr(draft_tok), _ptr(q_tok), _ptr(q_rows), _ptr(u), _ptr(w),
                                       _ptr(n_acc), _ptr(path), _ptr(out_tok), _ptr(new_len), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))


def sd_lmhead_accept_sampled_compact(batch: Batch, hidden, W, inv_temp: float, draft_tok, u, w, layers: LayerSet,
                                     lse, group_stats, n_acc, path, out_tok, new_len, workspace, status,
                                     stream=None) -> None:
    """LM-head statistics, acceptance at a sampling temperature and KV compaction in all layers: the
    LM-head tiles and one tail kernel."""
    M, Hd = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == Hd and M == batch.B * batch.T_max
    _check(lib.sd_lmhead_accept_sampled_compact(batch.ref(), _ptr(hidden), _ptr(W), int(Hd), int(V), C.c_float(inv_temp),
                                                _ptr(draft_tok), _ptr(u), _ptr(w), layers.layers, layers.L, layers.kt,
                                                layers.vt, _ptr(lse), _ptr(group_stats), _ptr(n_acc), _ptr(path),
                                                _ptr(out_tok), _ptr(new_len), _ptr(workspace),
                                                workspace.numel() * workspace.element_size(), _ptr(status),
                                                _stream(stream)))


def sd_draft_feature_attention(qp, k, v, H: int, scale: float, out, stream=None) -> None:
    """Meta-query cross-attention core: qp [Q,D], k and v [S,L,D], out [S,Q,D]; D = H * 128."""
    Q, D = qp.shape
    S, L, _ = k.shape
    _check(lib.sd_draft_feature_attention(_ptr(qp), _ptr(k), _ptr(v), int(S), int(L), int(Q), int(H), int(D),
                                          C.c_float(scale), _ptr(out), _stream(stream)))
