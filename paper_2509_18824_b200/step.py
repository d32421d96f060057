"""One whole verify step as a sequence of library calls.

Per layer: tree attention; then once: LM-head arg-max, greedy acceptance and
KV compaction over all layers.  This file only moves tensors to the device and
issues the C-ABI calls in order; it computes nothing itself.  (The layers'
projections, MLPs and norms of a real decoder are outside this library: q,
tree K/V and the final hidden states are inputs.)
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from . import binding as sd


def to_device(a: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy -> device tensor; bf16 bit patterns (uint16) travel as int16."""
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def pinned(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(np.ascontiguousarray(a)).pin_memory()


class VerifyStep:
    """Device-resident state (KV caches, LM-head weights, geometry) plus the
    per-step inputs and outputs of one batch."""

    def __init__(self, w, device="cuda", layers: Optional[List[int]] = None, keep_host_inputs=False):
        self.device = torch.device(device)
        self.w = w
        self.L = len(w.q)
        d = self.device
        self.batch = sd.Batch.of(w, device=d)
        self.status = sd.new_status(d)
        # resident state
        self.k_cache = [to_device(x, d) for x in w.k_cache]
        self.v_cache = [to_device(x, d) for x in w.v_cache]
        self.W = to_device(w.W, d) if w.W is not None else None
        # per-step inputs: q, tree K and tree V of all layers live in ONE device buffer (layer-major),
        # so that the end-to-end path can bring a whole group of layers over in a single copy
        B, T = w.B, w.T_max
        self._nq, self._nkv = B * T * w.Hq * w.D, B * T * w.Hkv * w.D       # bf16 elements per layer
        self._per_layer = self._nq + 2 * self._nkv
        self._in_dev = torch.empty(self.L * self._per_layer, dtype=torch.int16, device=d)
        self.q, self.k_tree, self.v_tree = self._layer_views(self._in_dev, w)
        for l in range(self.L):
            self.q[l].copy_(to_device(w.q[l], d)); self.k_tree[l].copy_(to_device(w.k_tree[l], d))
            self.v_tree[l].copy_(to_device(w.v_tree[l], d))
        self.hidden = to_device(w.hidden, d) if w.hidden is not None else None
        self.draft_tok = to_device(w.draft_tok, d) if w.draft_tok is not None else None
        # outputs
        self.out = [torch.zeros((B, T, w.Hq, w.D), dtype=torch.bfloat16, device=d) for _ in range(self.L)]
        self.lse = [torch.zeros((B, T, w.Hq), dtype=torch.float32, device=d) for _ in range(self.L)]
        M = B * T
        self.argmax = torch.zeros(M, dtype=torch.int32, device=d)
        self.maxlogit = torch.zeros(M, dtype=torch.float32, device=d)
        self.n_acc = torch.zeros(B, dtype=torch.int32, device=d)
        self.path = torch.zeros((B, T), dtype=torch.int32, device=d)
        self.out_tok = torch.zeros((B, T), dtype=torch.int32, device=d)
        self.new_len = torch.zeros(B, dtype=torch.int32, device=d)
        nbytes = sd.sd_workspace_bytes(self.batch, M if self.W is not None else 0, w.V if self.W is not None else 0)
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=d)
        self.caches = [sd.kv_layer(k, v) for k, v in zip(self.k_cache, self.v_cache)]
        self.layerset = sd.LayerSet(self.k_cache, self.v_cache, self.k_tree, self.v_tree)
        self.att_all = self._attention_set(0, self.L)
        self._att_groups = {}
        self.scale = float(w.scale)
        sd.sd_tree_prepare(self.batch, self.status)
        # pinned host copies for the end-to-end path
        self._copy_stream = None
        self.host = None
        if keep_host_inputs:
            self._in_host = torch.empty(self.L * self._per_layer, dtype=torch.int16).pin_memory()
            hq, hk, hv = self._layer_views(self._in_host, w)
            for l in range(self.L):
                hq[l].copy_(torch.from_numpy(w.q[l].view(np.int16)))
                hk[l].copy_(torch.from_numpy(w.k_tree[l].view(np.int16)))
                hv[l].copy_(torch.from_numpy(w.v_tree[l].view(np.int16)))
            self.host = dict(
                q=hq, k_tree=hk, v_tree=hv, hidden=pinned(w.hidden),
                draft_tok=pinned(w.draft_tok), parents=pinned(w.parents), n_nodes=pinned(w.n_nodes))
            self.host_out = dict(
                n_acc=torch.zeros(B, dtype=torch.int32).pin_memory(),
                path=torch.zeros((B, T), dtype=torch.int32).pin_memory(),
                out_tok=torch.zeros((B, T), dtype=torch.int32).pin_memory(),
                new_len=torch.zeros(B, dtype=torch.int32).pin_memory())
            # The end-to-end path double-buffers the per-step inputs on the device, so that the next
            # step's copies run while this step still computes.  Slot 0 is the set built above.
            self._slots = [self._slot_state()]
            self.batch = sd.Batch.of(w, device=d)
            self._in_dev = torch.empty_like(self._in_dev)
            self.q, self.k_tree, self.v_tree = self._layer_views(self._in_dev, w)
            self.hidden, self.draft_tok = torch.empty_like(self.hidden), torch.empty_like(self.draft_tok)
            self.layerset = sd.LayerSet(self.k_cache, self.v_cache, self.k_tree, self.v_tree)
            self.att_all = self._attention_set(0, self.L)
            self._att_groups = {}
            self._slots.append(self._slot_state())
            self._use_slot(0)
            self._step_no = 0

    _SLOT_FIELDS = ("batch", "_in_dev", "q", "k_tree", "v_tree", "hidden", "draft_tok", "layerset", "att_all",
                    "_att_groups")

    def _slot_state(self) -> dict:
        return {k: getattr(self, k) for k in self._SLOT_FIELDS}

    def _use_slot(self, i: int) -> None:
        """Make input set i the one the call wrappers below hand to the library."""
        for k, v in self._slots[i].items():
            setattr(self, k, v)

    def _layer_views(self, flat: torch.Tensor, w):
        """Per-layer q / tree K / tree V views of a flat layer-major buffer."""
        B, T = w.B, w.T_max
        q, kt, vt = [], [], []
        for l in range(self.L):
            o = l * self._per_layer
            q.append(flat[o:o + self._nq].view(B, T, w.Hq, w.D))
            kt.append(flat[o + self._nq:o + self._nq + self._nkv].view(B, T, w.Hkv, w.D))
            vt.append(flat[o + self._nq + self._nkv:o + self._per_layer].view(B, T, w.Hkv, w.D))
        return q, kt, vt

    # -- pieces ---------------------------------------------------------
    def attention(self, l: int, stream=None):
        sd.sd_verify_attention(self.batch, self.caches[l], self.q[l], self.k_tree[l], self.v_tree[l],
                               self.scale, self.out[l], self.lse[l], self.workspace, self.status, stream)

    def _attention_set(self, l0: int, l1: int):
        s = slice(l0, l1)
        return sd.AttentionLayerSet(self.k_cache[s], self.v_cache[s], self.q[s], self.k_tree[s], self.v_tree[s],
                                    self.out[s], self.lse[s])

    def attention_layers(self, l0: int = 0, l1: Optional[int] = None, stream=None):
        """Layers l0..l1-1 in one library call (all layers by default)."""
        l1 = self.L if l1 is None else l1
        if (l0, l1) == (0, self.L):
            ls = self.att_all
        else:
            ls = self._att_groups.get((l0, l1))
            if ls is None:
                ls = self._att_groups[(l0, l1)] = self._attention_set(l0, l1)
        sd.sd_verify_attention_layers(self.batch, ls, self.scale, self.workspace, self.status, stream)

    def lmhead(self, stream=None):
        sd.sd_lmhead_argmax(self.hidden, self.W, self.argmax, self.maxlogit, self.workspace, self.status, stream)

    def accept(self, target=None, stream=None):
        sd.sd_accept_tree(self.batch, self.draft_tok, self.argmax if target is None else target,
                          self.n_acc, self.path, self.out_tok, self.new_len, self.status, stream)

    def compact(self, stream=None):
        sd.sd_compact_kv(self.batch, self.layerset, self.n_acc, self.path, self.status, stream)

    def tail(self, stream=None):
        """LM head, acceptance and compaction through the one fused call."""
        sd.sd_lmhead_accept_compact(self.batch, self.hidden, self.W, self.draft_tok, self.layerset, self.argmax,
                                    self.maxlogit, self.n_acc, self.path, self.out_tok, self.new_len,
                                    self.workspace, self.status, stream)

    def tail_sampled(self, inv_temp: float, u: torch.Tensor, w: torch.Tensor, stream=None, fused=True):
        """The tail at a sampling temperature: LM head with log-sum-exp, the rejection walk with the
        given uniforms (u [B,T], w [B], device f32), the residual draw, then compaction; through the one
        fused call, or (fused=False) as the three separate calls it stands for."""
        if getattr(self, "lse_rows", None) is None:
            self.lse_rows = torch.zeros(self.w.B * self.w.T_max, dtype=torch.float32, device=self.device)
            self.group_stats = torch.zeros(sd.group_stats_shape(self.w.B * self.w.T_max, self.w.V),
                                           dtype=torch.float32, device=self.device)
            need = sd.sd_workspace_bytes(self.batch, self.w.B * self.w.T_max, self.w.V)
            if self.workspace.numel() < need:
                self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        if fused:
            sd.sd_lmhead_accept_sampled_compact(self.batch, self.hidden, self.W, inv_temp, self.draft_tok, u, w,
                                                self.layerset, self.lse_rows, self.group_stats, self.n_acc, self.path,
                                                self.out_tok, self.new_len, self.workspace, self.status, stream)
            return
        sd.sd_lmhead_stats(self.hidden, self.W, inv_temp, None, None, self.lse_rows,
                           self.workspace, self.status, stream, group_stats=self.group_stats)
        sd.sd_accept_tree_sampled(self.batch, self.hidden, self.W, inv_temp, self.lse_rows, self.draft_tok, u, w,
                                  self.n_acc, self.path, self.out_tok, self.new_len, self.workspace, self.status, stream,
                                  group_stats=self.group_stats)
        self.compact(stream)

    # -- the whole step -------------------------------------------------
    def run(self, stream=None, per_layer=True, fused_tail=True):
        """One attention call per layer, as a decoder issues them (layer l + 1's q, k and v depend on
        layer l's attention output), then LM head + acceptance + compaction in one call.
        per_layer=False puts all layers' attention into ONE call, which is only possible when every
        layer's q and tree K/V exist up front (an upper bound for a real decoder); fused_tail=False
        issues the three tail calls separately."""
        if per_layer:
            for l in range(self.L):
                self.attention(l, stream)
        else:
            self.attention_layers(stream=stream)
        if fused_tail:
            self.tail(stream)
        else:
            self.lmhead(stream)
            self.accept(None, stream)
            self.compact(stream)

    def capture(self, **run_args) -> "torch.cuda.CUDAGraph":
        """One run() recorded into a CUDA graph (the library calls only enqueue kernels on the stream
        they are given, so they can be captured); replay() then re-issues the step's launches without
        any host work per call.  One un-captured run comes first, so that per-kernel set-up is done."""
        self.run(**run_args)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.run(**run_args)
        return graph

    def launches_per_step(self, per_layer: bool = True) -> int:
        """Kernel launches of one run(): attention (one launch per layer, or per group of up to 32 layers
        in the all-layers call), the LM-head tiles and the fused merge/acceptance/compaction kernel."""
        att = self.L if per_layer else (self.L + sd.ATTENTION_LAYERS_PER_LAUNCH - 1) // sd.ATTENTION_LAYERS_PER_LAUNCH
        return att * sd.KERNELS_PER_ATTENTION + sd.KERNELS_PER_TAIL

    def h2d_bytes(self) -> int:
        h = self.host
        n = sum(t.numel() * t.element_size() for k in ("q", "k_tree", "v_tree") for t in h[k])
        return n + sum(h[k].numel() * h[k].element_size() for k in ("hidden", "draft_tok", "parents", "n_nodes"))

    def d2h_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.host_out.values())

    def run_from_host(self, group: int = 7, per_layer: bool = True):
        """End-to-end step: this step's inputs come from pinned host memory, the
        accepted tokens go back to the host; caches and weights stay resident.
        The host-to-device copies run on a second stream, ahead of the compute:
        attention is issued in groups of `group` layers, each group as soon as
        its layers' copies have landed (an event recorded behind them).  The
        device-side input buffers exist twice and alternate from step to step,
        so the copies of step i+1 overlap the last layers and the tail of step i
        and only wait for step i-1, which read the same buffers.  per_layer: one attention call
        per layer (a decoder computes layer l + 1's q, k, v from layer l's output) instead of one
        call per group of layers."""
        h = self.host
        main = torch.cuda.current_stream()
        if self._copy_stream is None:
            self._copy_stream = torch.cuda.Stream(device=self.device)
            self._ev_small = [torch.cuda.Event() for _ in range(2)]
            self._ev_layer = [[torch.cuda.Event() for _ in range(self.L)] for _ in range(2)]
            self._ev_done = [None, None]
            self._copy_stream.wait_stream(main)     # set-up work on the main stream has finished
        cs = self._copy_stream
        slot = self._step_no & 1
        self._step_no += 1
        self._use_slot(slot)
        if self._ev_done[slot] is not None:
            cs.wait_event(self._ev_done[slot])      # the step before last no longer reads this input set
        with torch.cuda.stream(cs):
            self.batch.parents.copy_(h["parents"], non_blocking=True)
            self.batch.n_nodes.copy_(h["n_nodes"], non_blocking=True)
            self._ev_small[slot].record(cs)
            for l0 in range(0, self.L, group):          # one copy per group of layers
                l1 = min(l0 + group, self.L)
                sl = slice(l0 * self._per_layer, l1 * self._per_layer)
                self._in_dev[sl].copy_(self._in_host[sl], non_blocking=True)
                self._ev_layer[slot][l1 - 1].record(cs)
            self.hidden.copy_(h["hidden"], non_blocking=True)
            self.draft_tok.copy_(h["draft_tok"], non_blocking=True)
            ev_last = torch.cuda.Event()
            ev_last.record(cs)
        main.wait_event(self._ev_small[slot])
        sd.sd_tree_prepare(self.batch, self.status)
        for l0 in range(0, self.L, group):
            l1 = min(l0 + group, self.L)
            main.wait_event(self._ev_layer[slot][l1 - 1])
            if per_layer:
                for l in range(l0, l1):
                    self.attention(l)
            else:
                self.attention_layers(l0, l1)
        main.wait_event(ev_last)        # hidden states and draft tokens have arrived
        self.tail()
        self.host_out["n_acc"].copy_(self.n_acc, non_blocking=True)
        self.host_out["path"].copy_(self.path, non_blocking=True)
        self.host_out["out_tok"].copy_(self.out_tok, non_blocking=True)
        self.host_out["new_len"].copy_(self.new_len, non_blocking=True)
        if self._ev_done[slot] is None:
            self._ev_done[slot] = torch.cuda.Event()
        self._ev_done[slot].record(main)

    def check_status(self):
        code = int(self.status.item())
        if code != 0:
            raise sd.SdError(code)
