"""Per-call measurements beyond the headline step: every workload's attention,
the LM head at several row counts, and the bandwidth-regime cases (chain
decoding, a compaction stress shape).  One JSON line per measurement.

    python -m paper_2509_18824_b200.supplements [attention] [attention_layers] [lmhead] [lmhead480] [sampled] [draft] [compact]
                                                [chain8] [compact512]        (small cases for profiler captures)

Timing: CUDA events on the launching stream, >= 3 warm-up calls, inputs rotated
over several layers so that the working set exceeds L2.
"""
from __future__ import annotations

import json
import os
import sys

import numpy as np
import torch

from . import binding as sd
from . import workloads as wl
from .step import to_device


def _peaks():
    fn = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(fn):
        p = json.load(open(fn))
        return float(p["hbm_gbs"]), float(p["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def _time(fn, reps):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def attention(configs=("c2", "c3", "c4", "c5", "chain11")):
    hbm, tens, src = _peaks()
    for cfg in configs:
        sp = wl.spec(cfg)
        sp.L = 4                                   # 4 distinct layers: > L2 for every config but c2
        w = wl.make_geometry(sp)
        wl.fill_attention(w)
        bt = sd.Batch.of(w)
        st = sd.new_status()
        sd.sd_tree_prepare(bt, st)
        kc = [to_device(x) for x in w.k_cache]; vc = [to_device(x) for x in w.v_cache]
        q = [to_device(x) for x in w.q]; kt = [to_device(x) for x in w.k_tree]; vt = [to_device(x) for x in w.v_tree]
        out = torch.zeros((w.B, w.T_max, w.Hq, w.D), dtype=torch.bfloat16, device="cuda")
        ws = torch.empty(sd.sd_workspace_bytes(bt), dtype=torch.uint8, device="cuda")
        caches = [sd.kv_layer(k, v) for k, v in zip(kc, vc)]

        def run():
            for l in range(w.L):
                sd.sd_verify_attention(bt, caches[l], q[l], kt[l], vt[l], w.scale, out, None, ws, st)
        ms = _time(run, 10) / w.L
        vis = sum(int((int(w.len[b]) + wl.node_depths(w.parents[b]) + 1).sum()) for b in range(w.B))
        flops = 4.0 * w.D * w.Hq * vis
        nbytes = (sum(int(w.len[b]) + w.T_max for b in range(w.B)) * w.Hkv * w.D * 4
                  + 2 * w.B * w.T_max * w.Hq * w.D * 2)
        print(json.dumps({"call": "sd_verify_attention", "workload": cfg, "us": ms * 1e3,
                          "tflops": flops / ms / 1e9, "frac_tensor_burst": flops / ms / 1e9 / tens,
                          "gbs": nbytes / ms / 1e6, "frac_hbm": nbytes / ms / 1e6 / hbm,
                          "frac_hbm_nominal_8TBs": nbytes / ms / 1e6 / 8000.0,
                          "flop_per_byte": flops / nbytes, "peaks": src, "status": int(st.item())}))
        del kc, vc, q, kt, vt
        torch.cuda.empty_cache()


def attention_layers(configs=("c5", "chain11", "tree28", "c4"), L=28):
    for r in measure_attention_layers(configs, L):
        print(json.dumps(r))


def measure_attention_layers(configs=("c5", "chain11", "tree28", "c4"), L=28, reps=20):
    """All L layers through sd_verify_attention_layers (one launch): the regime of a whole verify
    step, where per-launch costs are paid once.  chain11 is the bandwidth-bound case.  Yields one
    record per workload."""
    hbm, tens, src = _peaks()
    for cfg in configs:
        sp = wl.spec(cfg)
        sp.L = L if cfg != "c4" else 8             # c4's caches are 4x larger per layer
        w = wl.make_geometry(sp)
        wl.fill_attention(w)
        bt = sd.Batch.of(w)
        st = sd.new_status()
        sd.sd_tree_prepare(bt, st)
        kc = [to_device(x) for x in w.k_cache]; vc = [to_device(x) for x in w.v_cache]
        q = [to_device(x) for x in w.q]; kt = [to_device(x) for x in w.k_tree]; vt = [to_device(x) for x in w.v_tree]
        out = [torch.zeros((w.B, w.T_max, w.Hq, w.D), dtype=torch.bfloat16, device="cuda") for _ in range(w.L)]
        ws = torch.empty(sd.sd_workspace_bytes(bt), dtype=torch.uint8, device="cuda")
        ls = sd.AttentionLayerSet(kc, vc, q, kt, vt, out)
        ms = _time(lambda: sd.sd_verify_attention_layers(bt, ls, w.scale, ws, st), reps)
        vis = sum(int((int(w.len[b]) + wl.node_depths(w.parents[b]) + 1).sum()) for b in range(w.B))
        flops = 4.0 * w.D * w.Hq * vis * w.L
        nbytes = (sum(int(w.len[b]) + w.T_max for b in range(w.B)) * w.Hkv * w.D * 4
                  + 2 * w.B * w.T_max * w.Hq * w.D * 2) * w.L
        rec = {"call": "sd_verify_attention_layers", "workload": cfg, "layers": w.L, "us": ms * 1e3,
               "us_per_layer": ms * 1e3 / w.L,
               "tflops": flops / ms / 1e9, "frac_tensor_burst": flops / ms / 1e9 / tens,
               "algorithmic_bytes": nbytes, "gbs": nbytes / ms / 1e6, "frac_hbm": nbytes / ms / 1e6 / hbm,
               "frac_hbm_nominal_8TBs": nbytes / ms / 1e6 / 8000.0,
               "flop_per_byte": flops / nbytes, "peaks": src, "status": int(st.item())}
        del kc, vc, q, kt, vt, out, ls
        torch.cuda.empty_cache()
        yield rec


def lmhead(rows=(60, 240, 480, 960), V=152064, Hd=3584):
    hbm, tens, src = _peaks()
    W = to_device(wl.normal_bf16(7, "W", (V, Hd), 1.0 / np.sqrt(Hd)))
    for M in rows:
        h = to_device(wl.normal_bf16(7, f"h{M}", (M, Hd), 1.0 / np.sqrt(Hd)))
        am = torch.zeros(M, dtype=torch.int32, device="cuda")
        mx = torch.zeros(M, dtype=torch.float32, device="cuda")
        ws = torch.empty(sd.sd_workspace_bytes(None, M, V), dtype=torch.uint8, device="cuda")
        st = sd.new_status()
        ms = _time(lambda: sd.sd_lmhead_argmax(h, W, am, mx, ws, st), 10)
        flops = 2.0 * M * V * Hd
        nbytes = (V + M) * Hd * 2
        print(json.dumps({"call": "sd_lmhead_argmax", "rows": M, "us": ms * 1e3, "tflops": flops / ms / 1e9,
                          "frac_tensor_burst": flops / ms / 1e9 / tens, "gbs": nbytes / ms / 1e6,
                          "frac_hbm": nbytes / ms / 1e6 / hbm, "peaks": src, "status": int(st.item())}))


def sampled(cfg="c5", inv_temp=1.0):
    """The tail of a step at a sampling temperature (LM head with log-sum-exp, rejection walk, residual
    draw) next to the greedy tail, on the bench's shapes."""
    hbm, tens, src = _peaks()
    from .step import VerifyStep
    w = wl.make(cfg, attention=False, L=1)
    wl.fill_attention(w, [0])
    vs = VerifyStep(w)
    B, T, M = w.B, w.T_max, w.B * w.T_max
    g = torch.Generator(device="cuda"); g.manual_seed(0)
    u = torch.rand((B, T), device="cuda", generator=g)
    wv = torch.rand((B,), device="cuda", generator=g)
    lse = torch.zeros(M, dtype=torch.float32, device="cuda")
    ws = torch.empty(sd.sd_workspace_bytes(vs.batch, M, w.V), dtype=torch.uint8, device="cuda")
    st = vs.status
    flops = 2.0 * M * w.V * w.Hd
    ms_greedy = _time(lambda: sd.sd_lmhead_argmax(vs.hidden, vs.W, vs.argmax, vs.maxlogit, ws, st), 10)
    gs = torch.zeros(sd.group_stats_shape(M, w.V), dtype=torch.float32, device="cuda")
    ms_stats0 = _time(lambda: sd.sd_lmhead_stats(vs.hidden, vs.W, inv_temp, vs.argmax, vs.maxlogit, lse, ws, st), 10)
    ms_stats = _time(lambda: sd.sd_lmhead_stats(vs.hidden, vs.W, inv_temp, vs.argmax, vs.maxlogit, lse, ws, st,
                                                group_stats=gs), 10)
    ms_acc0 = _time(lambda: sd.sd_accept_tree_sampled(vs.batch, vs.hidden, vs.W, inv_temp, lse, vs.draft_tok, u, wv,
                                                      vs.n_acc, vs.path, vs.out_tok, vs.new_len, ws, st), 10)
    ms_acc = _time(lambda: sd.sd_accept_tree_sampled(vs.batch, vs.hidden, vs.W, inv_temp, lse, vs.draft_tok, u, wv,
                                                     vs.n_acc, vs.path, vs.out_tok, vs.new_len, ws, st, group_stats=gs), 10)
    ms_sep = _time(lambda: vs.tail_sampled(inv_temp, u, wv, fused=False), 10)
    ms_fused = _time(lambda: vs.tail_sampled(inv_temp, u, wv, fused=True), 10)
    wbytes = w.V * w.Hd * 2
    print(json.dumps({"call": "sampled tail", "workload": cfg, "rows": M,
                      "whole_tail_fused_call_us": ms_fused * 1e3, "whole_tail_separate_calls_us": ms_sep * 1e3,
                      "layers_compacted": vs.L,
                      "sd_lmhead_argmax_us": ms_greedy * 1e3, "sd_lmhead_stats_us": ms_stats * 1e3,
                      "stats_tflops": flops / ms_stats / 1e9, "stats_frac_tensor_burst": flops / ms_stats / 1e9 / tens,
                      "sd_lmhead_stats_without_group_table_us": ms_stats0 * 1e3,
                      "sd_accept_tree_sampled_us": ms_acc * 1e3,
                      "sd_accept_tree_sampled_second_pass_us": ms_acc0 * 1e3,
                      "second_pass_weight_stream_gbs": wbytes / ms_acc0 / 1e6,
                      "peaks": src, "status": int(st.item())}))


def chain_sampled(inv_temp=1.0):
    """sd_accept_chain_sampled on chain decoding shapes (root + 10 drafts, 8 sequences, vocabulary 152064):
    drafts and draft distributions are random here, which does not change the work."""
    from .step import VerifyStep
    w = wl.make("chain11", attention=False, L=1)
    wl.fill_attention(w, [0])
    vs = VerifyStep(w)
    B, T, M, V = w.B, w.T_max, w.B * w.T_max, w.V
    g = torch.Generator(device="cuda"); g.manual_seed(0)
    u = torch.rand((B, T), device="cuda", generator=g)
    wv = torch.rand((B,), device="cuda", generator=g)
    q = torch.rand((B, T, V), device="cuda", generator=g)
    q /= q.sum(dim=-1, keepdim=True)
    q_tok = torch.gather(q[:, : T - 1], 2, vs.draft_tok[:, 1:].long().unsqueeze(-1)).squeeze(-1)
    q_tok = torch.cat([torch.zeros((B, 1), device="cuda"), q_tok], dim=1).contiguous()
    lse = torch.zeros(M, dtype=torch.float32, device="cuda")
    ws = torch.empty(sd.sd_workspace_bytes(vs.batch, M, V), dtype=torch.uint8, device="cuda")
    st = vs.status
    ms_stats = _time(lambda: sd.sd_lmhead_stats(vs.hidden, vs.W, inv_temp, None, None, lse, ws, st), 10)
    ms_acc = _time(lambda: sd.sd_accept_chain_sampled(vs.batch, vs.hidden, vs.W, inv_temp, lse, vs.draft_tok, q_tok, q, u, wv,
                                                      vs.n_acc, vs.path, vs.out_tok, vs.new_len, ws, st), 10)
    logits = torch.empty((M, V), dtype=torch.float32, device="cuda")
    ms_stats_lg = _time(lambda: sd.sd_lmhead_stats_logits(vs.hidden, vs.W, inv_temp, None, None, lse, logits, ws, st), 10)
    ms_acc_lg = _time(lambda: sd.sd_accept_chain_sampled(vs.batch, vs.hidden, vs.W, inv_temp, lse, vs.draft_tok, q_tok, q, u, wv,
                                                         vs.n_acc, vs.path, vs.out_tok, vs.new_len, ws, st, logits=logits), 10)
    print(json.dumps({"call": "sd_accept_chain_sampled", "workload": "chain11", "rows": M,
                      "sd_lmhead_stats_logits_us": ms_stats_lg * 1e3, "sd_accept_chain_sampled_from_logits_us": ms_acc_lg * 1e3,
                      "sd_lmhead_stats_us": ms_stats * 1e3, "sd_accept_chain_sampled_us": ms_acc * 1e3,
                      "second_pass_weight_stream_gbs": V * w.Hd * 2 / ms_acc / 1e6, "status": int(st.item())}))


def tree_sampled_q(inv_temp=1.0):
    """sd_lmhead_stats_logits + sd_accept_tree_sampled_q on the bench's shapes (8 trees of 60 nodes,
    vocabulary 152064).  Random q and tokens: nearly every child is rejected, the expensive case."""
    from .step import VerifyStep
    w = wl.make("c5", attention=False, L=1)
    wl.fill_attention(w, [0])
    vs = VerifyStep(w)
    B, T, M, V = w.B, w.T_max, w.B * w.T_max, w.V
    g = torch.Generator(device="cuda"); g.manual_seed(0)
    u = torch.rand((B, T), device="cuda", generator=g)
    wv = torch.rand((B,), device="cuda", generator=g)
    q = torch.rand((B, T, V), device="cuda", generator=g)
    q /= q.sum(dim=-1, keepdim=True)
    lse = torch.zeros(M, dtype=torch.float32, device="cuda")
    logits = torch.empty((M, V), dtype=torch.float32, device="cuda")
    ws = torch.empty(sd.sd_workspace_bytes(vs.batch, M, V), dtype=torch.uint8, device="cuda")
    st = vs.status
    ms_stats = _time(lambda: sd.sd_lmhead_stats_logits(vs.hidden, vs.W, inv_temp, None, None, lse, logits, ws, st), 10)
    res = {}
    for name, uu in (("all_rejected", torch.full((B, T), 0.999, device="cuda")), ("random", u),
                     ("all_accepted", torch.zeros((B, T), device="cuda"))):
        res[name] = _time(lambda: sd.sd_accept_tree_sampled_q(vs.batch, inv_temp, lse, logits, vs.draft_tok, q, uu, wv,
                                                              vs.n_acc, vs.path, vs.out_tok, vs.new_len, st), 10) * 1e3
    print(json.dumps({"call": "sd_accept_tree_sampled_q", "workload": "c5", "rows": M,
                      "sd_lmhead_stats_logits_us": ms_stats * 1e3, "sd_accept_tree_sampled_q_us": res,
                      "logits_bytes": M * V * 4, "status": int(st.item())}))


def draft(S=4096, L=28, Q=4, H=28):
    """Draft-side feature aggregation on a 7B-shaped prefill: S tokens x 28 layer features of width 3584."""
    hbm, _, src = _peaks()
    D = H * 128
    g = torch.Generator(device="cuda"); g.manual_seed(0)
    qp = torch.randn((Q, D), device="cuda", generator=g).to(torch.bfloat16)
    k = torch.randn((S, L, D), device="cuda", generator=g).to(torch.bfloat16)
    v = torch.randn((S, L, D), device="cuda", generator=g).to(torch.bfloat16)
    out = torch.zeros((S, Q, D), dtype=torch.bfloat16, device="cuda")
    for name, vv in (("separate K and V", v), ("K = V (un-projected features)", k)):
        ms = _time(lambda: sd.sd_draft_feature_attention(qp, k, vv, H, 1.0 / np.sqrt(128.0), out), 10)
        nbytes = S * L * D * 2 * (2 if vv is v else 1) + S * Q * D * 2
        print(json.dumps({"call": "sd_draft_feature_attention", "workload": f"S={S} L={L} Q={Q} H={H}, {name}",
                          "us": ms * 1e3, "gbs": nbytes / ms / 1e6, "frac_hbm": nbytes / ms / 1e6 / hbm,
                          "frac_hbm_nominal_8TBs": nbytes / ms / 1e6 / 8000.0, "bytes": nbytes, "peaks": src}))


def compact(**kw):
    print(json.dumps(measure_compact(**kw)))


def measure_compact(B=1024, L=8, T=64, Hkv=4, D=128):
    """Stress shape for compaction: every node of every tree accepted (a 64-node chain), 1024
    sequences, 8 layers: 2 x 1.07 GB moved per call."""
    hbm, _, src = _peaks()
    g = np.random.default_rng(0)
    lens = g.integers(0, 64, size=B).astype(np.int32)
    table = np.arange(2 * B, dtype=np.int32).reshape(B, 2)
    parents = np.stack([wl.chain_tree(T)] * B)
    geo = type("G", (), dict(B=B, T_max=T, Hq=Hkv, Hkv=Hkv, D=D, block_table=table, len=lens,
                             n_nodes=np.full(B, T, np.int32), parents=parents))
    bt = sd.Batch.of(geo)
    st = sd.new_status()
    kc = [torch.zeros((2 * B, Hkv, 64, D), dtype=torch.int16, device="cuda") for _ in range(L)]
    vc = [torch.zeros((2 * B, Hkv, 64, D), dtype=torch.int16, device="cuda") for _ in range(L)]
    kt = [torch.randint(-30000, 30000, (B, T, Hkv, D), dtype=torch.int16, device="cuda") for _ in range(L)]
    vt = [torch.randint(-30000, 30000, (B, T, Hkv, D), dtype=torch.int16, device="cuda") for _ in range(L)]
    n_acc = torch.full((B,), T, dtype=torch.int32, device="cuda")
    path = torch.arange(T, dtype=torch.int32, device="cuda").repeat(B, 1).contiguous()
    ls = sd.LayerSet(kc, vc, kt, vt)
    ms = _time(lambda: sd.sd_compact_kv(bt, ls, n_acc, path, st), 10)
    moved = 2.0 * B * T * Hkv * D * 2 * 2 * L          # read + write, K and V
    ok = all(torch.equal(kc[l][2 * b + (int(lens[b]) + 5) // 64, :, (int(lens[b]) + 5) % 64], kt[l][b, 5])
             for l in (0, L - 1) for b in (0, B - 1))
    return {"call": "sd_compact_kv", "workload": f"stress B={B} L={L} all {T} nodes accepted",
            "us": ms * 1e3, "gbs": moved / ms / 1e6, "frac_hbm": moved / ms / 1e6 / hbm,
            "frac_hbm_nominal_8TBs": moved / ms / 1e6 / 8000.0, "bytes": moved, "peaks": src,
            "spot_check": bool(ok), "status": int(st.item())}


if __name__ == "__main__":
    what = sys.argv[1:] or ["attention", "attention_layers", "lmhead", "sampled", "draft", "compact"]
    if "attention" in what:
        attention()
    if "attention_layers" in what:
        attention_layers()
    if "lmhead" in what:
        lmhead()
    if "lmhead480" in what:                # the bench's LM-head launch alone (profiler captures)
        lmhead(rows=(480,))
    if "sampled" in what:
        sampled()
        chain_sampled()
        tree_sampled_q()
    if "draft" in what:
        draft()
    if "compact" in what:
        compact()
    if "chain8" in what:                   # chain decoding, 8 layers in one call (0.55 GB of K/V)
        for r in measure_attention_layers(("chain11",), L=8, reps=3):
            print(json.dumps(r))
    if "compact512" in what:               # half the stress shape: 1.07 GB moved per call
        compact(B=512)
