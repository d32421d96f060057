#!/usr/bin/env python
"""Benchmark of the whole draft-tree verify step.

One step = one pass of the complete hot path over one synthetic batch:
per-layer tree attention (28 layers), LM-head arg-max, greedy acceptance and
KV compaction in all layers.  Default workload "c5": batch 8, prefix 4096,
28 query / 4 KV heads, head_dim 128, 60-node depth-6 trees, vocabulary 152064,
hidden 3584, bf16, draft tokens planted along seeded paths of length 0..6.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched under torchrun) every rank runs an independent replica of
the same step on its own GPU; there is no collective on the data path.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum of attn_umma_kernel per layer, from the ncu capture
# summarised under profiles/.  Set an entry to None whenever the kernel changes until the counters
# are retaken.
ATTENTION_DRAM_BYTES_PER_LAYER = {"c5": 72.28e6}

METRIC = "tree_verify_steps_per_s"
UNIT = "steps/s"


def read_peaks():
    fn = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(fn):
        p = json.load(open(fn))
        return dict(hbm=float(p["hbm_gbs"]), tensor_burst=float(p["bf16_tflops"]),
                    tensor_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, tensor_burst=1590.0, tensor_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------
# algorithmic work of one step (what the method must move / compute)
# ----------------------------------------------------------------------------
def algorithmic_work(w):
    from paper_2509_18824_b200 import workloads as wl
    vis = 0                      # visible (query node, key) pairs summed over sequences
    kv_tokens = 0
    for b in range(w.B):
        n = int(w.n_nodes[b])
        d = wl.node_depths(w.parents[b][:n])
        vis += int((int(w.len[b]) + d + 1).sum())
        kv_tokens += int(w.len[b]) + n
    att_flops = 4.0 * w.D * w.Hq * vis                                  # QK^T and PV
    att_bytes = kv_tokens * w.Hkv * w.D * 2 * 2                          # K and V once per KV head
    att_bytes += 2 * w.B * w.T_max * w.Hq * w.D * 2                      # q read, out written
    lm_flops = 2.0 * w.M * w.Hd * w.V
    lm_bytes = (w.V + w.M) * w.Hd * 2
    return dict(att_flops=att_flops, att_bytes=att_bytes, lm_flops=lm_flops, lm_bytes=lm_bytes)


# ----------------------------------------------------------------------------
# clocks during the timed region
# ----------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={self.idx}", f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "50"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[5:9]):
                if v.strip().lower() == "active":
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------
# CPU baseline: the fp64 checker as it stands, on a bounded sample
# ----------------------------------------------------------------------------
def cpu_step_estimate(w, att_rows=6720, lm_rows=96):
    """Seconds the checker would need for one whole step, extrapolated from a sample:
    `att_rows` attention rows of layer 0, `lm_rows` LM-head rows, acceptance and one
    layer of compaction in full."""
    import oracle
    G = oracle.Geometry.of(w)
    g = np.random.default_rng(0)
    rows = np.stack([g.integers(0, w.B, att_rows), g.integers(0, w.T_max, att_rows),
                     g.integers(0, w.Hq, att_rows)], 1).astype(np.int32)
    t = time.perf_counter()
    oracle.attention_rows(G, w.k_cache[0], w.v_cache[0], w.q[0], w.k_tree[0], w.v_tree[0], w.scale, rows)
    t_att = (time.perf_counter() - t) / att_rows * (w.B * w.T_max * w.Hq) * w.L
    t = time.perf_counter()
    am, _, _ = oracle.lmhead(w.hidden, w.W, rows=list(range(lm_rows)))
    t_lm = (time.perf_counter() - t) / lm_rows * w.M
    target = g.integers(0, w.V, size=(w.B, w.T_max)).astype(np.int32)
    t = time.perf_counter()
    n_acc, path, _, _ = oracle.accept(G, w.draft_tok, target)
    t_acc = time.perf_counter() - t
    kc, vc = w.k_cache[0].copy(), w.v_cache[0].copy()
    t = time.perf_counter()
    oracle.compact(G, kc, vc, w.k_tree[0], w.v_tree[0], n_acc, path)
    t_cmp = (time.perf_counter() - t) * w.L
    total = t_att + t_lm + t_acc + t_cmp
    sample = (f"{att_rows} of {w.B * w.T_max * w.Hq * w.L} attention rows, {lm_rows} of {w.M} LM-head rows, "
              f"acceptance and 1 of {w.L} layers of compaction in full; scaled to one whole step")
    return total, sample, oracle.num_threads()


def max_over_ranks(values, device):
    """Slowest rank decides: element-wise maximum of `values` over all ranks (identity on one rank)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_throughput(world, steps, ms_total):
    """Whole-job steps/s of `world` independent replicas that each ran `steps` steps; `ms_total` is
    the slowest rank's time."""
    return world * steps / (ms_total * 1e-3)


def run_reference(args):
    """The fp64 CPU checker timed as the reference arm (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2509_18824_b200 import workloads as wl
    w = wl.make(args.config, layers=[0])
    times = []
    sample = ""
    cores = 1
    for i in range(args.warmup + args.steps):
        sec, sample, cores = cpu_step_estimate(w, att_rows=1344, lm_rows=16)
        if i >= args.warmup:
            times.append(sec)
    sec = sum(times) / len(times)
    val = 1.0 / sec
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, args),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(w, args):
    return {"workload": f"{args.config}: full verify step, batch {w.B}, prefix {int(w.len.max())}, "
                        f"{w.Hq}/{w.Hkv} heads, head_dim {w.D}, {w.T_max}-node trees, {w.L} layers, "
                        f"vocab {w.V}, hidden {w.Hd}, planted paths 0-6",
            "global_batch": int(w.B) * max(1, args.gpus), "layers": int(w.L),
            "l2": "inputs larger than L2 (KV caches 1.9 GB + LM-head weights 1.1 GB per step)",
            "parallelism": "replicas only (no sharding, no collective)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c5")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0,
                    help="override the number of layers (small cases for profiler captures only)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_2509_18824_b200 import workloads as wl
    from paper_2509_18824_b200 import binding as sd
    from paper_2509_18824_b200.step import VerifyStep

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # synthetic batch (each replica its own seed)
    over = {"L": args.layers} if args.layers > 0 else {}
    w = wl.make(args.config, seed=wl.spec(args.config).seed + 1000 * rank, **over)
    vs = VerifyStep(w, keep_host_inputs=True)
    # planted draft tokens follow the target's arg-max, taken here from the library's own LM head
    vs.lmhead()
    torch.cuda.synchronize()
    wl.plant(w, vs.argmax.cpu().numpy().reshape(w.B, w.T_max))
    vs.draft_tok.copy_(torch.from_numpy(w.draft_tok))
    vs.host["draft_tok"].copy_(torch.from_numpy(w.draft_tok))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        vs.run()
    barrier()
    vs.check_status()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        vs.run()
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)

    # per-call durations, same steps, events around every call (same stream)
    names = ["attention", "attention_single_layer_call", "tail", "tail_sampled", "lmhead", "accept", "compact"]
    ev = {n: [] for n in names}
    def timed(name, fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record()
        ev[name].append((a, b))
    for _ in range(args.steps):                           # the same two calls as the timed step
        timed("attention", vs.attention_layers)           # all layers, one library call
        timed("tail", vs.tail)                            # LM head + acceptance + compaction, one call
    gen = torch.Generator(device="cuda"); gen.manual_seed(rank)
    u_rand = torch.rand((w.B, w.T_max), device="cuda", generator=gen)
    w_rand = torch.rand((w.B,), device="cuda", generator=gen)
    vs.tail_sampled(1.0, u_rand, w_rand)                  # untimed: its first call allocates the statistics buffers
    for _ in range(max(1, args.steps // 10)):             # for comparison: the tail as three calls,
        timed("tail_sampled", lambda: vs.tail_sampled(1.0, u_rand, w_rand))   # the tail at temperature 1,
        timed("lmhead", vs.lmhead)                        # attention as one call per layer
        timed("accept", vs.accept)
        timed("compact", vs.compact)
        for l in range(vs.L):
            timed("attention_single_layer_call", lambda: vs.attention(l))
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    per_call_ms = {n: sum(a.elapsed_time(b) for a, b in ev[n]) / len(ev[n]) for n in names}

    # for comparison: the same step replayed from a CUDA graph (no host work per call)
    graph = vs.capture()
    for _ in range(3):
        graph.replay()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    g0.record()
    for _ in range(args.steps):
        graph.replay()
    g1.record()
    torch.cuda.synchronize()
    per_call_ms["graph_replay_step"] = g0.elapsed_time(g1) / args.steps
    del graph

    # end to end: this step's inputs from pinned host memory, results back to the host
    for _ in range(2):
        vs.run_from_host()
    barrier()
    t0 = time.perf_counter()
    e0.record()
    for _ in range(args.steps):
        vs.run_from_host()
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    vs.check_status()
    n_acc = vs.host_out["n_acc"].numpy().copy()
    assert (n_acc == w.planted_len + 1).all(), "planted paths were not recovered"

    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], "cuda")

    if rank == 0:
        peaks = read_peaks()
        work = algorithmic_work(w)
        ms_step = ms_total / args.steps
        value = job_throughput(world, args.steps, ms_total)
        tokens_per_step = int(n_acc.sum())
        n_att_launches = (vs.L + sd.ATTENTION_LAYERS_PER_LAUNCH - 1) // sd.ATTENTION_LAYERS_PER_LAUNCH
        layers_per_launch = vs.L / n_att_launches
        att_s = per_call_ms["attention"] * 1e-3 / n_att_launches          # one launch = layers_per_launch layers
        lm_s = per_call_ms["tail"] * 1e-3                  # LM-head tiles + the 18 us tail kernel
        att_tflops = work["att_flops"] * layers_per_launch / att_s / 1e12
        att_gbs = work["att_bytes"] * layers_per_launch / att_s / 1e9
        lm_tflops = work["lm_flops"] / lm_s / 1e12
        lm_gbs = work["lm_bytes"] / lm_s / 1e9
        # dominant kernel: tree attention, all layers of the step in one launch; at 60 nodes x 7
        # grouped heads per KV head its arithmetic intensity (~420 flop/B) puts it on the tensor roof
        traffic = ATTENTION_DRAM_BYTES_PER_LAYER.get(args.config)
        roofline = {"kernel": "sd_verify_attention_layers (attn_umma_kernel)", "bound": "tensor", "achieved": att_tflops,
                    "peak": peaks["tensor_sustained"], "unit": "TFLOP/s",
                    "frac": att_tflops / peaks["tensor_sustained"],
                    "traffic": traffic * layers_per_launch if traffic else None,
                    "traffic_unit": "bytes per launch (dram read + write; ncu capture of the 6.94-layer main launch of "
                                    "an 8-layer call, scaled by layers per launch)",
                    "layers_per_launch": layers_per_launch,
                    "algorithmic_bytes_per_launch": work["att_bytes"] * layers_per_launch,
                    "algorithmic_flops_per_launch": work["att_flops"] * layers_per_launch,
                    "peak_source": peaks["source"] + " (sustained bf16)",
                    "hbm_gbs": att_gbs, "hbm_frac_of_measured": att_gbs / peaks["hbm"],
                    "hbm_frac_of_nominal_8TBs": att_gbs / 8000.0,
                    "avg_launch_ms": att_s * 1e3}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": workload_config(w, args),
                "verified_tokens_per_s": value * tokens_per_step,
                "accepted_tokens_per_step": tokens_per_step,
                "clocks": clocks,
                "e2e": {"value": world * args.steps / (ms_e2e * 1e-3), "unit": UNIT,
                        "h2d_bytes_per_step": vs.h2d_bytes(), "d2h_bytes_per_step": vs.d2h_bytes()},
                "gpu_launches": vs.launches_per_step * args.steps,
                "roofline": roofline,
                "calls": {"attention_ms_all_layers": per_call_ms["attention"],
                          "attention_ms_per_layer": per_call_ms["attention"] / vs.L,
                          "attention_ms_single_layer_call": per_call_ms["attention_single_layer_call"],
                          "lmhead_accept_compact_ms": per_call_ms["tail"],
                          "sampled_tail_ms": per_call_ms["tail_sampled"],
                          "graph_replay_ms_per_step": per_call_ms["graph_replay_step"],
                          "lmhead_ms": per_call_ms["lmhead"], "accept_ms": per_call_ms["accept"],
                          "compact_ms": per_call_ms["compact"],
                          "lmhead_tflops": lm_tflops, "lmhead_frac_of_tensor_peak": lm_tflops / peaks["tensor_sustained"],
                          "lmhead_weight_gbs": lm_gbs}}
        if world == 1 and not args.no_cpu_baseline:
            sec, sample, cores = cpu_step_estimate(w)
            line["cpu_baseline"] = {"value": 1.0 / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": sample}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
