#!/usr/bin/env python
"""Benchmark of the whole draft-tree verify step.

One step = one pass of the complete hot path over one synthetic batch: tree
attention of every layer, ONE LIBRARY CALL PER LAYER (a decoder computes layer
l + 1's q, k and v from layer l's attention output, so that is how the calls
arrive), LM-head arg-max, greedy acceptance and KV compaction in all layers.
The step is recorded into a CUDA graph once and replayed.  Default workload
"c5": batch 8, prefix 4096, 28 query / 4 KV heads, head_dim 128, 60-node
depth-6 trees, 28 layers, vocabulary 152064, hidden 3584, bf16, draft tokens
planted along seeded paths of length 0..6.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

K steps are timed between a barrier + synchronize on both sides; the
measurement is repeated until about a second of timed work has run (so that the
clocks settle under load and the clock sampler sees the region) and the mean
over the repeats is reported.  With N > 1 (launched under torchrun) every rank
runs an independent replica of the same step on its own GPU; there is no
collective on the data path.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum of one single-layer launch of attn_umma_kernel, from the ncu
# capture summarised under profiles/.  Set an entry to None whenever the kernel changes until the counters
# are retaken.
ATTENTION_DRAM_BYTES_PER_LAUNCH = {"c5": 75.0e6}

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
    """Per LAYER of attention and per LM-head call."""
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
    """nvidia-smi polled every 50 ms into a file; mark() remembers how many samples exist, so that a
    region of the run can be summarised by itself."""
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

    def _rows(self):
        try:
            return [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        except Exception:
            return []

    def wait_first(self, timeout=5.0):
        """Blocks until the poller has delivered its first sample (it takes a while to start)."""
        t0 = time.time()
        while self.p is not None and not self._rows() and time.time() - t0 < timeout:
            time.sleep(0.02)

    def mark(self) -> int:
        return len(self._rows())

    def stop(self):
        if self.p is None:
            return
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()

    def summary(self, first: int = 0, last=None):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        rows = self._rows()[first:last]
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2])); pw.append(float(r[3]))
            except ValueError:
                continue
            for n, v in zip(names, r[5:9]):
                if v.strip().lower() == "active":
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "power_w": statistics.median(pw) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}

    def close(self):
        try:
            os.unlink(self.f.name)
        except Exception:
            pass


# ----------------------------------------------------------------------------
# CPU baseline: the fp64 checker as it stands, on a bounded sample
# ----------------------------------------------------------------------------
def cpu_step_estimate(w, lm_rows=None):
    """Seconds the checker needs for one whole step: ONE WHOLE LAYER of attention is timed and counted
    w.L times (the layers have identical shapes), the LM head over all rows (or `lm_rows` of them, scaled),
    acceptance in full, one layer of compaction counted w.L times."""
    import oracle
    G = oracle.Geometry.of(w)
    t = time.perf_counter()
    oracle.attention(G, w.k_cache[0], w.v_cache[0], w.q[0], w.k_tree[0], w.v_tree[0], w.scale)
    t_layer = time.perf_counter() - t
    rows = list(range(w.M if lm_rows is None else min(lm_rows, w.M)))
    t = time.perf_counter()
    oracle.lmhead(w.hidden, w.W, rows=rows)
    t_lm = (time.perf_counter() - t) / len(rows) * w.M
    g = np.random.default_rng(0)
    target = g.integers(0, w.V, size=(w.B, w.T_max)).astype(np.int32)
    t = time.perf_counter()
    n_acc, path, _, _ = oracle.accept(G, w.draft_tok, target)
    t_acc = time.perf_counter() - t
    kc, vc = w.k_cache[0].copy(), w.v_cache[0].copy()
    t = time.perf_counter()
    oracle.compact(G, kc, vc, w.k_tree[0], w.v_tree[0], n_acc, path)
    t_cmp = time.perf_counter() - t
    total = t_layer * w.L + t_lm + t_acc + t_cmp * w.L
    sample = (f"1 of {w.L} layers of attention in full ({t_layer:.2f} s, all {w.B * w.T_max * w.Hq} rows; "
              f"the layers have the same shape), {len(rows)} of {w.M} LM-head rows ({t_lm:.2f} s for all), "
              f"acceptance and 1 of {w.L} layers of compaction in full; one whole step = {total:.1f} s")
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
        sec, sample, cores = cpu_step_estimate(w, lm_rows=48)
        if i >= args.warmup:
            times.append(sec)
    sec = sum(times) / len(times)
    val = 1.0 / sec
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, args),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "every step of this run times: " + sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(w, args):
    return {"workload": f"{args.config}: full verify step, batch {w.B}, prefix {int(w.len.max())}, "
                        f"{w.Hq}/{w.Hkv} heads, head_dim {w.D}, {w.T_max}-node trees, {w.L} layers, "
                        f"vocab {w.V}, hidden {w.Hd}, planted paths 0-6",
            "attention_calls": "one library call per layer (28 per step); the step replayed from a CUDA graph",
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
    ap.add_argument("--no-supplements", action="store_true",
                    help="skip the chain-decoding and compaction-stress measurements (profiler captures)")
    ap.add_argument("--repeats", type=int, default=0,
                    help="measurements of K steps each (default: as many as make about a second of timed work)")
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
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()

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

    K, W = args.steps, max(args.warmup, 3)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed_repeats(step_fn, repeats):
        """`repeats` measurements of exactly K steps each (barrier + synchronize on both sides, CUDA
        events on the launching stream); returns the per-repeat durations in ms."""
        out = []
        for _ in range(repeats):
            e0, e1 = ev(), ev()
            barrier()
            e0.record()
            for _ in range(K):
                step_fn()
            e1.record()
            barrier()
            out.append(e0.elapsed_time(e1))
        return out

    # ---- the step: one attention call per layer + the fused tail, replayed from a CUDA graph
    graph = vs.capture(per_layer=True)
    for _ in range(W):
        graph.replay()
    barrier()
    vs.check_status()
    probe = timed_repeats(graph.replay, 1)[0]                    # untimed estimate: how many repeats make a second
    repeats = args.repeats if args.repeats > 0 else int(min(50, max(1, math.ceil(1000.0 / max(probe, 1e-3)))))
    if rank == 0:
        sampler.wait_first()
    m0 = sampler.mark() if rank == 0 else 0
    ms_step_runs = timed_repeats(graph.replay, repeats)
    m1 = sampler.mark() if rank == 0 else 0
    ms_total = sum(ms_step_runs)                                 # repeats x K steps

    # ---- per-call durations: events around every call, same stream, under the same sustained load
    names = ["attention_single_layer_call", "tail", "attention_all_layers_call", "tail_sampled", "lmhead", "accept", "compact"]
    evs = {n: [] for n in names}

    def timed(name, fn):
        a, b = ev(), ev()
        a.record(); fn(); b.record()
        evs[name].append((a, b))
    for _ in range(max(1, repeats // 2)):
        for _ in range(K):                                       # the same calls as the timed step
            for l in range(vs.L):
                timed("attention_single_layer_call", lambda: vs.attention(l))
            timed("tail", vs.tail)                               # LM head + acceptance + compaction, one call
        torch.cuda.synchronize()
    gen = torch.Generator(device="cuda"); gen.manual_seed(rank)
    u_rand = torch.rand((w.B, w.T_max), device="cuda", generator=gen)
    w_rand = torch.rand((w.B,), device="cuda", generator=gen)
    vs.tail_sampled(1.0, u_rand, w_rand)                         # untimed: its first call allocates the statistics buffers
    for _ in range(max(3, K // 4)):                              # for comparison: all layers in one call, the tail as
        timed("attention_all_layers_call", vs.attention_layers)  # three calls, the tail at temperature 1
        timed("tail_sampled", lambda: vs.tail_sampled(1.0, u_rand, w_rand))
        timed("lmhead", vs.lmhead)
        timed("accept", vs.accept)
        timed("compact", vs.compact)
    torch.cuda.synchronize()
    per_call_ms = {n: sum(a.elapsed_time(b) for a, b in evs[n]) / len(evs[n]) for n in names}

    # ---- upper bound: all layers' attention in ONE call (needs every layer's q, k, v up front)
    graph_all = vs.capture(per_layer=False)
    for _ in range(3):
        graph_all.replay()
    ms_all_runs = timed_repeats(graph_all.replay, max(1, repeats // 2))
    del graph_all

    # ---- end to end: this step's inputs from pinned host memory, results back to the host
    for _ in range(2):
        vs.run_from_host()
    ms_e2e_runs = timed_repeats(vs.run_from_host, max(1, repeats // 4))
    vs.check_status()
    n_acc = vs.host_out["n_acc"].numpy().copy()
    assert (n_acc == w.planted_len + 1).all(), "planted paths were not recovered"

    ms_total, ms_all, ms_e2e = max_over_ranks([ms_total, sum(ms_all_runs), sum(ms_e2e_runs)], "cuda")

    if rank == 0:
        sampler.stop()
        clocks = sampler.summary(m0, m1)
        clocks["timed_region_ms"] = sum(ms_step_runs)
        peaks = read_peaks()
        work = algorithmic_work(w)
        steps_total = K * repeats
        ms_step = ms_total / steps_total
        value = job_throughput(world, steps_total, ms_total)
        tokens_per_step = int(n_acc.sum())
        # dominant kernel: tree attention, one launch per layer; at 60 nodes x 7 grouped heads per KV head its
        # arithmetic intensity (~420 flop/B) puts it on the tensor roof.  The timed regions run for about a
        # second under load, so the sustained figure is the peak; the fraction of the burst figure is given too.
        att_s = per_call_ms["attention_single_layer_call"] * 1e-3
        att_tflops = work["att_flops"] / att_s / 1e12
        att_gbs = work["att_bytes"] / att_s / 1e9
        lm_s = per_call_ms["tail"] * 1e-3
        lm_tflops = work["lm_flops"] / lm_s / 1e12
        traffic = ATTENTION_DRAM_BYTES_PER_LAUNCH.get(args.config)
        roofline = {"kernel": "sd_verify_attention, one layer per launch (attn_umma_kernel<1>)", "bound": "tensor",
                    "achieved": att_tflops, "peak": peaks["tensor_sustained"], "unit": "TFLOP/s",
                    "frac": att_tflops / peaks["tensor_sustained"],
                    "frac_of_burst_peak": att_tflops / peaks["tensor_burst"], "burst_peak": peaks["tensor_burst"],
                    "traffic": traffic,
                    "traffic_unit": "bytes per launch (dram read + write, ncu)",
                    "algorithmic_bytes_per_launch": work["att_bytes"],
                    "algorithmic_flops_per_launch": work["att_flops"],
                    "peak_source": peaks["source"] + " (sustained bf16: about a second of back-to-back launches)",
                    "hbm_gbs": att_gbs, "hbm_frac_of_measured": att_gbs / peaks["hbm"],
                    "hbm_frac_of_nominal_8TBs": att_gbs / 8000.0,
                    "avg_launch_ms": att_s * 1e3, "launches_timed": len(evs["attention_single_layer_call"])}
        all_value = world * K * max(1, repeats // 2) / (ms_all * 1e-3)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
                "warmup": W, "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": workload_config(w, args),
                "repeats": repeats,
                "verified_tokens_per_s": value * tokens_per_step,
                "accepted_tokens_per_step": tokens_per_step,
                "clocks": clocks,
                "e2e": {"value": world * K * max(1, repeats // 4) / (ms_e2e * 1e-3), "unit": UNIT,
                        "h2d_bytes_per_step": vs.h2d_bytes(), "d2h_bytes_per_step": vs.d2h_bytes()},
                "gpu_launches": vs.launches_per_step(per_layer=True) * K,
                "roofline": roofline,
                "upper_bound_all_layers_in_one_call": {
                    "note": "sd_verify_attention_layers needs q and tree K/V of all layers before the call; a decoder "
                            "that computes layer l + 1 from layer l cannot use it, so this is not the headline",
                    "value": all_value, "unit": UNIT, "ms_per_step": 1e3 / all_value * world,
                    "gpu_launches_per_step": vs.launches_per_step(per_layer=False),
                    "attention_ms_all_layers": per_call_ms["attention_all_layers_call"],
                    "attention_tflops": work["att_flops"] * vs.L / (per_call_ms["attention_all_layers_call"] * 1e-3) / 1e12,
                    "attention_frac_of_sustained_peak": work["att_flops"] * vs.L / (per_call_ms["attention_all_layers_call"] * 1e-3) / 1e12 / peaks["tensor_sustained"],
                    "attention_frac_of_burst_peak": work["att_flops"] * vs.L / (per_call_ms["attention_all_layers_call"] * 1e-3) / 1e12 / peaks["tensor_burst"]},
                "calls": {"attention_ms_single_layer_call": per_call_ms["attention_single_layer_call"],
                          "lmhead_accept_compact_ms": per_call_ms["tail"],
                          "lmhead_accept_sampled_compact_ms": per_call_ms["tail_sampled"],
                          "lmhead_ms": per_call_ms["lmhead"], "accept_ms": per_call_ms["accept"],
                          "compact_ms": per_call_ms["compact"],
                          "lmhead_tflops": lm_tflops,
                          "lmhead_frac_of_sustained_peak": lm_tflops / peaks["tensor_sustained"],
                          "lmhead_frac_of_burst_peak": lm_tflops / peaks["tensor_burst"],
                          "lmhead_weight_gbs": work["lm_bytes"] / lm_s / 1e9}}
    del vs
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_supplements:
        # the two bandwidth-regime cases: chain decoding (the paper's own setting) through all 28 layers, and
        # compaction on a shape large enough to be bound by memory
        from paper_2509_18824_b200 import supplements as sup
        chain = next(sup.measure_attention_layers(("chain11",), L=28, reps=30))
        comp = sup.measure_compact()
        keep = ("workload", "layers", "us", "us_per_layer", "algorithmic_bytes", "bytes", "gbs", "frac_hbm",
                "frac_hbm_nominal_8TBs", "flop_per_byte", "tflops", "spot_check", "status")
        line["supplements"] = {
            "chain_decoding_attention": {k: chain[k] for k in keep if k in chain},
            "compaction_stress": {k: comp[k] for k in keep if k in comp},
            "note": "frac_hbm = algorithmic bytes / time / measured copy bandwidth; CUDA events, >= 3 warm-up calls"}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            sec, sample, cores = cpu_step_estimate(w)
            line["cpu_baseline"] = {"value": 1.0 / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": sample}
        print(json.dumps(line))
        sampler.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
