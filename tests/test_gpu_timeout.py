"""A bounded wait that runs out: the kernels give up, report SD_ERR_TIMEOUT through the status word and
return normally, and the next ordinary call on the same stream is correct.

The waits are made to run out from the host side only, through the library's test hooks (environment
variables read at every launch): SDV_TEST_WAIT_CYCLES shortens the bound of every barrier wait to about a
tenth of a millisecond, SDV_TEST_WITHHOLD=1 makes one role skip a single arrival (the softmax warps never
report their first tile / the MMA thread never reports its first accumulator), so that its consumer waits
for something that does not come.  Nothing faults, traps or spins without a bound; the grids are one CTA.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_18824_b200 import binding as sd
from paper_2509_18824_b200 import workloads as wl
from gpu_util import gpu_attention, check_attention, gpu_lmhead, check_argmax
from paper_2509_18824_b200.step import to_device

pytestmark = pytest.mark.gpu


def test_attention_wait_runs_out_and_the_next_call_is_fine(monkeypatch):
    w = wl.make("c1", lmhead=False, q_gain=45.0)                 # one sequence, one KV head, 32 rows: one CTA
    ref, _ = oracle.attention(oracle.Geometry.of(w), w.k_cache[0], w.v_cache[0], w.q[0], w.k_tree[0],
                              w.v_tree[0], w.scale)
    monkeypatch.setenv("SDV_TEST_CHUNKS", "1")                   # no key chunks: no cluster
    monkeypatch.setenv("SDV_TEST_WAIT_CYCLES", "200000")
    monkeypatch.setenv("SDV_TEST_WITHHOLD", "1")
    out, lse, status = gpu_attention(w, layer=0)                 # returns: the call and the synchronisation after it
    assert status == sd.SD_ERR_TIMEOUT
    monkeypatch.delenv("SDV_TEST_WITHHOLD")
    monkeypatch.delenv("SDV_TEST_WAIT_CYCLES")
    for _ in range(2):                                           # the context is intact: ordinary calls, right results
        out, lse, status = gpu_attention(w, layer=0)
        assert status == 0
        check_attention(out, ref, "after a timed-out call")


def test_lmhead_wait_runs_out_and_the_next_call_is_fine(monkeypatch):
    g = np.random.default_rng(1)
    M, Hd, V = 8, 128, 100                                       # at most 128 vocabulary rows: the single-CTA kernel
    h = wl.f32_to_bf16_bits(g.standard_normal((M, Hd)).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, Hd)) / np.sqrt(Hd)).astype(np.float32))
    hd, Wd = to_device(h), to_device(W)
    am = torch.full((M,), -5, dtype=torch.int32, device="cuda")
    ws = torch.empty(sd.sd_workspace_bytes(None, M, V), dtype=torch.uint8, device="cuda")
    st = sd.new_status()
    monkeypatch.setenv("SDV_TEST_WAIT_CYCLES", "200000")
    monkeypatch.setenv("SDV_TEST_WITHHOLD", "1")
    sd.sd_lmhead_argmax(hd, Wd, am, None, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == sd.SD_ERR_TIMEOUT
    monkeypatch.delenv("SDV_TEST_WITHHOLD")
    monkeypatch.delenv("SDV_TEST_WAIT_CYCLES")
    am2, mx2 = gpu_lmhead(h, W)
    ram, t1, t2 = oracle.lmhead(h, W)
    check_argmax(am2, mx2, ram, t1, t2)
