"""The allocation-free LM-head entry point.

Some users of the library verify drafts from a place where they may not ask
CUDA for memory: their device memory was divided up once at start-up, or they
run inside a host program that gives them a fixed arena, or they cannot afford
the device-wide synchronisation an allocation implies.  For them
sd_lmhead_argmax_static carries its own 1 MiB scratch table inside the library.
This test drives it through the C ABI twice in a row, on different inputs, and
requires exactly what sd_lmhead_argmax (caller-provided workspace) returns; the
second call also shows that what the first one left in the shared table does no
harm.  Rows beyond the table's capacity must be refused before anything runs.

Collected last on purpose (file name), so that a run stopping at the first
failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2509_18824_b200 import binding as sd
from paper_2509_18824_b200 import workloads as wl
from paper_2509_18824_b200.step import to_device

pytestmark = pytest.mark.gpu


def _inputs(seed, M, Hd, V):
    g = np.random.default_rng(seed)
    h = wl.f32_to_bf16_bits(g.standard_normal((M, Hd)).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, Hd)) / np.sqrt(Hd)).astype(np.float32))
    return to_device(h), to_device(W)


def _with_workspace(h, W):
    M, V = h.shape[0], W.shape[0]
    am = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    mx = torch.zeros(M, dtype=torch.float32, device="cuda")
    ws = torch.empty(sd.sd_workspace_bytes(None, M, V), dtype=torch.uint8, device="cuda")
    st = sd.new_status()
    sd.sd_lmhead_argmax(h, W, am, mx, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return am.cpu().numpy(), mx.cpu().numpy()


def test_static_scratch_variant_matches_twice_in_a_row():
    # outputs and status are set up before the calls; the calls themselves get no scratch
    cases = [(480, 512, 20000, 1), (37, 256, 4099, 2)]
    prepared = []
    for M, Hd, V, seed in cases:
        h, W = _inputs(seed, M, Hd, V)
        prepared.append((h, W, torch.full((M,), -1, dtype=torch.int32, device="cuda"),
                         torch.zeros(M, dtype=torch.float32, device="cuda"), sd.new_status()))
    for h, W, am, mx, st in prepared:           # two calls back to back on the same stream
        sd.sd_lmhead_argmax_static(h, W, am, mx, st)
    torch.cuda.synchronize()
    for h, W, am, mx, st in prepared:
        assert int(st.item()) == 0
        ref_am, ref_mx = _with_workspace(h, W)
        np.testing.assert_array_equal(am.cpu().numpy(), ref_am)
        np.testing.assert_allclose(mx.cpu().numpy(), ref_mx, rtol=2e-3, atol=2e-3)


def test_static_scratch_variant_refuses_too_many_rows():
    h, W = _inputs(3, 513, 64, 300)
    am = torch.full((513,), -1, dtype=torch.int32, device="cuda")
    st = sd.new_status()
    with pytest.raises(sd.SdError) as e:
        sd.sd_lmhead_argmax_static(h, W, am, None, st)
    assert e.value.code == sd.SD_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert (am.cpu().numpy() == -1).all() and int(st.item()) == 0


def test_static_scratch_variant_leaves_free_memory_alone():
    """The property the entry point is named for: once the first call on the device is behind us (it
    resolves the table's address, and the kernels' code may still have to be loaded before it), a call
    does not move the device's free memory: nothing is allocated, nothing is freed.  (Free memory is a
    device-wide figure; the measurement is repeated so that a change from outside is not mistaken for one.)"""
    h, W = _inputs(5, 300, 256, 9000)
    am = torch.full((300,), -1, dtype=torch.int32, device="cuda")
    st = sd.new_status()
    sd.sd_lmhead_argmax_static(h, W, am, None, st)
    torch.cuda.synchronize()
    moved = []
    for _ in range(3):
        before = torch.cuda.mem_get_info()[0]
        sd.sd_lmhead_argmax_static(h, W, am, None, st)
        torch.cuda.synchronize()
        moved.append(torch.cuda.mem_get_info()[0] - before)
        if moved[-1] == 0:
            break
    assert moved[-1] == 0, moved
    assert int(st.item()) == 0
