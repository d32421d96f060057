"""Helpers shared by the GPU parity tests: run the library on a workload-like
object and compare with the fp64 checker."""
import numpy as np
import torch

import oracle
from paper_2509_18824_b200 import binding as sd
from paper_2509_18824_b200 import workloads as wl
from paper_2509_18824_b200.step import to_device

# tolerances stated for bf16 inputs with fp32 accumulation
ATT_MAX_ABS = 1e-2
ATT_MEAN_ABS = 1e-3
ATT_REL_L2 = 2e-2
ARGMAX_BAND = 1e-3


def gpu_attention(p, layer=None):
    """p: object with geometry + q/k_tree/v_tree/k_cache/v_cache (arrays, or lists indexed by layer).
    Returns (out f32 [B,T,Hq,D], lse f32 [B,T,Hq], status int)."""
    pick = (lambda x: x) if layer is None else (lambda x: x[layer])
    bt = sd.Batch.of(p)
    st = sd.new_status()
    sd.sd_tree_prepare(bt, st)
    kc, vc = to_device(pick(p.k_cache)), to_device(pick(p.v_cache))
    q, kt, vt = to_device(pick(p.q)), to_device(pick(p.k_tree)), to_device(pick(p.v_tree))
    out = torch.full((p.B, p.T_max, p.Hq, p.D), 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((p.B, p.T_max, p.Hq), dtype=torch.float32, device="cuda")
    ws = torch.empty(sd.sd_workspace_bytes(bt), dtype=torch.uint8, device="cuda")
    sd.sd_verify_attention(bt, sd.kv_layer(kc, vc), q, kt, vt, float(p.scale), out, lse, ws, st)
    torch.cuda.synchronize()
    return out.float().cpu().numpy(), lse.cpu().numpy(), int(st.item())


def check_attention(got, ref, what=""):
    """got/ref arrays of equal shape (ref fp64)."""
    ok = np.isfinite(ref)
    d = np.abs(got[ok].astype(np.float64) - ref[ok])
    rel = np.sqrt((d ** 2).sum()) / max(np.sqrt((ref[ok] ** 2).sum()), 1e-30)
    assert np.isfinite(got[ok]).all(), what
    assert d.max() <= ATT_MAX_ABS, f"{what}: max abs err {d.max():.3e}"
    assert d.mean() <= ATT_MEAN_ABS, f"{what}: mean abs err {d.mean():.3e}"
    assert rel <= ATT_REL_L2, f"{what}: relative L2 err {rel:.3e}"
    return d.max(), d.mean(), rel


def gpu_lmhead(hidden, W):
    h, Wd = to_device(hidden), to_device(W)
    M, V = hidden.shape[0], W.shape[0]
    am = torch.full((M,), -5, dtype=torch.int32, device="cuda")
    mx = torch.zeros(M, dtype=torch.float32, device="cuda")
    ws = torch.empty(sd.sd_workspace_bytes(None, M, V), dtype=torch.uint8, device="cuda")
    st = sd.new_status()
    sd.sd_lmhead_argmax(h, Wd, am, mx, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return am.cpu().numpy(), mx.cpu().numpy()


def check_argmax(got_idx, got_max, ref_idx, ref_top1, ref_top2, require_all=False):
    """Identical except where the checker's top-2 logits are closer than the band;
    returns (rows in band, mismatches in band, mismatches outside band)."""
    gap = ref_top1 - ref_top2
    in_band = gap < ARGMAX_BAND
    mism = got_idx != ref_idx
    outside = int((mism & ~in_band).sum())
    assert outside == 0, f"{outside} argmax mismatches outside the {ARGMAX_BAND} band"
    if require_all:
        assert not mism.any()
    np.testing.assert_allclose(got_max, ref_top1, rtol=2e-3, atol=2e-3)
    return int(in_band.sum()), int((mism & in_band).sum()), outside
