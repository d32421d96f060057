"""GPU parity of the draft-side feature aggregation against oracle/draft_attention.py."""
import numpy as np
import pytest
import torch

from oracle.draft_attention import feature_attention
from paper_2509_18824_b200 import binding as sd
from paper_2509_18824_b200 import workloads as wl
from paper_2509_18824_b200.step import to_device

pytestmark = pytest.mark.gpu


def run(qp, k, v, H, scale):
    Q, D = qp.shape
    S = k.shape[0]
    out = torch.full((S, Q, D), 7.0, dtype=torch.bfloat16, device="cuda")
    same = v is k
    kd = to_device(k)
    vd = kd if same else to_device(v)
    sd.sd_draft_feature_attention(to_device(qp), kd, vd, H, scale, out)
    torch.cuda.synchronize()
    return out.float().cpu().numpy()


@pytest.mark.parametrize("S,L,Q,H,gain,same", [(1, 1, 1, 1, 1.0, False), (37, 28, 4, 3, 1.0, False),
                                               (5, 32, 8, 2, 6.0, False), (300, 7, 3, 28, 6.0, True),
                                               (2500, 28, 2, 1, 3.0, True)])
def test_feature_attention_matches_reference(S, L, Q, H, gain, same):
    g = np.random.default_rng(S + L)
    D = H * 128
    bf = lambda a: wl.f32_to_bf16_bits(a.astype(np.float32))
    qp = bf(g.standard_normal((Q, D)) * gain)
    k = bf(g.standard_normal((S, L, D)))
    v = k if same else bf(g.standard_normal((S, L, D)) * 3)
    scale = 1.0 / np.sqrt(128)
    got = run(qp, k, v, H, scale)
    ref = feature_attention(wl.bf16_bits_to_f64(qp), wl.bf16_bits_to_f64(k), wl.bf16_bits_to_f64(v), H, scale)
    d = np.abs(got - ref)
    # fp32 accumulation over 128-long dots and at most 32 layers, bf16 output (2^-9 relative)
    assert d.max() <= 2e-2 * max(1.0, np.abs(ref).max()) and d.mean() <= 2e-3 * max(1.0, np.abs(ref).mean() * 4)
    rel = np.sqrt((d ** 2).sum() / (ref ** 2).sum())
    assert rel <= 5e-3, rel


def test_feature_attention_unsupported_shapes():
    q = torch.zeros((9, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((2, 4, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((2, 9, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sd.SdError):
        sd.sd_draft_feature_attention(q, k, k, 1, 1.0, out)           # more than 8 meta queries
