"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sdverify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sd_[a-z_0-9]+)\s*\(", text)))


def test_library_loads_and_exports_the_header():
    from paper_2509_18824_b200 import build
    lib = ctypes.CDLL(build.build())
    syms = declared_symbols()
    assert {"sd_verify_attention", "sd_lmhead_argmax", "sd_accept_tree", "sd_compact_kv"} <= set(syms)
    for s in syms:
        assert hasattr(lib, s), s
    lib.sd_status_string.restype = ctypes.c_char_p
    assert lib.sd_status_string(0) == b"SD_OK"
    assert lib.sd_status_string(-7) == b"SD_ERR_BOUNDS"
    assert lib.sd_version() >= 100


def test_binding_matches_header():
    from paper_2509_18824_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()
    # host-side argument checks need no GPU: a null geometry is refused before any launch
    assert binding.lib.sd_tree_prepare(None, None, None) == binding.SD_ERR_INVALID_ARG
    bt = binding.sd_batch(1, 65, 4, 1, 128, 64, 4, 16, 16, 16, 16, 16)
    assert binding.lib.sd_tree_prepare(ctypes.byref(bt), 16, None) == binding.SD_ERR_UNSUPPORTED
    bt = binding.sd_batch(1, 8, 4, 1, 64, 64, 4, 16, 16, 16, 16, 16)
    assert binding.lib.sd_tree_prepare(ctypes.byref(bt), 16, None) == binding.SD_ERR_UNSUPPORTED
    bt = binding.sd_batch(1, 8, 4, 1, 128, 64, 4, 16, 16, 8, 16, 16)     # misaligned n_nodes
    assert binding.lib.sd_tree_prepare(ctypes.byref(bt), 16, None) == binding.SD_ERR_INVALID_ARG
    assert binding.sd_workspace_bytes(None, 60, 152064) > 0


def test_product_code_never_touches_the_checker():
    pkg = os.path.join(ROOT, "paper_2509_18824_b200")
    for dirpath, _, files in os.walk(pkg):
        if "_build" in dirpath:
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text, f
                assert "liboracle" not in text and "sd_oracle" not in text, f


def test_host_side_refusals_of_the_newer_calls():
    """Argument checks that need no GPU: every refusal comes back before anything is launched."""
    from paper_2509_18824_b200 import binding as b
    L = b.lib
    f = ctypes.c_float
    ok = 4096                                               # any 16-byte aligned, non-null stand-in address
    # draft feature aggregation: at most 8 meta queries, 32 layers, heads of 128
    assert L.sd_draft_feature_attention(ok, ok, ok, 4, 28, 9, 2, 256, f(1.0), ok, None) == b.SD_ERR_UNSUPPORTED
    assert L.sd_draft_feature_attention(ok, ok, ok, 4, 33, 4, 2, 256, f(1.0), ok, None) == b.SD_ERR_UNSUPPORTED
    assert L.sd_draft_feature_attention(ok, ok, ok, 4, 28, 4, 2, 200, f(1.0), ok, None) == b.SD_ERR_UNSUPPORTED
    assert L.sd_draft_feature_attention(ok, ok, ok, 4, 28, 4, 2, 256, f(0.0), ok, None) == b.SD_ERR_INVALID_ARG
    assert L.sd_draft_feature_attention(None, ok, ok, 4, 28, 4, 2, 256, f(1.0), ok, None) == b.SD_ERR_INVALID_ARG
    # soft-max statistics: temperature must be positive, the hidden size a multiple of 64, lse present
    assert L.sd_lmhead_stats(ok, ok, 8, 128, 100, f(0.0), None, None, ok, None, ok, 1 << 30, ok, None) == b.SD_ERR_INVALID_ARG
    assert L.sd_lmhead_stats(ok, ok, 8, 100, 100, f(1.0), None, None, ok, None, ok, 1 << 30, ok, None) == b.SD_ERR_UNSUPPORTED
    assert L.sd_lmhead_stats(ok, ok, 8, 128, 100, f(1.0), None, None, None, None, ok, 1 << 30, ok, None) == b.SD_ERR_INVALID_ARG
    assert L.sd_lmhead_stats(ok, ok, 8, 128, 100, f(1.0), None, None, ok, 4100, ok, 1 << 30, ok, None) == b.SD_ERR_INVALID_ARG
    # the workspace figure covers every call that takes one, and grows with the vocabulary
    bt = b.sd_batch(8, 60, 28, 4, 128, 64, 66, 16, 16, 16, 16, 16)
    small = L.sd_workspace_bytes(ctypes.byref(bt), 480, 1024)
    big = L.sd_workspace_bytes(ctypes.byref(bt), 480, 152064)
    assert big > small >= L.sd_workspace_bytes(None, 480, 1024) > 0
    assert big >= 8 * 152064 * 4                            # room for one probability row per sequence


def test_host_side_refusals_come_before_any_launch():
    """Host-detectable problems of the attention and the sampled-acceptance calls return their status with
    nothing enqueued (there is no GPU here: a launch attempt would come back as SD_ERR_CUDA instead)."""
    from paper_2509_18824_b200 import binding as b
    L = b.lib
    f = ctypes.c_float
    ok = 4096
    bt = b.sd_batch(2, 8, 4, 1, 128, 64, 4, ok, ok, ok, ok, ok)
    cache = b.sd_kv_layer(ok, ok, 8)
    need = L.sd_workspace_bytes(ctypes.byref(bt), 0, 0)
    assert need > 0
    # workspace smaller than sd_workspace_bytes: refused, for the one-layer and the all-layers call
    assert L.sd_verify_attention(ctypes.byref(bt), ctypes.byref(cache), ok, ok, ok, f(0.1), ok, None,
                                 ok, need - 1, ok, None) == b.SD_ERR_WORKSPACE
    ptrs = (ctypes.c_void_p * 1)(ok)
    assert L.sd_verify_attention_layers(ctypes.byref(bt), ctypes.byref(cache), 1, ptrs, ptrs, ptrs, f(0.1), ptrs, None,
                                        ok, need - 1, ok, None) == b.SD_ERR_WORKSPACE
    # sampled acceptance: a vocabulary beyond the residual draw's tables (8192 groups of 32 with the
    # group statistics, 4096 blocks of 256 without) is refused before the first kernel
    big = 1 << 40
    assert L.sd_accept_tree_sampled(ctypes.byref(bt), ok, ok, 128, 8192 * 32 + 1, f(1.0), ok, ok, ok, ok, ok,
                                    ok, ok, ok, ok, ok, big, ok, None) == b.SD_ERR_UNSUPPORTED
    assert L.sd_accept_tree_sampled(ctypes.byref(bt), ok, ok, 128, 4096 * 256 + 1, f(1.0), ok, None, ok, ok, ok,
                                    ok, ok, ok, ok, ok, big, ok, None) == b.SD_ERR_UNSUPPORTED
    assert L.sd_accept_tree_sampled(ctypes.byref(bt), ok, ok, 128, 1000, f(1.0), ok, None, ok, ok, ok,
                                    ok, ok, ok, ok, ok, 16, ok, None) == b.SD_ERR_WORKSPACE
    # chains drafted by sampling: the vocabulary limit of the block-wise draw, the distributions are required
    chain = lambda V, q_rows, ws_bytes: L.sd_accept_chain_sampled(
        ctypes.byref(bt), ok, ok, 128, V, f(1.0), ok, None, ok, ok, q_rows, ok, ok, ok, ok, ok, ok, ok, ws_bytes, ok, None)
    assert chain(4096 * 256 + 1, ok, big) == b.SD_ERR_UNSUPPORTED
    assert chain(1000, None, big) == b.SD_ERR_INVALID_ARG
    assert chain(1000, ok, 16) == b.SD_ERR_WORKSPACE
    assert L.sd_lmhead_stats_logits(ok, ok, 8, 128, 100, f(1.0), None, None, ok, None, ok, 1 << 30, ok, None) == b.SD_ERR_INVALID_ARG
    assert L.sd_lmhead_stats_logits(ok, ok, 8, 100, 100, f(1.0), None, None, ok, ok, ok, 1 << 30, ok, None) == b.SD_ERR_UNSUPPORTED
    # sampled trees: the vocabulary must fit eight shared-memory slices
    assert L.sd_accept_tree_sampled_q(ctypes.byref(bt), 8 * 20480 + 1, f(1.0), ok, ok, ok, ok, ok, ok, ok, ok, ok, ok, ok,
                                      None) == b.SD_ERR_UNSUPPORTED
    assert L.sd_accept_tree_sampled_q(ctypes.byref(bt), 1000, f(1.0), ok, None, ok, ok, ok, ok, ok, ok, ok, ok, ok,
                                      None) == b.SD_ERR_INVALID_ARG
    # the fused call at a temperature: the same vocabulary limit, the group table is required, workspace
    fused = lambda V, gs, ws_bytes: L.sd_lmhead_accept_sampled_compact(
        ctypes.byref(bt), ok, ok, 128, V, f(1.0), ok, ok, ok, ctypes.byref(cache), 1, ptrs, ptrs, ok, gs,
        ok, ok, ok, ok, ok, ws_bytes, ok, None)
    assert fused(8192 * 32 + 1, ok, big) == b.SD_ERR_UNSUPPORTED
    assert fused(1000, None, big) == b.SD_ERR_INVALID_ARG
    assert fused(1000, ok, 16) == b.SD_ERR_WORKSPACE
