"""The C-ABI library loads and exports every symbol include/forgestep.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "forgestep.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ft_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_boundary():
    syms = declared_symbols()
    for need in ("ft_workspace_bytes", "ft_init_model", "ft_train_step", "ft_train_step_host", "ft_forward_loss",
                 "ft_get_param", "ft_set_param", "ft_get_tap", "ft_apply_update", "ft_k_gemm", "ft_k_gemm_ws", "ft_k_attention_fwd",
                 "ft_k_attention_bwd"):
        assert need in syms


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2609_13645_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    for s in declared_symbols():
        assert hasattr(lib, s), s


def test_development_header_is_private_and_its_switches_are_exported():
    """The development switches live in a header of their own inside the package, none of them in the boundary, and the
    library exports each one (the kernel benchmarks and the ablation tests call them)."""
    text = open(os.path.join(ROOT, "paper_2609_13645_b200", "csrc", "forgestep_debug.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    dbg = sorted(set(re.findall(r"\b(ft_debug_[a-z_0-9]+)\s*\(", text)))
    assert len(dbg) >= 8 and not [s for s in declared_symbols() if s.startswith("ft_debug_")]
    from paper_2609_13645_b200 import build
    lib = ctypes.CDLL(build.build())
    for s in dbg:
        assert hasattr(lib, s), s


def test_workspace_size_and_config_validation_run_on_the_host():
    from paper_2609_13645_b200 import binding as B
    ok = B.make_config(1, 256, 4, 4, 64, 688, 1024, 2, 128)
    n = B.workspace_bytes(ok)
    assert n > 0 and n % 256 == 0
    assert B.workspace_bytes(B.make_config(1, 256, 4, 4, 64, 688, 1024, 4, 128)) > n
    for bad in (dict(head_dim=96), dict(d_model=100), dict(d_ffn=100), dict(n_kv_heads=3), dict(vocab=1001),
                dict(emb_scale=-1.0), dict(resid_scale=-0.5), dict(logit_scale=-2.0), dict(tie_embeddings=2),
                dict(qk_norm=3)):
        kw = dict(n_layers=1, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=688, vocab=1024, max_batch=2,
                  max_seq=128)
        kw.update(bad)
        assert B.workspace_bytes(B.make_config(**kw)) == 0, bad
    # model variants: a tied head drops the lm_head tensors from every arena; QK-Norm adds gains and the saved r; a
    # zero factor means 1 and changes nothing
    base = dict(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024, max_batch=2,
                max_seq=128)
    n0 = B.workspace_bytes(B.make_config(**base))
    assert B.workspace_bytes(B.make_config(**base, tie_embeddings=1)) < n0
    assert B.workspace_bytes(B.make_config(**base, qk_norm=1)) > n0
    assert B.workspace_bytes(B.make_config(**base, emb_scale=0.0, resid_scale=0.0, logit_scale=0.0)) == n0
    # a sharded optimizer state (ZeRO-1): masters and moments shrink to 1 / dp_world, nothing else changes
    n_params = 1024 * 256 * 2 + 2 * (256 * 512 + 256 * 256 + 2 * 688 * 256 + 256 * 688)
    for world in (2, 8):
        nw = B.workspace_bytes(B.make_config(**base, dp_world=world, dp_rank=world - 1))
        assert abs((n0 - nw) - 12 * n_params * (world - 1) / world) < 0.02 * 12 * n_params
    for bad in (dict(dp_world=3), dict(dp_world=64), dict(dp_world=2, dp_rank=2), dict(dp_world=0, dp_rank=1), dict(dp_world=2, debug_taps=1)):
        assert B.workspace_bytes(B.make_config(**base, **bad)) == 0, bad
    # the 1B-shaped workload fits one B200 with room to spare
    big = B.make_config(16, 2048, 16, 8, 128, 5632, 32000, 4, 2048)
    assert B.workspace_bytes(big) < 60 * 2 ** 30


def test_model_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2609_13645_b200 import binding as B
    with pytest.raises(RuntimeError):
        B.Model(B.make_config(1, 256, 4, 4, 64, 688, 1024, 2, 128))
