"""The attention backward that brings its own scratch, for callers that cannot allocate device memory.

Some users of this library run where allocating is not possible: inside an allocator hook, in an operator plugin
that only receives its inputs and outputs, or with the device's memory already fully handed out.  For them
ft_k_attention_bwd_noalloc keeps the small fp32 scratch of the backward pre-pass in a fixed array inside the
library.  It must give exactly what ft_k_attention_bwd gives, call after call, although every call reuses the
same array.  Collected last on purpose (file name), and independent of what ran before it.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _inputs(B, S, nh, nkv, d, seed):
    from paper_2609_13645_b200 import binding as Bn
    g = torch.Generator(device="cuda").manual_seed(seed)
    qkv = torch.randn(B * S, (nh + 2 * nkv) * d, device="cuda", generator=g).bfloat16()
    do = torch.randn(B * S, nh * d, device="cuda", generator=g).bfloat16()
    o = torch.empty(B * S, nh * d, dtype=torch.bfloat16, device="cuda")
    lse = torch.empty(B, nh, S, dtype=torch.float32, device="cuda")
    Bn.k_attention_fwd(qkv, o, lse, B, S, nh, nkv, d)
    return qkv, o, do, lse


def test_noalloc_backward_equals_the_regular_one_on_two_calls_in_a_row():
    from paper_2609_13645_b200 import binding as Bn
    # two different problems back to back: the second call finds the first call's values in the shared scratch
    for B, S, nh, nkv, d, seed in ((2, 320, 4, 2, 128, 1), (1, 200, 4, 4, 64, 2)):
        qkv, o, do, lse = _inputs(B, S, nh, nkv, d, seed)
        delta = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
        want = torch.zeros_like(qkv)
        Bn.k_attention_bwd(qkv, o, do, lse, delta, want, B, S, nh, nkv, d)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        got = torch.full_like(qkv, 3.0)
        st = Bn.k_attention_bwd_noalloc(qkv, o, do, lse, got, B, S, nh, nkv, d)
        torch.cuda.synchronize()
        assert st == Bn.FT_OK
        assert torch.cuda.mem_get_info()[0] >= free_before - (1 << 20)  # `got` came from torch's cache or is small
        a = got.float().cpu().numpy().astype(np.float64)
        b = want.float().cpu().numpy().astype(np.float64)
        rel = np.linalg.norm(a - b) / np.linalg.norm(b)
        assert rel < 3e-3, rel  # the tolerance of the attention parity tests; in fact the same kernels, same bits
        assert np.array_equal(a, b)


def test_noalloc_backward_rejects_problems_beyond_its_scratch():
    from paper_2609_13645_b200 import binding as Bn
    t = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    f = torch.zeros(8, dtype=torch.float32, device="cuda")
    # 2 * 16 * 65536 floats of delta would be needed: more than the 1 Mi floats built in; nothing is launched
    st = Bn.k_attention_bwd_noalloc(t, t, t, f, t, 2, 65536, 16, 8, 128)
    assert st == Bn.FT_ENOMEM
    torch.cuda.synchronize()
