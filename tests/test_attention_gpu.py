"""Flash-attention forward/backward kernels against the oracle's attention core (through the C ABI)."""
import math

import numpy as np
import pytest
import torch

from oracle import decoder as D

pytestmark = pytest.mark.gpu


def _to_bf16_cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).cuda()


def _f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _rel(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30)


def _case(B, S, nh, nkv, d, seed, qscale=1.0):
    rng = np.random.default_rng(seed)
    hq, hkv = nh * d, nkv * d
    qkv = D.bf16_round(rng.standard_normal((B, S, hq + 2 * hkv)) * np.concatenate(
        [np.full(hq, qscale), np.full(hkv, 1.0), np.full(hkv, 1.0)]))
    q = qkv[..., :hq].reshape(B, S, nh, d)
    k = qkv[..., hq:hq + hkv].reshape(B, S, nkv, d)
    v = qkv[..., hq + hkv:].reshape(B, S, nkv, d)
    return qkv, q, k, v


@pytest.mark.parametrize("B,S,nh,nkv,d", [(2, 128, 4, 4, 64), (1, 320, 4, 2, 128), (2, 200, 2, 1, 64),
                                          (1, 77, 2, 2, 128), (1, 1, 2, 1, 64)])
def test_forward_matches_oracle(B, S, nh, nkv, d):
    from paper_2609_13645_b200 import binding as Bn
    qkv, q, k, v = _case(B, S, nh, nkv, d, seed=S, qscale=2.0)
    o_ref, lse_ref = D.attention_fwd(q, k, v, nh // nkv, D.bf16_round, True)
    tq = _to_bf16_cuda(qkv.reshape(B * S, -1))
    o = torch.zeros(B * S, nh * d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
    Bn.k_attention_fwd(tq, o, lse, B, S, nh, nkv, d)
    torch.cuda.synchronize()
    got = _f64(o).reshape(B, S, nh, d)
    assert _rel(got, o_ref) < 2e-3
    assert np.mean(got != o_ref) < 0.02  # same roundings except ties
    assert np.max(np.abs(_f64(lse) - lse_ref)) < 2e-5


def test_forward_is_independent_of_key_block_order_effects():
    """Rows with a large spread of scores (reference jumps between key blocks) still match the one-shot definition."""
    from paper_2609_13645_b200 import binding as Bn
    B, S, nh, nkv, d = 1, 512, 2, 2, 64
    qkv, q, k, v = _case(B, S, nh, nkv, d, seed=5, qscale=6.0)
    o_ref, lse_ref = D.attention_fwd(q, k, v, 1, D.bf16_round, True)
    tq = _to_bf16_cuda(qkv.reshape(B * S, -1))
    o = torch.zeros(B * S, nh * d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
    Bn.k_attention_fwd(tq, o, lse, B, S, nh, nkv, d)
    torch.cuda.synchronize()
    got = _f64(o).reshape(B, S, nh, d)
    assert _rel(got, o_ref) < 2e-3 and np.mean(got != o_ref) < 0.02
    assert np.max(np.abs(_f64(lse) - lse_ref)) < 1e-4


@pytest.mark.parametrize("B,S,nh,nkv,d,rope", [(2, 128, 4, 4, 64, False), (1, 320, 4, 2, 128, True),
                                               (2, 200, 4, 1, 64, True), (1, 77, 2, 2, 128, False)])
def test_backward_matches_oracle(B, S, nh, nkv, d, rope):
    from paper_2609_13645_b200 import binding as Bn
    qkv, q, k, v = _case(B, S, nh, nkv, d, seed=100 + S)
    rng = np.random.default_rng(7)
    n_rep = nh // nkv
    o_ref, lse_ref = D.attention_fwd(q, k, v, n_rep, D.bf16_round, True)
    do = D.bf16_round(rng.standard_normal((B, S, nh, d)))
    lse32 = lse_ref.astype(np.float32).astype(np.float64)
    dq, dk, dv = D.attention_bwd(q, k, v, o_ref, do, lse32, n_rep, D.bf16_round)
    cos = sin = None
    if rope:
        c, s = D.rope_tables(S, d, 1e4)
        dq = D.rope_apply_transpose(dq, c, s)
        dk = D.rope_apply_transpose(dk, c, s)
        cos = torch.from_numpy(c.astype(np.float32)).cuda()
        sin = torch.from_numpy(s.astype(np.float32)).cuda()
    dq, dk, dv = D.bf16_round(dq), D.bf16_round(dk), D.bf16_round(dv)
    tq = _to_bf16_cuda(qkv.reshape(B * S, -1))
    to = _to_bf16_cuda(o_ref.reshape(B * S, -1))
    tdo = _to_bf16_cuda(do.reshape(B * S, -1))
    tl = torch.from_numpy(lse_ref.astype(np.float32)).cuda()
    delta = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
    dqkv = torch.zeros(B * S, (nh + 2 * nkv) * d, dtype=torch.bfloat16, device="cuda")
    Bn.k_attention_bwd(tq, to, tdo, tl, delta, dqkv, B, S, nh, nkv, d, cos, sin)
    torch.cuda.synchronize()
    got = _f64(dqkv).reshape(B, S, -1)
    hq, hkv = nh * d, nkv * d
    g_dq, g_dk, g_dv = got[..., :hq], got[..., hq:hq + hkv], got[..., hq + hkv:]
    assert _rel(g_dv, dv.reshape(B, S, hkv)) < 3e-3
    assert _rel(g_dq, dq.reshape(B, S, hq)) < 3e-3
    assert _rel(g_dk, dk.reshape(B, S, hkv)) < 3e-3
    d_ref = np.einsum("bsnd,bsnd->bns", do, o_ref)
    assert np.max(np.abs(_f64(delta) - d_ref)) < 1e-4 * max(1.0, np.max(np.abs(d_ref)))


@pytest.mark.parametrize("B,S,nh,nkv,d", [(2, 384, 4, 2, 128), (4, 2048, 16, 8, 128), (8, 1024, 12, 12, 64)])
def test_forward_and_backward_are_bit_identical_run_to_run(B, S, nh, nkv, d):
    """Large shapes on purpose: with every SM holding several CTAs, warps of one CTA drift a block apart, which is
    where an ordering mistake between the softmax warps and the MMA issuer shows."""
    from paper_2609_13645_b200 import binding as Bn
    qkv, q, k, v = _case(B, S, nh, nkv, d, seed=9)
    rng = np.random.default_rng(1)
    tq = _to_bf16_cuda(qkv.reshape(B * S, -1))
    tdo = _to_bf16_cuda(D.bf16_round(rng.standard_normal((B * S, nh * d))))
    outs = []
    for _ in range(3):
        o = torch.zeros(B * S, nh * d, dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
        Bn.k_attention_fwd(tq, o, lse, B, S, nh, nkv, d)
        delta = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
        dqkv = torch.zeros(B * S, (nh + 2 * nkv) * d, dtype=torch.bfloat16, device="cuda")
        Bn.k_attention_bwd(tq, o, tdo, lse, delta, dqkv, B, S, nh, nkv, d)
        torch.cuda.synchronize()
        outs.append((o.view(torch.int16).cpu().numpy().copy(), lse.cpu().numpy().copy(),
                     dqkv.view(torch.int16).cpu().numpy().copy()))
    for other in outs[1:]:
        for a, b in zip(outs[0], other):
            assert np.array_equal(a, b)


@pytest.mark.parametrize("B,S,nh,nkv,d,rope", [(2, 128, 4, 4, 64, False), (1, 384, 4, 2, 128, True),
                                               (2, 256, 4, 1, 64, True), (1, 640, 2, 2, 128, True)])
def test_backward_with_stored_ds_matches_oracle(B, S, nh, nkv, d, rope):
    """dK/dV kernel leaves dS^T in a scratch array and dQ is a batched contraction over it: same oracle, same bars."""
    from paper_2609_13645_b200 import binding as Bn
    qkv, q, k, v = _case(B, S, nh, nkv, d, seed=300 + S)
    rng = np.random.default_rng(11)
    n_rep = nh // nkv
    o_ref, lse_ref = D.attention_fwd(q, k, v, n_rep, D.bf16_round, True)
    do = D.bf16_round(rng.standard_normal((B, S, nh, d)))
    lse32 = lse_ref.astype(np.float32).astype(np.float64)
    dq, dk, dv = D.attention_bwd(q, k, v, o_ref, do, lse32, n_rep, D.bf16_round)
    cos = sin = None
    if rope:
        c, s = D.rope_tables(S, d, 1e4)
        dq = D.rope_apply_transpose(dq, c, s)
        dk = D.rope_apply_transpose(dk, c, s)
        cos = torch.from_numpy(c.astype(np.float32)).cuda()
        sin = torch.from_numpy(s.astype(np.float32)).cuda()
    dq, dk, dv = D.bf16_round(dq), D.bf16_round(dk), D.bf16_round(dv)
    tq = _to_bf16_cuda(qkv.reshape(B * S, -1))
    to = _to_bf16_cuda(o_ref.reshape(B * S, -1))
    tdo = _to_bf16_cuda(do.reshape(B * S, -1))
    tl = torch.from_numpy(lse_ref.astype(np.float32)).cuda()
    delta = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
    # NaN-filled scratch and output: every element the contraction reads must have been written by the dK/dV kernel
    ds = torch.full((B * nh, S, S), float("nan"), dtype=torch.bfloat16, device="cuda")
    dqkv = torch.full((B * S, (nh + 2 * nkv) * d), float("nan"), dtype=torch.bfloat16, device="cuda")
    Bn.k_attention_bwd_ws(tq, to, tdo, tl, delta, dqkv, ds, B, S, nh, nkv, d, cos, sin)
    torch.cuda.synchronize()
    got = _f64(dqkv).reshape(B, S, -1)
    assert np.all(np.isfinite(got))
    hq, hkv = nh * d, nkv * d
    g_dq, g_dk, g_dv = got[..., :hq], got[..., hq:hq + hkv], got[..., hq + hkv:]
    assert _rel(g_dv, dv.reshape(B, S, hkv)) < 3e-3
    assert _rel(g_dq, dq.reshape(B, S, hq)) < 3e-3
    assert _rel(g_dk, dk.reshape(B, S, hkv)) < 3e-3
    # dK and dV do not depend on the path: bit for bit those of the recomputing backward
    ref = torch.zeros_like(dqkv)
    Bn.k_attention_bwd(tq, to, tdo, tl, delta, ref, B, S, nh, nkv, d, cos, sin)
    torch.cuda.synchronize()
    assert torch.equal(ref[:, hq:].view(torch.int16), dqkv[:, hq:].view(torch.int16))
    assert _rel(_f64(ref[:, :hq]), _f64(dqkv[:, :hq])) < 2e-3


def test_backward_with_stored_ds_falls_back_when_it_cannot_apply():
    """A sequence that is not a multiple of 128, or a scratch array that is too small, takes the recomputing kernels."""
    from paper_2609_13645_b200 import binding as Bn
    for (B, S, nh, nkv, d, short) in [(1, 200, 2, 1, 64, False), (1, 256, 2, 2, 64, True)]:
        qkv, q, k, v = _case(B, S, nh, nkv, d, seed=5)
        rng = np.random.default_rng(2)
        tq = _to_bf16_cuda(qkv.reshape(B * S, -1))
        tdo = _to_bf16_cuda(D.bf16_round(rng.standard_normal((B * S, nh * d))))
        o = torch.zeros(B * S, nh * d, dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
        Bn.k_attention_fwd(tq, o, lse, B, S, nh, nkv, d)
        delta = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
        ds = torch.zeros(B * nh * S * S // (2 if short else 1), dtype=torch.bfloat16, device="cuda")
        a = torch.zeros(B * S, (nh + 2 * nkv) * d, dtype=torch.bfloat16, device="cuda")
        b = torch.zeros_like(a)
        Bn.k_attention_bwd_ws(tq, o, tdo, lse, delta, a, ds, B, S, nh, nkv, d)
        Bn.k_attention_bwd(tq, o, tdo, lse, delta, b, B, S, nh, nkv, d)
        torch.cuda.synchronize()
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
        assert not bool(ds.any())


@pytest.mark.parametrize("B,S,nh,nkv,d", [(2, 384, 4, 2, 128), (4, 2048, 16, 8, 128), (8, 1024, 12, 12, 64)])
def test_backward_with_stored_ds_is_bit_identical_run_to_run(B, S, nh, nkv, d):
    from paper_2609_13645_b200 import binding as Bn
    qkv, q, k, v = _case(B, S, nh, nkv, d, seed=9)
    rng = np.random.default_rng(1)
    tq = _to_bf16_cuda(qkv.reshape(B * S, -1))
    tdo = _to_bf16_cuda(D.bf16_round(rng.standard_normal((B * S, nh * d))))
    o = torch.zeros(B * S, nh * d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
    Bn.k_attention_fwd(tq, o, lse, B, S, nh, nkv, d)
    outs = []
    for _ in range(3):
        delta = torch.zeros(B, nh, S, dtype=torch.float32, device="cuda")
        ds = torch.empty(B * nh, S, S, dtype=torch.bfloat16, device="cuda")
        dqkv = torch.zeros(B * S, (nh + 2 * nkv) * d, dtype=torch.bfloat16, device="cuda")
        Bn.k_attention_bwd_ws(tq, o, tdo, lse, delta, dqkv, ds, B, S, nh, nkv, d)
        torch.cuda.synchronize()
        outs.append(dqkv.view(torch.int16).cpu().numpy().copy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
