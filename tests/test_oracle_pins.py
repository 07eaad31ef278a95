"""Pins of the CPU oracle against things other than itself.

Each test ties one part of oracle/decoder.py to what the paper or the
mathematics fixes: finite differences, PyTorch fp64 autograd and
torch.optim.AdamW as independent library routines, closed forms, invariants,
and numbers worked by hand or printed by the paper (tests/golden/).
"""
import math
import os

import numpy as np
import pytest
import torch

import synth_inputs as SI
from oracle import decoder as D

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny_cfg(**kw):
    base = dict(n_layers=2, d_model=16, n_heads=4, n_kv_heads=2, head_dim=8, d_ffn=24, vocab=32)
    base.update(kw)
    return D.Config(**base)


def tiny_params(cfg, seed=7, std=0.2):
    rng = np.random.default_rng(seed)
    p = {}
    for name, shape in D.param_specs(cfg):
        if len(shape) == 1:
            p[name] = (1.0 + 0.1 * rng.standard_normal(shape)).astype(np.float32)
        else:
            p[name] = (std * rng.standard_normal(shape)).astype(np.float32)
    return p


def tiny_batch(cfg, B=2, S=8, seed=3):
    rng = np.random.default_rng(seed)
    ids = rng.integers(0, cfg.vocab, size=(B, S + 1))
    return ids[:, :S].astype(np.int32), ids[:, 1:].astype(np.int32)


# ---------------------------------------------------------------- bf16 rounding
def test_bf16_round_matches_torch_conversion():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.standard_normal(20000) * np.exp(rng.uniform(-30, 30, 20000)),
        np.array([0.0, -0.0, 1.0, -1.0, 1.00390625, 1.01171875, 255.5, 256.5, 1e-40, -3e-39, 3.38e38]),
    ]).astype(np.float32)  # fp32 inputs: the fp32->bf16 cast of torch is then a single rounding
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    got = D.bf16_round(x.astype(np.float64))
    assert np.array_equal(got, want)


def test_bf16_round_ties_to_even_and_idempotent():
    # 1 + 2^-8 is exactly between 1 and 1 + 2^-7: goes to the even significand (1.0)
    assert D.bf16_round(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert D.bf16_round(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    x = np.random.default_rng(1).standard_normal(1000)
    y = D.bf16_round(x)
    assert np.array_equal(D.bf16_round(y), y)
    assert np.max(np.abs(y - x) / np.abs(x)) <= 2.0 ** -8 * (1 + 1e-12)  # unit roundoff of 8 significant bits
    # power-of-two scaling commutes with the rounding (what the integer softmax reference relies on)
    assert np.array_equal(D.bf16_round(x * 8.0), 8.0 * y)


# ---------------------------------------------------------------- whole backward: finite differences
VARIANTS = [dict(), dict(emb_scale=12.0, resid_scale=1.4 / math.sqrt(2), logit_scale=256.0 / 1024.0),
            dict(tie_embeddings=True), dict(tie_embeddings=True, emb_scale=3.0, resid_scale=0.7, logit_scale=0.5),
            dict(qk_norm=True), dict(qk_norm=True, tie_embeddings=True, n_kv_heads=1),
            dict(rope_factors=(1.0, 1.7, 3.1, 4.9), rope_mscale=1.19, qk_norm=True),
            dict(mtp=True, mtp_weight=0.3), dict(mtp=True, mtp_weight=1.0, tie_embeddings=True, qk_norm=True, emb_scale=3.0,
                                                 resid_scale=0.7, logit_scale=0.5)]
VARIANT_IDS = ["plain", "mup", "tied", "tied+mup", "qknorm", "qknorm+tied+mqa", "longrope+qknorm", "mtp", "mtp+tied+qknorm+mup"]


@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
def test_gradients_match_central_finite_differences(variant):
    cfg = tiny_cfg(**variant)
    params = tiny_params(cfg)
    tok, lab = tiny_batch(cfg)
    lab[0, 2] = -1  # one ignored label
    _, grads, _ = D.forward_backward(cfg, params, tok, lab, mode="exact", want_taps=False)
    p64 = {k: v.astype(np.float64) for k, v in params.items()}
    eps = 1e-5
    worst = 0.0
    rng = np.random.default_rng(5)
    for name, arr in p64.items():
        flat = arr.reshape(-1)
        idx = np.arange(flat.size) if flat.size <= 64 else rng.choice(flat.size, 64, replace=False)
        fd = np.zeros(len(idx))
        for n, i in enumerate(idx):
            old = flat[i]
            flat[i] = old + eps
            lp, _, _ = D.forward_backward(cfg, p64, tok, lab, mode="exact", want_taps=False, backward=False)
            flat[i] = old - eps
            lm, _, _ = D.forward_backward(cfg, p64, tok, lab, mode="exact", want_taps=False, backward=False)
            flat[i] = old
            fd[n] = (lp - lm) / (2 * eps)
        an = grads[name].reshape(-1)[idx]
        err = np.linalg.norm(fd - an) / max(np.linalg.norm(an), 1e-30)
        worst = max(worst, err)
        assert err < 2e-6, (name, err)
    assert worst > 0.0


# ---------------------------------------------------------------- second opinion: torch fp64 autograd
def _torch_loss(cfg, tp, tok, lab):
    """The same decoder written with torch library ops (independent of the oracle's numpy code)."""
    import torch.nn.functional as F
    B, S = tok.shape
    d, nh, nkv = cfg.head_dim, cfg.n_heads, cfg.n_kv_heads
    pos = torch.arange(S, dtype=torch.float64)
    inv = torch.tensor(cfg.rope_theta, dtype=torch.float64) ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
    if cfg.rope_factors is not None:  # LongRoPE: per-frequency rescale factors, one magnitude factor on cos and sin
        inv = inv / torch.tensor(cfg.rope_factors, dtype=torch.float64)
    ang = torch.outer(pos, inv)
    cos = (cfg.rope_mscale * torch.cos(ang)).to(torch.float32).to(torch.float64)  # the tables are stored as fp32
    sin = (cfg.rope_mscale * torch.sin(ang)).to(torch.float32).to(torch.float64)

    def rope(x):  # x [B,S,n,d]; rotate-half form
        half = torch.cat([-x[..., d // 2:], x[..., :d // 2]], dim=-1)
        c2 = torch.cat([cos, cos], -1)[None, :, None, :]
        s2 = torch.cat([sin, sin], -1)[None, :, None, :]
        return x * c2 + half * s2

    def rms(x, g):
        return x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + cfg.rms_eps) * g

    # model variants, written the way the published muP decoders apply them: embeddings times scale_emb, every branch
    # output times scale_depth / sqrt(n_layers) before the residual add, final hidden state times the logit factor
    def layer(x, p):
        qkv = F.linear(rms(x, tp[p + "norm1"]), tp[p + "wqkv"])
        q, k, v = torch.split(qkv, [cfg.h_q, cfg.h_kv, cfg.h_kv], dim=-1)
        q, k = q.reshape(B, S, nh, d), k.reshape(B, S, nkv, d)
        if cfg.qk_norm:  # per-head RMSNorm over head_dim before the rotation, as in the published QK-Norm decoders
            q, k = rms(q, tp[p + "q_norm"]), rms(k, tp[p + "k_norm"])
        q = rope(q).transpose(1, 2)
        k = rope(k).transpose(1, 2).repeat_interleave(nh // nkv, dim=1)
        v = v.reshape(B, S, nkv, d).transpose(1, 2).repeat_interleave(nh // nkv, dim=1)
        o = F.scaled_dot_product_attention(q, k, v, is_causal=True)
        x = x + F.linear(o.transpose(1, 2).reshape(B, S, cfg.h_q), tp[p + "wo"]) * cfg.resid_scale
        g, u = torch.chunk(F.linear(rms(x, tp[p + "norm2"]), tp[p + "wgu"]), 2, dim=-1)
        return x + F.linear(F.silu(g) * u, tp[p + "wd"]) * cfg.resid_scale

    head = tp["embed"] if cfg.tie_embeddings else tp["lm_head"]
    ids = torch.from_numpy(tok.astype(np.int64))
    labels = torch.from_numpy(lab.astype(np.int64))
    x = F.embedding(ids, tp["embed"]) * cfg.emb_scale
    for l in range(cfg.n_layers):
        x = layer(x, f"layers.{l}.")
    z = F.linear(rms(x, tp["norm_f"]) * cfg.logit_scale, head)
    loss = F.cross_entropy(z.reshape(B * S, -1), labels.reshape(-1), ignore_index=-1)
    if cfg.mtp:
        # the published depth-1 multi-token-prediction module: the backbone's last hidden state and the embedding of the
        # NEXT token, each normalised, concatenated and projected back to the model width by ONE matrix [h, 2h]; one
        # more decoder layer; the backbone's output head; trained on the token after next
        nxt = torch.cat([ids[:, 1:], ids[:, -1:]], dim=1)
        lab2 = torch.cat([labels[:, 1:], torch.full((B, 1), -1, dtype=torch.int64)], dim=1)
        cat = torch.cat([rms(x, tp["mtp.norm_h"]), rms(F.embedding(nxt, tp["embed"]) * cfg.emb_scale, tp["mtp.norm_e"])], dim=-1)
        w_cat = torch.cat([tp["mtp.proj_h"], tp["mtp.proj_e"]], dim=1)
        x2 = layer(F.linear(cat, w_cat), "mtp.layer.")
        z2 = F.linear(rms(x2, tp["mtp.norm_f"]) * cfg.logit_scale, head)
        loss = loss + cfg.mtp_weight * F.cross_entropy(z2.reshape(B * S, -1), lab2.reshape(-1), ignore_index=-1)
    return loss, z


@pytest.mark.parametrize("variant", VARIANTS[1:], ids=VARIANT_IDS[1:])
def test_model_variants_match_torch_autograd(variant):
    cfg = tiny_cfg(**variant)
    params = tiny_params(cfg, seed=21)
    assert ("lm_head" in params) == (not cfg.tie_embeddings)
    tok, lab = tiny_batch(cfg, B=2, S=7, seed=22)
    loss, grads, taps = D.forward_backward(cfg, params, tok, lab, mode="exact", keep_logits=True)
    tp = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in params.items()}
    tl, z = _torch_loss(cfg, tp, tok, lab)
    tl.backward()
    assert abs(loss - tl.item()) < 1e-12
    assert np.allclose(taps["logits"], z.detach().numpy(), rtol=0, atol=1e-11)
    for name in params:
        tg = tp[name].grad.numpy()
        assert np.linalg.norm(grads[name] - tg) / np.linalg.norm(tg) < 1e-11, name
    # all factors 1 and untied is the plain decoder bit for bit
    plain = tiny_cfg()
    pp = tiny_params(plain, seed=21)
    a = D.forward_backward(plain, pp, tok, lab, mode="contract")
    b = D.forward_backward(tiny_cfg(emb_scale=1.0, resid_scale=1.0, logit_scale=1.0, tie_embeddings=False), pp, tok, lab,
                           mode="contract")
    assert a[0] == b[0] and all(np.array_equal(a[1][k], b[1][k]) for k in a[1])


@pytest.mark.parametrize("nkv", [4, 2, 1])
def test_loss_and_gradients_match_torch_autograd(nkv):
    cfg = tiny_cfg(n_kv_heads=nkv)
    params = tiny_params(cfg, seed=11)
    tok, lab = tiny_batch(cfg, B=3, S=9, seed=12)
    lab[1, 4] = -1
    loss, grads, taps = D.forward_backward(cfg, params, tok, lab, mode="exact", keep_logits=True)
    tp = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in params.items()}
    tl, z = _torch_loss(cfg, tp, tok, lab)
    tl.backward()
    assert abs(loss - tl.item()) < 1e-12
    assert np.allclose(taps["logits"], z.detach().numpy(), rtol=0, atol=1e-12)
    for name in params:
        tg = tp[name].grad.numpy()
        err = np.linalg.norm(grads[name] - tg) / np.linalg.norm(tg)
        assert err < 1e-12, (name, err)


def test_train_steps_match_torch_adamw():
    """Three full steps (exact-mode gradients) against torch.optim.AdamW in fp64."""
    cfg = tiny_cfg()
    params = tiny_params(cfg, seed=21)
    st = D.TrainState(cfg, params)
    tp = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in params.items()}
    decay = [tp[k] for k in tp if tp[k].ndim == 2]
    nodecay = [tp[k] for k in tp if tp[k].ndim == 1]
    opt = torch.optim.AdamW([dict(params=decay, weight_decay=cfg.weight_decay), dict(params=nodecay, weight_decay=0.0)],
                            lr=cfg.lr, betas=(cfg.beta1, cfg.beta2), eps=cfg.adam_eps)
    for step in range(3):
        tok, lab = tiny_batch(cfg, seed=100 + step)
        # keep the oracle's masters in fp64-equal lockstep: its state is fp32, so feed torch the same values
        with torch.no_grad():
            for k in tp:
                tp[k].copy_(torch.from_numpy(st.params[k].astype(np.float64)))
        for grp in opt.param_groups:
            for q in grp["params"]:
                if q in opt.state and "exp_avg" in opt.state[q]:
                    name = [k for k in tp if tp[k] is q][0]
                    opt.state[q]["exp_avg"].copy_(torch.from_numpy(st.m[name].astype(np.float64)))
                    opt.state[q]["exp_avg_sq"].copy_(torch.from_numpy(st.v[name].astype(np.float64)))
        loss, gn, grads, _ = st.train_step(tok, lab, mode="exact")
        opt.zero_grad()
        tl, _ = _torch_loss(cfg, tp, tok, lab)
        tl.backward()
        tgn = math.sqrt(sum(float((q.grad ** 2).sum()) for q in tp.values()))
        opt.step()
        assert abs(loss - tl.item()) < 1e-12
        assert abs(gn - tgn) / tgn < 1e-12
        for k in tp:
            want = tp[k].detach().numpy()
            assert np.allclose(st.params[k], want.astype(np.float32), rtol=0, atol=1e-9), k
            err = np.linalg.norm(st.params[k].astype(np.float64) - want) / np.linalg.norm(want)
            assert err < 1e-7, (k, err)  # only the fp32 storage of the oracle's state separates them


# ---------------------------------------------------------------- AdamW and clipping: worked numbers
def test_adamw_hand_worked_trajectory():
    cfg = tiny_cfg()
    rows = [l.split() for l in open(os.path.join(GOLDEN, "adamw_hand_worked.txt")) if l.strip() and l[0] != "#"]
    p = np.array([0.02]); m = np.zeros(1); v = np.zeros(1)
    for case, step, g, wp, wm, wv in rows:
        if case != "traj":
            continue
        p, m, v = D.adamw_update(p, np.array([float(g)]), m, v, int(step), cfg, cfg.weight_decay)
        assert abs(p[0] - float(wp)) < 2e-10 and abs(m[0] - float(wm)) < 1e-12 and abs(v[0] - float(wv)) < 1e-12
    z = [r for r in rows if r[0] == "zero"][0]
    p, m, v = D.adamw_update(np.array([0.02]), np.zeros(1), np.zeros(1), np.zeros(1), 1, cfg, cfg.weight_decay)
    assert abs(p[0] - float(z[3])) < 1e-15 and m[0] == 0.0 and v[0] == 0.0


def test_gains_get_no_weight_decay_and_clip_scales_gradients():
    cfg = tiny_cfg(max_grad_norm=0.5)
    params = tiny_params(cfg)
    st = D.TrainState(cfg, params)
    grads = {k: np.zeros(v.shape) for k, v in params.items()}
    st.apply_gradients(grads)
    for k, v in params.items():
        if v.ndim == 1:
            assert np.array_equal(st.params[k], v)  # zero gradient, no decay: unchanged
        else:
            assert np.allclose(st.params[k], v * (1 - cfg.lr * cfg.weight_decay), rtol=1e-6)
    # clip coefficient = min(1, max_norm/(norm+eps)) as in the device-side listing
    assert D.clip_coeff(0.25, cfg) == 1.0
    assert abs(D.clip_coeff(2.0, cfg) - 0.5 / (2.0 + 1e-6)) < 1e-15
    assert D.clip_coeff(123.0, tiny_cfg()) == 1.0  # clipping off
    # a clipped update equals the unclipped update of the pre-scaled gradient
    g = np.array([0.3, -2.0]); p0 = np.array([0.1, 0.2])
    a = D.adamw_update(p0, g, np.zeros(2), np.zeros(2), 1, cfg, 0.1, clip=0.25)
    b = D.adamw_update(p0, 0.25 * g, np.zeros(2), np.zeros(2), 1, cfg, 0.1)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


# ---------------------------------------------------------------- attention invariants
def _rand_qkv(B=2, S=12, nh=4, nkv=2, d=8, seed=0):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((B, S, nh, d)), rng.standard_normal((B, S, nkv, d)),
            rng.standard_normal((B, S, nkv, d)))


def test_attention_matches_brute_force_rows_and_mask():
    q, k, v = _rand_qkv()
    o, lse = D.attention_fwd(q, k, v, 2, D._identity, False)
    B, S, nh, d = q.shape
    for b in range(B):
        for n in range(nh):
            for i in range(S):
                s = np.array([q[b, i, n] @ k[b, j, n // 2] / math.sqrt(d) for j in range(i + 1)])
                p = np.exp(s - s.max()); p /= p.sum()
                assert abs(p.sum() - 1) < 1e-12
                want = sum(p[j] * v[b, j, n // 2] for j in range(i + 1))
                assert np.allclose(o[b, i, n], want, atol=1e-13)
                assert abs(lse[b, n, i] - math.log(np.exp(s).sum())) < 1e-12


def test_attention_special_cases():
    q, k, v = _rand_qkv(S=1)
    o, _ = D.attention_fwd(q, k, v, 2, D._identity, False)
    assert np.allclose(o, np.repeat(v, 2, axis=2))  # one key: o = v
    q, k, v = _rand_qkv(S=10)
    o, lse = D.attention_fwd(np.zeros_like(q), k, v, 2, D._identity, False)  # equal scores: running mean of v
    want = np.cumsum(v, axis=1) / np.arange(1, 11)[None, :, None, None]
    assert np.allclose(o, np.repeat(want, 2, axis=2), atol=1e-13)
    assert np.allclose(lse, np.log(np.arange(1, 11))[None, None, :])


def test_integer_reference_does_not_change_unrounded_softmax_and_lse():
    q, k, v = _rand_qkv(S=33, seed=4)
    o0, l0 = D.attention_fwd(q * 3, k, v, 2, D._identity, False)
    o1, l1 = D.attention_fwd(q * 3, k, v, 2, D._identity, True)  # ceil'ed reference, no rounding
    assert np.allclose(o0, o1, atol=1e-13) and np.allclose(l0, l1, atol=1e-12)


def test_gqa_with_duplicated_kv_equals_mha():
    q, k, v = _rand_qkv(nh=4, nkv=2)
    o_g, _ = D.attention_fwd(q, k, v, 2, D._identity, False)
    o_m, _ = D.attention_fwd(q, np.repeat(k, 2, axis=2), np.repeat(v, 2, axis=2), 1, D._identity, False)
    assert np.array_equal(o_g, o_m)


def test_future_tokens_do_not_change_earlier_logits():
    cfg = tiny_cfg()
    params = tiny_params(cfg)
    tok, lab = tiny_batch(cfg)
    _, _, t0 = D.forward_backward(cfg, params, tok, lab, backward=False, keep_logits=True)
    tok2 = tok.copy(); tok2[:, 5:] = (tok2[:, 5:] + 7) % cfg.vocab
    _, _, t1 = D.forward_backward(cfg, params, tok2, lab, backward=False, keep_logits=True)
    assert np.array_equal(t0["logits"][:, :5], t1["logits"][:, :5])
    assert not np.array_equal(t0["logits"][:, 5:], t1["logits"][:, 5:])


# ---------------------------------------------------------------- RoPE, RMSNorm, SwiGLU, CE
def test_rope_properties():
    S, d = 16, 8
    c, s = D.rope_tables(S + 5, d, 1e4)
    assert np.array_equal(c[0], np.ones(d // 2)) and np.array_equal(s[0], np.zeros(d // 2))
    rng = np.random.default_rng(2)
    x = rng.standard_normal((1, S, 3, d)); y = rng.standard_normal((1, S, 3, d))
    rx = D.rope_apply(x, c[:S], s[:S])
    assert np.array_equal(rx[:, 0], x[:, 0])  # position 0: identity
    assert np.allclose(np.linalg.norm(rx, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-6)
    # q_m . k_n depends on m - n only: shift every position by 5
    ry = D.rope_apply(y, c[:S], s[:S])
    rx5 = D.rope_apply(x, c[5:S + 5], s[5:S + 5]); ry5 = D.rope_apply(y, c[5:S + 5], s[5:S + 5])
    g0 = np.einsum("bmnd,bknd->bnmk", rx, ry); g5 = np.einsum("bmnd,bknd->bnmk", rx5, ry5)
    assert np.allclose(g0, g5, atol=2e-6)  # tables are stored in fp32
    # the backward rotation is the transpose: <rope(x), y> = <x, rope^T(y)>
    assert abs(np.sum(rx * y) - np.sum(x * D.rope_apply_transpose(y, c[:S], s[:S]))) < 1e-10
    # angle of (p, i) is p * theta^(-2i/d)
    assert abs(c[3, 1] - np.float32(math.cos(3 * 1e4 ** (-2 / 8)))) < 1e-7
    # LongRoPE form: angle / lambda_i, magnitude factor on both tables: norms scale by it, the relative-position
    # property and the transpose survive, factors of 1 change nothing
    lam, ms = (1.0, 2.0, 3.5, 8.0), 1.25
    c2, s2 = D.rope_tables(S + 5, d, 1e4, lam, ms)
    assert abs(c2[3, 1] - np.float32(ms * math.cos(3 * 1e4 ** (-2 / 8) / 2.0))) < 1e-7
    assert abs(s2[7, 3] - np.float32(ms * math.sin(7 * 1e4 ** (-6 / 8) / 8.0))) < 1e-7
    r2 = D.rope_apply(x, c2[:S], s2[:S])
    assert np.allclose(np.linalg.norm(r2, axis=-1), ms * np.linalg.norm(x, axis=-1), rtol=1e-6)
    a0 = np.einsum("bmnd,bknd->bnmk", r2, D.rope_apply(y, c2[:S], s2[:S]))
    a5 = np.einsum("bmnd,bknd->bnmk", D.rope_apply(x, c2[5:S + 5], s2[5:S + 5]), D.rope_apply(y, c2[5:S + 5], s2[5:S + 5]))
    assert np.allclose(a0, a5, atol=4e-6)
    assert abs(np.sum(r2 * y) - np.sum(x * D.rope_apply_transpose(y, c2[:S], s2[:S]))) < 1e-10
    c1, s1 = D.rope_tables(S, d, 1e4, (1.0,) * (d // 2), 1.0)
    assert np.array_equal(c1, c[:S]) and np.array_equal(s1, s[:S])


def test_rmsnorm_properties():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 32))
    y, r = D.rmsnorm_fwd(x, np.ones(32), 0.0)
    assert np.allclose(np.sqrt(np.mean(y * y, -1)), 1.0)
    y2, _ = D.rmsnorm_fwd(7.5 * x, np.ones(32), 0.0)
    assert np.allclose(y, y2)
    g = rng.standard_normal(32)
    y3, _ = D.rmsnorm_fwd(x, g, 1e-5)
    assert np.allclose(y3, x / np.sqrt((x * x).mean(-1, keepdims=True) + 1e-5) * g)


def test_swiglu_derivative_points():
    assert D.sigmoid(np.array([0.0]))[0] == 0.5
    # silu(0) = 0, silu'(0) = 1/2: through the decoder's backward formula sg*(1+G*(1-sg)) at G=0
    G = np.array([0.0]); sg = D.sigmoid(G)
    assert (G * sg)[0] == 0.0 and (sg * (1 + G * (1 - sg)))[0] == 0.5


def test_cross_entropy_closed_forms():
    cfg = tiny_cfg()
    params = tiny_params(cfg)
    params["lm_head"] = np.zeros_like(params["lm_head"])  # uniform logits
    tok, lab = tiny_batch(cfg)
    loss, grads, taps = D.forward_backward(cfg, params, tok, lab, mode="exact")
    assert abs(loss - math.log(cfg.vocab)) < 1e-14
    # d loss / d lm_head rows sum to zero over the vocabulary (softmax - onehot sums to 0 per token)
    assert np.allclose(grads["lm_head"].sum(axis=0), 0.0, atol=1e-15)


def test_loss_at_initialisation_is_ln_vocab_plus_half_variance():
    w = SI.WORKLOADS["c1_tiny"]
    cfg = D.Config(**{k: w[k] for k in SI.MODEL_KEYS})
    params = D.init_params(cfg, SI.WEIGHT_SEED)
    tok, lab = SI.workload_batch("c1_tiny")
    loss, _, _ = D.forward_backward(cfg, params, tok, lab, backward=False, want_taps=False)
    # hF has RMS 1, so logits ~ N(0, 0.02^2 h): E[lse] ~= ln V + sigma^2/2 (6.983 for this shape)
    expect = math.log(cfg.vocab) + 0.5 * 0.02 ** 2 * cfg.d_model
    assert abs(loss - expect) < 0.03
    for name, arr in params.items():
        if arr.ndim == 2:
            assert abs(arr.std() - 0.02) < 3e-4 and abs(arr.mean()) < 2e-4
            z = arr.reshape(-1) / 0.02
            assert abs(np.mean(z ** 4) - 3.0) < 0.1  # normal kurtosis
        else:
            assert np.all(arr == 1.0)


def test_contract_mode_is_a_bf16_sized_perturbation_of_exact_mode():
    w = SI.WORKLOADS["c1_tiny"]
    cfg = D.Config(**{k: w[k] for k in SI.MODEL_KEYS})
    params = D.init_params(cfg, SI.WEIGHT_SEED)
    tok, lab = SI.workload_batch("c1_tiny")
    lc, gc, tc = D.forward_backward(cfg, params, tok, lab, mode="contract")
    le, ge, te = D.forward_backward(cfg, params, tok, lab, mode="exact")
    assert abs(lc - le) < 1e-3
    for k in ("layers.0.h1", "layers.0.q", "layers.0.o", "layers.0.x_out", "hF"):
        e = np.linalg.norm(tc[k] - te[k]) / np.linalg.norm(te[k])
        assert 3e-4 < e < 1e-2, (k, e)
    for k in gc:
        e = np.linalg.norm(gc[k] - ge[k]) / np.linalg.norm(ge[k])
        assert 1e-4 < e < 3e-2, (k, e)


# ---------------------------------------------------------------- inputs and the MFU numerator
def test_zipf_stream_matches_closed_form_frequencies():
    V = 32000
    ids = SI.token_stream(V, 64, 4096, "zipf", seed=1, step=0).reshape(-1)
    w = np.arange(1, V + 1, dtype=np.float64) ** -1.1
    p = w / w.sum()
    assert abs(p[0] - 0.14203) < 1e-4
    n = ids.size
    f0 = np.mean(ids == 0)
    assert abs(f0 - p[0]) < 4 * math.sqrt(p[0] * (1 - p[0]) / n)
    assert abs(np.mean(ids < 10) - p[:10].sum()) < 4 * math.sqrt(0.25 / n)
    assert ids.min() >= 0 and ids.max() < V
    u = SI.token_stream(1024, 8, 4096, "uniform", seed=1).reshape(-1)
    assert abs(u.mean() - 511.5) < 10 and u.min() >= 0 and u.max() < 1024
    t, l = SI.batch(1024, 2, 16, "uniform")
    assert np.array_equal(t[:, 1:], l[:, :-1])  # labels are the next token


def test_flop_formula_reproduces_the_papers_tables():
    from paper_2609_13645_b200.flops import flops_per_token
    for line in open(os.path.join(GOLDEN, "paper_flops_tables.txt")):
        if not line.strip() or line[0] == "#":
            continue
        left, right = line.split("|")
        name, L, h, f, nh, nkv, d, V, s = left.split()
        ffn, core, head, proj, total = map(float, right.split())
        fl = flops_per_token(int(L), int(h), int(nh), int(nkv), int(d), int(f), int(V), int(s))
        for key, want in (("ffn", ffn), ("core", core), ("head", head), ("proj", proj), ("total", total)):
            assert abs(fl[key] / 1e9 - want) < 6e-4, (name, key, fl[key] / 1e9, want)


def test_flop_formula_with_the_mtp_head_reproduces_the_papers_row():
    """The printed 1.452 GFLOP/token of the MTP row fixes what the head consists of: one more layer, a second output
    head and a [h, 2h] projection (a layer plus a head alone gives 1.423)."""
    from paper_2609_13645_b200.flops import flops_per_token
    for line in open(os.path.join(GOLDEN, "paper_flops_mtp.txt")):
        if not line.strip() or line[0] == "#":
            continue
        left, right = line.split("|")
        name, L, h, f, nh, nkv, d, V, s = left.split()
        ffn, core, head, proj, mtp, total = map(float, right.split())
        fl = flops_per_token(int(L), int(h), int(nh), int(nkv), int(d), int(f), int(V), int(s), mtp=True)
        for key, want in (("ffn", ffn), ("core", core), ("head", head), ("proj", proj), ("mtp", mtp), ("total", total)):
            assert abs(fl[key] / 1e9 - want) < 6e-4, (name, key, fl[key] / 1e9, want)
        layer_and_head = fl["mtp"] - 3 * 2 * (2 * int(h)) * int(h)
        assert abs(layer_and_head / 1e9 - mtp) > 0.02


def test_mtp_head_properties():
    """What the reading of the one-layer MTP head implies without any arithmetic of its own: weight 0 switches it off for
    the backbone; its loss ignores the first label of a sequence and the last position; it adds exactly weight * its own
    mean cross-entropy; at initialisation that cross-entropy is close to ln V like the backbone's."""
    cfg = tiny_cfg(mtp=True, mtp_weight=0.0)
    params = tiny_params(cfg)
    tok, lab = tiny_batch(cfg)
    plain = tiny_cfg()
    pp = {k: v for k, v in params.items() if not k.startswith("mtp.")}
    l0, g0, _ = D.forward_backward(plain, pp, tok, lab, mode="exact")
    l1, g1, t1 = D.forward_backward(cfg, params, tok, lab, mode="exact")
    assert l0 == l1
    for k in g0:
        assert np.array_equal(g0[k], g1[k]), k
    assert all(not np.any(g1[k]) for k in g1 if k.startswith("mtp."))
    # weight w adds w * (the head's own loss), which does not see labels[:, 0] nor anything at the last position
    cfg_w = tiny_cfg(mtp=True, mtp_weight=0.7)
    lw, _, tw = D.forward_backward(cfg_w, params, tok, lab, mode="exact", backward=False)
    assert abs(lw - (l0 + 0.7 * tw["mtp.loss"])) < 1e-12
    lab2 = lab.copy(); lab2[:, 0] = (lab2[:, 0] + 1) % cfg.vocab
    _, _, ta = D.forward_backward(cfg_w, params, tok, lab2, mode="exact", backward=False)
    assert ta["mtp.loss"] == tw["mtp.loss"]
    tok2 = tok.copy(); tok2[:, -1] = (tok2[:, -1] + 1) % cfg.vocab  # the last token only feeds the uncounted last position...
    _, _, tb = D.forward_backward(cfg_w, params, tok2, lab, mode="exact", backward=False)
    # ... as itself and as position S-2's "next token": so the head's loss may move, but only through rows that are causal
    # successors of S-2; the backbone rows before the last are untouched
    assert np.array_equal(tb["ce_lse"][:, :-1], tw["ce_lse"][:, :-1])
    # at the real initialisation scale the head starts at ln V
    c = D.Config(n_layers=1, d_model=64, n_heads=2, n_kv_heads=1, head_dim=32, d_ffn=96, vocab=512, mtp=True)
    p = D.init_params(c, 3)
    t, l = tiny_batch(c, B=2, S=16)
    _, _, tt = D.forward_backward(c, p, t, l, mode="contract", backward=False)
    assert abs(tt["mtp.loss"] - np.log(512)) < 0.05
