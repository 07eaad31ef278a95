"""Helpers shared by the GPU parity tests: run the same seeded step through the oracle and the library."""
import numpy as np

import synth_inputs as SI
from oracle import decoder as D


def f32(x):
    return float(np.float32(x))


def oracle_config(**kw):
    """Oracle config whose hyper-parameters carry the fp32 values the C struct holds."""
    c = D.Config(**kw)
    for k in ("rms_eps", "rope_theta", "lr", "beta1", "beta2", "adam_eps", "weight_decay", "max_grad_norm", "emb_scale",
              "resid_scale", "logit_scale", "mtp_weight"):
        setattr(c, k, f32(getattr(c, k)))
    return c


def lib_config(B, ocfg, max_batch, max_seq, **extra):
    return B.make_config(ocfg.n_layers, ocfg.d_model, ocfg.n_heads, ocfg.n_kv_heads, ocfg.head_dim, ocfg.d_ffn,
                         ocfg.vocab, max_batch, max_seq, rms_eps=ocfg.rms_eps, rope_theta=ocfg.rope_theta, lr=ocfg.lr,
                         beta1=ocfg.beta1, beta2=ocfg.beta2, adam_eps=ocfg.adam_eps, weight_decay=ocfg.weight_decay,
                         max_grad_norm=ocfg.max_grad_norm, emb_scale=ocfg.emb_scale, resid_scale=ocfg.resid_scale,
                         logit_scale=ocfg.logit_scale, tie_embeddings=int(ocfg.tie_embeddings), qk_norm=int(ocfg.qk_norm),
                         mtp=int(ocfg.mtp), mtp_weight=ocfg.mtp_weight, **extra)


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64).reshape(-1)
    b = np.asarray(b, dtype=np.float64).reshape(-1)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def load_params(model, params):
    for name, arr in params.items():
        model.set_param(name, arr)


def to_dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


# oracle tap name -> (library tap name, slicer on the library's flat array)
def lib_tap(model, ocfg, name, layer, T):
    hq, hkv, f = ocfg.h_q, ocfg.h_kv, ocfg.d_ffn
    n = hq + 2 * hkv
    if name in ("q", "k", "v"):
        a = model.get_tap("qkv", layer).reshape(T, n)
        return {"q": a[:, :hq], "k": a[:, hq:hq + hkv], "v": a[:, hq + hkv:]}[name]
    if name in ("G", "U"):
        a = model.get_tap("gu", layer).reshape(T, 2 * f)
        return a[:, :f] if name == "G" else a[:, f:]
    if name in ("d_q", "d_k", "d_v"):
        a = model.get_tap("d_qkv", layer).reshape(T, n)
        return {"d_q": a[:, :hq], "d_k": a[:, hq:hq + hkv], "d_v": a[:, hq + hkv:]}[name]
    if name in ("d_G", "d_U"):
        a = model.get_tap("d_gu", layer).reshape(T, 2 * f)
        return a[:, :f] if name == "d_G" else a[:, f:]
    return model.get_tap(name, layer)


FWD_TAPS = ("x_in", "h1", "q", "k", "v", "attn_lse", "o", "x_mid", "h2", "G", "U", "a", "x_out")
BWD_TAPS = ("d_x_out", "d_a", "d_G", "d_U", "d_h2", "d_x_mid", "d_o", "d_q", "d_k", "d_v", "d_h1", "d_x_in")
