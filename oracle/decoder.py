"""Plain CPU oracle of one training step of a Llama-style dense decoder.

TEST INFRASTRUCTURE: slow, obviously-correct numpy in fp64.  It is the
definition the CUDA library is compared against and shares no code with it.

What it follows in the paper
  * architecture: decoder-only, grouped-query attention, SwiGLU feed-forward,
    pre-normalisation RMSNorm, RoPE, untied output head (Appendix
    "Model Architectures", architecture tables);
  * which contractions exist (Q/K/V/O projections, gate/up/down, causal
    attention core, output head): Appendix "Model-FLOPs Utilization";
  * the optimizer: the fused clip + Adam + bf16 write-back listing and the
    device-side clip-coefficient listing in the appendix on framework-level
    optimisation ("Deep customization"), restated here from their arithmetic;
  * precision: bf16 compute copies written back from fp32 masters, weight
    gradients kept in fp32 (Section "Operator-Level Forging", kernel table caption).

The decoder arithmetic itself is the textbook definition; the paper does not
restate it.  Two modes share one code path:
  * mode="contract": R(.) = round-to-nearest-even to bfloat16 is applied to the
    tensors a bf16 training step stores (listed where they are produced);
  * mode="exact":    R(.) = identity (used for finite differences).

Pins (see tests): finite differences, PyTorch fp64 autograd + torch.optim.AdamW
on a tiny model, attention/RoPE/RMSNorm/CE invariants, a hand-computed AdamW
trajectory, loss at initialisation.  What nothing external pins is *where* the
bf16 roundings of contract mode sit: that placement is a recorded choice
("parity unpinned" for the placement only; the value each rounding produces is
pinned by the bfloat16 format itself).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import numpy as np

LOG2E = 1.4426950408889634
LN2 = 0.6931471805599453


@dataclasses.dataclass
class Config:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 1e4
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.95
    adam_eps: float = 1e-8
    weight_decay: float = 0.1
    max_grad_norm: float = 0.0  # <= 0: clipping off
    clip_eps: float = 1e-6
    # Variants of the paper's model families (appendix "Model Architectures", rows "Tied input/output embeddings" and
    # "muP (scale_emb, dim_model_base, scale_depth)").  The paper gives the three muP numbers, not where they act;
    # the reading taken here is the published MiniCPM convention, reduced to three plain factors:
    #   emb_scale   (scale_emb)                     x_0 = R(emb_scale * E[token])
    #   resid_scale (scale_depth / sqrt(n_layers))  x <- R(x + resid_scale * branch) for both branches of a layer
    #   logit_scale (dim_model_base / d_model)      z = logit_scale * (h_F W^T)
    # All 1 (and untied) reproduces the plain decoder exactly.
    emb_scale: float = 1.0
    resid_scale: float = 1.0
    logit_scale: float = 1.0
    tie_embeddings: bool = False  # the output head reads the embedding table; its gradient is the sum of both uses
    # Per-head QK-Norm (appendix "Model Architectures", Qwen3 column: "RoPE (theta = 1e6, QK-Norm)"): the d entries of
    # every query and key head are RMS-normalised with a learned gain of d entries (one for all query heads, one for all
    # key heads of a layer; eps = rms_eps) before the rotation.  The paper names it without a formula; this is the
    # published Qwen3 definition.
    qk_norm: bool = False
    # LongRoPE (appendix "Model Architectures", MiniCPM4 rows: "Position encoding: LongRoPE"): the paper names it
    # without its constants; reading = the published method's form, a per-frequency rescale factor lambda_i and one
    # magnitude factor: angle(p, i) = p * theta^(-2i/d) / lambda_i, and cos, sin are multiplied by rope_mscale.
    # None / 1 is plain RoPE.  (Which lambda_i a checkpoint uses is model data, passed in like the weights.)
    rope_factors: Optional[Tuple[float, ...]] = None
    rope_mscale: float = 1.0
    # One-layer multi-token-prediction (Eagle) head (appendix "Model Architectures", row "MTP / Eagle head: On (1 layer)";
    # appendix "Ascend Model-FLOPs Utilization": its FLOP count is one more backbone layer, attention core, projections
    # and feed-forward, plus one more output head).  The paper fixes that much and no more; reading = the published
    # depth-1 MTP module:
    #   h'_i = R(R(hn_i Wh^T) + en_i We^T),  hn = R(rmsnorm(x_L; g_h)),  en = R(rmsnorm(R(emb_scale E[tok_{i+1}]); g_e)),
    #   x' = one more decoder layer on h' (parameters "mtp.layer.*"), z' = logit_scale * R(rmsnorm(x'; g_f)) W_head^T
    #   with the backbone's output head, trained on the token after next: label'_i = label_{i+1}; the last position of a
    #   sequence has no successor and does not count.  loss = loss_backbone + mtp_weight * mean CE(z', label').
    mtp: bool = False
    mtp_weight: float = 1.0

    @property
    def h_q(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def h_kv(self) -> int:
        return self.n_kv_heads * self.head_dim


# --------------------------------------------------------------------------
# bfloat16 rounding (the "R" of contract mode)
# --------------------------------------------------------------------------
def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round fp64 values to the nearest bfloat16 (ties to even), returned as fp64.

    bfloat16 has 8 significant bits and fp32's exponent range.  For
    x = m * 2**e with 0.5 <= |m| < 1 the spacing of representable values is
    2**(e-8); below the smallest normal (2**-126) the spacing stays 2**-133.
    """
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)
    e = np.maximum(e, -125)
    q = np.ldexp(1.0, e - 8)
    with np.errstate(invalid="ignore", over="ignore"):
        y = np.rint(x / q) * q
    big = np.abs(y) > 3.3895313892515355e38  # largest finite bfloat16
    if np.any(big):
        y = np.where(big, np.sign(y) * np.inf, y)
    return y


def _identity(x):
    return np.asarray(x, dtype=np.float64)


def _rounder(mode: str):
    if mode == "contract":
        return bf16_round
    if mode == "exact":
        return _identity
    raise ValueError("mode must be 'contract' or 'exact'")


# --------------------------------------------------------------------------
# parameters
# --------------------------------------------------------------------------
def param_specs(cfg: Config) -> List[Tuple[str, Tuple[int, ...]]]:
    """Names and logical [out, in] shapes, in the library's parameter order."""
    specs: List[Tuple[str, Tuple[int, ...]]] = [("embed", (cfg.vocab, cfg.d_model))]
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        specs += [
            (p + "norm1", (cfg.d_model,)),
            (p + "wqkv", (cfg.h_q + 2 * cfg.h_kv, cfg.d_model)),  # rows: q heads, k heads, v heads
            (p + "wo", (cfg.d_model, cfg.h_q)),
            (p + "norm2", (cfg.d_model,)),
            (p + "wgu", (2 * cfg.d_ffn, cfg.d_model)),  # rows: gate 0..f-1, then up 0..f-1
            (p + "wd", (cfg.d_model, cfg.d_ffn)),
        ]
        if cfg.qk_norm:
            specs += [(p + "q_norm", (cfg.head_dim,)), (p + "k_norm", (cfg.head_dim,))]
    specs += [("norm_f", (cfg.d_model,))]
    if not cfg.tie_embeddings:
        specs += [("lm_head", (cfg.vocab, cfg.d_model))]
    if cfg.mtp:
        p = "mtp.layer."
        specs += [
            ("mtp.norm_h", (cfg.d_model,)),
            ("mtp.norm_e", (cfg.d_model,)),
            ("mtp.proj_h", (cfg.d_model, cfg.d_model)),
            ("mtp.proj_e", (cfg.d_model, cfg.d_model)),
            (p + "norm1", (cfg.d_model,)),
            (p + "wqkv", (cfg.h_q + 2 * cfg.h_kv, cfg.d_model)),
            (p + "wo", (cfg.d_model, cfg.h_q)),
            (p + "norm2", (cfg.d_model,)),
            (p + "wgu", (2 * cfg.d_ffn, cfg.d_model)),
            (p + "wd", (cfg.d_model, cfg.d_ffn)),
        ]
        if cfg.qk_norm:
            specs += [(p + "q_norm", (cfg.head_dim,)), (p + "k_norm", (cfg.head_dim,))]
        specs += [("mtp.norm_f", (cfg.d_model,))]
    return specs


_M64 = (1 << 64) - 1


def _splitmix64(z: np.ndarray) -> np.ndarray:
    """The splitmix64 finaliser on uint64 arrays (wrap-around arithmetic)."""
    z = (z + np.uint64(0x9E3779B97F4A7C15)).astype(np.uint64)
    z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def init_normal(seed: int, tensor_id: int, n: int, std: float = 0.02) -> np.ndarray:
    """Counter-based N(0, std^2) draws, one per element index, as fp32.

    key = splitmix64(seed ^ (tensor_id+1)*C1 ^ elem*C2); its top and next 24
    bits give two uniforms u1 in (0,1], u2 in [0,1); Box-Muller in fp64:
    sqrt(-2 ln u1) * cos(2 pi u2) * std, stored as fp32.
    """
    with np.errstate(over="ignore"):
        elem = np.arange(n, dtype=np.uint64)
        k = np.uint64(seed & _M64) ^ (np.uint64(tensor_id + 1) * np.uint64(0xD1B54A32D192ED03)) ^ (
            elem * np.uint64(0x8CB92BA72F3D8DD7)
        )
        r = _splitmix64(k)
    a = (r >> np.uint64(40)).astype(np.float64)  # top 24 bits
    b = ((r >> np.uint64(16)) & np.uint64(0xFFFFFF)).astype(np.float64)  # next 24 bits
    u1 = (a + 1.0) / 16777216.0
    u2 = b / 16777216.0
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return (z * std).astype(np.float32)


def init_params(cfg: Config, seed: int) -> Dict[str, np.ndarray]:
    """fp32 masters: every matrix ~ N(0, 0.02^2), every RMSNorm gain = 1."""
    out: Dict[str, np.ndarray] = {}
    for tid, (name, shape) in enumerate(param_specs(cfg)):
        if len(shape) == 1:
            out[name] = np.ones(shape, dtype=np.float32)
        else:
            out[name] = init_normal(seed, tid, shape[0] * shape[1]).reshape(shape)
    return out


# --------------------------------------------------------------------------
# building blocks (each in fp64, inputs already carry any contract rounding)
# --------------------------------------------------------------------------
def rope_tables(S: int, d: int, theta: float, factors=None, mscale: float = 1.0) -> Tuple[np.ndarray, np.ndarray]:
    """mscale * cos/sin of p * theta**(-2i/d) / factors_i, p = 0..S-1, i = 0..d/2-1: fp64 values stored as fp32."""
    i = np.arange(d // 2, dtype=np.float64)
    inv_freq = np.power(float(theta), -2.0 * i / d)
    if factors is not None:
        inv_freq = inv_freq / np.asarray(factors, dtype=np.float64)
    ang = np.arange(S, dtype=np.float64)[:, None] * inv_freq[None, :]
    c = (float(mscale) * np.cos(ang)).astype(np.float32).astype(np.float64)
    s = (float(mscale) * np.sin(ang)).astype(np.float32).astype(np.float64)
    return c, s


def rope_apply(x: np.ndarray, c: np.ndarray, s: np.ndarray) -> np.ndarray:
    """Half-split pairing on x[..., S, n, d]: (x_i, x_{i+d/2}) rotated by the angle of (p, i)."""
    d = x.shape[-1]
    x1, x2 = x[..., : d // 2], x[..., d // 2 :]
    cc, ss = c[:, None, :], s[:, None, :]
    return np.concatenate([x1 * cc - x2 * ss, x2 * cc + x1 * ss], axis=-1)


def rope_apply_transpose(dy: np.ndarray, c: np.ndarray, s: np.ndarray) -> np.ndarray:
    """Gradient of rope_apply with respect to x (rotation by the negative angle)."""
    d = dy.shape[-1]
    y1, y2 = dy[..., : d // 2], dy[..., d // 2 :]
    cc, ss = c[:, None, :], s[:, None, :]
    return np.concatenate([y1 * cc + y2 * ss, y2 * cc - y1 * ss], axis=-1)


def rmsnorm_fwd(x: np.ndarray, g: np.ndarray, eps: float) -> Tuple[np.ndarray, np.ndarray]:
    """y = x * r * g with r = (mean_k x_k^2 + eps)^(-1/2); returns (y, r)."""
    r = 1.0 / np.sqrt(np.mean(x * x, axis=-1) + eps)
    return x * r[..., None] * g, r


def rmsnorm_bwd(dy: np.ndarray, x: np.ndarray, r: np.ndarray, g: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """dx_k = r g_k dy_k - x_k r^3 (1/h) sum_j g_j dy_j x_j ;  dg_k = sum_t dy_tk x_tk r_t."""
    h = x.shape[-1]
    gdy = dy * g
    dot = np.sum(gdy * x, axis=-1)
    dx = gdy * r[..., None] - x * (r ** 3 * dot / h)[..., None]
    dg = np.sum((dy * x * r[..., None]).reshape(-1, h), axis=0)
    return dx, dg


def sigmoid(x: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-x))


def swiglu_fwd(G: np.ndarray, U: np.ndarray) -> np.ndarray:
    """a = silu(G) U = G sigmoid(G) U (the SwiGLU feed-forward's gate, appendix "Model Architectures")."""
    return G * sigmoid(G) * U


def swiglu_bwd(d_a: np.ndarray, G: np.ndarray, U: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """(dG, dU) of a = G s U with s = sigmoid(G): dU = d_a G s, dG = d_a U s (1 + G (1 - s)).  Unrounded."""
    sg = sigmoid(G)
    return d_a * U * sg * (1.0 + G * (1.0 - sg)), d_a * G * sg


def attention_fwd(q, k, v, n_rep: int, R, contract: bool):
    """Causal softmax(q k^T / sqrt(d)) v per batch and head.

    q [B,S,n_h,d]; k,v [B,S,n_kv,d]; query head n reads kv head n // n_rep.
    Row i, valid keys j <= i:  S_ij = q_i.k_j / sqrt(d);
    P~_ij = 2^(S_ij log2e - c_i) with reference c_i = ceil(max_j S_ij log2e) in
    contract mode (any constant reference gives the same softmax; an integer one
    makes the bf16 rounding of P~ independent of the order keys are visited in);
    l_i = sum_j P~_ij (unrounded); o_i = R( (sum_j R(P~_ij) v_j) / l_i );
    LSE_i = (c_i + log2 l_i) ln 2 = log sum_j exp(S_ij).
    """
    B, S, n_h, d = q.shape
    scale = 1.0 / math.sqrt(d)
    o = np.empty_like(q)
    lse = np.empty((B, n_h, S), dtype=np.float64)
    rows_per = 2048  # rows are independent; blocks of rows only bound the memory of the score matrix
    for b in range(B):
        for n in range(n_h):
            kk = k[b, :, n // n_rep, :]
            vv = v[b, :, n // n_rep, :]
            for i0 in range(0, S, rows_per):
                i1 = min(S, i0 + rows_per)
                sc = (q[b, i0:i1, n, :] @ kk[:i1].T) * scale  # keys beyond i1-1 are masked for all rows
                rows = np.arange(i0, i1)[:, None]
                cols = np.arange(i1)[None, :]
                valid = cols <= rows
                s2 = np.where(valid, sc * LOG2E, -np.inf)
                c = np.max(s2, axis=1)
                if contract:
                    c = np.ceil(c)
                pt = np.exp2(s2 - c[:, None])  # masked entries -> exactly 0
                l = np.sum(pt, axis=1)
                o[b, i0:i1, n, :] = R((R(pt) @ vv[:i1]) / l[:, None])
                lse[b, n, i0:i1] = (c + np.log2(l)) * LN2
    return o, lse


def attention_bwd(q, k, v, o, do, lse, n_rep: int, R):
    """Gradients of the causal attention core.

    D_i = sum_k do_ik o_ik;  P_ij = exp(S_ij - LSE_i);  dV_j = sum_i R(P_ij) do_i;
    dP_ij = do_i . v_j;  dS_ij = R(P_ij (dP_ij - D_i));
    dQ_i = (1/sqrt d) sum_j dS_ij k_j;  dK_j = (1/sqrt d) sum_i dS_ij q_i;
    dK, dV are summed over the query heads that share a kv head.  Returned
    unrounded (the caller rotates dq, dk back and rounds).
    """
    B, S, n_h, d = q.shape
    scale = 1.0 / math.sqrt(d)
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    rows_per = 2048
    for b in range(B):
        for n in range(n_h):
            g = n // n_rep
            kk = k[b, :, g, :]
            vv = v[b, :, g, :]
            for i0 in range(0, S, rows_per):
                i1 = min(S, i0 + rows_per)
                qi = q[b, i0:i1, n, :]
                doi = do[b, i0:i1, n, :]
                sc = (qi @ kk[:i1].T) * scale
                rows = np.arange(i0, i1)[:, None]
                cols = np.arange(i1)[None, :]
                valid = cols <= rows
                p = np.where(valid, np.exp(sc - lse[b, n, i0:i1, None]), 0.0)
                D = np.sum(doi * o[b, i0:i1, n, :], axis=1)
                dp = doi @ vv[:i1].T
                ds = R(p * (dp - D[:, None]))
                dv[b, :i1, g, :] += R(p).T @ doi
                dq[b, i0:i1, n, :] = (ds @ kk[:i1]) * scale
                dk[b, :i1, g, :] += (ds.T @ qi) * scale
    return dq, dk, dv


# --------------------------------------------------------------------------
# forward + backward of the whole decoder
# --------------------------------------------------------------------------
def forward_backward(cfg: Config, params: Dict[str, np.ndarray], tokens: np.ndarray, labels: np.ndarray,
                     mode: str = "contract", want_taps: bool = True, backward: bool = True,
                     keep_logits: bool = False):
    """Loss, gradients (fp64, never rounded) and named intermediate tensors.

    tokens, labels: int [B, S]; labels < 0 do not count in the loss.
    Returns (loss, grads, taps).  Taps are keyed "name" or "layers.{l}.name".
    """
    R = _rounder(mode)
    contract = mode == "contract"
    B, S = tokens.shape
    T = B * S
    h, nh, nkv, d, f, V = cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn, cfg.vocab
    hq, hkv = cfg.h_q, cfg.h_kv
    n_rep = nh // nkv
    taps: Dict[str, np.ndarray] = {}

    def tap(name, val):
        if want_taps:
            taps[name] = val

    # 1. compute copies: W^b = R(W) for every parameter (matrices and gains)
    W = {k_: R(np.asarray(v_, dtype=np.float64)) for k_, v_ in params.items()}
    cos, sin = rope_tables(S, d, cfg.rope_theta, cfg.rope_factors, cfg.rope_mscale)

    # 2. embedding: row copy (exact when emb_scale is 1: R of a bf16 value is itself)
    s_e, s_r, s_l = float(cfg.emb_scale), float(cfg.resid_scale), float(cfg.logit_scale)
    head = "embed" if cfg.tie_embeddings else "lm_head"
    x = R(s_e * W["embed"][tokens])  # [B,S,h]
    def layer_fwd(x_in, p):
        """One decoder layer with the parameters named p + "...": returns (x_out, what its backward needs)."""
        y, r1 = rmsnorm_fwd(x_in, W[p + "norm1"], cfg.rms_eps)
        h1 = R(y)
        qkv = h1 @ W[p + "wqkv"].T  # unrounded accumulators
        q = qkv[..., :hq].reshape(B, S, nh, d)
        k = qkv[..., hq:hq + hkv].reshape(B, S, nkv, d)
        v = qkv[..., hq + hkv:].reshape(B, S, nkv, d)
        if cfg.qk_norm:  # per-head RMSNorm of the unrounded accumulators, then the rotation, then one rounding
            q, rq = rmsnorm_fwd(q, W[p + "q_norm"], cfg.rms_eps)  # rq [B,S,n_h]; q is now the normalised, gained value
            k, rk = rmsnorm_fwd(k, W[p + "k_norm"], cfg.rms_eps)
            q_hat, k_hat = q / W[p + "q_norm"], k / W[p + "k_norm"]  # unit-RMS values (pre-gain) for the backward pass
        q = R(rope_apply(q, cos, sin))  # RoPE on the unrounded q, k; one rounding after it
        k = R(rope_apply(k, cos, sin))
        v = R(v)
        o, lse = attention_fwd(q, k, v, n_rep, R, contract)
        o2 = o.reshape(B, S, hq)
        x_mid = R(x_in + s_r * (o2 @ W[p + "wo"].T))
        y, r2 = rmsnorm_fwd(x_mid, W[p + "norm2"], cfg.rms_eps)
        h2 = R(y)
        gu = h2 @ W[p + "wgu"].T
        G = R(gu[..., :f])
        U = R(gu[..., f:])
        a = R(swiglu_fwd(G, U))
        x_out = R(x_mid + s_r * (a @ W[p + "wd"].T))
        sv = dict(x_in=x_in, r1=r1, h1=h1, q=q, k=k, v=v, o=o, lse=lse, x_mid=x_mid, r2=r2, h2=h2, G=G, U=U, a=a)
        if cfg.qk_norm:
            sv.update(q_hat=q_hat, k_hat=k_hat, rq=rq, rk=rk)
        for nm, val in (("x_in", x_in), ("h1", h1), ("q", q), ("k", k), ("v", v), ("attn_lse", lse), ("o", o2),
                        ("x_mid", x_mid), ("h2", h2), ("G", G), ("U", U), ("a", a), ("x_out", x_out)):
            tap(p + nm, val)
        return x_out, sv

    saved = []
    for l in range(cfg.n_layers):
        x, sv = layer_fwd(x, f"layers.{l}.")
        saved.append(sv)

    def head_fwd(hF_, labels_):
        """Logits (unrounded), per-row log-sum-exp and the mean loss over the counted labels."""
        z_ = s_l * (hF_ @ W[head].T)
        zmax = np.max(z_, axis=-1, keepdims=True)
        lse_ = (zmax + np.log(np.sum(np.exp(z_ - zmax), axis=-1, keepdims=True)))[..., 0]
        counted_ = labels_ >= 0
        n_ = int(np.sum(counted_))
        safe_ = np.where(counted_, labels_, 0)
        z_y = np.take_along_axis(z_, safe_[..., None], axis=-1)[..., 0]
        loss_ = float(np.sum(np.where(counted_, lse_ - z_y, 0.0)) / max(n_, 1))
        return z_, lse_, loss_, (counted_, n_, safe_)

    def head_bwd(z_, lse_, hF_, meta, weight):
        """B1: dz = R(weight * logit_scale (softmax(z) - onehot(y)) / n_counted), zero rows for ignored labels: the
        gradient with respect to the unscaled product h_F W^T, rounded once.  Returns (d_hF, head gradient)."""
        counted_, n_, safe_ = meta
        pz = np.exp(z_ - lse_[..., None])
        onehot = np.zeros_like(pz)
        np.put_along_axis(onehot, safe_[..., None], 1.0, axis=-1)
        dz = R(np.where(counted_[..., None], weight * s_l * (pz - onehot) / max(n_, 1), 0.0))
        return R(dz @ W[head]), dz.reshape(T, V).T @ hF_.reshape(T, h)

    x_L = x
    y, rF = rmsnorm_fwd(x_L, W["norm_f"], cfg.rms_eps)
    hF = R(y)
    z, ce_lse, loss, meta = head_fwd(hF, labels)
    tap("hF", hF)
    tap("ce_lse", ce_lse)
    if keep_logits:
        taps["logits"] = z
    if cfg.mtp:
        # the token after next: ids shifted by one inside every sequence, the last position does not count
        tok2 = np.concatenate([tokens[:, 1:], tokens[:, -1:]], axis=1)
        lab2 = np.concatenate([labels[:, 1:], np.full((B, 1), -1, dtype=labels.dtype)], axis=1)
        y, r_h = rmsnorm_fwd(x_L, W["mtp.norm_h"], cfg.rms_eps)
        hn = R(y)
        xe = R(s_e * W["embed"][tok2])
        y, r_e = rmsnorm_fwd(xe, W["mtp.norm_e"], cfg.rms_eps)
        en = R(y)
        u1 = R(hn @ W["mtp.proj_h"].T)
        hp = R(u1 + en @ W["mtp.proj_e"].T)
        x2, sv2 = layer_fwd(hp, "mtp.layer.")
        y, rF2 = rmsnorm_fwd(x2, W["mtp.norm_f"], cfg.rms_eps)
        hF2 = R(y)
        z2, lse2, loss2, meta2 = head_fwd(hF2, lab2)
        tap("mtp.hn", hn); tap("mtp.en", en); tap("mtp.h_in", hp); tap("mtp.hF", hF2); tap("mtp.ce_lse", lse2)
        taps["mtp.loss"] = loss2
        loss = loss + float(cfg.mtp_weight) * loss2
    if not backward:
        return loss, {}, taps

    grads: Dict[str, np.ndarray] = {}

    def layer_bwd(dx, sv, p):
        """Backward of layer_fwd: gradient of the layer's input; parameter gradients go to grads[p + ...]."""
        tap(p + "d_x_out", dx)
        # the branch output entered the residual stream times resid_scale: its gradient is resid_scale * dx (not rounded)
        d_a = R((s_r * dx) @ W[p + "wd"])
        grads[p + "wd"] = (s_r * dx).reshape(T, h).T @ sv["a"].reshape(T, f)
        G, U = sv["G"], sv["U"]
        dG, dU = swiglu_bwd(d_a, G, U)
        dG, dU = R(dG), R(dU)
        dGU = np.concatenate([dG, dU], axis=-1)
        d_h2 = R(dGU @ W[p + "wgu"])
        grads[p + "wgu"] = dGU.reshape(T, 2 * f).T @ sv["h2"].reshape(T, h)
        dxn, grads[p + "norm2"] = rmsnorm_bwd(d_h2, sv["x_mid"], sv["r2"], W[p + "norm2"])
        d_x_mid = R(dx + dxn)
        d_o = R((s_r * d_x_mid) @ W[p + "wo"])
        grads[p + "wo"] = (s_r * d_x_mid).reshape(T, h).T @ sv["o"].reshape(T, hq)
        dq, dk, dv = attention_bwd(sv["q"], sv["k"], sv["v"], sv["o"], d_o.reshape(B, S, nh, d), sv["lse"],
                                   n_rep, R)
        dq = R(rope_apply_transpose(dq, cos, sin))
        dk = R(rope_apply_transpose(dk, cos, sin))
        dv = R(dv)
        if cfg.qk_norm:
            # backward of y = x_hat * g with x_hat = x r: dx = r (g dy - x_hat mean_k(g dy x_hat)), dg = sum dy x_hat;
            # dy is the rounded gradient above, dx is rounded once more (it is what the projection's backward reads)
            def head_norm_bwd(dy, x_hat, r, g):
                gdy = dy * g
                dxh = r[..., None] * (gdy - x_hat * np.mean(gdy * x_hat, axis=-1, keepdims=True))
                return dxh, np.sum((dy * x_hat).reshape(-1, d), axis=0)
            dq, grads[p + "q_norm"] = head_norm_bwd(dq, sv["q_hat"], sv["rq"], W[p + "q_norm"])
            dk, grads[p + "k_norm"] = head_norm_bwd(dk, sv["k_hat"], sv["rk"], W[p + "k_norm"])
            dq, dk = R(dq), R(dk)
        dqkv = np.concatenate([dq.reshape(B, S, hq), dk.reshape(B, S, hkv), dv.reshape(B, S, hkv)], axis=-1)
        d_h1 = R(dqkv @ W[p + "wqkv"])
        grads[p + "wqkv"] = dqkv.reshape(T, hq + 2 * hkv).T @ sv["h1"].reshape(T, h)
        dxn, grads[p + "norm1"] = rmsnorm_bwd(d_h1, sv["x_in"], sv["r1"], W[p + "norm1"])
        d_x_in = R(d_x_mid + dxn)
        for nm, val in (("d_a", d_a), ("d_G", dG), ("d_U", dU), ("d_h2", d_h2), ("d_x_mid", d_x_mid),
                        ("d_o", d_o), ("d_q", dq.reshape(B, S, hq)), ("d_k", dk.reshape(B, S, hkv)),
                        ("d_v", dv.reshape(B, S, hkv)), ("d_h1", d_h1), ("d_x_in", d_x_in)):
            tap(p + nm, val)
        return d_x_in

    d_hF, g_head = head_bwd(z, ce_lse, hF, meta, 1.0)
    tap("d_hF", d_hF)
    dE = np.zeros((V, h), dtype=np.float64)
    d_xL_mtp = 0.0
    if cfg.mtp:
        d_hF2, g_head2 = head_bwd(z2, lse2, hF2, meta2, float(cfg.mtp_weight))
        g_head = g_head + g_head2
        dxn, grads["mtp.norm_f"] = rmsnorm_bwd(d_hF2, x2, rF2, W["mtp.norm_f"])
        d_hp = layer_bwd(R(dxn), sv2, "mtp.layer.")
        # h' = R(u1 + en We^T), u1 = R(hn Wh^T): the add passes the gradient to both terms unchanged
        d_en = R(d_hp @ W["mtp.proj_e"])
        grads["mtp.proj_e"] = d_hp.reshape(T, h).T @ en.reshape(T, h)
        d_hn = R(d_hp @ W["mtp.proj_h"])
        grads["mtp.proj_h"] = d_hp.reshape(T, h).T @ hn.reshape(T, h)
        dxn, grads["mtp.norm_e"] = rmsnorm_bwd(d_en, xe, r_e, W["mtp.norm_e"])
        np.add.at(dE, tok2.reshape(-1), R(dxn).reshape(T, h))
        dxn, grads["mtp.norm_h"] = rmsnorm_bwd(d_hn, x_L, r_h, W["mtp.norm_h"])
        d_xL_mtp = R(dxn)  # joins the backbone's gradient of x_L below, inside its one rounding
        tap("mtp.d_hF", d_hF2); tap("mtp.d_h_in", d_hp); tap("mtp.d_x_L", d_xL_mtp)
    if not cfg.tie_embeddings:
        grads["lm_head"] = g_head
    dxn, grads["norm_f"] = rmsnorm_bwd(d_hF, x_L, rF, W["norm_f"])
    dx = R(dxn + d_xL_mtp)

    for l in reversed(range(cfg.n_layers)):
        dx = layer_bwd(dx, saved[l], f"layers.{l}.")
        saved[l] = None

    # B10: dE[v,:] = sum over positions holding token v
    np.add.at(dE, tokens.reshape(-1), dx.reshape(T, h))
    grads["embed"] = s_e * dE + (g_head if cfg.tie_embeddings else 0.0)
    return loss, grads, taps


# --------------------------------------------------------------------------
# optimizer
# --------------------------------------------------------------------------
def grad_norm(grads: Dict[str, np.ndarray]) -> float:
    return math.sqrt(sum(float(np.sum(np.asarray(g, dtype=np.float64) ** 2)) for g in grads.values()))


def clip_coeff(gnorm: float, cfg: Config) -> float:
    """min(1, max_norm / (norm + eps)); 1 when clipping is off."""
    if cfg.max_grad_norm <= 0.0:
        return 1.0
    return min(1.0, cfg.max_grad_norm / (gnorm + cfg.clip_eps))


def adamw_update(p, g, m, v, step: int, cfg: Config, wd: float, clip: float = 1.0):
    """One fused clip + Adam + decoupled-decay update of one tensor (fp64 arithmetic).

    g <- g*clip;  m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;
    update = (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps) + wd p;  p <- p - lr update.
    Returns the new (p, m, v) in fp64; the caller stores them as fp32.
    """
    p = np.asarray(p, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64) * clip
    m = cfg.beta1 * np.asarray(m, dtype=np.float64) + (1.0 - cfg.beta1) * g
    v = cfg.beta2 * np.asarray(v, dtype=np.float64) + (1.0 - cfg.beta2) * g * g
    bc1 = 1.0 - cfg.beta1 ** step
    bc2 = 1.0 - cfg.beta2 ** step
    update = (m / bc1) / (np.sqrt(v / bc2) + cfg.adam_eps) + wd * p
    return p - cfg.lr * update, m, v


class TrainState:
    """fp32 masters and Adam moments per parameter name, plus the step counter."""

    def __init__(self, cfg: Config, params: Dict[str, np.ndarray]):
        self.cfg = cfg
        self.params = {k: np.array(v, dtype=np.float32) for k, v in params.items()}
        self.m = {k: np.zeros_like(v) for k, v in self.params.items()}
        self.v = {k: np.zeros_like(v) for k, v in self.params.items()}
        self.step = 0

    def apply_gradients(self, grads: Dict[str, np.ndarray]) -> float:
        """Global grad norm, clip coefficient, then the update of every tensor.  Returns the norm."""
        cfg = self.cfg
        gn = grad_norm(grads)
        coeff = clip_coeff(gn, cfg)
        self.step += 1
        for name in self.params:
            wd = cfg.weight_decay if self.params[name].ndim == 2 else 0.0  # no decay on RMSNorm gains
            p, m, v = adamw_update(self.params[name], grads[name], self.m[name], self.v[name], self.step, cfg, wd,
                                   coeff)
            self.params[name] = p.astype(np.float32)
            self.m[name] = m.astype(np.float32)
            self.v[name] = v.astype(np.float32)
        return gn

    def train_step(self, tokens, labels, mode: str = "contract", want_taps: bool = False):
        loss, grads, taps = forward_backward(self.cfg, self.params, tokens, labels, mode, want_taps)
        gn = self.apply_gradients(grads)
        return loss, gn, grads, taps
