"""Model-FLOP count per token (the MFU numerator).

Follows the paper's appendix "Model-FLOPs Utilization": a multiply-accumulate is
two FLOPs; forward per token
  attention projections 2h(h_q + 2h_kv) + 2 h_q h,   FFN 2(2hf) + 2fh,
  attention core (causal, factor 1/2 folded in) 2 n_h s d,   output head 2hV;
every per-layer term is counted three times (forward + two backward) and summed
over L layers, the head three times once.  The one-layer MTP (Eagle) head of the
appendix "Ascend Model-FLOPs Utilization" is a row of its own: one more layer
(projections, FFN, attention core), a second output head and the projection of
the concatenated [hidden state; next-token embedding] back to the model width,
2 (2h) h; with the 1B geometry printed there this gives the table's 1.452 GFLOP/token.
"""
from __future__ import annotations


def flops_per_token(n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, seq, mtp=False):
    """dict of forward+backward FLOPs per token by operator class, plus 'total'."""
    h, f, d = d_model, d_ffn, head_dim
    hq, hkv = n_heads * d, n_kv_heads * d
    proj = 2 * h * (hq + 2 * hkv) + 2 * hq * h
    ffn = 2 * (2 * h * f) + 2 * f * h
    core = 2 * n_heads * seq * d
    head = 2 * h * vocab
    out = {
        "proj": 3 * n_layers * proj,
        "ffn": 3 * n_layers * ffn,
        "core": 3 * n_layers * core,
        "head": 3 * head,
    }
    if mtp:
        out["mtp"] = 3 * (proj + ffn + core + head + 2 * (2 * h) * h)
    out["total"] = sum(out.values())
    return out
