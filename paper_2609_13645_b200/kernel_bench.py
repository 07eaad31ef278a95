"""Times one kernel of the library through the C ABI with CUDA events (also the target of ncu captures).

    python -m paper_2609_13645_b200.kernel_bench gemm --M 8192 --N 11264 --K 2048 --layout tn --iters 20
    python -m paper_2609_13645_b200.kernel_bench attn_fwd --B 4 --S 2048 --nh 16 --nkv 8 --d 128
    python -m paper_2609_13645_b200.kernel_bench attn_bwd --B 4 --S 2048 --nh 16 --nkv 8 --d 128
    python -m paper_2609_13645_b200.kernel_bench step --workload c3_1b --layers 1 --iters 3

`step` runs whole train steps of a workload cut down to --layers layers (a few GB on the device): the in-situ target
for ncu captures of the kernels that have no entry point of their own (norms, SwiGLU backward, cross-entropy, the
weight-gradient GEMM with AdamW in its epilogue, the leftover optimizer pass).

Inputs are random bf16; between timed launches a 256 MB buffer is rewritten so the operands do not sit in L2.
Prints one JSON line with the mean launch time and the achieved TFLOP/s.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main():
    import torch
    from paper_2609_13645_b200 import binding as B

    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["gemm", "attn_fwd", "attn_bwd", "step"])
    ap.add_argument("--workload", default="c3_1b")
    ap.add_argument("--layers", type=int, default=1)
    ap.add_argument("--qk-norm", action="store_true", help="step: per-head QK-Norm variant")
    ap.add_argument("--unfused", action="store_true", help="step: separate optimizer pass instead of the fused epilogue")
    ap.add_argument("--M", type=int, default=8192)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--K", type=int, default=2048)
    ap.add_argument("--layout", default="tn", choices=["tn", "nn", "wgrad"])
    ap.add_argument("--B", type=int, default=4)
    ap.add_argument("--S", type=int, default=2048)
    ap.add_argument("--nh", type=int, default=16)
    ap.add_argument("--nkv", type=int, default=8)
    ap.add_argument("--d", type=int, default=128)
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--out", default="auto", choices=["auto", "bf16", "resid", "f32", "f32acc"], help="GEMM epilogue")
    ap.add_argument("--bn", type=int, default=0, help="force the GEMM tile width (development)")
    ap.add_argument("--ws", action="store_true", help="GEMM with a scratch buffer (split-K / balanced-K schedules); attn_bwd with the dS^T scratch")
    ap.add_argument("--pairs", type=int, default=1, help="0: single-CTA GEMM kernel only (development)")
    a = ap.parse_args()
    torch.manual_seed(0)
    if a.bn:
        B.lib().ft_debug_gemm_tile(a.bn)
    B.lib().ft_debug_gemm_pairs(a.pairs)
    dev = "cuda"
    if a.kernel == "step":
        import synth_inputs as SI
        w = SI.WORKLOADS[a.workload]
        Bsz, S = w["batch"], w["seq"]
        cfg = B.make_config(a.layers, w["d_model"], w["n_heads"], w["n_kv_heads"], w["head_dim"], w["d_ffn"], w["vocab"],
                            Bsz, S, recompute=w.get("recompute", 0), qk_norm=int(a.qk_norm))
        model = B.Model(cfg, seed=SI.WEIGHT_SEED)
        model.set_fused_update(not a.unfused)
        total = 0.0
        for it in range(a.warmup + a.iters):
            tok, lab = SI.batch(w["vocab"], Bsz, S, w["dist"], step=it)
            tok, lab = torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); model.train_step(tok, lab, want_loss=False); e1.record()
            torch.cuda.synchronize()
            if it >= a.warmup:
                total += e0.elapsed_time(e1)
        print(json.dumps(dict(kernel="step", workload=a.workload, layers=a.layers, fused=not a.unfused, ms=total / a.iters,
                              iters=a.iters)))
        model.close()
        return
    flush = None if a.no_flush else torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)

    if a.kernel == "gemm":
        M, N, K = a.M, a.N, a.K
        if a.layout == "tn":
            A = torch.randn(M, K, device=dev).bfloat16(); Bm = torch.randn(N, K, device=dev).bfloat16()
            out = torch.empty(M, N, dtype=torch.bfloat16, device=dev); amn, bmn, kind = 0, 0, 0
        elif a.layout == "nn":
            A = torch.randn(M, K, device=dev).bfloat16(); Bm = torch.randn(K, N, device=dev).bfloat16()
            out = torch.empty(M, N, dtype=torch.bfloat16, device=dev); amn, bmn, kind = 0, 1, 0
        else:
            A = torch.randn(K, M, device=dev).bfloat16(); Bm = torch.randn(K, N, device=dev).bfloat16()
            out = torch.empty(M, N, dtype=torch.float32, device=dev); amn, bmn, kind = 1, 1, 2
        resid = None
        if a.out != "auto":
            kind = {"bf16": 0, "resid": 1, "f32": 2, "f32acc": 3}[a.out]
            out = torch.zeros(M, N, dtype=torch.bfloat16 if kind < 2 else torch.float32, device=dev)
            if kind == 1:
                resid = torch.randn(M, N, device=dev).bfloat16()
        flops = 2.0 * M * N * K
        run = lambda: B.k_gemm(A, amn, Bm, bmn, out, kind, M, N, K, err, resid)
        if a.ws:
            scratch = torch.empty(6 << 20, dtype=torch.float32, device=dev)
            run = lambda: B.k_gemm_ws(A, amn, Bm, bmn, out, kind, M, N, K, scratch, err, resid)
        desc = dict(kernel="gemm", layout=a.layout, out=a.out, M=M, N=N, K=K, ws=bool(a.ws))
    else:
        Bsz, S, nh, nkv, d = a.B, a.S, a.nh, a.nkv, a.d
        qkv = torch.randn(Bsz * S, (nh + 2 * nkv) * d, device=dev).bfloat16()
        o = torch.empty(Bsz * S, nh * d, dtype=torch.bfloat16, device=dev)
        lse = torch.empty(Bsz, nh, S, dtype=torch.float32, device=dev)
        B.k_attention_fwd(qkv, o, lse, Bsz, S, nh, nkv, d)
        fwd_flops = 2.0 * Bsz * nh * S * S * d  # causal: half of 4 B n_h S^2 d
        if a.kernel == "attn_fwd":
            flops = fwd_flops
            run = lambda: B.k_attention_fwd(qkv, o, lse, Bsz, S, nh, nkv, d)
        else:
            do = torch.randn(Bsz * S, nh * d, device=dev).bfloat16()
            delta = torch.empty(Bsz, nh, S, dtype=torch.float32, device=dev)
            dqkv = torch.empty_like(qkv)
            flops = 2.0 * fwd_flops  # model count of the backward (the paper's 1:2 ratio)
            run = lambda: B.k_attention_bwd(qkv, o, do, lse, delta, dqkv, Bsz, S, nh, nkv, d)
            if a.ws:
                ds = torch.empty(Bsz * nh, S, S, dtype=torch.bfloat16, device=dev)
                run = lambda: B.k_attention_bwd_ws(qkv, o, do, lse, delta, dqkv, ds, Bsz, S, nh, nkv, d)
        desc = dict(kernel=a.kernel, B=Bsz, S=S, n_heads=nh, n_kv=nkv, d=d, ws=bool(a.ws))

    for _ in range(a.warmup):
        run()
    torch.cuda.synchronize()
    total = 0.0
    for _ in range(a.iters):
        if flush is not None:
            flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); run(); e1.record()
        torch.cuda.synchronize()
        total += e0.elapsed_time(e1)
    ms = total / a.iters
    assert int(err.item()) == 0
    desc.update(ms=ms, tflops=flops / (ms * 1e-3) / 1e12, iters=a.iters)
    print(json.dumps(desc))


if __name__ == "__main__":
    main()
