#!/usr/bin/env python
"""Benchmark of the train step (forward + backward + AdamW) of a Llama-style dense decoder on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3_1b] [--impl reference]

One "step" is one pass of the whole hot path over one synthetic batch.  Prints ONE JSON line: tokens/s
(whole job), MFU against the measured and the nominal dense-bf16 peak, the end-to-end figure through the
host-buffer entry point, a roofline object for the dominant kernel class (the tcgen05 GEMMs) taken from CUDA
events recorded around every launch inside the timed region, and the CPU oracle timed on a bounded sample.

With --gpus N > 1 (launched by torch.distributed.run, or by this script itself when no launcher set WORLD_SIZE) every
rank trains an independent replica on its own batch stream: the path is single-GPU by design, so there is no data-path collective; NCCL only carries the
barrier and the max-over-ranks of the device time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

import synth_inputs as SI
from paper_2609_13645_b200.flops import flops_per_token

NOMINAL_BF16_TFLOPS = 2250.0  # vendor's dense bf16 figure for B200, context only
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms",
                 "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# DRAM read + write bytes of one launch of the dominant kernel, from the committed ncu capture of the gate/up GEMM
# (dram__bytes_read.sum 96.7 MB + dram__bytes_write.sum 158.9 MB in the latest capture; the algorithmic bytes of that launch
# are 264.3 MB)
NCU_GEMM_TRAFFIC_BYTES = 255.6e6
NCU_GEMM_TRAFFIC_OF = ("one launch of gemm_tc_pair_kernel at M 8192, N 11264, K 2048 (gate/up projection of c3_1b), ncu capture "
                       "summarised in profiles/gemm_tc_pair_kernel_tn_8192x11264x2048.md; algorithmic bytes 264.3e6")


def variant_kwargs(args, w):
    """--variant mup_tied: the muP factors of the paper's MiniCPM rows (scale_emb 12, scale_depth 1.4, dim_model_base 256)
    and tied input/output embeddings on top of the workload's shape; --variant qknorm_tied: per-head QK-Norm and tied
    embeddings (the paper's Qwen3 row); the default is the plain decoder."""
    if args.variant == "plain":
        return {}
    if args.variant == "qknorm_tied":  # the Qwen3 column: per-head QK-Norm, tied embeddings, no muP
        return dict(qk_norm=1, tie_embeddings=1)
    if args.variant == "mup_mtp":  # the MiniCPM5 1B column: muP factors, untied, one-layer MTP (Eagle) head
        return dict(emb_scale=12.0, resid_scale=1.4 / w["n_layers"] ** 0.5, logit_scale=256.0 / w["d_model"], mtp=1, mtp_weight=1.0)
    return dict(emb_scale=12.0, resid_scale=1.4 / w["n_layers"] ** 0.5, logit_scale=256.0 / w["d_model"], tie_embeddings=1)


def max_over_ranks(values, world, device=None):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank defines a multi-GPU time)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_tokens_per_s(tokens_per_step_per_rank, world, ms_total, steps):
    """Whole-job throughput of `world` independent replicas that all took ms_total (max over ranks) for `steps` steps."""
    return world * tokens_per_step_per_rank / (ms_total / 1e3 / steps)


def model_flops(w, seq, mtp=False):
    return flops_per_token(w["n_layers"], w["d_model"], w["n_heads"], w["n_kv_heads"], w["head_dim"], w["d_ffn"],
                           w["vocab"], seq, mtp=mtp)


# ------------------------------------------------------------------------------------------ CPU oracle legs
def oracle_sample_run(workload: str, n_layers: int, B: int, S: int, steps: int, warmup: int):
    """Times the CPU oracle, as it stands, on a cut-down sample of the workload.  Returns per-step seconds."""
    from oracle import decoder as D
    w = dict(SI.WORKLOADS[workload])
    cfg = D.Config(**{k: w[k] for k in SI.MODEL_KEYS})
    cfg.n_layers = n_layers
    rng = np.random.default_rng(0)
    params = {}
    for name, shape in D.param_specs(cfg):
        params[name] = (np.ones(shape, dtype=np.float32) if len(shape) == 1
                        else (0.02 * rng.standard_normal(shape, dtype=np.float32)))
    st = D.TrainState(cfg, params)
    times = []
    for i in range(warmup + steps):
        tok, lab = SI.batch(cfg.vocab, B, S, w["dist"], step=i)
        t0 = time.perf_counter()
        st.train_step(tok, lab, mode="contract", want_taps=False)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    w["n_layers"] = n_layers
    return times, model_flops(w, S)["total"] * B * S


def cpu_baseline(workload: str):
    """Oracle on a bounded sample: same shape with 2 layers, 1 x 256 tokens, one step.  The oracle's achieved
    model-FLOP/s on the sample is converted to tokens/s of the full workload with the same FLOP formula."""
    w = SI.WORKLOADS[workload]
    nl, B, S = oracle_sample_shape(workload)
    times, fl = oracle_sample_run(workload, nl, B, S, steps=1, warmup=0)
    rate = fl / times[0]
    full = model_flops(w, w["seq"])["total"]
    return {"value": rate / full, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{workload} shape with {nl} of {w['n_layers']} layers, batch {B} x seq {S}, one oracle train "
                      f"step ({times[0]:.1f} s, {rate / 1e9:.1f} model GFLOP/s), converted with the workload's "
                      f"FLOPs/token"}


def oracle_sample_shape(workload: str):
    """The bounded sample both oracle legs time: the workload's shape with 2 of its layers, batch 1 x 256 tokens."""
    w = SI.WORKLOADS[workload]
    return min(2, w["n_layers"]), 1, min(256, w["seq"])


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    w = SI.WORKLOADS[args.workload]
    nl, B, S = oracle_sample_shape(args.workload)
    times, fl = oracle_sample_run(args.workload, nl, B, S, steps=args.steps, warmup=args.warmup)
    t = sum(times) / len(times)
    rate = fl / t
    full = model_flops(w, w["seq"])["total"]
    val = rate / full
    sample = (f"{args.workload} shape with {nl} of {w['n_layers']} layers, batch {B} x seq {S} per step; model-FLOP/s "
              f"converted to tokens/s with the workload's FLOPs/token")
    line = {"impl": "reference", "metric": "train_tokens_per_sec", "value": val, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": sample},
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------------ the CUDA arm
def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2609_13645_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    w = SI.WORKLOADS[args.workload]
    Bsz, S = w["batch"], w["seq"]
    cfg = B.make_config(w["n_layers"], w["d_model"], w["n_heads"], w["n_kv_heads"], w["head_dim"], w["d_ffn"],
                        w["vocab"], Bsz, S, recompute=w["recompute"], **variant_kwargs(args, w))
    # The model lives on its own (capturable) stream; everything below is enqueued and timed on that stream.
    side = torch.cuda.Stream()
    torch.cuda.set_stream(side)
    model = B.Model(cfg, seed=SI.WEIGHT_SEED)
    model.set_graph(not args.no_graph)
    model.set_overlap(not args.no_overlap)
    model.set_fused_update(not args.no_fused_update)
    model.set_fused_swiglu_bwd(not args.no_fused_swiglu_bwd)
    model.set_streaming_ce(args.streaming_ce)
    n_batches = args.steps + args.warmup
    host_batches = [SI.batch(w["vocab"], Bsz, S, w["dist"], seed=SI.DATA_SEED + 1000 * rank, step=i)
                    for i in range(n_batches)]
    dev_batches = [(torch.from_numpy(t).cuda(), torch.from_numpy(l).cuda()) for t, l in host_batches]
    tokens_per_step = Bsz * S
    peaks, peak_kind = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- (1) the headline: K steps, inputs resident in HBM, whole-step graph replay, no host sync inside
    # the graph is captured on the second step of a shape: with fewer than two warm-up steps the capture would land in
    # the timed region, so the missing ones are run first (untimed, on the first batch)
    priming = max(0, 2 - args.warmup) if not args.no_graph else 0
    for i in range(priming):
        model.train_step(*dev_batches[0], want_loss=False)
    for i in range(args.warmup):
        model.train_step(*dev_batches[i], want_loss=False)
    barrier()
    launches0 = model.launch_count
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for i in range(args.steps):
        model.train_step(*dev_batches[args.warmup + i], want_loss=False)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    launches = model.launch_count - launches0
    graph_replays = model.graph_replays

    # ---- (2) end to end: host buffers in, loss out, every step (directly after the headline pass, so that both see
    # the GPU in the same thermal state)
    pinned = [(torch.from_numpy(t).pin_memory(), torch.from_numpy(l).pin_memory()) for t, l in host_batches]
    for i in range(min(2, args.warmup)):  # through the same calls as the timed loop: their one-time set-up (the pinned
        model.submit_step_host(pinned[i][0].numpy(), pinned[i][1].numpy())  # result ring, its events) happens here
        model.collect_step()
    barrier()
    ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev2.record()
    # The loop a trainer runs: submit step i (ids copied from pinned host memory, the step, its scalars copied back),
    # then read the loss of step i-1, so the device never waits for the host; every step's loss is read inside the
    # timed region, the last one before it closes.
    e2e_loss = None
    for i in range(args.steps):
        t, l = pinned[args.warmup + i]
        model.submit_step_host(t.numpy(), l.numpy())
        if i > 0:
            e2e_loss, _ = model.collect_step()
    e2e_loss, _ = model.collect_step()
    ev3.record()
    barrier()
    ms_e2e = ev2.elapsed_time(ev3)


    # ---- (3) the same K steps launch by launch with CUDA events around every kernel: per-class times and roofline
    model.set_profiling(True)
    ev4, ev5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev4.record()
    for i in range(args.steps):
        model.train_step(*dev_batches[args.warmup + i], want_loss=False)
    ev5.record()
    barrier()
    ms_prof = ev4.elapsed_time(ev5)
    prof = model.get_profile()
    gemm_shapes = model.get_gemm_profile()
    model.set_profiling(False)
    loss_check = model.forward_loss(*dev_batches[0])

    ms_total, ms_e2e, ms_prof = max_over_ranks([ms_total, ms_e2e, ms_prof], world, device="cuda")

    if rank == 0:
        fl = model_flops(w, S, mtp=args.variant == "mup_mtp")  # the MTP head's own row of the paper's FLOP table
        step_s = ms_total / 1e3 / args.steps
        tok_s = job_tokens_per_s(tokens_per_step, world, ms_total, args.steps)
        model_tflops = fl["total"] * tokens_per_step / step_s / 1e12
        g = prof["gemm"]
        gemm_tflops = g["work"] / (g["ms"] / 1e3) / 1e12 if g["ms"] > 0 else None
        peak_tf = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
        roof = {"bound": "tensor", "kernel": "gemm_tc_kernel (all tcgen05 GEMMs of the step)",
                "achieved": gemm_tflops, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": gemm_tflops / peak_tf if gemm_tflops else None, "traffic": NCU_GEMM_TRAFFIC_BYTES,
                "traffic_of": NCU_GEMM_TRAFFIC_OF,
                "peak_kind": f"{peak_kind} sustained bf16 (kernels timed inside a long step)",
                "share_of_step": g["ms"] / ms_prof,
                "measured_in": "the profiled pass (same K steps, CUDA events around every launch, no graph)"}
        classes = {k: {"ms_per_step": v["ms"] / args.steps, "share": v["ms"] / ms_prof, "launches_per_step":
                       v["launches"] / args.steps,
                       ("tflops" if k in ("gemm", "attn_fwd", "attn_bwd") else "gbs"):
                       (v["work"] / (v["ms"] / 1e3) / (1e12 if k in ("gemm", "attn_fwd", "attn_bwd") else 1e9)
                        if v["ms"] > 0 else None)} for k, v in prof.items()}
        line = {
            "metric": "train_tokens_per_sec", "value": tok_s, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "batch": Bsz, "seq_len": S, "tokens_per_step_per_gpu": tokens_per_step,
                       "parallelism": "replicas only (single-GPU path, no collectives)" if world > 1 else "1 GPU",
                       "recompute": w["recompute"], "cuda_graph": graph_replays > 0, "graph_priming_steps": priming,
                       "variant": args.variant,
                       "l2": "no flush needed: weights + activations touched per step are far larger than the 126 MB L2",
                       "token_ids": w["dist"]},
            "mfu": {"model_tflops": model_tflops, "model_gflop_per_token": fl["total"] / 1e9,
                    "vs_measured_burst": model_tflops / peaks["bf16_tflops"],
                    "vs_measured_sustained": model_tflops / peak_tf,
                    "vs_nominal_2250": model_tflops / NOMINAL_BF16_TFLOPS, "peaks": peak_kind},
            "roofline": roof, "ms_per_step_profiled": ms_prof / args.steps, "kernel_classes": classes,
            "e2e": {"value": job_tokens_per_s(tokens_per_step, world, ms_e2e, args.steps), "unit": "tokens/s",
                    "h2d_bytes_per_step": 2 * tokens_per_step * 4, "d2h_bytes_per_step": 64,
                    "ms_per_step": ms_e2e / args.steps, "last_loss": e2e_loss,
                    "api": "submit_step_host + collect_step: step i is enqueued before the loss of step i-1 is read"},
            "gemm_shapes": [dict(g, ms_per_step=g["ms"] / args.steps, launches_per_step=g["launches"] / args.steps)
                            for g in sorted(gemm_shapes, key=lambda g: -g["ms"])],
            "gpu_launches": launches, "clocks": clocks, "loss_after_run": loss_check,
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(args.workload)
        print(json.dumps(line))
    model.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def run_dp(args):
    """Opt-in (--dp): the same workload as ONE data-parallel job over all ranks (paper_2609_13645_b200/dp.py): bucketed
    reduce-scatter behind the backward pass, sharded AdamW, per-bucket all-gather.  The default arm stays replicas.
    Every step reads its loss (the driver's collect), so this is an end-to-end style number."""
    import torch
    import torch.distributed as dist
    from paper_2609_13645_b200 import binding as B
    from paper_2609_13645_b200.dp import DataParallel, LibraryBackend

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29771", rank=0, world_size=1)
    w = SI.WORKLOADS[args.workload]
    Bsz, S = w["batch"], w["seq"]
    cfg = B.make_config(w["n_layers"], w["d_model"], w["n_heads"], w["n_kv_heads"], w["head_dim"], w["d_ffn"],
                        w["vocab"], Bsz, S, recompute=w["recompute"], **variant_kwargs(args, w))
    side = torch.cuda.Stream()
    torch.cuda.set_stream(side)
    model = B.Model(cfg, seed=SI.WEIGHT_SEED)
    dp = DataParallel(LibraryBackend(model))
    n_batches = args.steps + args.warmup
    batches = [SI.batch(w["vocab"], Bsz, S, w["dist"], seed=SI.DATA_SEED + 1000 * rank, step=i) for i in range(n_batches)]
    batches = [(torch.from_numpy(t).cuda(), torch.from_numpy(l).cuda()) for t, l in batches]
    for i in range(args.warmup):
        dp.step(*batches[i])
    dist.barrier(); torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    loss = None
    for i in range(args.steps):
        loss, gnorm = dp.step(*batches[args.warmup + i])
    ev1.record()
    dist.barrier(); torch.cuda.synchronize()
    ms = max_over_ranks([ev0.elapsed_time(ev1)], world, device="cuda")[0]
    if rank == 0:
        print(json.dumps({
            "metric": "train_tokens_per_sec", "value": job_tokens_per_s(Bsz * S, world, ms, args.steps), "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "batch_per_gpu": Bsz, "seq_len": S, "global_batch": Bsz * world,
                       "parallelism": f"dp{world}: reduce-scatter per gradient bucket behind the backward pass, sharded AdamW, "
                                      "all-gather of the bf16 copy per bucket", "buckets": len(dp.buckets)},
            "last_loss": loss, "mode": "dp"}))
    dist.barrier()
    dist.destroy_process_group()


def relaunch_under_torchrun(n: int) -> int:
    """`python bench.py --gpus N` run plainly (no launcher in the environment): start N ranks of this same command line
    under torch.distributed.run on this node and hand back its exit code.  Rank 0 of the child job prints the JSON line."""
    import socket
    with socket.socket() as sock:  # a free port for the rendezvous
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c3_1b", choices=sorted(SI.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dp", action="store_true", help="one data-parallel job over the ranks instead of independent replicas")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel separately in the timed region")
    ap.add_argument("--variant", default="plain", choices=["plain", "mup_tied", "qknorm_tied", "mup_mtp"],
                    help="model variant on the workload's shape (default: the plain decoder the metric is quoted on)")
    ap.add_argument("--no-overlap", action="store_true", help="ablation: weight-gradient GEMMs on the main stream")
    ap.add_argument("--no-fused-update", action="store_true", help="ablation: separate AdamW pass over all parameters")
    ap.add_argument("--no-fused-swiglu-bwd", action="store_true",
                    help="ablation: SwiGLU backward as a kernel of its own instead of the data-gradient GEMM's epilogue")
    ap.add_argument("--streaming-ce", action="store_true", help="cross-entropy inside the logits GEMM's epilogues (GEMM runs twice)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return relaunch_under_torchrun(args.gpus)
    if args.impl == "reference":
        return run_reference(args)
    if args.dp:
        return run_dp(args)
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
