"""Writes the stored expected values of whole train steps at a benchmark workload's full size.

Runs consecutive oracle steps (contract mode, fresh synthetic batch every step, weights from the seeded
initialiser) and stores a compact summary per step: the loss, the global gradient norm, the L2 norm of every
gradient and of every updated master, and a fixed random sample (seeded by the tensor's name) of every gradient, updated
master and both Adam moments.  Imports nothing but the oracle and the seeded input generators; the GPU tests read the file and
never write it.

    python tests/golden/make_full_size_golden.py c2_124m --steps 10
    python tests/golden/make_full_size_golden.py c3_1b --steps 1

Output: tests/golden/full_size_<workload>.npz (keys: meta, loss, gnorm, sample_steps, and per tensor name
"gl2/<name>", "pl2/<name>" [steps], "idx/<name>" [n], "g/<name>", "p/<name>", "m/<name>", "v/<name>"
[len(sample_steps), n] as fp32).  The committed files were written with --samples 2048 and then passed through
--shrink-from (1024 samples of gradients and masters; the moment samples dropped) to keep them small.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time
import zlib

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth_inputs as SI  # noqa: E402
from oracle import decoder as D  # noqa: E402

HYPER = ("rms_eps", "rope_theta", "lr", "beta1", "beta2", "adam_eps", "weight_decay")


def sample_index(name: str, size: int, n: int) -> np.ndarray:
    """n distinct flat positions (logical [out, in] order) of a tensor, drawn uniformly from a generator seeded by the
    tensor's name (a fixed stride would walk down one column whenever it is a multiple of the row length); all of the
    tensor when it is smaller."""
    if size <= n:
        return np.arange(size, dtype=np.int64)
    rng = np.random.default_rng(zlib.crc32(name.encode()))
    return np.sort(rng.choice(size, size=n, replace=False)).astype(np.int64)


def oracle_config(name: str) -> D.Config:
    w = SI.WORKLOADS[name]
    cfg = D.Config(**{k: w[k] for k in SI.MODEL_KEYS})
    for k in HYPER:  # the values a C struct of floats holds
        setattr(cfg, k, float(np.float32(getattr(cfg, k))))
    return cfg


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("workload")
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--samples", type=int, default=2048)
    ap.add_argument("--sample-steps", type=str, default="", help="1-based steps whose samples are kept (default: all)")
    ap.add_argument("--out", type=str, default="")
    ap.add_argument("--shrink-from", type=str, default="",
                    help="instead of running the oracle: rewrite an earlier output of this script with every other sample "
                         "and without the moment samples (the stored values stay the oracle's)")
    a = ap.parse_args()
    if a.shrink_from:
        src = np.load(a.shrink_from)
        keep_arrays = {}
        for k in src.files:
            if k[:2] in ("m/", "v/"):
                continue
            v = src[k]
            if k.startswith("idx/"):
                v = v[::2]
            elif k[:2] in ("g/", "p/"):
                v = v[:, ::2]
            keep_arrays[k] = v
        meta = json.loads(str(src["meta"]))
        meta["samples"] = int(meta["samples"]) // 2
        keep_arrays["meta"] = np.array(json.dumps(meta))
        path = a.out or os.path.join(HERE, f"full_size_{a.workload}.npz")
        np.savez_compressed(path, **keep_arrays)
        print("wrote", path, os.path.getsize(path), "bytes")
        return
    cfg = oracle_config(a.workload)
    keep = sorted({int(s) for s in a.sample_steps.split(",") if s}) or list(range(1, a.steps + 1))
    params = D.init_params(cfg, SI.WEIGHT_SEED)
    st = D.TrainState(cfg, params)
    names = list(st.params)
    idx = {n: sample_index(n, st.params[n].size, a.samples) for n in names}
    out = {"loss": [], "gnorm": []}
    for n in names:
        out["gl2/" + n], out["pl2/" + n] = [], []
        for k in "gpmv":
            out[k + "/" + n] = []
    secs = []
    for step in range(a.steps):
        tok, lab = SI.workload_batch(a.workload, step=step)
        t0 = time.time()
        loss, gn, grads, _ = st.train_step(tok, lab)
        secs.append(time.time() - t0)
        out["loss"].append(loss)
        out["gnorm"].append(gn)
        for n in names:
            out["gl2/" + n].append(float(np.linalg.norm(grads[n].astype(np.float64))))
            out["pl2/" + n].append(float(np.linalg.norm(st.params[n].astype(np.float64))))
            if step + 1 in keep:
                out["g/" + n].append(np.asarray(grads[n]).reshape(-1)[idx[n]].astype(np.float32))
                out["p/" + n].append(st.params[n].reshape(-1)[idx[n]])
                out["m/" + n].append(st.m[n].reshape(-1)[idx[n]])
                out["v/" + n].append(st.v[n].reshape(-1)[idx[n]])
        del grads
        print(f"step {step + 1}: loss {loss:.6f} gnorm {gn:.6f} ({secs[-1]:.0f} s)", flush=True)
    meta = dict(workload=a.workload, steps=a.steps, weight_seed=SI.WEIGHT_SEED, data_seed=SI.DATA_SEED,
                samples=a.samples, seconds_per_step=secs, cores=os.cpu_count(),
                hyper={k: getattr(cfg, k) for k in HYPER})
    arrays = {"meta": np.array(json.dumps(meta)), "sample_steps": np.array(keep, dtype=np.int64)}
    for k, v in out.items():
        arrays[k] = np.asarray(v, dtype=np.float32 if k[:2] in ("g/", "p/", "m/", "v/") else np.float64)
    for n in names:
        arrays["idx/" + n] = idx[n]
    path = a.out or os.path.join(HERE, f"full_size_{a.workload}.npz")
    np.savez_compressed(path, **arrays)
    print("wrote", path, os.path.getsize(path), "bytes")


if __name__ == "__main__":
    main()
