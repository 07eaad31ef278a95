"""Whole train steps at a benchmark workload's full size against stored oracle results.

tests/golden/full_size_<workload>.npz is written by tests/golden/make_full_size_golden.py, which runs consecutive
oracle steps (contract mode, a fresh synthetic batch per step) and calls nothing but the oracle.  Here the library takes
the same steps from the same initial weights in the configuration bench.py times (whole-step graph, AdamW and SwiGLU
backward in GEMM epilogues, weight gradients on a second stream, recomputation where the workload asks for it) and is
compared end to end: loss abs 1e-2 and gradient norm every step; on the sampled steps every gradient (its L2 norm and a
fixed strided sample, rel-L2 <= 2e-2) and every updated master (sample rel-L2: step 1 within the sign-flip ceiling of a
cold Adam step, later steps within the bound measured and fixed below).
"""
import json
import os

import numpy as np
import pytest
import torch

import synth_inputs as SI
from oracle import decoder as D
from tests.parity_util import lib_config, oracle_config, rel_l2, to_dev

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
TOL_LOSS, TOL_GRAD = 1e-2, 2e-2
# updated masters, rel-L2 on the sample: a cold first step is sign(g) (see tests/test_train_step_gpu.py); afterwards the
# two trajectories drift apart by rounding noise fed through Adam, measured per workload and held to a fixed ceiling
MASTER_CEILING = {1: 6e-3, "later": 1e-2}


@pytest.mark.parametrize("name", ["c2_124m", "c3_1b"])
def test_whole_steps_at_full_size_match_the_stored_oracle_results(name):
    from paper_2609_13645_b200 import binding as B
    path = os.path.join(GOLDEN, f"full_size_{name}.npz")
    if not os.path.exists(path):
        pytest.skip(f"no stored oracle result for {name}")
    gold = np.load(path)
    meta = json.loads(str(gold["meta"]))
    assert meta["weight_seed"] == SI.WEIGHT_SEED and meta["data_seed"] == SI.DATA_SEED
    w = SI.WORKLOADS[name]
    ocfg = oracle_config(**{k: w[k] for k in SI.MODEL_KEYS})
    need = B.workspace_bytes(lib_config(B, ocfg, w["batch"], w["seq"], recompute=w["recompute"])) + (6 << 30)
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip(f"needs {need >> 30} GiB of free device memory")
    sample_steps = [int(s) for s in gold["sample_steps"]]
    report = {}
    side = torch.cuda.Stream()  # a capturable stream, as in bench.py
    with torch.cuda.stream(side):
        model = B.Model(lib_config(B, ocfg, w["batch"], w["seq"], recompute=w["recompute"]), seed=SI.WEIGHT_SEED)
        model.set_graph(True)
        params = D.init_params(ocfg, SI.WEIGHT_SEED)
        names = list(params)
        for n in names:
            model.set_param(n, params[n])
        del params
        for step in range(1, meta["steps"] + 1):
            tok, lab = SI.workload_batch(name, step=step - 1)
            tok_d, lab_d = to_dev(tok), to_dev(lab)
            sampled = step in sample_steps
            k = sample_steps.index(step) if sampled else -1
            if sampled:
                # the step itself consumes its weight gradients in the GEMM epilogues: read them from a pass without update
                model.forward_backward(tok_d, lab_d)
                worst_g = 0.0
                for n in names:
                    g = model.get_param(n, B.KIND_GRAD).astype(np.float64).reshape(-1)
                    nrm = float(np.linalg.norm(g))
                    ref = float(gold["gl2/" + n][step - 1])
                    assert abs(nrm - ref) <= 1e-2 * ref + 1e-12, (step, n, nrm, ref)
                    e = rel_l2(g[gold["idx/" + n]], gold["g/" + n][k])
                    worst_g = max(worst_g, e)
                    assert e < TOL_GRAD, (step, "grad", n, e)
                report[f"step{step}.grad"] = worst_g
            loss, gn = model.train_step(tok_d, lab_d)
            assert abs(loss - float(gold["loss"][step - 1])) < TOL_LOSS, (step, loss, float(gold["loss"][step - 1]))
            assert abs(gn - float(gold["gnorm"][step - 1])) < 1e-2 * float(gold["gnorm"][step - 1]), (step, gn)
            if sampled:
                worst_p = 0.0
                for n in names:
                    p = model.get_param(n, B.KIND_MASTER).astype(np.float64).reshape(-1)
                    nrm = float(np.linalg.norm(p))
                    ref = float(gold["pl2/" + n][step - 1])
                    assert abs(nrm - ref) <= 1e-3 * ref, (step, n, nrm, ref)
                    e = rel_l2(p[gold["idx/" + n]], gold["p/" + n][k])
                    worst_p = max(worst_p, e)
                    assert e < MASTER_CEILING.get(step, MASTER_CEILING["later"]), (step, "master", n, e)
                report[f"step{step}.master"] = worst_p
        side.synchronize()
        assert model.step == meta["steps"]
        assert model.graph_replays >= meta["steps"] - 2 or meta["steps"] < 3
        model.close()
        model.workspace = None
    print(name, "worst sampled rel-L2 per step:", {k: float(f"{v:.3g}") for k, v in report.items()})
