"""Whole train step (forward, backward, AdamW) of the CUDA library against the CPU oracle, through the C ABI.

Tolerances: loss abs 1e-2, per-tensor relative L2 <= 2e-2 on activations and gradients, <= 1e-3 on updated fp32
masters (asserted where Adam's moments are warm; the very first update is g / (|g| + eps) = sign(g), where a gradient
entry of the wrong sign moves a master by 2 lr, so step 1 is held to the sign-flip bound with a fixed ceiling);
run-to-run results are bit-identical.
"""
import numpy as np
import pytest
import torch

import synth_inputs as SI
from oracle import decoder as D
from tests.parity_util import (BWD_TAPS, FWD_TAPS, lib_config, lib_tap, load_params, oracle_config, rel_l2, to_dev)
from tests.parity_util import f32 as parity_f32

pytestmark = pytest.mark.gpu

TOL_LOSS, TOL_ACT, TOL_MASTER = 1e-2, 2e-2, 1e-3
# step 1 only (cold moments): ceiling on the master error whatever the sign-flip prediction says, so that a regression in
# the gradients or the update cannot widen its own tolerance (measured worst case over the shapes and variants of this file: 4.5e-3)
MASTER_CEILING_STEP1 = 6e-3


def _c1():
    w = SI.WORKLOADS["c1_tiny"]
    return oracle_config(**{k: w[k] for k in SI.MODEL_KEYS}), w


def _small_gqa():
    # two layers, GQA 4/2 with head_dim 128, ragged ffn; a shape no single tile covers
    return oracle_config(n_layers=2, d_model=512, n_heads=4, n_kv_heads=2, head_dim=128, d_ffn=720, vocab=2048)


def _check_step(ocfg, tok, lab, params, debug=True, recompute=0, report=None, stored_ds=True, streaming_ce=False):
    from paper_2609_13645_b200 import binding as B
    Bsz, S = tok.shape
    T = Bsz * S
    model = B.Model(lib_config(B, ocfg, Bsz, S, debug_taps=1 if debug else 0, recompute=recompute), seed=1)
    if ocfg.rope_factors is not None or ocfg.rope_mscale != 1.0:
        model.set_rope_scaling(ocfg.rope_factors, ocfg.rope_mscale)
    model.set_attention_stored_ds(stored_ds)
    model.set_streaming_ce(streaming_ce)
    if not debug:  # gradients are compared below: keep them (the fused epilogues consume them; their bits are tested apart)
        model.set_fused_update(False)
    load_params(model, params)
    st = D.TrainState(ocfg, params)
    loss_o, gn_o, grads_o, taps_o = st.train_step(tok, lab, mode="contract", want_taps=True)
    loss_g, gn_g = model.train_step(to_dev(tok), to_dev(lab))
    worst = {}
    assert abs(loss_g - loss_o) < TOL_LOSS, (loss_g, loss_o)
    assert abs(gn_g - gn_o) / gn_o < 2e-3, (gn_g, gn_o)
    if debug:
        for l in range(ocfg.n_layers):
            for nm in FWD_TAPS + BWD_TAPS:
                e = rel_l2(lib_tap(model, ocfg, nm, l, T), taps_o[f"layers.{l}.{nm}"])
                worst[f"{l}.{nm}"] = e
                assert e < TOL_ACT, (l, nm, e)
        for nm in ("hF", "ce_lse", "d_hF"):
            e = rel_l2(model.get_tap(nm, -1), taps_o[nm])
            worst[nm] = e
            assert e < TOL_ACT, (nm, e)
    for name in params:
        e = rel_l2(model.get_param(name, B.KIND_GRAD), grads_o[name])
        worst["grad." + name] = e
        assert e < TOL_ACT, ("grad", name, e)
    # The update itself adds nothing: the oracle's AdamW applied to the LIBRARY's gradients reproduces the
    # library's masters to fp32 rounding.
    st_g = D.TrainState(ocfg, params)
    st_g.apply_gradients({k: model.get_param(k, B.KIND_GRAD).astype(np.float64) for k in params})
    for name in params:
        assert rel_l2(model.get_param(name, B.KIND_MASTER), st_g.params[name]) < 1e-6, ("update", name)
        assert rel_l2(model.get_param(name, B.KIND_ADAM_M), st_g.m[name]) < 1e-6
        assert rel_l2(model.get_param(name, B.KIND_ADAM_V), st_g.v[name]) < 1e-6
    # End to end against the oracle's masters.  On step 1 Adam's update is g/(|g|+eps) ~ sign(g), so a gradient
    # entry whose sign differs moves the master by 2 lr.  With gradient error rho (rel-L2) a fraction ~rho/pi of
    # the entries flips, i.e. a master error of (2 lr / rms p) sqrt(rho/pi): the stated 1e-3 needs rho <= 3e-4,
    # below the rounding noise of a bf16 step, so the bound asserted is the larger of the two (2.5x: gradient entries are not Gaussian).
    for name in params:
        e = rel_l2(model.get_param(name, B.KIND_MASTER), st.params[name])
        worst["master." + name] = e
        rho = worst["grad." + name]
        rms_p = float(np.sqrt(np.mean(st.params[name].astype(np.float64) ** 2)))
        predicted = 2.0 * ocfg.lr / rms_p * np.sqrt(rho / np.pi)
        assert e < max(TOL_MASTER, min(2.5 * predicted, MASTER_CEILING_STEP1)), ("master", name, e, predicted)
        # the bf16 compute copy is the rounded new master
        got_b = model.get_param(name, B.KIND_BF16)
        assert np.array_equal(got_b, D.bf16_round(model.get_param(name, B.KIND_MASTER)).astype(np.float32))
    assert model.step == 1
    if report is not None:
        report.update(worst)
    model.close()
    return worst


def test_config1_step_matches_oracle_on_every_tap_gradient_and_master():
    ocfg, w = _c1()
    params = D.init_params(ocfg, SI.WEIGHT_SEED)
    tok, lab = SI.workload_batch("c1_tiny")
    worst = _check_step(ocfg, tok, lab, params)
    print("worst rel-L2:", sorted(worst.items(), key=lambda kv: -kv[1])[:8])


def test_gqa_head_dim_128_two_layers_with_ignored_labels():
    ocfg = _small_gqa()
    params = D.init_params(ocfg, 99)
    tok, lab = SI.batch(ocfg.vocab, 2, 200, "zipf", seed=5)
    lab = lab.copy()
    lab[0, :7] = -1
    _check_step(ocfg, tok, lab, params)


@pytest.mark.parametrize("shape,recompute", [("c1", 0), ("gqa_ragged_ffn", 0), ("gqa_ragged_ffn", 1)])
def test_default_path_without_taps_matches_oracle_on_loss_every_gradient_and_master(shape, recompute):
    """Without debug taps the step takes the paths a training run takes (SwiGLU backward inside the data-gradient
    epilogue, no stored d_a); loss, every parameter gradient and the updated masters against the oracle."""
    if shape == "c1":
        ocfg, _ = _c1()
        params = D.init_params(ocfg, SI.WEIGHT_SEED)
        tok, lab = SI.workload_batch("c1_tiny")
    else:
        ocfg = _small_gqa()
        params = D.init_params(ocfg, 99)
        tok, lab = SI.batch(ocfg.vocab, 2, 200, "zipf", seed=5)
        lab = lab.copy()
        lab[1, -5:] = -1
    _check_step(ocfg, tok, lab, params, debug=False, recompute=recompute)


@pytest.mark.parametrize("one_pass", [True, False])
def test_output_head_over_several_row_chunks_matches_oracle_in_both_forms(one_pass):
    """5 x 1024 tokens: the logits are formed in two chunks of rows (4096 + 1024).  By default the logit gradient of all
    rows is kept and the head's data and weight gradients are one contraction each over all rows; with the buffer limit
    at 0 they are formed per chunk and the weight gradient accumulates in memory.  Both against the oracle: loss, hF, the
    log-sum-exp of every row, d_hF, every gradient, masters."""
    import ctypes as C
    from paper_2609_13645_b200 import binding as B
    ocfg, _ = _c1()
    params = D.init_params(ocfg, SI.WEIGHT_SEED)
    tok, lab = SI.batch(ocfg.vocab, 5, 1024, "zipf", seed=3)
    lab = lab.copy()
    lab[4, 1000:] = -1
    L = B.lib()
    L.ft_debug_head_dz_limit.argtypes = [C.c_uint64]
    L.ft_debug_head_dz_limit.restype = None
    L.ft_debug_head_dz_limit(C.c_uint64(4 << 30 if one_pass else 0))
    try:
        _check_step(ocfg, tok, lab, params)
    finally:
        L.ft_debug_head_dz_limit(C.c_uint64(4 << 30))


@pytest.mark.parametrize("variant", ["mtp", "mtp+tied+qknorm+mup", "mtp+ragged+streaming"])
def test_mtp_head_step_matches_oracle_on_loss_every_gradient_and_master(variant):
    """The one-layer MTP (Eagle) head of the paper's 1B configuration: the normalised last hidden state and the normalised
    embedding of the next token, projected, through one more decoder layer and the backbone's output head, trained on
    the token after next with its own weight.  Full-step parity with the oracle: loss, every gradient (backbone, head,
    embedding table with its three contributions when tied, all mtp.* tensors), AdamW, masters."""
    import math
    kw = dict(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024, mtp=True, mtp_weight=0.3)
    Bsz, S = 2, 128
    streaming = False
    if "tied" in variant:
        kw.update(tie_embeddings=True, qk_norm=True, emb_scale=12.0, resid_scale=1.4 / math.sqrt(2), logit_scale=0.5,
                  mtp_weight=1.0)
    if "ragged" in variant:
        kw.update(vocab=1000, d_ffn=720)
        Bsz, S, streaming = 3, 70, True
    ocfg = oracle_config(**kw)
    params = D.init_params(ocfg, SI.WEIGHT_SEED)
    assert "mtp.proj_e" in params and "mtp.layer.wgu" in params
    tok, lab = SI.batch(ocfg.vocab, Bsz, S, "zipf", seed=31)
    lab = lab.copy(); lab[0, 5:9] = -1
    _check_step(ocfg, tok, lab, params, debug=False, streaming_ce=streaming)


def test_mtp_head_step_is_bit_identical_with_graph_recomputation_second_stream_and_fused_update():
    from paper_2609_13645_b200 import binding as B
    ocfg = oracle_config(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024, mtp=True,
                         mtp_weight=0.5)
    Bsz, S = 2, 128
    batches = [SI.batch(ocfg.vocab, Bsz, S, "zipf", step=i) for i in range(4)]
    outs = []
    for recompute, overlap, graph, fused in [(0, False, False, False), (1, True, False, True), (0, True, True, True),
                                             (0, False, False, True)]:
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            model = B.Model(lib_config(B, ocfg, Bsz, S, recompute=recompute), seed=5)
            model.set_overlap(overlap)
            model.set_fused_update(fused)
            model.set_graph(graph)
            losses = [model.train_step(to_dev(t), to_dev(l))[0] for t, l in batches]
            side.synchronize()
            state = [model.get_param(n, B.KIND_MASTER).view(np.uint32).copy() for n, _ in model.params]
            if graph:
                assert model.graph_replays >= 2
            model.close()
        outs.append((np.float32(losses).view(np.uint32), state))
    for o in outs[1:]:
        assert np.array_equal(o[0], outs[0][0])
        for a, b in zip(o[1], outs[0][1]):
            assert np.array_equal(a, b)


@pytest.mark.parametrize("shape", ["c1", "ragged_tied_mup"])
def test_streaming_cross_entropy_matches_oracle_and_the_default_path(shape):
    """Cross-entropy inside the logits GEMM's epilogues (per-tile max / sum pairs, then the GEMM again for dz): the same
    parity bars as the default path, and losses / gradients that agree with it to rounding.  The ragged case has a
    vocabulary that ends inside a 256-column tile, rows that end inside a 128-row tile, ignored labels, tied
    embeddings and a logit factor."""
    from paper_2609_13645_b200 import binding as B
    if shape == "c1":
        ocfg, w = _c1()
        tok, lab = SI.workload_batch("c1_tiny")
    else:
        ocfg = oracle_config(n_layers=1, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1000,
                             tie_embeddings=True, logit_scale=0.5, emb_scale=4.0)
        tok, lab = SI.batch(ocfg.vocab, 3, 70, "zipf", seed=21)
        lab = lab.copy(); lab[1, 3:11] = -1
    params = D.init_params(ocfg, SI.WEIGHT_SEED)
    _check_step(ocfg, tok, lab, params, streaming_ce=True)
    Bsz, S = tok.shape
    out = []
    for streaming in (False, True):
        m = B.Model(lib_config(B, ocfg, Bsz, S), seed=1)
        load_params(m, params)
        m.set_streaming_ce(streaming)
        loss = m.forward_backward(to_dev(tok), to_dev(lab))
        out.append((loss, {n: m.get_param(n, B.KIND_GRAD) for n in params}))
        m.close()
    assert abs(out[0][0] - out[1][0]) < 2e-6 * abs(out[0][0])
    for n in params:
        assert rel_l2(out[1][1][n], out[0][1][n]) < 3e-3, n


@pytest.mark.parametrize("stored_ds", [False, True])
def test_both_attention_backward_paths_match_oracle_on_a_multi_tile_sequence(stored_ds):
    """S = 384 is a multiple of 128, so the step may keep dS^T and compute dQ as one batched contraction; with the
    switch off it recomputes S and dP in a dQ kernel.  Same parity bars either way."""
    ocfg = _small_gqa()
    params = D.init_params(ocfg, 99)
    tok, lab = SI.batch(ocfg.vocab, 1, 384, "zipf", seed=6)
    _check_step(ocfg, tok, lab, params, stored_ds=stored_ds)


@pytest.mark.parametrize("variant", ["mup", "tied", "tied+mup", "qknorm", "qknorm128+tied+mup", "longrope+qknorm"])
def test_model_variants_match_oracle_on_every_tap_gradient_and_master(variant):
    """The paper's model families differ from the plain decoder by tied input/output embeddings and by the muP factors
    on the embedding, the residual branches and the logits: same full-step parity as configuration 1."""
    import math
    kw = dict(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024)
    if "mup" in variant:  # MiniCPM's numbers: scale_emb 12, scale_depth 1.4, dim_model_base 256 (here d_model = 256 -> 0.5 used)
        kw.update(emb_scale=12.0, resid_scale=1.4 / math.sqrt(2), logit_scale=0.5)
    if "tied" in variant:
        kw.update(tie_embeddings=True)
    if "qknorm" in variant:  # the Qwen3 column: per-head RMSNorm of q and k before the rotation
        kw.update(qk_norm=True)
    if "128" in variant:
        kw.update(d_model=512, head_dim=128)
    if "longrope" in variant:  # per-frequency rescale factors growing with the index, magnitude factor on cos / sin
        kw.update(rope_factors=tuple(float(np.float32(1.0 + 0.2 * i)) for i in range(kw["head_dim"] // 2)),
                  rope_mscale=float(np.float32(1.1)))
    ocfg = oracle_config(**kw)
    params = D.init_params(ocfg, SI.WEIGHT_SEED)
    if ocfg.qk_norm:  # gains away from 1, so that a missing or misplaced gain shows
        rng = np.random.default_rng(3)
        for l in range(ocfg.n_layers):
            for nm in ("q_norm", "k_norm"):
                params[f"layers.{l}.{nm}"] = (1.0 + 0.25 * rng.standard_normal(ocfg.head_dim)).astype(np.float32)
    assert ("lm_head" in params) == ("tied" not in variant)
    tok, lab = SI.batch(ocfg.vocab, 2, 128, "uniform", step=0)
    _check_step(ocfg, tok, lab, params)


def test_seeded_initialisation_matches_the_oracles_generator():
    from paper_2609_13645_b200 import binding as B
    ocfg, w = _c1()
    model = B.Model(lib_config(B, ocfg, 2, 128), seed=SI.WEIGHT_SEED)
    want = D.init_params(ocfg, SI.WEIGHT_SEED)
    for name, arr in want.items():
        got = model.get_param(name)
        assert got.shape == arr.shape
        assert np.allclose(got, arr, rtol=2.5e-7, atol=1e-12), name  # libm differences of the two sides: <= 1 ulp of fp32
        assert np.mean(got != arr) < 1e-3
    assert model.step == 0
    tok, lab = SI.workload_batch("c1_tiny")
    loss = model.forward_loss(to_dev(tok), to_dev(lab))
    assert abs(loss - (np.log(1024) + 0.5 * 0.02 ** 2 * 256)) < 0.03
    model.close()


def test_adamw_in_isolation_matches_oracle_to_1e6():
    from paper_2609_13645_b200 import binding as B
    ocfg, _ = _c1()
    ocfg.max_grad_norm = D.Config.__dataclass_fields__["max_grad_norm"].default
    rng = np.random.default_rng(3)
    params = D.init_params(ocfg, 5)
    for clip in (0.0, 0.5):
        ocfg.max_grad_norm = clip
        model = B.Model(lib_config(B, ocfg, 2, 128), seed=1)
        load_params(model, params)
        st = D.TrainState(ocfg, params)
        for step in range(3):
            grads = {k: (rng.standard_normal(v.shape) * 10.0 ** rng.uniform(-6, -2)).astype(np.float32)
                     for k, v in params.items()}
            for k, g in grads.items():
                model.set_param(k, g, B.KIND_GRAD)
            gn_o = st.apply_gradients({k: g.astype(np.float64) for k, g in grads.items()})
            gn_g = model.apply_update()
            assert abs(gn_g - gn_o) / gn_o < 1e-5
            for k in params:
                assert rel_l2(model.get_param(k), st.params[k]) < 1e-6, (clip, step, k)
                assert rel_l2(model.get_param(k, B.KIND_ADAM_M), st.m[k]) < 1e-6
                assert rel_l2(model.get_param(k, B.KIND_ADAM_V), st.v[k]) < 1e-6
        assert model.step == 3
        model.close()


def _run_steps(ocfg, params, n, recompute=0, Bsz=2, S=128, start=0, model=None):
    from paper_2609_13645_b200 import binding as B
    if model is None:
        model = B.Model(lib_config(B, ocfg, Bsz, S, recompute=recompute), seed=1)
        load_params(model, params)
    losses = []
    for s in range(start, start + n):
        tok, lab = SI.batch(ocfg.vocab, Bsz, S, "uniform", step=s)
        losses.append(model.train_step(to_dev(tok), to_dev(lab)))
    return model, losses


def _state_bits(model):
    from paper_2609_13645_b200 import binding as B
    out = []
    for name, _ in model.params:
        for kind in (B.KIND_MASTER, B.KIND_ADAM_M, B.KIND_ADAM_V, B.KIND_BF16):
            out.append(model.get_param(name, kind).view(np.uint32).copy())
    return out


def test_bit_identical_run_to_run_and_with_recomputation():
    ocfg, _ = _c1()
    params = D.init_params(ocfg, SI.WEIGHT_SEED)
    m1, l1 = _run_steps(ocfg, params, 3)
    m2, l2 = _run_steps(ocfg, params, 3)
    m3, l3 = _run_steps(ocfg, params, 3, recompute=1)
    assert np.array_equal(np.float32(l1).view(np.uint32), np.float32(l2).view(np.uint32))
    assert np.array_equal(np.float32(l1).view(np.uint32), np.float32(l3).view(np.uint32))
    for a, b, c in zip(_state_bits(m1), _state_bits(m2), _state_bits(m3)):
        assert np.array_equal(a, b) and np.array_equal(a, c)
    for m in (m1, m2, m3):
        m.close()


def test_resume_from_saved_state_is_bit_identical():
    from paper_2609_13645_b200 import binding as B
    ocfg, _ = _c1()
    params = D.init_params(ocfg, SI.WEIGHT_SEED)
    straight, ls = _run_steps(ocfg, params, 4)
    first, l_a = _run_steps(ocfg, params, 2)
    fresh = B.Model(lib_config(B, ocfg, 2, 128), seed=777)
    for name, _ in first.params:
        for kind in (B.KIND_MASTER, B.KIND_ADAM_M, B.KIND_ADAM_V):
            fresh.set_param(name, first.get_param(name, kind), kind)
    fresh.step = first.step
    _, l_b = _run_steps(ocfg, params, 2, start=2, model=fresh)
    assert np.array_equal(np.float32(ls).view(np.uint32), np.float32(l_a + l_b).view(np.uint32))
    for a, b in zip(_state_bits(straight), _state_bits(fresh)):
        assert np.array_equal(a, b)
    for m in (straight, first, fresh):
        m.close()


def test_host_buffer_entry_point_equals_device_entry_point():
    ocfg, _ = _c1()
    params = D.init_params(ocfg, SI.WEIGHT_SEED)
    from paper_2609_13645_b200 import binding as B
    tok, lab = SI.workload_batch("c1_tiny")
    a = B.Model(lib_config(B, ocfg, 2, 128), seed=1)
    b = B.Model(lib_config(B, ocfg, 2, 128), seed=1)
    load_params(a, params)
    load_params(b, params)
    la = a.train_step(to_dev(tok), to_dev(lab))
    lb = b.train_step_host(tok, lab)
    assert la == lb
    for x, y in zip(_state_bits(a), _state_bits(b)):
        assert np.array_equal(x, y)
    a.close()
    b.close()


def test_pipelined_host_steps_equal_the_synchronous_host_steps_bit_for_bit():
    """submit_step_host / collect_step keep one step in flight; losses, norms and the final state are those of
    train_step_host, and the in-flight limit and the empty collect are reported, not silently accepted."""
    from paper_2609_13645_b200 import binding as B
    ocfg, w = _c1()
    Bsz, S = w["batch"], w["seq"]
    batches = [SI.batch(ocfg.vocab, Bsz, S, "zipf", step=i) for i in range(5)]
    pinned = [(torch.from_numpy(t).pin_memory(), torch.from_numpy(l).pin_memory()) for t, l in batches]

    def run(pipelined):
        model = B.Model(lib_config(B, ocfg, Bsz, S), seed=3)
        out = []
        if not pipelined:
            for t, l in pinned:
                out.append(model.train_step_host(t.numpy(), l.numpy()))
        else:
            with pytest.raises(B.ForgeStepError) as ei:
                model.collect_step()
            assert ei.value.status == B.FT_ENOTFOUND
            for i, (t, l) in enumerate(pinned):
                model.submit_step_host(t.numpy(), l.numpy())
                if i > 0:
                    out.append(model.collect_step())
            out.append(model.collect_step())
            # the limit: two submits are accepted, the third is refused and enqueues nothing
            model.submit_step_host(pinned[0][0].numpy(), pinned[0][1].numpy())
            model.submit_step_host(pinned[1][0].numpy(), pinned[1][1].numpy())
            with pytest.raises(B.ForgeStepError) as ei:
                model.submit_step_host(pinned[2][0].numpy(), pinned[2][1].numpy())
            assert ei.value.status == B.FT_EINVAL
            model._pending.pop()
            extra = [model.collect_step(), model.collect_step()]
            assert all(np.isfinite(x[0]) for x in extra) and model.step == 7
            model.close()
            return out, None
        state = {n: model.get_param(n, B.KIND_MASTER) for n, _ in model.params}
        model.close()
        return out, state

    sync_out, sync_state = run(False)
    pipe_out, _ = run(True)
    assert sync_out == pipe_out
    # and the state after the same five pipelined steps
    model = B.Model(lib_config(B, ocfg, Bsz, S), seed=3)
    for t, l in pinned:
        model.submit_step_host(t.numpy(), l.numpy())
        model.collect_step()
    for n, _ in model.params:
        assert np.array_equal(model.get_param(n, B.KIND_MASTER), sync_state[n])
    model.close()


def test_error_paths_return_codes_and_keep_the_context_usable():
    from paper_2609_13645_b200 import binding as B
    ocfg, _ = _c1()
    model = B.Model(lib_config(B, ocfg, 2, 128), seed=1)
    tok, lab = SI.workload_batch("c1_tiny")
    big = to_dev(np.zeros((4, 128), dtype=np.int32))
    with pytest.raises(B.ForgeStepError) as e:
        model.train_step(big, big)
    assert e.value.status == B.FT_EINVAL
    with pytest.raises(B.ForgeStepError):
        model.get_tap("no_such_tap", 0)
    for bad in ((None, 0.0), (np.zeros(ocfg.head_dim // 2), 1.0), (-np.ones(ocfg.head_dim // 2), 1.0)):
        with pytest.raises(B.ForgeStepError) as e:
            model.set_rope_scaling(*bad)
        assert e.value.status == B.FT_EINVAL
    # a non-finite master makes the loss non-finite: reported, not fatal
    w = model.get_param("norm_f")
    w[0] = np.inf
    model.set_param("norm_f", w)
    with pytest.raises(B.ForgeStepError) as e:
        model.forward_loss(to_dev(tok), to_dev(lab))
    assert e.value.status == B.FT_ENONFINITE
    w[0] = 1.0
    model.set_param("norm_f", w)
    assert np.isfinite(model.forward_loss(to_dev(tok), to_dev(lab)))
    model.close()


def test_whole_step_graph_replay_is_bit_identical_to_plain_launches():
    from paper_2609_13645_b200 import binding as B
    ocfg, _ = _c1()
    params = D.init_params(ocfg, SI.WEIGHT_SEED)
    plain, l_plain = _run_steps(ocfg, params, 5)
    side = torch.cuda.Stream()  # the legacy default stream cannot be captured
    with torch.cuda.stream(side):
        graphed = B.Model(lib_config(B, ocfg, 2, 128), seed=1)
        load_params(graphed, params)
        graphed.set_graph(True)
        _, l_graph = _run_steps(ocfg, params, 5, model=graphed)
        side.synchronize()
        assert graphed.graph_replays >= 3  # step 1 plain, step 2 captured and replayed, steps 3..5 replayed
        assert np.array_equal(np.float32(l_plain).view(np.uint32), np.float32(l_graph).view(np.uint32))
        for a, b in zip(_state_bits(plain), _state_bits(graphed)):
            assert np.array_equal(a, b)
        assert graphed.step == 5
        graphed.close()
    plain.close()


@pytest.mark.parametrize("shape", ["c1", "gqa", "gqa_clip"])
def test_masters_after_a_step_with_warm_moments_meet_the_1e_3_bound(shape):
    """The stated bound on updated masters, rel-L2 <= 1e-3 per tensor, in the regime where it can hold: the state
    (masters, both moments, step counter) of five oracle steps is loaded into the library, both sides take one more step
    on the same fresh batch.  With warm moments the update is m_hat / (sqrt(v_hat) + eps), a smooth function of the
    gradient, so the bf16-level gradient differences (rho ~ 1e-3) move a master by ~ lr * 0.1 * rho, far below the bound.
    Also: gradients of that step within 2e-2, moments within 1e-3, and the step counter restored and advanced."""
    from paper_2609_13645_b200 import binding as B
    if shape == "c1":
        ocfg, w = _c1()
        Bsz, S, dist = w["batch"], w["seq"], "uniform"
    else:
        ocfg = _small_gqa()
        if shape == "gqa_clip":
            ocfg.max_grad_norm = parity_f32(0.5)
        Bsz, S, dist = 2, 200, "zipf"
    params = D.init_params(ocfg, 4321)
    st = D.TrainState(ocfg, params)
    for k in range(5):
        tok, lab = SI.batch(ocfg.vocab, Bsz, S, dist, seed=77, step=k)
        st.train_step(tok, lab)
    model = B.Model(lib_config(B, ocfg, Bsz, S), seed=1)
    model.set_fused_update(False)  # the gradients of the step are compared too
    for name in params:
        model.set_param(name, st.params[name], B.KIND_MASTER)
        model.set_param(name, st.m[name], B.KIND_ADAM_M)
        model.set_param(name, st.v[name], B.KIND_ADAM_V)
    model.step = st.step
    assert model.step == 5
    tok, lab = SI.batch(ocfg.vocab, Bsz, S, dist, seed=77, step=5)
    loss_o, gn_o, grads_o, _ = st.train_step(tok, lab)
    loss_g, gn_g = model.train_step(to_dev(tok), to_dev(lab))
    assert abs(loss_g - loss_o) < TOL_LOSS
    assert abs(gn_g - gn_o) / gn_o < 5e-3
    worst = {}
    for name in params:
        assert rel_l2(model.get_param(name, B.KIND_GRAD), grads_o[name]) < TOL_ACT, name
        e = rel_l2(model.get_param(name, B.KIND_MASTER), st.params[name])
        worst[name] = e
        assert e < TOL_MASTER, ("master", name, e)
        assert rel_l2(model.get_param(name, B.KIND_ADAM_M), st.m[name]) < 5e-3, ("m", name)
        assert rel_l2(model.get_param(name, B.KIND_ADAM_V), st.v[name]) < 5e-3, ("v", name)
    print("warm-moment master rel-L2, worst:", sorted(worst.items(), key=lambda kv: -kv[1])[:4])
    assert model.step == 6
    model.close()


def test_ten_step_loss_and_gradient_norm_trajectory_matches_oracle():
    """Ten consecutive steps on fresh batches: per-step loss within 1e-2, gradient norm within 1 %, and the masters
    after ten steps within 8e-3 (measured 6.8e-3 on the embedding table, 4e-3 on the projections: the cold first step's
    sign flips plus the drift of two bf16 trajectories, which Adam's normalisation keeps from piling up)."""
    from paper_2609_13645_b200 import binding as B
    ocfg = oracle_config(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=352, vocab=512)
    params = D.init_params(ocfg, 2024)
    st = D.TrainState(ocfg, params)
    model = B.Model(lib_config(B, ocfg, 2, 96), seed=1)
    load_params(model, params)
    for step in range(10):
        tok, lab = SI.batch(ocfg.vocab, 2, 96, "zipf", step=step)
        loss_o, gn_o, _, _ = st.train_step(tok, lab)
        loss_g, gn_g = model.train_step(to_dev(tok), to_dev(lab))
        assert abs(loss_g - loss_o) < TOL_LOSS, (step, loss_g, loss_o)
        assert abs(gn_g - gn_o) / gn_o < 1e-2, (step, gn_g, gn_o)
    assert model.step == 10
    worst = {}
    for name in params:
        e = rel_l2(model.get_param(name), st.params[name])
        worst[name] = e
        assert e < 8e-3, (name, e)
    print("ten-step master rel-L2, worst:", sorted(worst.items(), key=lambda kv: -kv[1])[:4])
    model.close()


@pytest.mark.parametrize("shape", ["c1", "split_k", "balanced", "tied_mup"])
def test_adamw_inside_the_weight_gradient_epilogue_equals_the_separate_optimizer_pass(shape):
    """Clipping is off, so the train step applies AdamW where the weight gradient is finished (GEMM epilogue, split-K
    reduction, or the epilogue that completes a tile divided along K).  Same update function, same gradient bits:
    parameters, moments, bf16 copies and losses must equal the unfused step bit for bit over several steps; the
    gradient norm is summed in another order and agrees to rounding."""
    from paper_2609_13645_b200 import binding as B
    if shape == "c1":
        ocfg, _ = _c1()
        Bsz, S = 2, 128
    elif shape == "tied_mup":  # the head's gradient joins the table's: it stays with the separate pass; factors in the epilogues
        ocfg = oracle_config(n_layers=2, d_model=512, n_heads=4, n_kv_heads=2, head_dim=128, d_ffn=1024, vocab=2048,
                             tie_embeddings=True, emb_scale=12.0, resid_scale=0.99, logit_scale=0.5, qk_norm=True)
        Bsz, S = 2, 1024
    elif shape == "split_k":   # weight gradients with few tiles and 2048 tokens: K split over 4 parts
        ocfg = oracle_config(n_layers=2, d_model=512, n_heads=4, n_kv_heads=2, head_dim=128, d_ffn=1024, vocab=2048)
        Bsz, S = 2, 1024
    else:                      # gate/up gradient of 18 x 5 = 90 tiles over 3072 tokens (48 K blocks): the 16 tiles past the 74 pairs are divided
        ocfg = oracle_config(n_layers=1, d_model=1280, n_heads=10, n_kv_heads=2, head_dim=128, d_ffn=2304, vocab=2048)
        Bsz, S = 3, 1024
    runs = []
    for fused in (True, False):
        model = B.Model(lib_config(B, ocfg, Bsz, S), seed=3)
        model.set_fused_update(fused)
        out = []
        for s in range(3):
            tok, lab = SI.batch(ocfg.vocab, Bsz, S, "uniform", step=s)
            out.append(model.train_step(to_dev(tok), to_dev(lab)))
        runs.append((model, out))
    (mf, lf), (mu, lu) = runs
    assert np.array_equal(np.float32([x[0] for x in lf]).view(np.uint32), np.float32([x[0] for x in lu]).view(np.uint32))
    for (_, gf), (_, gu) in zip(lf, lu):
        assert abs(gf - gu) <= 1e-5 * gu
    for a, b in zip(_state_bits(mf), _state_bits(mu)):
        assert np.array_equal(a, b)
    assert mf.step == 3 and mu.step == 3
    mf.close()
    mu.close()


@pytest.mark.parametrize("shape", ["c1", "ragged_ffn", "one_cta", "balanced", "mup_recompute"])
def test_swiglu_backward_inside_the_data_gradient_epilogue_changes_no_bit(shape):
    """By default the down projection's data-gradient GEMM never stores d_a: its epilogue rounds the accumulator to bf16,
    reads gate and up, and writes d_gate | d_up.  Same element function on the same rounded value as the separate
    elementwise pass, so losses, norms and the whole optimizer state must equal that path bit for bit.  Shapes: the
    CTA-pair kernel; an ffn width whose last 32-column chunk is half empty; few tokens (single-CTA kernel); a tile count
    that divides the last wave along K (partials completed before the epilogue); muP factors with recomputation.  The
    fused epilogue has two forms (gate / up and the result moved as TMA tiles through shared memory, or one row per thread
    with plain loads and stores): both are run."""
    from paper_2609_13645_b200 import binding as B
    kw, recompute = {}, 0
    if shape == "c1":
        ocfg, _ = _c1()
        Bsz, S = 2, 128
    elif shape == "ragged_ffn":
        ocfg = oracle_config(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024, max_grad_norm=0.5)
        Bsz, S = 3, 160
    elif shape == "one_cta":
        ocfg = oracle_config(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=1040, vocab=1024)
        Bsz, S = 1, 136
    elif shape == "balanced":  # 8 x 10 = 80 tiles of d_a on 74 pairs, contraction over d_model = 2560 (40 K blocks): the last 6 are divided along K
        ocfg = oracle_config(n_layers=1, d_model=2560, n_heads=20, n_kv_heads=4, head_dim=128, d_ffn=2560, vocab=2048)
        Bsz, S = 2, 1024
    else:
        ocfg = oracle_config(n_layers=3, d_model=512, n_heads=4, n_kv_heads=2, head_dim=128, d_ffn=1024, vocab=2048,
                             emb_scale=12.0, resid_scale=0.7, logit_scale=0.5, max_grad_norm=1.0)
        Bsz, S, recompute = 2, 512, 1
    runs = []
    # fused with the epilogue's tiles moved by TMA (the default), fused with one row per thread, separate pass
    for fused, tma in ((True, 1), (True, 0), (False, 1)):
        B.lib().ft_debug_gemm_swiglu_tma(tma)
        try:
            model = B.Model(lib_config(B, ocfg, Bsz, S, recompute=recompute), seed=9)
            model.set_fused_swiglu_bwd(fused)
            out = []
            for s in range(3):
                tok, lab = SI.batch(ocfg.vocab, Bsz, S, "zipf", step=s)
                out.append(model.train_step(to_dev(tok), to_dev(lab)))
        finally:
            B.lib().ft_debug_gemm_swiglu_tma(1)
        runs.append((model, out))
    (mf, lf), (mr, lr), (mu, lu) = runs
    assert lf == lu and lr == lu
    for a, b, c in zip(_state_bits(mf), _state_bits(mr), _state_bits(mu)):
        assert np.array_equal(a, c) and np.array_equal(b, c)
    mf.close()
    mr.close()
    mu.close()


@pytest.mark.parametrize("shape", ["gqa_ragged", "wide", "balanced_tail"])
def test_two_weight_gradients_in_one_launch_match_one_launch_each(shape):
    """A layer's weight gradients run as two grouped launches (down + gate/up projection, output + qkv projection): the
    second problem's tiles follow the first's in one persistent schedule.  Every whole tile is computed exactly as a launch
    of its own computes it; the tiles of the last wave that the balanced schedule divides along K, and outputs of few tiles,
    which a launch of their own splits along K, are summed in another order.  So against one launch per gradient: every
    gradient agrees to fp32 summation order (rel-L2 < 1e-5; measured up to 2.5e-6 over 3072 tokens); of three fused steps the first loss is identical and the later ones
    agree to 1e-3.  (Parity of the grouped path with the oracle is what every
    other test of this file checks, since it is the default.)"""
    from paper_2609_13645_b200 import binding as B
    if shape == "gqa_ragged":  # outputs of 256 x 688, 1376 x 256, 256 x 256, 512 x 256: ragged column tiles
        ocfg = oracle_config(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024)
        Bsz, S = 3, 160
    elif shape == "wide":
        ocfg = oracle_config(n_layers=2, d_model=512, n_heads=4, n_kv_heads=2, head_dim=128, d_ffn=1536, vocab=2048,
                             emb_scale=12.0, resid_scale=0.7, logit_scale=0.5)  # resid_scale: the two problems' factors differ
        Bsz, S = 2, 512
    else:  # 12 x 4 + 24 x 4 = 144 tiles on 74 pairs with 48 K blocks: the last 70 tiles stay whole, wave sizes differ from single launches
        ocfg = oracle_config(n_layers=1, d_model=1024, n_heads=8, n_kv_heads=8, head_dim=128, d_ffn=3072, vocab=2048)
        Bsz, S = 3, 1024
    grads, losses = [], []
    for group in (1, 0):
        B.lib().ft_debug_gemm_group(group)
        try:
            model = B.Model(lib_config(B, ocfg, Bsz, S), seed=11)
            tok, lab = SI.batch(ocfg.vocab, Bsz, S, "zipf", step=0)
            model.forward_backward(to_dev(tok), to_dev(lab))
            grads.append({n: model.get_param(n, B.KIND_GRAD).astype(np.float64) for n, _ in model.params})
            out = []
            for s in range(3):
                tok, lab = SI.batch(ocfg.vocab, Bsz, S, "zipf", step=s)
                out.append(model.train_step(to_dev(tok), to_dev(lab))[0])
            losses.append(out)
            model.close()
        finally:
            B.lib().ft_debug_gemm_group(1)
    for n in grads[0]:
        assert rel_l2(grads[0][n], grads[1][n]) < 1e-5, (n, rel_l2(grads[0][n], grads[1][n]))
    # the first loss precedes any update; later ones see bf16 weights that a last-bit difference in a gradient can move
    assert losses[0][0] == losses[1][0] and np.allclose(losses[0], losses[1], rtol=0, atol=1e-3), (losses[0], losses[1])


@pytest.mark.parametrize("recompute", [0, 1])
def test_weight_gradients_on_the_second_stream_change_no_bit(recompute):
    """The weight-gradient GEMMs run on a second stream, concurrent with the rest of the backward pass; events order
    them against the producers of their inputs and against later writers of the buffers they read (with recomputation
    all layers share one activation slot).  Three steps of a three-layer model must equal the single-stream run."""
    from paper_2609_13645_b200 import binding as B
    ocfg = oracle_config(n_layers=3, d_model=512, n_heads=4, n_kv_heads=2, head_dim=128, d_ffn=1024, vocab=2048)
    Bsz, S = 2, 512
    runs = []
    for overlap in (True, False):
        model = B.Model(lib_config(B, ocfg, Bsz, S, recompute=recompute), seed=5)
        model.set_overlap(overlap)
        out = []
        for s in range(3):
            tok, lab = SI.batch(ocfg.vocab, Bsz, S, "uniform", step=s)
            out.append(model.train_step(to_dev(tok), to_dev(lab)))
        runs.append((model, out))
    (mo, lo), (ms, ls) = runs
    assert lo == ls
    for a, b in zip(_state_bits(mo), _state_bits(ms)):
        assert np.array_equal(a, b)
    mo.close()
    ms.close()
