"""The data-parallel driver over the real library hooks on one GPU.

(1) A one-rank NCCL group: the reduce-scatter and the all-gather move nothing, so what is checked is the library side of
    the recipe (buckets that tile the arena in completion order, per-bucket events, AdamW applied range by range on a
    second stream, the label-count override, the norm from per-slice sums): without clipping the result must be the plain
    unfused train step bit for bit.
(2) The same path against the ORACLE at the stated tolerances, clipping on and off, from a state with warm moments.
(3) Two ranks with a SHARDED optimizer state (dp_world = 2), emulated as two host threads on the one GPU with the
    collectives done by hand (tests/local_ranks.py): each rank trains on its half of the batch, holds masters and moments
    only for its own slices, and after every step all ranks' bf16 copies and the assembled masters must match ONE oracle
    process that trained on the whole batch.
"""
import numpy as np
import pytest
import torch

import synth_inputs as SI
from oracle import decoder as D
from tests.local_ranks import run_ranks
from tests.parity_util import lib_config, oracle_config, rel_l2

pytestmark = pytest.mark.gpu
TOL_LOSS, TOL_GRAD, TOL_MASTER = 1e-2, 2e-2, 1e-3


@pytest.fixture(scope="module")
def one_rank_group():
    import torch.distributed as dist
    if not dist.is_initialized():
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29761", rank=0, world_size=1)
    yield dist
    dist.destroy_process_group()


def _cfg(clip=0.0, tied=False, qk_norm=False, mtp=False):
    return oracle_config(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024,
                         max_grad_norm=clip, tie_embeddings=tied, qk_norm=qk_norm, mtp=mtp, mtp_weight=0.4)


def _batches(ocfg, Bsz, S, n, first=0):
    out = []
    for i in range(first, first + n):
        t, l = SI.batch(ocfg.vocab, Bsz, S, "zipf", step=i)
        l = l.copy()
        l[0, :9] = -1
        out.append((t, l))
    return out


@pytest.mark.parametrize("tied,recompute,qk_norm,mtp", [(False, 0, False, False), (True, 0, False, False),
                                                        (False, 1, False, False), (True, 0, True, False),
                                                        (False, 0, False, True)])
def test_one_rank_data_parallel_steps_equal_plain_steps_bit_for_bit(one_rank_group, tied, recompute, qk_norm, mtp):
    from paper_2609_13645_b200 import binding as B
    from paper_2609_13645_b200.dp import DataParallel, LibraryBackend
    ocfg = _cfg(0.0, tied, qk_norm, mtp)
    Bsz, S = 2, 128
    batches = [(torch.from_numpy(t).cuda(), torch.from_numpy(l).cuda()) for t, l in _batches(ocfg, Bsz, S, 3)]
    plain = B.Model(lib_config(B, ocfg, Bsz, S, recompute=recompute), seed=11)
    plain.set_fused_update(False)
    ref = []
    for t, l in batches:
        loss = plain.forward_backward(t, l)
        ref.append((loss, plain.apply_update()))
    model = B.Model(lib_config(B, ocfg, Bsz, S, recompute=recompute), seed=11)
    be = LibraryBackend(model)
    dp = DataParallel(be)
    # the buckets tile the arena exactly once, in 128-element units
    spans = sorted(dp.buckets)
    assert spans[0][0] == 0 and all(a[0] + a[1] == b[0] for a, b in zip(spans, spans[1:]))
    assert spans[-1][0] + spans[-1][1] == be.grad().numel() and all(c % 128 == 0 for _, c in spans)
    assert len(dp.buckets) == ocfg.n_layers + (2 if tied else 3) + (1 if mtp else 0)
    got = [dp.step(t, l) for t, l in batches]
    torch.cuda.synchronize()
    for (l0, g0), (l1, g1) in zip(ref, got):
        assert l0 == l1
        assert abs(g0 - g1) <= 2e-6 * g0  # the norm is summed per slice
    for name, _ in model.params:
        for kind in (B.KIND_MASTER, B.KIND_ADAM_M, B.KIND_ADAM_V, B.KIND_BF16):
            assert np.array_equal(plain.get_param(name, kind), model.get_param(name, kind)), (name, kind)
    assert model.step == 3
    # and the ordinary step still works on the same model afterwards (the count override is only the driver's)
    model._check(B.lib().ft_dp_set_label_count_device(model._h, None))
    loss, _ = model.train_step(*batches[0])
    assert np.isfinite(loss)
    model.close(); plain.close()


def _warm_oracle(ocfg, Bsz, S, steps=5):
    params = D.init_params(ocfg, 4242)
    st = D.TrainState(ocfg, params)
    for t, l in _batches(ocfg, Bsz, S, steps):
        st.train_step(t, l)
    return st


def _load_state(B, setter, st):
    for name in st.params:
        setter(name, st.params[name], B.KIND_MASTER)
        setter(name, st.m[name], B.KIND_ADAM_M)
        setter(name, st.v[name], B.KIND_ADAM_V)


@pytest.mark.parametrize("clip,tied,mtp", [(0.0, False, False), (0.5, False, False), (0.5, True, True)])
def test_one_rank_data_parallel_steps_match_the_oracle(one_rank_group, clip, tied, mtp):
    """The data-parallel path against the oracle itself (not against the plain step): state with warm moments from five
    oracle steps, then two more steps on both sides.  Loss 1e-2, gradient norm, every updated master rel-L2 <= 1e-3,
    moments, and the bf16 copy equal to the rounded master."""
    from paper_2609_13645_b200 import binding as B
    from paper_2609_13645_b200.dp import DataParallel, LibraryBackend
    ocfg = _cfg(clip, tied, False, mtp)
    Bsz, S = 2, 128
    st = _warm_oracle(ocfg, Bsz, S)
    model = B.Model(lib_config(B, ocfg, Bsz, S), seed=11)
    _load_state(B, model.set_param, st)
    model.step = st.step
    dp = DataParallel(LibraryBackend(model))
    for t, l in _batches(ocfg, Bsz, S, 2, first=5):
        loss_o, gn_o, _, _ = st.train_step(t, l)
        loss_g, gn_g = dp.step(torch.from_numpy(t).cuda(), torch.from_numpy(l).cuda())
        assert abs(loss_g - loss_o) < TOL_LOSS
        assert abs(gn_g - gn_o) < 5e-3 * gn_o
        for name in st.params:
            p = model.get_param(name, B.KIND_MASTER)
            assert rel_l2(p, st.params[name]) < TOL_MASTER, ("master", name)
            assert rel_l2(model.get_param(name, B.KIND_ADAM_M), st.m[name]) < 5e-3, ("m", name)
            assert rel_l2(model.get_param(name, B.KIND_ADAM_V), st.v[name]) < 5e-3, ("v", name)
            assert np.array_equal(model.get_param(name, B.KIND_BF16), D.bf16_round(p).astype(np.float32)), name
    assert model.step == 7
    model.close()


@pytest.mark.parametrize("clip,tied,mtp,recompute", [(0.0, False, False, 0), (0.5, False, False, 1), (0.0, True, True, 0)])
def test_two_ranks_with_sharded_optimizer_state_match_one_oracle_on_the_whole_batch(clip, tied, mtp, recompute):
    from paper_2609_13645_b200 import binding as B
    from paper_2609_13645_b200.dp import DataParallel, LibraryBackend
    world, Bsz, S = 2, 2, 128
    ocfg = _cfg(clip, tied, False, mtp)
    st = _warm_oracle(ocfg, world * Bsz, S)
    whole = B.workspace_bytes(lib_config(B, ocfg, Bsz, S, recompute=recompute))
    part = B.workspace_bytes(lib_config(B, ocfg, Bsz, S, recompute=recompute, dp_world=world, dp_rank=1))
    n_state = sum(int(np.prod(v.shape)) for v in st.params.values())
    assert 0.45 * 12 * n_state < whole - part < 0.55 * 12 * n_state  # masters and moments: half of 12 bytes per parameter
    steps = _batches(ocfg, world * Bsz, S, 2, first=5)
    refs = []
    for t, l in steps:
        loss_o, gn_o, _, _ = st.train_step(t, l)
        refs.append((loss_o, gn_o, {k: v.copy() for k, v in st.params.items()}, {k: v.copy() for k, v in st.m.items()}))
    st0 = _warm_oracle(ocfg, world * Bsz, S)  # the warm state again, to load into the ranks

    def rank_main(rank, dist):
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            model = B.Model(lib_config(B, ocfg, Bsz, S, recompute=recompute, dp_world=world, dp_rank=rank), seed=11)
            with pytest.raises(B.ForgeStepError):  # a sharded model has no single-rank step
                model.train_step(torch.zeros(Bsz, S, dtype=torch.int32, device="cuda"), torch.zeros(Bsz, S, dtype=torch.int32, device="cuda"))
            dp = DataParallel(LibraryBackend(model), dist=dist)
            for name in st0.params:
                dp.set_state(name, st0.params[name], B.KIND_MASTER)
                dp.set_state(name, st0.m[name], B.KIND_ADAM_M)
                dp.set_state(name, st0.v[name], B.KIND_ADAM_V)
            model.step = st0.step
            out = []
            for (t, l), (loss_o, gn_o, p_o, m_o) in zip(steps, refs):
                lo, hi = rank * Bsz, (rank + 1) * Bsz
                loss, gn = dp.step(torch.from_numpy(t[lo:hi].copy()).cuda(), torch.from_numpy(l[lo:hi].copy()).cuda())
                masters = {n: dp.get_state(n, B.KIND_MASTER).cpu().numpy() for n in p_o}
                moments = {n: dp.get_state(n, B.KIND_ADAM_M).cpu().numpy() for n in p_o}
                copies = {n: model.get_param(n, B.KIND_BF16) for n in p_o}
                own = {n: model.get_param(n, B.KIND_MASTER) for n in p_o}
                out.append((loss, gn, masters, moments, copies, own))
            side.synchronize()
            model.close()
        return out

    res = run_ranks(world, rank_main)
    for k, (loss_o, gn_o, p_o, m_o) in enumerate(refs):
        for rank in range(world):
            loss, gn, masters, moments, copies, own = res[rank][k]
            assert abs(loss - loss_o) < TOL_LOSS and abs(gn - gn_o) < 5e-3 * gn_o
            for n in p_o:
                assert rel_l2(masters[n], p_o[n]) < TOL_MASTER, ("master", k, rank, n)
                assert rel_l2(moments[n], m_o[n]) < 5e-3, ("m", k, rank, n)
                # the all-gathered compute copy is the rounded assembled master, on every rank
                assert np.array_equal(copies[n], D.bf16_round(masters[n]).astype(np.float32)), (k, rank, n)
                # a rank returns its own elements and 0 elsewhere; the two ranks' parts tile the tensor
                mine = own[n] != 0
                assert np.array_equal(own[n][mine], masters[n][mine])
        a, b = res[0][k][5], res[1][k][5]
        for n in p_o:
            assert not np.any((a[n] != 0) & (b[n] != 0)), n
        assert res[0][k][0] == res[1][k][0] and res[0][k][1] == res[1][k][1]  # both ranks report the same loss and norm
