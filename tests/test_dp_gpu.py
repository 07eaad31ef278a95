"""The data-parallel driver over the real library hooks on one GPU: a one-rank NCCL group.

With one rank the reduce-scatter and the all-gather move nothing, so what is checked is the library side of the
recipe: buckets that tile the arena in completion order, per-bucket events, AdamW applied range by range on a second
stream, the label-count override, the norm from per-slice sums.  The result must be the plain (unfused) train step:
bit for bit in losses, masters, moments and compute copy; the norm agrees to rounding (it is summed per slice).
"""
import numpy as np
import pytest
import torch

import synth_inputs as SI
from tests.parity_util import lib_config, oracle_config, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def one_rank_group():
    import torch.distributed as dist
    if not dist.is_initialized():
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29761", rank=0, world_size=1)
    yield dist
    dist.destroy_process_group()


@pytest.mark.parametrize("clip,tied,recompute,qk_norm,mtp", [(0.0, False, 0, False, False), (0.5, False, 0, False, False),
                                                             (0.0, True, 0, False, False), (0.0, False, 1, False, False),
                                                             (0.0, True, 0, True, False), (0.0, False, 0, False, True),
                                                             (0.5, True, 0, False, True)])
def test_one_rank_data_parallel_steps_equal_plain_steps(one_rank_group, clip, tied, recompute, qk_norm, mtp):
    from paper_2609_13645_b200 import binding as B
    from paper_2609_13645_b200.dp import DataParallel, LibraryBackend
    ocfg = oracle_config(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024,
                         max_grad_norm=clip, tie_embeddings=tied, qk_norm=qk_norm, mtp=mtp, mtp_weight=0.4)
    Bsz, S = 2, 128
    batches = []
    for i in range(3):
        t, l = SI.batch(ocfg.vocab, Bsz, S, "zipf", step=i)
        l = l.copy(); l[0, :9] = -1
        batches.append((torch.from_numpy(t).cuda(), torch.from_numpy(l).cuda()))

    plain = B.Model(lib_config(B, ocfg, Bsz, S, recompute=recompute), seed=11)
    plain.set_fused_update(False)
    ref = []
    for t, l in batches:
        loss = plain.forward_backward(t, l)
        gn = plain.apply_update()
        ref.append((loss, gn))

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
    for i, ((l0, g0), (l1, g1)) in enumerate(zip(ref, got)):
        if clip > 0 and i > 0:
            # after a clipped update the two runs hold parameters that differ in last bits (see below), and so do
            # their next losses and norms
            assert abs(l0 - l1) <= 1e-5 * abs(l0) and abs(g0 - g1) <= 1e-4 * g0
        else:
            assert l0 == l1
            assert abs(g0 - g1) <= 2e-6 * g0
    for name, _ in model.params:
        for kind in (B.KIND_MASTER, B.KIND_ADAM_M, B.KIND_ADAM_V, B.KIND_BF16):
            a, b = plain.get_param(name, kind), model.get_param(name, kind)
            if clip > 0:
                # The coefficient comes from a norm summed in another order and differs in its last bits.  Moments follow
                # to rounding; a master moves by lr * g / (|g| + eps)-like terms, which turn that last bit into a visible
                # fraction of one update where |g| is of the order of eps (rows of the table few tokens touch).
                # From the second step on the two runs hold parameters that differ in such last bits, and a bf16 step
                # amplifies that to its rounding noise floor: the moments then agree to about 1e-3 (measured up to 1.1e-3 on
                # a gain whose gradient is a sum of cancelling terms), not to 1e-7.  A wrong slice or a missed update is O(1).
                if kind in (B.KIND_ADAM_M, B.KIND_ADAM_V):
                    assert rel_l2(b, a) < 5e-3, (name, kind)
                else:
                    # measured up to 0.08 lr per step on elements whose gradient is tiny; a skipped or doubled update of
                    # one step is a whole lr (|m / sqrt(v)| is about 1 in the first steps)
                    tol = 0.2 * ocfg.lr * len(batches)
                    if kind == B.KIND_BF16:  # a master that moved by less than that can still cross a bf16 boundary: one ulp
                        tol = max(tol, 2.0 ** -7 * float(np.max(np.abs(a))))  # a bf16 ulp is up to 2^-7 of the value
                    assert np.max(np.abs(a - b)) <= tol, (name, kind)
            else:
                assert np.array_equal(a, b), (name, kind)
    assert model.step == 3
    # and the ordinary step still works on the same model afterwards (the count override is only the driver's)
    model._check(B.lib().ft_dp_set_label_count_device(model._h, None))
    loss, _ = model.train_step(*batches[0])
    assert np.isfinite(loss)
    model.close(); plain.close()
