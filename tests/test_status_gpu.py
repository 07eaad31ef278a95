"""Device-side problems are reported as status codes and leave the context usable: a bounded wait that runs out, token
ids or labels outside the vocabulary.  Nothing here faults, traps or hangs: the wait that runs out is a 2-millisecond
wait on a barrier that nothing signals, made by a probe kernel with the library's own bounded-wait routine."""
import ctypes as C

import numpy as np
import pytest
import torch

import synth_inputs as SI
from tests.parity_util import lib_config, oracle_config, to_dev

pytestmark = pytest.mark.gpu


def _model(B):
    w = SI.WORKLOADS["c1_tiny"]
    ocfg = oracle_config(**{k: w[k] for k in SI.MODEL_KEYS})
    return B.Model(lib_config(B, ocfg, w["batch"], w["seq"]), seed=SI.WEIGHT_SEED), ocfg


def _wait_probe(B, model, cycles):
    L = B.lib()
    L.ft_debug_wait_probe.argtypes = [C.c_void_p, C.c_int64]
    L.ft_debug_wait_probe.restype = C.c_int
    return L.ft_debug_wait_probe(model._h, cycles)


def test_a_wait_that_runs_out_is_reported_once_and_the_model_keeps_working():
    from paper_2609_13645_b200 import binding as B
    model, _ = _model(B)
    ref, _ = _model(B)
    tok, lab = SI.workload_batch("c1_tiny")
    tok_d, lab_d = to_dev(tok), to_dev(lab)
    first = model.train_step(tok_d, lab_d)
    assert first == ref.train_step(tok_d, lab_d)
    assert _wait_probe(B, model, 0) == B.FT_EINVAL          # limits outside [1, 2e7] cycles are refused
    assert _wait_probe(B, model, 10 ** 9) == B.FT_EINVAL
    assert _wait_probe(B, model, 4_000_000) == B.FT_OK       # about 2 ms of SM clocks
    # the step after the probe runs normally, and its synchronising read reports the wait that ran out
    with pytest.raises(B.ForgeStepError) as e:
        model.train_step(tok_d, lab_d)
    assert e.value.status == B.FT_ETIMEOUT
    ref.train_step(tok_d, lab_d)
    # reported once; the context and the model are intact: the following step equals the undisturbed model's, bit for bit
    third = model.train_step(tok_d, lab_d)
    assert third == ref.train_step(tok_d, lab_d)
    for name, _ in model.params:
        assert np.array_equal(model.get_param(name).view(np.uint32), ref.get_param(name).view(np.uint32)), name
    # the pipelined entry reports it the same way
    pinned = (torch.from_numpy(tok).pin_memory(), torch.from_numpy(lab).pin_memory())
    assert _wait_probe(B, model, 1_000_000) == B.FT_OK
    model.submit_step_host(pinned[0].numpy(), pinned[1].numpy())
    with pytest.raises(B.ForgeStepError) as e:
        model.collect_step()
    assert e.value.status == B.FT_ETIMEOUT
    model.submit_step_host(pinned[0].numpy(), pinned[1].numpy())
    loss, _ = model.collect_step()
    assert np.isfinite(loss)
    torch.cuda.synchronize()
    model.close()
    ref.close()


def test_ids_outside_the_vocabulary_are_reported_and_do_not_count():
    from paper_2609_13645_b200 import binding as B
    model, ocfg = _model(B)
    tok, lab = SI.workload_batch("c1_tiny")
    good = model.forward_loss(to_dev(tok), to_dev(lab))
    # a label >= vocab: FT_EINVAL; it is ignored by the loss AND by the count, like a negative label
    lab_bad = lab.copy()
    lab_bad[0, 3] = ocfg.vocab + 5
    with pytest.raises(B.ForgeStepError) as e:
        model.forward_loss(to_dev(tok), to_dev(lab_bad))
    assert e.value.status == B.FT_EINVAL
    lab_ign = lab.copy()
    lab_ign[0, 3] = -1
    ign = model.forward_loss(to_dev(tok), to_dev(lab_ign))
    # the loss value of the flagged call is that of the batch with the label ignored
    tok_d, lab_bad_d = to_dev(tok), to_dev(lab_bad)
    loss = C.c_float()
    st = B.lib().ft_forward_loss(model._h, C.c_void_p(tok_d.data_ptr()), C.c_void_p(lab_bad_d.data_ptr()), 2, 128, C.byref(loss))
    assert st == B.FT_EINVAL and np.float32(loss.value) == np.float32(ign) and ign != good
    # a token id out of range (negative, or >= vocab): reported; the context stays usable
    for bad_id in (-7, ocfg.vocab):
        tok_bad = tok.copy()
        tok_bad[1, 100] = bad_id
        with pytest.raises(B.ForgeStepError) as e:
            model.train_step(to_dev(tok_bad), to_dev(lab))
        assert e.value.status == B.FT_EINVAL
    assert np.isfinite(model.train_step(to_dev(tok), to_dev(lab))[0])
    model.close()


def test_single_kernel_status_word_reads_clean_after_attention_calls():
    from paper_2609_13645_b200 import binding as B
    L = B.lib()
    L.ft_k_status.argtypes = [C.c_void_p]
    L.ft_k_status.restype = C.c_int
    Bsz, S, nh, nkv, d = 1, 256, 4, 2, 64
    qkv = (torch.randn(Bsz * S, (nh + 2 * nkv) * d, device="cuda") * 0.5).to(torch.bfloat16)
    o = torch.empty(Bsz * S, nh * d, device="cuda", dtype=torch.bfloat16)
    lse = torch.empty(Bsz, nh, S, device="cuda", dtype=torch.float32)
    B.k_attention_fwd(qkv, o, lse, Bsz, S, nh, nkv, d)
    assert L.ft_k_status(C.c_void_p(torch.cuda.current_stream().cuda_stream)) == B.FT_OK
    assert torch.isfinite(lse).all()
