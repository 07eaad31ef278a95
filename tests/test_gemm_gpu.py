"""tcgen05 GEMM family against the fp64 contraction of the same bf16 inputs (through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import decoder as D

pytestmark = pytest.mark.gpu


def _bf16_tensor(rng, shape, scale=1.0):
    a = D.bf16_round(rng.standard_normal(shape) * scale)
    return a, torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).cuda()


def _run(M, N, K, a_mn, b_mn, out_kind, seed=0, ws=False):
    from paper_2609_13645_b200 import binding as B
    rng = np.random.default_rng(seed)
    A, At = _bf16_tensor(rng, (K, M) if a_mn else (M, K))
    Bm, Bt = _bf16_tensor(rng, (K, N) if b_mn else (N, K))
    ref = (A.T if a_mn else A) @ (Bm if b_mn else Bm.T)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    resid = None
    if out_kind in (0, 1):
        out = torch.full((M, N), 7.0, dtype=torch.bfloat16, device="cuda")
        if out_kind == 1:
            R_, resid = _bf16_tensor(rng, (M, N))
            ref = ref + R_
        ref = D.bf16_round(ref)
    else:
        out = torch.full((M, N), 0.5, dtype=torch.float32, device="cuda")
        if out_kind == 3:
            ref = ref + 0.5
    if ws:
        scratch = torch.full((5 << 20,), float("nan"), dtype=torch.float32, device="cuda")
        B.k_gemm_ws(At, a_mn, Bt, b_mn, out, out_kind, M, N, K, scratch, err, resid)
    else:
        B.k_gemm(At, a_mn, Bt, b_mn, out, out_kind, M, N, K, err, resid)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    got = out.float().cpu().numpy().astype(np.float64)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    return rel, got, ref


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (256, 256, 256), (384, 768, 320), (200, 136, 72), (1000, 1376, 256),
                                   (256, 256, 688)])
def test_forward_layout_bf16_out(M, N, K):
    rel, got, ref = _run(M, N, K, 0, 0, 0)
    assert rel < 2e-3, rel
    # apart from roundings that flip at a tie, every element is the correctly rounded fp64 result
    assert np.mean(got != ref) < 0.02
    assert np.max(np.abs(got - ref) / (np.abs(ref) + 1e-3)) < 2.0 ** -6


@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (200, 136, 1376), (512, 688, 256)])
def test_data_gradient_layout(M, N, K):
    rel, got, ref = _run(M, N, K, 0, 1, 0)
    assert rel < 2e-3, rel
    assert np.mean(got != ref) < 0.02


@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (768, 256, 200), (256, 688, 1000), (1376, 256, 264)])
def test_weight_gradient_layout_fp32_out(M, N, K):
    rel, got, ref = _run(M, N, K, 1, 1, 2)
    assert rel < 1e-5, rel


def test_fp32_accumulate_and_residual_epilogues():
    rel, _, _ = _run(256, 384, 192, 1, 1, 3)
    assert rel < 1e-5, rel
    rel, got, ref = _run(300, 256, 128, 0, 0, 1)
    assert rel < 2e-3 and np.mean(got != ref) < 0.02
    rel, _, _ = _run(256, 1024, 256, 0, 0, 2)
    assert rel < 1e-5


def test_large_tile_variant_many_tiles():
    # enough 128x256 tiles to fill every SM: the wide-tile kernel with its double-buffered accumulator
    rel, got, ref = _run(2048, 4096, 512, 0, 0, 0, seed=3)
    assert rel < 2e-3 and np.mean(got != ref) < 0.02
    rel, _, _ = _run(4096, 2048, 384, 1, 1, 2, seed=4)
    assert rel < 1e-5
    rel, got, ref = _run(2048, 4096, 520, 0, 1, 0, seed=5)
    assert rel < 2e-3


def test_bad_arguments_are_rejected_without_launching():
    from paper_2609_13645_b200 import binding as B
    a = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    c = torch.zeros(128, 128, dtype=torch.bfloat16, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.ForgeStepError):
        B.k_gemm(a, 0, a, 0, c, 0, 128, 124, 64, err)  # N not a multiple of 8
    with pytest.raises(B.ForgeStepError):
        B.k_gemm(a, 1, a, 0, c, 0, 64, 128, 128, err)  # mn-major A with k-major B is not offered


@pytest.mark.parametrize("M,N,K,acc", [(768, 768, 8192, False), (512, 256, 4096, True), (1000, 520, 2056, True),
                                       (256, 256, 1024, False), (768, 2304, 8192, False), (256, 256, 960, True)])
def test_split_k_weight_gradient_matches_the_contraction_and_repeats_bit_for_bit(M, N, K, acc):
    """Few output tiles, long K: the K range is divided over concurrent CTA pairs and the parts are added in a
    fixed order.  Checked against the fp64 contraction, against run-to-run bit identity, and (ragged K, ragged
    tiles) against the padding rules of the single-pass kernel."""
    from paper_2609_13645_b200 import binding as B
    rng = np.random.default_rng(11)
    A, At = _bf16_tensor(rng, (K, M))
    Bm, Bt = _bf16_tensor(rng, (K, N))
    ref = A.T @ Bm + (0.5 if acc else 0.0)
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    scratch = torch.full((256 + 8 * M * N,), float("nan"), dtype=torch.float32, device="cuda")
    outs = []
    for _ in range(2):
        out = torch.full((M, N), 0.5, dtype=torch.float32, device="cuda")
        B.k_gemm_ws(At, 1, Bt, 1, out, 3 if acc else 2, M, N, K, scratch, err)
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        outs.append(out.cpu().numpy())
    assert np.array_equal(outs[0], outs[1])
    got = outs[0].astype(np.float64)
    assert np.all(np.isfinite(got))
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 1e-5
    # a scratch buffer too small for two parts falls back to the single-pass kernel and still gives the result
    out = torch.full((M, N), 0.5, dtype=torch.float32, device="cuda")
    B.k_gemm_ws(At, 1, Bt, 1, out, 3 if acc else 2, M, N, K, scratch[:M * N], err)
    torch.cuda.synchronize()
    got1 = out.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got1 - ref) / np.linalg.norm(ref) < 1e-5


# Shapes with more 256 x 256 tiles than the 74 SM pairs, a last wave of at most 37 tiles and a contraction of at least 40
# K blocks (K >= 2560): the balanced schedule divides that wave into 2 .. 8 K parts.  Ragged M, N and K (parts of unequal
# length) included; the last two shapes stay below the K limit and take the plain schedule with the same scratch.
BALANCED = [(2048, 2560, 2560), (2048, 2560, 4096), (4096, 4096, 2600), (2000, 2568, 3000), (8192, 2048, 2816),
            (2304, 2304, 6144), (2560, 2560, 8192), (2048, 2560, 1024), (8192, 2048, 704)]


@pytest.mark.parametrize("M,N,K", BALANCED)
@pytest.mark.parametrize("a_mn,b_mn,kind", [(0, 0, 0), (0, 1, 0), (1, 1, 2), (1, 1, 3), (0, 0, 1)])
def test_balanced_k_schedule_matches_the_contraction(M, N, K, a_mn, b_mn, kind):
    rel, got, ref = _run(M, N, K, a_mn, b_mn, kind, seed=21, ws=True)
    assert np.all(np.isfinite(got))
    if kind >= 2:
        assert rel < 1e-5, rel
    else:
        assert rel < 2e-3 and np.mean(got != ref) < 0.02
        # one bf16 rounding of a sum whose fp32 accumulation error is far below the typical magnitude sqrt(K)
        assert np.all(np.abs(got - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-2)


def test_balanced_k_schedule_repeats_bit_for_bit_and_leaves_its_counters_clear():
    from paper_2609_13645_b200 import binding as B
    M, N, K = 2048, 2560, 4096
    rng = np.random.default_rng(5)
    _, At = _bf16_tensor(rng, (M, K))
    _, Bt = _bf16_tensor(rng, (N, K))
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    scratch = torch.full((5 << 20,), float("nan"), dtype=torch.float32, device="cuda")
    outs = []
    for _ in range(3):
        out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        B.k_gemm_ws(At, 0, Bt, 0, out, 0, M, N, K, scratch, err)
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        assert int(scratch[:256].view(torch.int32).abs().sum().item()) == 0
        outs.append(out.view(torch.int16).cpu().numpy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


@pytest.mark.parametrize("M,N,K,a_mn,b_mn,ws", [(1000, 1376, 256, 0, 0, False), (300, 328, 128, 0, 0, False),
                                                 (2048, 4096, 512, 0, 0, False), (512, 688, 256, 0, 1, False),
                                                 (8192, 2560, 2560, 0, 1, True), (4096, 768, 768, 0, 1, False)])
def test_bf16_output_through_tensor_stores_changes_no_bit(M, N, K, a_mn, b_mn, ws):
    """The plain bf16 epilogue of the CTA-pair kernel has two forms: tiles of 32 rows x 64 columns packed in shared memory
    and sent off as TMA tensor stores (default), or one row per thread with 32-byte stores.  Same accumulators, same
    rounding: the outputs must be equal bit for bit, ragged rows and columns, a balanced (K-divided) last wave and a
    short contraction included."""
    from paper_2609_13645_b200 import binding as B
    outs = []
    for on in (1, 0):
        B.lib().ft_debug_gemm_tma_out(on)
        try:
            rel, got, _ = _run(M, N, K, a_mn, b_mn, 0, seed=5, ws=ws)
        finally:
            B.lib().ft_debug_gemm_tma_out(1)
        assert rel < 2e-3, rel
        outs.append(got)
    assert np.array_equal(outs[0], outs[1])
