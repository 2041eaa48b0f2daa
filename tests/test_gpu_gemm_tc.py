"""The tcgen05 tile kernel alone, through br_gemm_bf16, against a float64 contraction of the same
bf16 inputs (products of bf16 values are exact in fp32, so only the accumulation order differs)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _operand(rng, rows, K, mn_major, torch):
    """Returns (device tensor as stored, float64 matrix of logical shape rows x K)."""
    x = torch.from_numpy(rng.standard_normal((rows, K)).astype(np.float32)).to(torch.bfloat16)
    logical = x.double().numpy()
    stored = x.t().contiguous() if mn_major else x.contiguous()
    return stored.cuda(), logical


@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (1, 1), (0, 1), (1, 0)])
@pytest.mark.parametrize("Md,Nd,K", [(128, 256, 64), (256, 512, 256), (200, 328, 136), (8, 8, 8), (1024, 1024, 1000)])
def test_single_pair_all_majors(a_mn, b_mn, Md, Nd, K):
    import torch
    import paper_2602_03515_b200 as br
    rng = np.random.default_rng(Md * 7 + Nd * 3 + K + a_mn * 2 + b_mn)
    A, Ar = _operand(rng, Md, K, a_mn, torch)
    B, Br = _operand(rng, Nd, K, b_mn, torch)
    D = torch.full((Md, Nd), float("nan"), device="cuda")
    lda = Md if a_mn else K
    ldb = Nd if b_mn else K
    br.br_gemm_bf16(0, Md, Nd, K, [A.data_ptr()], [B.data_ptr()], a_mn, b_mn, lda, ldb, D.data_ptr(), Nd, 1.0, 0.0)
    ref = Ar @ Br.T
    got = D.cpu().double().numpy()
    assert np.all(np.isfinite(got))
    assert np.max(np.abs(got - ref)) <= 1e-5 * np.sqrt(K) * max(1.0, np.max(np.abs(ref)))


def test_three_pairs_and_axpby():
    import torch
    import paper_2602_03515_b200 as br
    rng = np.random.default_rng(5)
    Md, Nd, K = 384, 264, 520
    As, Bs, ref = [], [], np.zeros((Md, Nd))
    keep = []
    for p in range(3):
        A, Ar = _operand(rng, Md, K, 1, torch)
        B, Br = _operand(rng, Nd, K, 1, torch)
        keep += [A, B]
        As.append(A.data_ptr()); Bs.append(B.data_ptr())
        ref += Ar @ Br.T
    D0 = torch.randn(Md, Nd, device="cuda")
    D = D0.clone()
    br.br_gemm_bf16(0, Md, Nd, K, As, Bs, 1, 1, Md, Nd, D.data_ptr(), Nd, 0.25, -1.5)
    want = 0.25 * ref - 1.5 * D0.cpu().double().numpy()
    assert np.max(np.abs(D.cpu().double().numpy() - want)) <= 2e-5 * np.sqrt(3 * K) * np.max(np.abs(want))


def test_many_tiles_persistent_loop():
    """More tiles than CTAs, ragged in both directions: exercises the stage ring and the two
    accumulators across tile boundaries."""
    import torch
    import paper_2602_03515_b200 as br
    rng = np.random.default_rng(9)
    Md, Nd, K = 3080, 2824, 192          # 25 x 12 = 300 tiles
    A, Ar = _operand(rng, Md, K, 0, torch)
    B, Br = _operand(rng, Nd, K, 1, torch)
    D = torch.zeros(Md, Nd, device="cuda")
    br.br_gemm_bf16(0, Md, Nd, K, [A.data_ptr()], [B.data_ptr()], 0, 1, K, Nd, D.data_ptr(), Nd, 1.0, 0.0)
    ref = Ar @ Br.T
    assert np.max(np.abs(D.cpu().double().numpy() - ref)) <= 1e-5 * np.sqrt(K) * np.max(np.abs(ref))


def test_rejects_bad_arguments():
    import torch
    import paper_2602_03515_b200 as br
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    d = torch.zeros(64, 64, device="cuda")
    with pytest.raises(br.BrError):
        br.br_gemm_bf16(0, 60, 64, 64, [x.data_ptr()], [x.data_ptr()], 0, 0, 64, 64, d.data_ptr(), 64)


@pytest.mark.parametrize("Md,Nd,K,a_mn,b_mn", [(8192 + 72, 520, 4096, 0, 1), (6000, 6000, 3592, 1, 0)])
def test_tile_walks_with_partial_groups(Md, Nd, K, a_mn, b_mn):
    """Shapes whose operand panels exceed the share of L2 a tile group may take, so that the walk
    is cut into several groups (the last one partial): a tall result with a small second operand is
    walked in groups of column-blocks, a large square one in groups of row-blocks.  Checked on sampled
    rows (all columns) against a float64 contraction."""
    import torch
    import paper_2602_03515_b200 as br
    rng = np.random.default_rng(Md + Nd + K)
    A, Ar = _operand(rng, Md, K, a_mn, torch)
    B, Br = _operand(rng, Nd, K, b_mn, torch)
    D = torch.full((Md, Nd), float("nan"), device="cuda")
    lda = Md if a_mn else K
    ldb = Nd if b_mn else K
    br.br_gemm_bf16(0, Md, Nd, K, [A.data_ptr()], [B.data_ptr()], a_mn, b_mn, lda, ldb, D.data_ptr(), Nd, 1.0, 0.0)
    assert bool(torch.isfinite(D).all())
    rows = np.unique(np.concatenate([np.arange(0, Md, 97), np.arange(Md - 8, Md), np.arange(248, 264)]))
    ref = Ar[rows] @ Br.T
    got = D[torch.from_numpy(rows).cuda()].cpu().double().numpy()
    assert np.max(np.abs(got - ref)) <= 1e-5 * np.sqrt(K) * np.max(np.abs(ref))
