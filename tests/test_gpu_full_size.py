"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration the
benchmark times (tensor-core path, grouped launches over several layers, gradients read through
the delay ring).

Free-running trajectories with refreshes inside them are in tests/test_gpu_free_running.py; here the
step and the refresh are checked separately, at the largest shapes:

* step: the bases are set to seeded random orthogonal matrices on both sides (teacher-forced), the
  delayed step runs for two updates, and the whole weight change, the momentum and the second moment
  are compared with the oracle element by element (tolerance of the bf16 tensor-core path, 2e-2);
* refresh: a forced refresh from given factors is compared with the oracle's Power() at orders
  1024, 2560, 4224 and 6912 (the largest of the benchmark), and there also against the properties
  that define the result at any size: Q^T Q = I, and R = Q^T (F Q0) upper triangular with a positive
  diagonal (checked on sampled columns in float64).
"""
from dataclasses import replace

import numpy as np
import pytest

from workloads import LayerSpec, Workload, get_workload
from workloads.configs import GEOM_BI, GEOM_UNI, SRC_SECOND

pytestmark = pytest.mark.gpu

TOL_DW = 2e-2
# Factors: bf16 gradients are exact operands, the error is the fp32 accumulation in the tensor cores
# (one rounding toward zero per 16-deep slice): on the diagonal, a sum of up to 32000 squares, that is a
# one-sided error of about (32000 / 16) x 2^-24 = 1.2e-4 of the sum; 3e-4 leaves a factor of 2.5.
TOL_FACTOR = 3e-4


def _orthogonal(k, seed):
    rng = np.random.default_rng(seed)
    q, r = np.linalg.qr(rng.standard_normal((k, k)))
    return (q * np.sign(np.diag(r))).astype(np.float32)


def _teacher_forced_steps(w, updates=2):
    import paper_2602_03515_b200 as br
    from tests.parity_util import SideBySide, rel_l2
    sbs = SideBySide(w, gemm_prec=br.BR_GEMM_BF16)
    try:
        import torch
        for li, lay in enumerate(sbs.oracle.layers):
            if lay.U is not None:
                q = _orthogonal(lay.U.shape[0], 100 + li)
                lay.U = q.astype(np.float64)
                sbs.opt.set_state(li, br.BR_BUF_U, torch.from_numpy(q))
            if lay.V is not None:
                q = _orthogonal(lay.V.shape[0], 200 + li)
                lay.V = q.astype(np.float64)
                sbs.opt.set_state(li, br.BR_BUF_V, torch.from_numpy(q))
        done = 0
        while done < updates:
            st_g, st_o, dg, do = sbs.step(w.tau)
            assert st_g == st_o
            for li, (a, b) in enumerate(zip(dg, do)):
                if b is None:
                    assert not np.any(a)
                    continue
                e = rel_l2(a, b)
                assert e <= TOL_DW, (li, e)
            done += 0 if do[0] is None else 1
            for li in range(len(w.layers)):
                assert sbs.opt.counters(li) == sbs.oracle.counters(li)
        assert sbs.opt.sync_status() == br.BR_OK
        for li, lay in enumerate(sbs.oracle.layers):
            assert rel_l2(sbs.state(li, br.BR_BUF_V2), lay.V2) < 2e-2
            assert rel_l2(sbs.state(li, br.BR_BUF_M), lay.M) < 1e-3
            if lay.L is not None:
                assert rel_l2(sbs.state(li, br.BR_BUF_L), lay.L) < TOL_FACTOR
            if lay.R is not None:
                assert rel_l2(sbs.state(li, br.BR_BUF_R), lay.R) < TOL_FACTOR
    finally:
        sbs.close()


def test_c2_full_size_block_teacher_forced_bases():
    """The four matrices of the d_model = 1024, ffn = 4096 block (1024x3072, 1024x1024, 1024x4096,
    4096x1024), bilateral, bf16 low-rank-plus-noise gradients, one grouped launch per phase."""
    w = replace(get_workload("c2"), tau=1, freq=10 ** 6)
    w = replace(w, layers=[replace(l, tau_max=1) for l in w.layers])
    _teacher_forced_steps(w, updates=2)


def test_c5_shapes_full_size_teacher_forced_bases():
    """One matrix of each distinct shape of the ~3B layer set: 2560x2560, 2560x6912, 6912x2560
    bilateral and the 32000x2560 embedding (unilateral, right factor), rank-32 signal + 0.05 noise."""
    layers = [LayerSpec("wq", 2560, 2560, GEOM_BI, SRC_SECOND, 1), LayerSpec("wup", 2560, 6912, GEOM_BI, SRC_SECOND, 1),
              LayerSpec("wdown", 6912, 2560, GEOM_BI, SRC_SECOND, 1), LayerSpec("emb", 32000, 2560, GEOM_UNI, SRC_SECOND, 1)]
    base = get_workload("c5", n_layers=1, tau=1)
    w = replace(base, layers=layers, tau=1, freq=10 ** 6)
    _teacher_forced_steps(w, updates=1)


def _forced_refresh(k, F, Q0):
    import torch
    import paper_2602_03515_b200 as br
    w = torch.zeros(k, 8, device="cuda")
    opt = br.BasisRotation([LayerSpec("W", k, 8, GEOM_BI, SRC_SECOND, 0)], [w], grad_dtype="bf16",
                           gemm_prec=br.BR_GEMM_BF16, freq=10 ** 6)
    try:
        assert opt.step([(torch.randn(k, 8, device="cuda") * 0.01).to(torch.bfloat16)], 0) == br.BR_OK
        opt.set_state(0, br.BR_BUF_L, torch.from_numpy(F))
        opt.set_state(0, br.BR_BUF_U, torch.from_numpy(Q0))
        opt.refresh_basis(0)
        assert opt.sync_status() == br.BR_OK
        return opt.get_state(0, br.BR_BUF_U).numpy().astype(np.float64)
    finally:
        opt.close()


def _lowrank_noise_factor(k, rank, seed, samples=3):
    """EMA-like factor of a rank-`rank` signal plus 0.05 noise stream: sum of a few G G^T."""
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((k, rank))
    F = np.zeros((k, k))
    n = 256
    B = rng.standard_normal((n, rank))
    for _ in range(samples * (k // n + 1)):
        G = A @ B.T + 0.05 * rng.standard_normal((k, n))
        F += G @ G.T
    return (F / np.abs(F).max()).astype(np.float32)


def test_refresh_order_1024_against_oracle_power():
    from oracle import br_oracle as O
    from tests.parity_util import basis_err
    k = 1024
    F = _lowrank_noise_factor(k, 16, 31)
    Q0 = np.eye(k, dtype=np.float32)
    U = _forced_refresh(k, F, Q0)
    ref, deficient = O.power(F.astype(np.float64), Q0.astype(np.float64))
    assert not deficient
    assert basis_err(U, ref) < 1e-3
    assert np.max(np.abs(U.T @ U - np.eye(k))) < 1e-5


@pytest.mark.parametrize("k", [4224, 2560])
def test_refresh_tensor_core_projections(k):
    """Third refresh of a basis of order 4224 / 2560 in one handle (orders from 2048 use the tensor-core
    forms: deflated power product, block projections with at least 2^18 coefficients).  The first (from U = I) is ill-conditioned, the second runs in fp64 and notes that
    no column shrank much, so the third runs its large block projections on the tensor cores
    (three-term bf16 splits, applied twice).  Compared with the oracle's Power(F, U2): at order 2560 in
    its written-out Householder form (about a minute of interpreted loops), at order 4224 -- where that
    form would take some five minutes -- with the library QR routine as the step (`qr_pos_lapack`, pinned
    against the written-out form at small orders)."""
    import torch
    import paper_2602_03515_b200 as br
    from oracle import br_oracle as O
    from tests.parity_util import basis_err
    F = _lowrank_noise_factor(k, 16, 33, samples=3)      # 13,000 noise samples: the noise part is well conditioned
    w = torch.zeros(k, 8, device="cuda")
    opt = br.BasisRotation([LayerSpec("W", k, 8, GEOM_BI, SRC_SECOND, 0)], [w], grad_dtype="bf16",
                           gemm_prec=br.BR_GEMM_BF16, freq=10 ** 6)
    try:
        assert opt.step([(torch.randn(k, 8, device="cuda") * 0.01).to(torch.bfloat16)], 0) == br.BR_OK
        opt.set_state(0, br.BR_BUF_L, torch.from_numpy(F))
        opt.refresh_basis(0)
        assert br.br_get_basis_flags(opt.handle, 0) & 1 == 0       # from the identity: columns shrink by 1e4
        opt.refresh_basis(0)
        assert br.br_get_basis_flags(opt.handle, 0) & 1 == 1       # tracking
        U2 = opt.get_state(0, br.BR_BUF_U).numpy()
        opt.refresh_basis(0)                                        # large block projections on the tensor cores
        assert opt.sync_status() == br.BR_OK
        U3 = opt.get_state(0, br.BR_BUF_U).numpy().astype(np.float64)
        ref, deficient = O.power(F.astype(np.float64), U2.astype(np.float64),
                                 qr=O.qr_pos if k <= 2560 else O.qr_pos_lapack)
        assert not deficient
        assert basis_err(U3, ref) < 1e-5
        assert np.max(np.abs(U3.T @ U3 - np.eye(k))) < 1e-5
    finally:
        opt.close()


def test_refresh_order_6912_against_oracle_power_and_properties():
    """The largest order of the ~3B layer set.  First refresh from U = I (ill-conditioned: columns lose
    up to 1e-5 of their length), second from the first one's result (the basis tracks the factor).  Both
    are compared with the oracle's Power() (library QR routine as its step at this order), and with the
    properties that define the result whatever computes it, on sampled columns in float64: Q^T Q = I and
    R = Q^T (F Q0) upper triangular with a positive diagonal."""
    from oracle import br_oracle as O
    from tests.parity_util import basis_err
    k = 6912
    F = _lowrank_noise_factor(k, 32, 32, samples=2)      # 14,000 noise samples for order 6912: full rank with margin
    Q0 = np.eye(k, dtype=np.float32)
    U1 = _forced_refresh(k, F, Q0)                      # ill-conditioned first refresh
    U1f = U1.astype(np.float32)
    U2 = _forced_refresh(k, F, U1f)                     # second refresh: the basis tracks the factor
    rng = np.random.default_rng(0)
    cols = np.unique(np.concatenate([np.arange(64), np.arange(k - 64, k), rng.integers(0, k, 384)]))
    F64 = F.astype(np.float64)
    for Qin, U, tol in ((Q0.astype(np.float64), U1, 1e-3), (U1f.astype(np.float64), U2, 1e-5)):
        assert np.all(np.isfinite(U))
        ref, deficient = O.power(F64, Qin, qr=O.qr_pos_lapack)
        assert not deficient
        assert basis_err(U, ref) < tol, basis_err(U, ref)
        assert np.max(np.abs(U.T @ U[:, cols] - np.eye(k)[:, cols])) < 1e-5
        A = F64 @ Qin[:, cols]                           # sampled columns of F Q0
        R = U.T @ A                                      # column j of R: zero below row cols[j], positive there
        scale = np.linalg.norm(A, axis=0)
        below = np.arange(k)[:, None] > cols[None, :]
        assert np.max(np.abs(R * below) / scale[None, :]) < 1e-5
        assert np.all(R[cols, np.arange(len(cols))] > 0)


def test_c3_full_size_block_unilateral_first_moment():
    """The block of C3 at full size: unilateral rotation of the smaller side (left for 1024x3072,
    1024x1024, 1024x4096; right for 4096x1024), S = 1st, teacher-forced bases, two updates."""
    w = replace(get_workload("c3"), tau=1, freq=10 ** 6)
    w = replace(w, layers=[replace(l, tau_max=1) for l in w.layers])
    _teacher_forced_steps(w, updates=2)


def test_c4_shapes_full_size_student_t_gradients():
    """One matrix of each distinct shape of C4 (d_model 2048, ffn 5632, embedding 32000x2048 unilateral)
    with the heavy-tailed gradients of that configuration (1e-3 x Student-t, 3 degrees of freedom)."""
    layers = [LayerSpec("wq", 2048, 2048, GEOM_BI, SRC_SECOND, 1), LayerSpec("wup", 2048, 5632, GEOM_BI, SRC_SECOND, 1),
              LayerSpec("wdown", 5632, 2048, GEOM_BI, SRC_SECOND, 1), LayerSpec("emb", 32000, 2048, GEOM_UNI, SRC_SECOND, 1)]
    base = get_workload("c4", n_layers=1, tau=1)
    w = replace(base, layers=layers, tau=1, freq=10 ** 6)
    _teacher_forced_steps(w, updates=1)
