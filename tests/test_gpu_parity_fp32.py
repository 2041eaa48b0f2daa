"""GPU parity of the accurate (fp32 FFMA + fp64 refresh) path against the float64 oracle, through
the C-ABI.  Tolerances: per-step parameter update relative L2 <= 1e-4, bases (sign-normalised)
max-abs <= 1e-3, integer state bit-exact."""
from dataclasses import replace

import numpy as np
import pytest

from workloads import get_workload, LayerSpec, Workload
from workloads.configs import GEOM_BI, GEOM_NONE, GEOM_UNI, SRC_FIRST, SRC_SECOND

pytestmark = pytest.mark.gpu

TOL_DW, TOL_BASIS = 1e-4, 1e-3


def _run(w, calls, tau=-1, **kw):
    from tests.parity_util import SideBySide, basis_err, rel_l2
    import paper_2602_03515_b200 as br
    sbs = SideBySide(w, **kw)
    worst_dw, worst_q = 0.0, 0.0
    try:
        for c in range(calls):
            before = [lay.refresh_count for lay in sbs.oracle.layers]
            sbs.remember_bases()
            st_g, st_o, dg, do = sbs.step(tau)
            assert st_g == st_o or (st_g == br.BR_OK and st_o == 2), (c, st_g, st_o)
            for li, (a, b) in enumerate(zip(dg, do)):
                if b is None:
                    assert not np.any(a), "warm-up call changed the weights"
                    continue
                worst_dw = max(worst_dw, rel_l2(a, b))
            for li, lay in enumerate(sbs.oracle.layers):
                assert sbs.opt.counters(li) == sbs.oracle.counters(li)
                if lay.refresh_count != before[li] and st_o != 2:
                    # a refresh happened inside this call: bases and V~ against the oracle's, now
                    sbs.check_bases(li, TOL_BASIS, 1e-3, where=f"call {c + 1}, refresh {lay.refresh_count},", tensor_core=False)
        for li, lay in enumerate(sbs.oracle.layers):
            for which, ref in ((br.BR_BUF_U, lay.U), (br.BR_BUF_V, lay.V)):
                if ref is not None and lay.refresh_count > 0:
                    worst_q = max(worst_q, basis_err(sbs.state(li, which), ref))
            assert rel_l2(sbs.state(li, br.BR_BUF_M), lay.M) < 1e-5
            assert rel_l2(sbs.state(li, br.BR_BUF_V2), lay.V2) < 1e-3
            assert rel_l2(sbs.state(li, br.BR_BUF_W), lay.W) < 1e-5
            if lay.L is not None:
                assert rel_l2(sbs.state(li, br.BR_BUF_L), lay.L) < 1e-5
            if lay.R is not None:
                assert rel_l2(sbs.state(li, br.BR_BUF_R), lay.R) < 1e-5
        assert sbs.opt.sync_status() in (br.BR_OK, br.BR_WARN_RANK_DEFICIENT)
    finally:
        sbs.close()
    assert worst_dw <= TOL_DW, worst_dw
    assert worst_q <= TOL_BASIS, worst_q
    return worst_dw, worst_q


def test_c1_full_trajectory():
    """64x32 fp32, bilateral, S=2nd, tau=2, refresh every 5, 20 calls."""
    w = get_workload("c1")
    _run(w, w.calls, tau=2)


def test_small_matrix_update_is_a_single_launch():
    """A matrix with both dimensions <= 128 on the fp32 path is bound by launch latency: an update on which
    no refresh is due is one launch of the library (the refresh calls of C1, every fifth update, take the
    general path); parity of that kernel is what test_c1_full_trajectory and the strategy grid assert."""
    import torch
    import paper_2602_03515_b200 as br
    from workloads import GradientStream, initial_weight
    w = get_workload("c1")
    wt = torch.from_numpy(initial_weight(w, 0).copy()).cuda()
    opt = br.BasisRotation.from_workload(w, [wt])
    gs = GradientStream(w, 0)
    try:
        per_call = []
        for c in range(1, 9):
            n0, _ = opt.launch_stats()
            opt.step([torch.from_numpy(gs(c)).cuda()], 2)
            per_call.append(opt.launch_stats()[0] - n0)
        # calls 1-2: warm-up (no update); updates t = 1..6 at calls 3..8; t = 5 (call 7) refreshes
        assert per_call[:2] == [0, 0] and per_call[2:6] == [1, 1, 1, 1] and per_call[6] > 10 and per_call[7] == 1
        assert opt.sync_status() == br.BR_OK
    finally:
        opt.close()


def _small(geom, src, m, n, dtype="f32", kind="iid_normal", tau=1, freq=3, scale=0.05, **kw):
    return Workload("small", [LayerSpec("W", m, n, geom, src, tau)], dtype, kind, scale, 4, tau=tau,
                    freq=freq, calls=10, gemm_prec="f32", seed=3, **kw)


@pytest.mark.parametrize("geom,src", [(GEOM_BI, SRC_SECOND), (GEOM_BI, SRC_FIRST), (GEOM_UNI, SRC_SECOND),
                                      (GEOM_UNI, SRC_FIRST), (GEOM_NONE, SRC_SECOND)])
@pytest.mark.parametrize("m,n", [(37, 53), (96, 40), (130, 130)])
def test_strategy_grid_ragged_shapes(geom, src, m, n):
    # (bilateral S=1st on a rectangular matrix: M M^T or M^T M is rank-deficient on the larger side, and
    # the basis is completed from the previous one -- same rule in the oracle and in the library)
    _run(_small(geom, src, m, n), 10, tau=1)


def test_bf16_gradients_lowrank_fp32_gemm():
    # noise 0.5 against a rank-4 signal: the first refresh then has min_j R_jj/|a_j| ~ 4e-3, so the
    # fp32 rounding of the stored factors (1e-7 relative) stays below the 1e-4 update tolerance.
    # (With noise 0.05 the same quantity is 4e-5 and fp32 factor state alone costs ~5e-4.)
    w = _small(GEOM_BI, SRC_SECOND, 72, 104, dtype="bf16", kind="lowrank_noise", tau=2, freq=4, scale=0.5)
    _run(w, 12, tau=2)


def test_weight_decay_and_on_refresh_accumulation():
    # The literal placement of the accumulation inside the refresh feeds only every freq-th
    # gradient into the factor, so the first refresh sees a single G G^T: a wide unilateral layer
    # (24 x 96, left factor) keeps that factor full rank and well conditioned.
    w = _small(GEOM_UNI, SRC_SECOND, 24, 96, tau=0, freq=2, weight_decay=0.1)
    _run(w, 8, tau=0, accum="on_refresh")


def test_global_norm_clipping_mixed_layers_and_delays():
    """Clipping threshold well below the joint gradient norm, rotated and plain layers, per-layer
    delays: each update must use the factor of the call its gradient was submitted with."""
    layers = [LayerSpec("a", 40, 56, GEOM_BI, SRC_SECOND, 2), LayerSpec("b", 24, 64, GEOM_UNI, SRC_FIRST, 1),
              LayerSpec("c", 20, 20, GEOM_NONE, SRC_SECOND, 0)]
    w = Workload("clip", layers, "f32", "iid_normal", 0.05, tau=2, freq=3, calls=12, gemm_prec="f32", seed=15)
    _run(w, 12, tau=-1, clip_norm=0.5)


def test_power_iters_2():
    _run(_small(GEOM_BI, SRC_SECOND, 40, 56, tau=0, freq=3), 7, tau=0, power_iters=2)


def test_multi_layer_per_layer_tau_and_freq():
    layers = [LayerSpec("a", 33, 65, GEOM_BI, SRC_SECOND, 3, 2), LayerSpec("b", 64, 16, GEOM_UNI, SRC_SECOND, 1, 3),
              LayerSpec("c", 20, 20, GEOM_NONE, SRC_SECOND, 0, 0), LayerSpec("d", 24, 80, GEOM_UNI, SRC_FIRST, 2, 0)]
    w = Workload("multi", layers, "f32", "iid_normal", 0.02, tau=3, freq=4, calls=12, gemm_prec="f32", seed=5)
    _run(w, 12, tau=-1)


def test_variable_tau_per_call():
    from tests.parity_util import SideBySide, rel_l2
    w = _small(GEOM_BI, SRC_SECOND, 32, 48, tau=3, freq=3)
    sbs = SideBySide(w)
    try:
        for tau in (3, 3, 3, 3, 1, 2, 0, 3, 2):
            st_g, st_o, dg, do = sbs.step(tau)
            assert st_g == st_o
            if do[0] is not None:
                assert rel_l2(dg[0], do[0]) < TOL_DW
            assert sbs.opt.counters(0) == sbs.oracle.counters(0)
    finally:
        sbs.close()


def test_qr_many_panels_teacher_forced():
    """Forced refresh from a given L, U (set through the API) against the oracle's Power():
    k = 200 spans 4 panels of 64 columns with a ragged last one; the factor has a 1e4 spread of
    eigenvalues."""
    import torch
    import paper_2602_03515_b200 as br
    from oracle import br_oracle as O
    from tests.parity_util import basis_err
    k, n = 200, 16
    rng = np.random.default_rng(11)
    Qe, _ = np.linalg.qr(rng.standard_normal((k, k)))
    lam = np.logspace(0, -4, k)
    F = ((Qe * lam) @ Qe.T).astype(np.float32)
    U0, _ = np.linalg.qr(rng.standard_normal((k, k)))
    U0 = U0.astype(np.float32)
    w = torch.zeros(k, n, device="cuda")
    spec = LayerSpec("W", k, n, GEOM_UNI, SRC_SECOND, 0)
    spec = replace(spec, geom=GEOM_BI)
    opt = br.BasisRotation([spec], [w], grad_dtype="f32", gemm_prec=br.BR_GEMM_FP32, freq=1000)
    try:
        g = torch.randn(k, n, device="cuda") * 0.01
        assert opt.step([g], 0) == br.BR_OK          # t = 1 so that a forced refresh is allowed
        opt.set_state(0, br.BR_BUF_L, torch.from_numpy(F))
        opt.set_state(0, br.BR_BUF_U, torch.from_numpy(U0))
        opt.refresh_basis(0)
        assert opt.sync_status() == br.BR_OK
        U = opt.get_state(0, br.BR_BUF_U).numpy().astype(np.float64)
        ref, deficient = O.power(F.astype(np.float64), U0.astype(np.float64))
        assert not deficient
        assert np.max(np.abs(U.T @ U - np.eye(k))) < 1e-5
        assert basis_err(U, ref) < 1e-5
        assert opt.counters(0)["refresh_count"] == 1 and opt.counters(0)["t"] == 1
    finally:
        opt.close()


@pytest.mark.parametrize("start", ["identity", "tracking"])
def test_qr_wide_panels_split_contractions(start):
    """k = 1160: nine 128-column panels and a ragged 8-column one, contractions split over K.
    "identity": Power(F, I) for a factor with a 1e5 spread of eigenvalues, the ill-conditioned
    first refresh (every column of F is dominated by the leading eigenvectors; both Cholesky-QR
    passes run).  "tracking": the basis already holds approximate eigenvectors, so the columns of
    F Q are nearly orthogonal and the second pass is cancelled by the device-side flag."""
    import torch
    import paper_2602_03515_b200 as br
    from oracle import br_oracle as O
    from tests.parity_util import basis_err
    k, n = 1160, 8
    rng = np.random.default_rng(5)
    Qe, _ = np.linalg.qr(rng.standard_normal((k, k)))
    lam = np.logspace(0, -5, k)
    F = ((Qe * lam) @ Qe.T).astype(np.float32)
    if start == "identity":
        U0 = np.eye(k, dtype=np.float32)
    else:
        pert, _ = np.linalg.qr(np.eye(k) + 1e-3 * rng.standard_normal((k, k)))
        U0 = (Qe @ pert).astype(np.float32)
    w = torch.zeros(k, n, device="cuda")
    opt = br.BasisRotation([LayerSpec("W", k, n, GEOM_BI, SRC_SECOND, 0)], [w], grad_dtype="f32",
                           gemm_prec=br.BR_GEMM_FP32, freq=1000)
    try:
        assert opt.step([torch.randn(k, n, device="cuda") * 0.01], 0) == br.BR_OK
        opt.set_state(0, br.BR_BUF_L, torch.from_numpy(F))
        opt.set_state(0, br.BR_BUF_U, torch.from_numpy(U0))
        opt.refresh_basis(0)
        assert opt.sync_status() == br.BR_OK
        U = opt.get_state(0, br.BR_BUF_U).numpy().astype(np.float64)
        ref, deficient = O.power(F.astype(np.float64), U0.astype(np.float64))
        assert not deficient
        assert np.max(np.abs(U.T @ U - np.eye(k))) < 1e-5
        assert basis_err(U, ref) < 1e-5
    finally:
        opt.close()


def test_host_side_errors_leave_handle_usable():
    import torch
    import paper_2602_03515_b200 as br
    w = torch.zeros(16, 8, device="cuda")
    opt = br.BasisRotation([LayerSpec("W", 16, 8, GEOM_BI, SRC_SECOND, 2)], [w], grad_dtype="f32",
                           gemm_prec=br.BR_GEMM_FP32)
    try:
        g = torch.randn(16, 8, device="cuda")
        with pytest.raises(br.BrError) as e:
            opt.step([g], 5)
        assert e.value.status == br.BR_ERR_TAU
        with pytest.raises(br.BrError) as e:
            opt.refresh_basis(0)
        assert e.value.status == br.BR_ERR_STATE
        with pytest.raises(br.BrError) as e:
            br.br_step(opt.handle, [0], 0)
        assert e.value.status == br.BR_ERR_INVALID
        assert opt.counters(0)["calls"] == 0
        assert opt.step([g], 2) == br.BR_WARMUP
        assert opt.counters(0) == dict(calls=1, t=0, ring_slot=1, refresh_count=0, next_refresh_t=10)
    finally:
        opt.close()


def test_checkpoint_resume_bit_identical():
    """run 9 calls == run 5, save, destroy, create, load, run 4 (all buffers and counters)."""
    import torch
    import paper_2602_03515_b200 as br
    from workloads import GradientStream, initial_weight
    w = _small(GEOM_BI, SRC_SECOND, 40, 24, tau=2, freq=3)
    gs = GradientStream(w, 0)
    bufs = [br.BR_BUF_W, br.BR_BUF_M, br.BR_BUF_V2, br.BR_BUF_U, br.BR_BUF_V, br.BR_BUF_L, br.BR_BUF_R, br.BR_BUF_RING]

    def fresh():
        wt = torch.from_numpy(initial_weight(w, 0).copy()).cuda()
        return wt, br.BasisRotation.from_workload(w, [wt], gemm_prec=br.BR_GEMM_FP32)

    wt, a = fresh()
    for c in range(1, 10):
        a.step([torch.from_numpy(gs(c)).cuda()], 2)
    final = {b: a.get_state(0, b).clone() for b in bufs}
    ca = a.counters(0)
    a.close()
    wt, b1 = fresh()
    for c in range(1, 6):
        b1.step([torch.from_numpy(gs(c)).cuda()], 2)
    saved = {b: b1.get_state(0, b).clone() for b in bufs}
    cnt = b1.counters(0)
    b1.close()
    wt, b2 = fresh()
    for b in bufs:
        b2.set_state(0, b, saved[b])
    br.br_set_counters(b2.handle, 0, cnt["calls"], cnt["t"], cnt["refresh_count"])
    for c in range(6, 10):
        b2.step([torch.from_numpy(gs(c)).cuda()], 2)
    assert b2.counters(0) == ca
    for b in bufs:
        assert torch.equal(b2.get_state(0, b), final[b]), b
    b2.close()


def test_closed_loop_quadratic_against_oracle_and_the_papers_claim():
    """Closed loop: the gradient of f(W) = 1/2 tr(W^T P W Q) is computed from the library's own
    current weights at every call and applied two calls later.  The loss trajectory follows the
    oracle's own closed loop, and the paper's toy claim holds on the GPU path too: rotation on the
    misaligned problem ends as low as plain Adam on the aligned one, plain Adam on the misaligned
    problem far higher."""
    import torch
    import paper_2602_03515_b200 as br
    from oracle import br_oracle as O
    from workloads.closed_loop import kronecker_quadratic, loss
    tau, steps = 2, 300

    def gpu_run(geom, aligned):
        P, Q, W0 = kronecker_quadratic(aligned=aligned)
        Pd, Qd = torch.from_numpy(P).float().cuda(), torch.from_numpy(Q).float().cuda()
        w = torch.from_numpy(W0).float().cuda().contiguous()
        opt = br.BasisRotation([LayerSpec("W", 32, 16, geom, SRC_SECOND, tau)], [w], grad_dtype="f32", lr=0.02,
                               beta1=0.0, beta2=0.9, eps=1e-12, freq=5, gemm_prec=br.BR_GEMM_FP32)
        lay = O.OracleLayer(W0.astype(np.float32).astype(np.float64), geom, O.SRC_SECOND, tau)
        f32 = lambda x: float(np.float32(x))
        orc = O.Oracle([lay], O.Hyper(lr=f32(0.02), beta1=0.0, beta2=f32(0.9), eps=f32(1e-12), freq=5))
        worst = 0.0
        try:
            for c in range(steps):
                opt.step([(Pd @ w @ Qd).contiguous()], tau)
                orc.step([P @ lay.W @ Q], tau)
                # parity while the problem is well posed: over the first 100 calls the loss falls by three
                # orders of magnitude.  Later the gradients are confined to a few directions and the factors
                # are rank-deficient up to the rounding of their storage only: the float64 oracle then meets
                # pivots below 1e-12 and completes the basis, while the same factor stored in fp32 has full
                # rank at the 6e-8 level and is factorised as it stands (an exactly deficient factor is
                # completed by both, see test_numerically_rank_deficient_refresh_...).  The two closed loops
                # then differ in directions that carry next to no loss (18 % of a loss 1e-4 of the initial one
                # after 300 calls).
                if c in (24, 49, 74, 99):
                    lg, lo = loss(P, Q, w.double().cpu().numpy()), loss(P, Q, lay.W)
                    worst = max(worst, abs(lg - lo) / lo)
            # (late in the run the gradients are confined to a few directions: the factor may be
            # numerically rank-deficient, which the library reports)
            assert opt.sync_status() in (br.BR_OK, br.BR_WARN_RANK_DEFICIENT)
            return loss(P, Q, w.double().cpu().numpy()), worst
        finally:
            opt.close()

    aligned, e1 = gpu_run(GEOM_NONE, True)
    misaligned, e2 = gpu_run(GEOM_NONE, False)
    rotated, e3 = gpu_run(GEOM_BI, False)
    assert max(e1, e2, e3) < 5e-2, (e1, e2, e3)          # closed loops amplify rounding: loss within 5 %
    assert misaligned > 5.0 * aligned and rotated < 2.0 * aligned


def test_closed_loop_spiral_plain_adam_through_the_ring():
    """The spiral loss of Sec. 2.2 / App. D.1 in closed loop: two parameters, geometry none (Eq. (adam)),
    learning rate 0.1, beta1 = 0, beta2 = 0.9; the gradient is computed from the library's own current
    weights at every call, and from call 40 on it is applied one call late (tau = 1, through the ring).
    The iterates follow the oracle's own closed loop while rounding has not been amplified yet (a
    float64 emulation with fp32 weights and moments separates from the float64 run by 1e-4 within 60
    steps of this oscillating trajectory and by 4e-4 within 100), and the oscillation statistics agree
    afterwards."""
    import torch
    import paper_2602_03515_b200 as br
    from oracle import br_oracle as O
    from workloads.closed_loop import spiral_grad, spiral_valley_excess
    steps, delay_from = 500, 40
    for p0 in ([8.0, 0.0], [5.0, 5.0]):
        w = torch.tensor([p0], dtype=torch.float32, device="cuda")
        opt = br.BasisRotation([LayerSpec("p", 1, 2, GEOM_NONE, SRC_SECOND, 1)], [w], grad_dtype="f32", lr=0.1, beta1=0.0,
                               beta2=0.9, eps=1e-8, gemm_prec=br.BR_GEMM_FP32)
        f32 = lambda x: float(np.float32(x))
        lay = O.OracleLayer(np.array([p0], dtype=np.float64), O.GEOM_NONE, O.SRC_SECOND, 1)
        orc = O.Oracle([lay], O.Hyper(lr=f32(0.1), beta1=0.0, beta2=f32(0.9), eps=f32(1e-8), freq=10))
        ex_g, ex_o = [], []
        try:
            for c in range(steps):
                tau = 0 if c < delay_from else 1
                pg = w.double().cpu().numpy()[0]
                g = torch.from_numpy(spiral_grad(pg)[None, :].astype(np.float32)).cuda()
                assert opt.step([g], tau) == br.BR_OK
                orc.step([spiral_grad(lay.W[0])[None, :]], tau)
                assert opt.counters(0) == orc.counters(0)
                if c < 60:
                    assert np.max(np.abs(w.double().cpu().numpy()[0] - lay.W[0])) < 1e-3, c
                if c >= 100:
                    ex_g.append(spiral_valley_excess(w.double().cpu().numpy()[0]))
                    ex_o.append(spiral_valley_excess(lay.W[0]))
            assert opt.sync_status() == br.BR_OK
        finally:
            opt.close()
        assert abs(np.mean(ex_g) / np.mean(ex_o) - 1.0) < 0.1, (np.mean(ex_g), np.mean(ex_o))


@pytest.mark.parametrize("path,m,n", [("fp32", 64, 48), ("bf16", 264, 136)])
def test_numerically_rank_deficient_refresh_is_completed_in_the_same_call(path, m, n):
    """Gradients confined to rank-4 row and column spaces (no noise): L and R have exactly rank 4, which
    the host cannot know beforehand (the factors have seen enough gradients to be full rank).  The
    library finds it in the factorisation itself, with the oracle's criterion (some |R_jj| <= 1e-12 of
    the largest), and factorises the completed product F Q + 1e-6 ||(F Q)_j|| Q_j in the same refresh:
    BR_WARN_RANK_DEFICIENT is there after the very call in which the oracle reports it, the bases are
    orthonormal, and they agree with the oracle's in every column (the completed product has full
    rank, so its Q factor is unique).  Entries are small integers times a power of two and the
    factor EMA runs with rate 1/2, so that the stored fp32 factors are exact: a factor that is
    rank-deficient only up to its own fp32 rounding (6e-8) is, for the 1e-12 criterion, a full-rank one."""
    import paper_2602_03515_b200 as br
    from tests.parity_util import SideBySide, basis_err, rel_l2
    tc = path == "bf16"
    w = Workload("rank4", [LayerSpec("W", m, n, GEOM_BI, SRC_SECOND, 0)], "bf16" if tc else "f32", "integer_subspace",
                 2.0 ** -6, 4, tau=0, freq=3, calls=5, gemm_prec="bf16" if tc else "f32", seed=23)
    sbs = SideBySide(w, beta_factor=0.5)
    try:
        seen = 0
        for c in range(5):
            sbs.remember_bases()
            st_g, st_o, dg, do = sbs.step(0)
            assert st_g == br.BR_OK
            word = sbs.opt.sync_status()                     # the status word of this very call
            assert word == (br.BR_WARN_RANK_DEFICIENT if st_o == 2 else br.BR_OK), (c, word, st_o)
            lay = sbs.oracle.layers[0]
            if st_o == 2:
                seen += 1
                for which, ref, k in ((br.BR_BUF_U, lay.U, m), (br.BR_BUF_V, lay.V, n)):
                    q = sbs.state(0, which)
                    assert np.max(np.abs(q.T @ q - np.eye(k))) < 1e-5
                    assert basis_err(q[:, :4], ref[:, :4]) < 1e-5            # the range of the factor
                    assert basis_err(q, ref) < 1e-3                          # and the completed columns
                assert br.br_get_basis_flags(sbs.opt.handle, 0) & 12 == 12
            assert rel_l2(dg[0], do[0]) <= (2e-2 if tc else 1e-4), (c, rel_l2(dg[0], do[0]))
            assert sbs.opt.counters(0) == sbs.oracle.counters(0)
        assert seen == 1
    finally:
        sbs.close()
