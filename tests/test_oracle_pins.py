"""Pins of the float64 oracle against what the paper and the mathematics fix.

Each test is chosen so that a plausible slip in the oracle (a dropped term, a
transposed operand, a wrong index or sign) fails at least one of them.
"""
import numpy as np
import pytest

from oracle import br_oracle as O


def rng(seed):
    return np.random.default_rng(seed)


def rand_orth(k, seed):
    q, r = np.linalg.qr(rng(seed).standard_normal((k, k)))
    return q * np.sign(np.diag(r))[None, :]


def run(layer_kwargs, hp, grads, tau=-1, W0=None):
    m, n = grads[0].shape
    W0 = np.zeros((m, n)) if W0 is None else W0
    lay = O.OracleLayer(W0, **layer_kwargs)
    orc = O.Oracle([lay], hp)
    dws = []
    for g in grads:
        orc.step([g], tau)
        dws.append(None if lay.last_dW is None else lay.last_dW.copy())
    return orc, lay, dws


# P1 -- Q^T Q = I to 1e-10 after every refresh, both factors (Sec. 3.2, Power = matmul + QR)
@pytest.mark.parametrize("geom,src", [(O.GEOM_BI, O.SRC_SECOND), (O.GEOM_BI, O.SRC_FIRST),
                                      (O.GEOM_UNI, O.SRC_SECOND), (O.GEOM_UNI, O.SRC_FIRST)])
def test_p1_orthonormal_after_every_refresh(geom, src):
    r = rng(1)
    m, n = 24, 40
    lay = O.OracleLayer(np.zeros((m, n)), geom=geom, src=src, tau_max=0)
    orc = O.Oracle([lay], O.Hyper(freq=3))
    for c in range(12):
        orc.step([r.standard_normal((m, n))], 0)
        for Q in (lay.U, lay.V):
            if Q is not None:
                assert np.max(np.abs(Q.T @ Q - np.eye(Q.shape[0]))) < 1e-10
    assert lay.refresh_count == 4


# P2 -- with U = V = I the step is exactly Eq. (adam): eps inside the sqrt, no bias correction
def test_p2_identity_basis_is_plain_adam_bit_exact():
    r = rng(2)
    m, n, T = 7, 5, 9
    grads = [r.standard_normal((m, n)) for _ in range(T)]
    W0 = r.standard_normal((m, n))
    hp = O.Hyper(lr=3e-3, beta1=0.8, beta2=0.95, eps=1e-6, freq=10 ** 6)
    _, lay, _ = run(dict(geom=O.GEOM_BI, src=O.SRC_SECOND), hp, grads, 0, W0)
    # independently written Adam (scalar loops)
    w, mm, vv = W0.copy(), np.zeros((m, n)), np.zeros((m, n))
    for g in grads:
        for i in range(m):
            for j in range(n):
                mm[i, j] = 0.8 * mm[i, j] + (1 - 0.8) * g[i, j]
                vv[i, j] = 0.95 * vv[i, j] + (1 - 0.95) * g[i, j] * g[i, j]
                w[i, j] = w[i, j] + (-3e-3 * mm[i, j] / np.sqrt(vv[i, j] + 1e-6))
    assert np.array_equal(lay.W, w)
    assert np.array_equal(lay.M, mm) and np.array_equal(lay.V2, vv)
    # geometry NONE takes the plain-Adam branch and must agree too
    _, lay0, _ = run(dict(geom=O.GEOM_NONE), hp, grads, 0, W0)
    assert np.array_equal(lay0.W, w)


def test_p2_closed_form_constant_gradient():
    # constant g: m_t = (1-b1^t) g, v_t = (1-b2^t) g^2 -> closed-form update
    g = np.array([[0.5, -2.0], [1.5, 0.25]])
    hp = O.Hyper(lr=0.1, beta1=0.9, beta2=0.99, eps=0.0, freq=10 ** 6)
    _, lay, dws = run(dict(geom=O.GEOM_NONE), hp, [g] * 6, 0)
    for t, dw in enumerate(dws, start=1):
        expect = -0.1 * (1 - 0.9 ** t) * g / np.sqrt((1 - 0.99 ** t) * g * g)
        assert np.allclose(dw, expect, rtol=1e-13, atol=0)


# P3 -- basis-aligned (diagonal) problem: the coordinate basis is recovered (Sec. 2.2 / 3.1)
def test_p3_diagonal_factors_recover_coordinate_basis():
    m, n = 6, 4
    d1 = np.array([3.0, 2.5, 2.0, 1.5, 1.0, 0.5])
    d2 = np.array([2.0, 1.5, 1.0, 0.5])
    grads = []
    for c in range(12):
        P = np.zeros((m, n))
        for j in range(n):
            P[(j + c) % m, j] = 1.0          # sub-permutation: G G^T and G^T G are diagonal
        grads.append(d1[:, None] * P * d2[None, :])
    hp = O.Hyper(freq=6)
    _, lay, dws = run(dict(geom=O.GEOM_BI, src=O.SRC_SECOND), hp, grads, 0)
    assert lay.refresh_count == 2
    assert np.array_equal(lay.U, np.eye(m)) and np.array_equal(lay.V, np.eye(n))
    _, lay0, dws0 = run(dict(geom=O.GEOM_NONE), hp, grads, 0)
    assert np.allclose(lay.W, lay0.W, rtol=0, atol=1e-15)


def test_p3_stochastic_diagonal_covariance():
    # G = D1 Z D2 with iid Z: E[G G^T] = tr(D2^2) D1^2, eigenvectors are +-e_i sorted by D1
    r = rng(3)
    m, n = 5, 4
    d1 = np.array([5.0, 4.0, 3.0, 2.0, 1.0])
    d2 = np.array([4.0, 3.0, 2.0, 1.0])
    lay = O.OracleLayer(np.zeros((m, n)), geom=O.GEOM_BI, src=O.SRC_SECOND)
    orc = O.Oracle([lay], O.Hyper(beta2=0.9995, freq=500, power_iters=1))
    for c in range(20000):
        orc.step([d1[:, None] * r.standard_normal((m, n)) * d2[None, :]], 0)
    assert np.max(np.abs(np.abs(lay.U) - np.eye(m))) < 5e-2
    assert np.max(np.abs(np.abs(lay.V) - np.eye(n))) < 5e-2


# P4 -- Adam in the rotated space == rotate, scale, rotate back (App. C)
def test_p4_fixed_rotation_equivalence():
    r = rng(4)
    m, n, T = 9, 6, 15
    U, V = rand_orth(m, 40), rand_orth(n, 41)
    grads = [r.standard_normal((m, n)) for _ in range(T)]
    W0 = r.standard_normal((m, n))
    hp = O.Hyper(lr=1e-2, beta1=0.9, beta2=0.99, eps=1e-8, freq=10 ** 6)
    lay = O.OracleLayer(W0, geom=O.GEOM_BI, src=O.SRC_SECOND)
    lay.U, lay.V = U.copy(), V.copy()
    orc = O.Oracle([lay], hp)
    # plain Adam on the pre-rotated problem
    wt, mt, vt = U.T @ W0 @ V, np.zeros((m, n)), np.zeros((m, n))
    for g in grads:
        orc.step([g], 0)
        wt, mt, vt, _ = O.plain_adam_update(wt, mt, vt, U.T @ g @ V, 1e-2, 0.9, 0.99, 1e-8)
    back = U @ wt @ V.T
    assert np.linalg.norm(lay.W - back) / np.linalg.norm(back) < 1e-12


# P5 -- delay is an index shift for weight-independent gradients (App. B, Eq. delayed_grad)
@pytest.mark.parametrize("tau", [1, 3])
def test_p5_delay_is_index_shift_and_counters(tau):
    r = rng(5)
    m, n, T = 8, 6, 14
    grads = [r.standard_normal((m, n)) for _ in range(T)]
    hp = O.Hyper(freq=4)
    orc_d, lay_d, dws_d = run(dict(geom=O.GEOM_BI, src=O.SRC_SECOND, tau_max=tau), hp, grads, tau)
    orc_0, lay_0, dws_0 = run(dict(geom=O.GEOM_BI, src=O.SRC_SECOND, tau_max=0), hp, grads[:T - tau], 0)
    assert all(d is None for d in dws_d[:tau])
    for a, b in zip(dws_d[tau:], dws_0):
        assert np.array_equal(a, b)
    assert np.array_equal(lay_d.W, lay_0.W) and np.array_equal(lay_d.U, lay_0.U)
    c = orc_d.counters(0)
    assert c["calls"] == T and c["t"] == T - tau and c["ring_slot"] == T % tau
    assert c["refresh_count"] == (T - tau) // 4
    assert c["next_refresh_t"] == ((T - tau) // 4 + 1) * 4


def test_p5_warmup_status_and_variable_tau():
    r = rng(6)
    m, n = 4, 3
    lay = O.OracleLayer(np.zeros((m, n)), tau_max=3)
    orc = O.Oracle([lay], O.Hyper())
    gs = [r.standard_normal((m, n)) for _ in range(6)]
    assert [orc.step([g], 3) for g in gs[:3]] == [O.STATUS_WARMUP] * 3
    m_before = lay.M.copy()
    assert orc.step([gs[3]], 3) == O.STATUS_OK        # consumes g_1
    assert np.allclose(lay.M - 0.9 * m_before, 0.1 * gs[0])
    m_before = lay.M.copy()
    assert orc.step([gs[4]], 1) == O.STATUS_OK        # tau=1 -> consumes g_4
    assert np.allclose(lay.M - 0.9 * m_before, 0.1 * gs[3])


# P6 -- brute-force eigendecomposition and a library QR as pins for Power()
@pytest.mark.parametrize("k,ratio,iters", [(8, 0.5, 60), (17, 0.5, 60), (32, 0.75, 160)])
def test_p6_power_iteration_converges_to_eigh(k, ratio, iters):
    # error after `iters` steps is O(ratio^iters); the spectrum is kept within ~1e-5 of its top so
    # that the dense eigensolver itself is accurate to the asserted level
    Qe = rand_orth(k, 60 + k)
    lam = ratio ** np.arange(k)
    F = (Qe * lam[None, :]) @ Qe.T
    Q, deficient = O.power(F, np.eye(k), iters=iters)
    w, vec = np.linalg.eigh(F)
    vec = vec[:, ::-1]                       # descending eigenvalues
    assert not deficient
    assert np.max(np.abs(O.sign_normalise(Q) - O.sign_normalise(vec))) < 1e-10


@pytest.mark.parametrize("shape", [(5, 5), (12, 12), (33, 33), (20, 7)])
def test_p6_qr_pos_matches_library_qr(shape):
    A = rng(7).standard_normal(shape)
    Q, R, deficient = O.qr_pos(A)
    q, r_ = np.linalg.qr(A)
    s = np.sign(np.diag(r_))
    assert not deficient
    assert np.all(np.diag(R) > 0)
    assert np.allclose(Q, q * s[None, :], atol=1e-12) and np.allclose(R, r_ * s[:, None], atol=1e-12)
    assert np.allclose(Q @ R, A, atol=1e-12)


def test_p6_qr_pos_hand_example():
    # classic 3x3 example: A = [[12,-51,4],[6,167,-68],[-4,24,-41]] -> R = [[14,21,-14],[0,175,-70],[0,0,35]]
    A = np.array([[12.0, -51, 4], [6, 167, -68], [-4, 24, -41]])
    Q, R, _ = O.qr_pos(A)
    assert np.allclose(R, [[14, 21, -14], [0, 175, -70], [0, 0, 35]], atol=1e-10)
    assert np.allclose(Q, np.array([[6 / 7, -69 / 175, -58 / 175], [3 / 7, 158 / 175, 6 / 175],
                                    [-2 / 7, 6 / 35, -33 / 35]]), atol=1e-12)


@pytest.mark.parametrize("shape", [(3, 3), (40, 40), (257, 257), (64, 20)])
def test_p6_library_qr_variant_equals_the_written_out_one(shape):
    """`qr_pos_lapack` (what `Hyper.qr = "lapack"` selects for orders in the thousands) against the
    written-out Householder `qr_pos`, and against what defines the result whatever computes it:
    Q^T Q = I, Q R = A, R upper triangular with a positive diagonal (unique for full column rank)."""
    A = rng(17).standard_normal(shape)
    Q0, R0, d0 = O.qr_pos(A)
    Q1, R1, d1 = O.qr_pos_lapack(A)
    assert not d0 and not d1
    assert np.max(np.abs(Q0 - Q1)) < 1e-11 and np.max(np.abs(R0 - R1)) < 1e-11 * np.max(np.abs(R0))
    assert np.max(np.abs(Q1.T @ Q1 - np.eye(shape[1]))) < 1e-12
    assert np.max(np.abs(Q1 @ R1 - A)) < 1e-12 * np.max(np.abs(A)) * shape[0]
    assert np.all(np.diag(R1) > 0) and np.array_equal(R1, np.triu(R1))


def test_p6_library_qr_variant_hand_example_flag_and_trajectory():
    A = np.array([[12.0, -51, 4], [6, 167, -68], [-4, 24, -41]])
    Q, R, _ = O.qr_pos_lapack(A)
    assert np.allclose(R, [[14, 21, -14], [0, 175, -70], [0, 0, 35]], atol=1e-10)
    B = rng(8).standard_normal((6, 2)) @ rng(9).standard_normal((2, 6))   # rank 2
    assert O.qr_pos_lapack(B)[2] and O.qr_pos(B)[2]
    assert O.qr_pos_lapack(np.zeros((4, 4)))[2]
    # a whole trajectory through three refreshes: the two variants agree to rounding
    out = []
    for impl in ("householder", "lapack"):
        lay = O.OracleLayer(rng(3).standard_normal((24, 40)) * 0.02, O.GEOM_BI, O.SRC_SECOND, 0)
        orc = O.Oracle([lay], O.Hyper(freq=4, qr=impl))
        g = rng(4)
        for _ in range(13):
            orc.step([g.standard_normal((24, 40)) * 0.01], 0)
        out.append((lay.W.copy(), lay.U.copy(), lay.V.copy()))
    for a, b in zip(*out):
        assert np.max(np.abs(a - b)) < 1e-9


def test_p6_power_sensitivity_diagnostic():
    """The conditioning diagnostic: zero for a diagonal factor (a relative perturbation keeps it diagonal,
    so Power(F, I) stays I), first order in the size of the perturbation, and far larger for a
    low-rank-plus-noise factor started from the identity than for a well-separated one."""
    assert O.power_sensitivity(np.diag(np.logspace(0, -3, 16)), np.eye(16)) == 0.0
    Qe, _ = np.linalg.qr(rng(31).standard_normal((24, 24)))
    F = (Qe * (0.5 ** np.arange(24))) @ Qe.T
    s1, s2 = O.power_sensitivity(F, np.eye(24), rel=1e-9), O.power_sensitivity(F, np.eye(24), rel=2e-9)
    assert 0.0 < s1 < 1e-3 and abs(s2 / s1 - 2.0) < 1e-3
    B = rng(32).standard_normal((64, 4))
    noisy = 1e4 * B @ B.T + np.cov(rng(33).standard_normal((64, 640)))
    easy = (Qe * np.linspace(2.0, 1.0, 24)) @ Qe.T
    assert O.power_sensitivity(noisy, np.eye(64)) > 1e3 * O.power_sensitivity(easy, np.eye(24))


def test_p6_rank_deficient_flag_and_orthonormality():
    A = rng(8).standard_normal((6, 2)) @ rng(9).standard_normal((2, 6))   # rank 2
    Q, R, deficient = O.qr_pos(A)
    assert deficient
    assert np.max(np.abs(Q.T @ Q - np.eye(6))) < 1e-12
    Qz, _, dz = O.qr_pos(np.zeros((4, 4)))
    assert dz and np.allclose(Qz.T @ Qz, np.eye(4))


def test_p6_rank_deficient_completion_from_the_previous_basis():
    """Power(F, Q) with a rank-2 F of order 7: the first two columns are the unique Q factor of the
    range (they match LAPACK's QR of F Q); the other five complete the basis from the previous one:
    the whole result equals LAPACK's QR of F Q + 1e-6 Q diag(||(F Q)_j||) (full rank, hence unique) after the
    sign fix, it is orthonormal, and the completed columns span the orthogonal complement of the range."""
    k, r = 7, 2
    B = rng(21).standard_normal((k, r))
    F = B @ B.T
    Qprev, _ = np.linalg.qr(rng(22).standard_normal((k, k)))
    Q, deficient = O.power(F, Qprev)
    assert deficient
    assert np.max(np.abs(Q.T @ Q - np.eye(k))) < 1e-9
    A = F @ Qprev
    q0, r0 = np.linalg.qr(A[:, :r])
    assert np.max(np.abs(Q[:, :r] - q0 * np.sign(np.diag(r0)))) < 1e-4     # moved by the 1e-6 term only
    q1, r1 = np.linalg.qr(A + 1e-6 * Qprev * np.linalg.norm(A, axis=0)[None, :])
    assert np.max(np.abs(Q - q1 * np.sign(np.diag(r1)))) < 1e-8
    # the leading columns span the range of F, the completed ones its orthogonal complement
    lead, rest = Q[:, :r], Q[:, r:]
    assert np.linalg.norm(F - lead @ (lead.T @ F)) < 1e-4 * np.linalg.norm(F)
    assert np.linalg.norm(F @ rest) < 1e-4 * np.linalg.norm(F)
    # a full-rank product is left alone (bit for bit the plain factorisation)
    F2 = F + np.eye(k)
    Q2, d2 = O.power(F2, Qprev)
    assert not d2 and np.array_equal(Q2, O.qr_pos(F2 @ Qprev)[0])


# P7 -- Kronecker-factored covariance (Theorem 3.1 and its lemma)
def test_p7_kronecker_structure_and_norm_chain():
    r = rng(10)
    m, n = 4, 3
    def spd(k, s):
        X = rng(s).standard_normal((k, k))
        return X @ X.T + 0.1 * np.eye(k)
    A, B = spd(n, 70), spd(m, 71)                      # cov(vec(G)) = A (x) B, column-major vec
    # exact expectations by summing over a basis: E[G G^T] = sum_j sum_j' A_jj' ... use sampling-free identity
    C = np.kron(A, B)
    EGGt = np.zeros((m, m)); EGtG = np.zeros((n, n))
    idx = lambda i, j: j * m + i                       # column-major position of G_ij
    for i in range(m):
        for i2 in range(m):
            EGGt[i, i2] = sum(C[idx(i, j), idx(i2, j)] for j in range(n))
    for j in range(n):
        for j2 in range(n):
            EGtG[j, j2] = sum(C[idx(i, j), idx(i, j2)] for i in range(m))
    assert np.allclose(EGGt, np.trace(A) * B, atol=1e-12)
    assert np.allclose(EGtG, np.trace(B) * A, atol=1e-12)
    # eigenvectors via the oracle's Power() on those factors
    U, _ = O.power(EGGt, np.eye(m), iters=400)
    V, _ = O.power(EGtG, np.eye(n), iters=400)
    n11 = lambda X: np.sum(np.abs(X))
    H = C
    HU = np.kron(np.eye(n), U.T) @ H @ np.kron(np.eye(n), U)
    HUV = np.kron(V.T, U.T) @ H @ np.kron(V, U)
    assert n11(HUV) <= n11(HU) + 1e-9 <= n11(H) + 2e-9
    assert abs(n11(HUV) - np.sum(np.linalg.eigvalsh(C))) < 1e-6     # diagonalised: sum of eigenvalues


# P8 -- vec(U^T G V) = (V^T (x) U^T) vec(G): pins sides and transposes of rotate()
def test_p8_two_sided_rotation_is_kronecker_rotation():
    r = rng(11)
    m, n = 5, 3
    lay = O.OracleLayer(np.zeros((m, n)), geom=O.GEOM_BI)
    lay.U, lay.V = rand_orth(m, 80), rand_orth(n, 81)
    G = r.standard_normal((m, n))
    vec = lambda X: X.reshape(-1, order="F")
    assert np.allclose(vec(lay.rotate(G)), np.kron(lay.V.T, lay.U.T) @ vec(G), atol=1e-13)
    assert np.allclose(vec(lay.rotate_back(G)), np.kron(lay.V, lay.U) @ vec(G), atol=1e-13)


# P9 -- round trip, invariances, unilateral == bilateral with identity, memory table (App. H)
def test_p9_round_trip_and_sign_flip_invariance():
    r = rng(12)
    m, n = 7, 9
    lay = O.OracleLayer(np.zeros((m, n)), geom=O.GEOM_BI)
    lay.U, lay.V = rand_orth(m, 90), rand_orth(n, 91)
    G = r.standard_normal((m, n))
    assert np.allclose(lay.rotate_back(lay.rotate(G)), G, atol=1e-12)
    # flipping column signs of U, V leaves the update unchanged
    grads = [r.standard_normal((m, n)) for _ in range(5)]
    outs = []
    for flip in (False, True):
        l2 = O.OracleLayer(np.zeros((m, n)), geom=O.GEOM_BI)
        su = np.where(np.arange(m) % 2 == 0, -1.0, 1.0) if flip else np.ones(m)
        sv = np.where(np.arange(n) % 3 == 0, -1.0, 1.0) if flip else np.ones(n)
        l2.U, l2.V = lay.U * su[None, :], lay.V * sv[None, :]
        orc = O.Oracle([l2], O.Hyper(freq=10 ** 6))
        for g in grads:
            orc.step([g], 0)
        outs.append(l2.W.copy())
    assert np.allclose(outs[0], outs[1], atol=1e-14)


def test_p9_power_scale_invariance_and_eps0_gradient_scale_invariance():
    r = rng(13)
    k = 10
    X = r.standard_normal((k, k)); F = X @ X.T
    Q0 = rand_orth(k, 92)
    Q1, _ = O.power(F, Q0)
    Q2, _ = O.power(37.5 * F, Q0)
    assert np.allclose(Q1, Q2, atol=1e-12)
    m, n = 6, 8
    grads = [r.standard_normal((m, n)) for _ in range(8)]
    hp = O.Hyper(eps=0.0, freq=3)
    _, l1, _ = run(dict(geom=O.GEOM_BI), hp, grads, 0)
    _, l2, _ = run(dict(geom=O.GEOM_BI), hp, [1e3 * g for g in grads], 0)
    assert np.allclose(l1.W, l2.W, rtol=1e-9, atol=1e-12)


def test_p9_unilateral_side_and_equivalence():
    r = rng(14)
    for (m, n) in [(6, 10), (10, 6), (7, 7)]:
        grads = [r.standard_normal((m, n)) for _ in range(7)]
        hp = O.Hyper(freq=3)
        _, lu, _ = run(dict(geom=O.GEOM_UNI, src=O.SRC_SECOND), hp, grads, 0)
        left = m <= n
        assert (lu.U is not None) == left and (lu.V is not None) == (not left)
        # before any refresh the unilateral layer is plain Adam
        hp2 = O.Hyper(freq=10 ** 6)
        _, lu2, _ = run(dict(geom=O.GEOM_UNI, src=O.SRC_SECOND), hp2, grads, 0)
        _, ln2, _ = run(dict(geom=O.GEOM_NONE), hp2, grads, 0)
        assert np.allclose(lu2.W, ln2.W, atol=1e-15)
        # with a given rotation on the rotated side, uni equals bi with identity elsewhere
        Qs = rand_orth(m if left else n, 95)
        la = O.OracleLayer(np.zeros((m, n)), geom=O.GEOM_UNI)
        lb = O.OracleLayer(np.zeros((m, n)), geom=O.GEOM_BI)
        if left:
            la.U = Qs.copy(); lb.U = Qs.copy()
        else:
            la.V = Qs.copy(); lb.V = Qs.copy()
        oa, ob = O.Oracle([la], hp2), O.Oracle([lb], hp2)
        for g in grads:
            oa.step([g], 0); ob.step([g], 0)
        assert np.allclose(la.W, lb.W, atol=1e-14)


def test_p9_first_moment_source_uses_updated_momentum():
    # S=1st: U <- Power(M_t M_t^T, U) with the momentum that already contains G_t (Alg. 1 passes M_t)
    r = rng(15)
    m, n = 5, 8
    grads = [r.standard_normal((m, n)) for _ in range(2)]
    hp = O.Hyper(freq=2, beta1=0.5)
    _, lay, _ = run(dict(geom=O.GEOM_UNI, src=O.SRC_FIRST), hp, grads, 0)
    M2 = 0.5 * (0.5 * grads[0]) + 0.5 * grads[1]
    q, r_ = np.linalg.qr(M2 @ M2.T)
    assert np.allclose(lay.U, q * np.sign(np.diag(r_))[None, :], atol=1e-12)
    assert lay.L is None and lay.R is None


def test_p9_accumulate_on_refresh_variant():
    # literal Algorithm 2: only the gradients of refresh steps enter L
    r = rng(16)
    m, n = 4, 9
    grads = [r.standard_normal((m, n)) for _ in range(6)]
    hp = O.Hyper(freq=3, accum="on_refresh", beta2=0.9)
    _, lay, _ = run(dict(geom=O.GEOM_BI, src=O.SRC_SECOND), hp, grads, 0)
    L = 0.9 * (0.1 * grads[2] @ grads[2].T) + 0.1 * grads[5] @ grads[5].T
    assert np.allclose(lay.L, L, atol=1e-14)
    hp = O.Hyper(freq=3, accum="every_step", beta2=0.9)
    _, lay, _ = run(dict(geom=O.GEOM_BI, src=O.SRC_SECOND), hp, grads, 0)
    L = np.zeros((m, m)); Rr = np.zeros((n, n))
    for g in grads:
        L = 0.9 * L + 0.1 * g @ g.T
        Rr = 0.9 * Rr + 0.1 * g.T @ g
    assert np.allclose(lay.L, L, atol=1e-14) and np.allclose(lay.R, Rr, atol=1e-14)


def test_p9_memory_table_app_h():
    # golden values: tests/golden/memory_table.txt (App. H, Table 2; GiB per matrix, fp32)
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "memory_table.txt")
    geoms = {"Bi": O.GEOM_BI, "Uni": O.GEOM_UNI}
    srcs = {"2nd": O.SRC_SECOND, "1st": O.SRC_FIRST}
    rows = 0
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        s, g, attn, mlp = line.split()
        for (m, n), printed in (((4096, 4096), float(attn)), ((4096, 14336), float(mlp))):
            rot, mom = O.overhead_elements(m, n, geoms[g], srcs[s])
            gib = 4.0 * (rot + mom) / 2 ** 30
            assert abs(gib - printed) < 0.0051, (line, gib)
        rows += 1
    assert rows == 4


def test_weight_decay_is_decoupled():
    g = np.ones((2, 2)); W0 = np.full((2, 2), 2.0)
    hp = O.Hyper(lr=0.1, weight_decay=0.5, eps=0.0, freq=10 ** 6)
    _, lay, dws = run(dict(geom=O.GEOM_BI), hp, [g], 0, W0)
    m1, v1 = 0.1, 0.001
    assert np.allclose(lay.W, (1 - 0.05) * 2.0 - 0.1 * m1 / np.sqrt(v1))


def test_forced_refresh_matches_scheduled_and_rejects_t0():
    r = rng(17)
    m, n = 6, 5
    grads = [r.standard_normal((m, n)) for _ in range(4)]
    lay = O.OracleLayer(np.zeros((m, n)), geom=O.GEOM_BI)
    orc = O.Oracle([lay], O.Hyper(freq=10 ** 6))
    with pytest.raises(ValueError):
        orc.refresh_basis()
    for g in grads:
        orc.step([g], 0)
    t = lay.t
    orc.refresh_basis(0)
    q, r_ = np.linalg.qr(lay.L)       # U was I: Power(L, I) = qr(L)
    assert np.allclose(lay.U, q * np.sign(np.diag(r_))[None, :], atol=1e-12)
    assert lay.t == t and lay.refresh_count == 1


def test_stage_aware_frequency_rule_hand_values():
    """App. I with P = 32 (mid = 15) and f0 = 10, worked by hand from the printed rule:
    tau = 31: n = -16, 1 - n/mid = 31/15, f = floor(150/31) = 4;   tau = 16: n = -1, f = floor(150/16) = 9;
    tau = 15: n = 1, f = floor(150/14) = 10;   tau = 8: n = 8, f = floor(150/7) = 21;   tau = 2: n = 14, f = 150.
    tau = 1 divides by zero and tau = 0 goes negative: undefined.  The period shrinks as the delay grows."""
    for tau, want in ((31, 4), (16, 9), (15, 10), (8, 21), (2, 150)):
        assert O.stage_aware_freq(32, tau, 10) == want
    for tau in (0, 1):
        with pytest.raises(ValueError):
            O.stage_aware_freq(32, tau, 10)
    with pytest.raises(ValueError):
        O.stage_aware_freq(3, 1, 10)
    fs = [O.stage_aware_freq(32, tau, 10) for tau in range(2, 32)]
    assert all(a >= b for a, b in zip(fs, fs[1:]))
    assert O.stage_aware_freq(32, 15, 14) == 15          # exactly 14 / (14/15): no floating-point floor slip


def test_effective_delay_closed_forms():
    """Eq. (effective-delay): one group gives its own delay; equal constants give the root mean square;
    a group with a zero constant does not count; scaling all constants changes nothing."""
    assert O.effective_delay([3.0], [7]) == pytest.approx(7.0)
    assert O.effective_delay([1, 1, 1, 1], [0, 1, 2, 3]) == pytest.approx(np.sqrt(14 / 4))
    assert O.effective_delay([2.0, 0.0], [5, 100]) == pytest.approx(5.0)
    assert O.effective_delay([1, 2, 3], [3, 2, 1]) == pytest.approx(O.effective_delay([10, 20, 30], [3, 2, 1]))
    assert O.effective_delay([1, 2, 3], [3, 2, 1]) == pytest.approx(np.sqrt((9 + 16 + 9) / 14))


def test_global_norm_clipping_closed_forms():
    """App. D.2 clipping: (a) a threshold above the joint norm changes nothing, bit for bit; (b) below
    it, the momentum after the first update has joint norm (1 - beta1) * clip exactly as a closed form
    (M0 = 0, so M1 = (1 - beta1) * s * g with s = clip / ||g||); (c) a clipped trajectory is invariant to
    rescaling every gradient by a > 1 (the clipped gradient is clip * g / ||g||); (d) the factor travels
    with its call through the delay: with tau = 2 the update at call 3 uses the factor of call 1."""
    shapes = [(6, 4), (3, 5)]
    def run(clip, scale=1.0, tau=0, calls=3, tmax=0):
        layers = [O.OracleLayer(np.zeros(s), O.GEOM_NONE, O.SRC_SECOND, tmax) for s in shapes]
        orc = O.Oracle(layers, O.Hyper(lr=1e-2, clip_norm=clip, freq=10 ** 6))
        r = rng(40)
        for c in range(calls):
            orc.step([scale * (c + 1) * r.standard_normal(s) for s in shapes], tau)
        return orc
    a, b = run(0.0), run(1e6)
    for x, y in zip(a.layers, b.layers):
        assert np.array_equal(x.W, y.W) and np.array_equal(x.M, y.M)
    one = run(0.5, calls=1)
    joint = np.sqrt(sum(np.sum(l.M ** 2) for l in one.layers))
    assert joint == pytest.approx((1 - 0.9) * 0.5, rel=1e-12)
    c1, c2 = run(0.5), run(0.5, scale=7.0)
    for x, y in zip(c1.layers, c2.layers):
        assert np.allclose(x.W, y.W, rtol=1e-12, atol=0)
    d = run(0.5, tau=2, calls=3, tmax=2)
    assert d.layers[0].t == 1 and set(d.clip_of_call) == {1, 2, 3}
    g1 = [1 * x for x in [rng(40).standard_normal(shapes[0])]][0]     # the first draw of call 1
    n1 = np.sqrt(sum(np.sum(x ** 2) for x in (lambda r: [r.standard_normal(s) for s in shapes])(rng(40))))
    assert d.clip_of_call[1] == pytest.approx(0.5 / n1, rel=1e-12)
    assert np.allclose(d.layers[0].M, (1 - 0.9) * d.clip_of_call[1] * g1, rtol=1e-12, atol=0)


def test_lr_warmup_cosine_schedule_values():
    """App. D.2 schedule, 1000 steps with 1.2 % warm-up (W = 12): linear ramp reaching base_lr at step
    11, base_lr again at step 12 (cosine of 0), the mid-point of the decay halfway, monotone decay."""
    f = lambda t: O.lr_warmup_cosine(t, 1000, 0.012, 1e-3, 1e-5)
    assert f(0) == pytest.approx(1e-3 / 12) and f(5) == pytest.approx(6e-3 / 12) and f(11) == pytest.approx(1e-3)
    assert f(12) == pytest.approx(1e-3)
    assert f(12 + 494) == pytest.approx(1e-5 + (1e-3 - 1e-5) * 0.5)
    vals = [f(t) for t in range(12, 1000)]
    assert all(a >= b for a, b in zip(vals, vals[1:])) and vals[-1] > 1e-5


def _closed_loop_oracle(geom, aligned, tau, steps=300):
    from workloads.closed_loop import kronecker_quadratic, loss
    P, Q, W0 = kronecker_quadratic(aligned=aligned)
    lay = O.OracleLayer(W0.copy(), geom, O.SRC_SECOND, tau)
    orc = O.Oracle([lay], O.Hyper(lr=0.02, beta1=0.0, beta2=0.9, eps=1e-12, freq=5))
    for _ in range(steps):
        orc.step([P @ lay.W @ Q], tau)          # the gradient at the CURRENT weights, applied tau calls later
    return loss(P, Q, lay.W)


def test_closed_loop_quadratic_rotation_removes_the_delay_penalty():
    """The paper's toy claim (Sec. 2.2, Fig. 2; Sec. 3.1), on a Kronecker quadratic with genuinely
    stale gradients (tau = 2): Adam on the misaligned problem is much worse than on the aligned one,
    and the basis-rotated step on the misaligned problem is as good as Adam on the aligned one."""
    aligned = _closed_loop_oracle(O.GEOM_NONE, True, 2)
    misaligned = _closed_loop_oracle(O.GEOM_NONE, False, 2)
    rotated = _closed_loop_oracle(O.GEOM_BI, False, 2)
    assert misaligned > 5.0 * aligned
    assert rotated < 2.0 * aligned
    # and delay itself hurts plain Adam on the misaligned problem
    assert _closed_loop_oracle(O.GEOM_NONE, False, 0) < 0.5 * misaligned


def _spiral_run(p0, steps, delay_from=None):
    """Plain Adam of Eq. (adam) on the spiral loss with the paper's settings (App. D.1: learning rate 0.1,
    beta1 = 0, beta2 = 0.9), gradient computed from the current iterate; from call `delay_from` on the
    applied gradient is one call old (tau = 1 through the ring)."""
    from workloads.closed_loop import spiral_grad
    lay = O.OracleLayer(np.array([p0], dtype=np.float64), O.GEOM_NONE, O.SRC_SECOND, 1)
    orc = O.Oracle([lay], O.Hyper(lr=0.1, beta1=0.0, beta2=0.9, eps=1e-8, freq=10 ** 9))
    traj = [lay.W[0].copy()]
    for c in range(steps):
        orc.step([spiral_grad(lay.W[0])[None, :]], 0 if (delay_from is None or c < delay_from) else 1)
        traj.append(lay.W[0].copy())
    return np.array(traj)


def test_spiral_loss_definition_and_the_papers_alignment_claim():
    """Spiral loss of Sec. 2.2 / App. D.1.  Definition: the gradient equals central differences of
    f(r, theta) = r^2 + (20 sin(4r - theta) + 1)^2, and on the valley 20 sin(4r - theta) = -1 the loss is
    r^2.  The paper's observation, in the form that can be checked without its figure: without delay Adam
    sits higher up the valley walls (oscillates more) where the Hessian eigenbasis is misaligned with the
    coordinate axes than where it is aligned, and a delay of one step raises that further in both."""
    from workloads.closed_loop import spiral_grad, spiral_loss, spiral_misalignment, spiral_valley_excess
    for p in ([3.0, -1.0], [-0.7, 5.2], [6.0, 6.0]):
        p = np.array(p)
        fd = np.array([(spiral_loss(p + e) - spiral_loss(p - e)) / 2e-6 for e in (np.array([1e-6, 0]), np.array([0, 1e-6]))])
        assert np.allclose(spiral_grad(p), fd, rtol=1e-6, atol=1e-5)
    th = 0.3
    r = (np.arcsin(-1.0 / 20.0) + th + 4 * np.pi) / 4.0
    on_valley = np.array([r * np.cos(th), r * np.sin(th)])
    assert abs(spiral_loss(on_valley) - r * r) < 1e-9 and abs(spiral_valley_excess(on_valley)) < 1e-9
    stats = {}
    for name, p0 in (("aligned", [8.0, 0.0]), ("misaligned", [5.0, 5.0])):
        free, delayed = _spiral_run(p0, 1000), _spiral_run(p0, 1000, delay_from=600)
        assert np.array_equal(free[:601], delayed[:601])                   # identical until the delay starts
        stats[name] = (spiral_misalignment(free[600]),
                       np.mean([spiral_valley_excess(p) for p in free[600:]]),
                       np.mean([spiral_valley_excess(p) for p in delayed[600:]]))
    assert stats["aligned"][0] < 0.05 and stats["misaligned"][0] > 0.9
    assert stats["misaligned"][1] > 1.5 * stats["aligned"][1]              # misalignment: more oscillation
    for name in stats:
        assert stats[name][2] > 2.0 * stats[name][1]                      # delay: more again


def test_golden_c1_trajectory_is_reproduced():
    """tests/golden/c1_trajectory.txt (written by tests/golden/make_c1_trajectory.py from the oracle alone):
    the oracle of today reproduces the stored C1 trajectory -- counters exactly, values to 1e-9 relative (the host BLAS may order its sums differently).
    Not a pin to the paper (it prints no worked example); a guard against accidental changes of the
    oracle's arithmetic, e.g. while a faster QR step is added beside the written-out one."""
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_c1_trajectory", os.path.join(here, "make_c1_trajectory.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = [l.split() for l in open(os.path.join(here, "c1_trajectory.txt")) if not l.startswith("#")]
    now = list(mod.rows())
    assert len(stored) == len(now) == 20
    for line, (c, st, t, rc, vals) in zip(stored, now):
        assert [int(x) for x in line[:4]] == [c, st, t, rc]
        ref = np.array([float(x) for x in line[4:]])
        assert np.all(np.abs(np.array(vals) - ref) <= 1e-9 * np.abs(ref) + 1e-300)
