"""Float64 CPU oracle of the rotated Adam step on delayed gradients.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA path is checked against.  It shares no code with the CUDA path and must
never be imported by the product package; only tests, the smoke check and the
benchmark's CPU-baseline legs use it.

What it follows (all in the paper's notation, W in R^{m x n}):

* Algorithm 1 ("Adam with Basis Rotation"): M_t, the refresh test
  ``t mod freq == 0``, G~ = U^T G V, M~ = U^T M V, V~ EMA, and the weight
  write W <- W - eta U (M~ / sqrt(V~ + eps)) V^T.
* Algorithm 2 ("Eigenbasis-Estimation"): source S in {1st, 2nd}, geometry in
  {unilateral, bilateral}; L, R are EMAs of G G^T and G^T G with rate beta2.
* Sec. 3.2: Power(A, Q) is one power-iteration step followed by a QR
  decomposition, Q <- qr(A Q).Q; the unilateral variant rotates the smaller
  dimension only.
* Eq. (adam): plain Adam as the paper writes it, eps inside the square root
  and no bias correction.
* App. B, Eq. (delayed_grad): the gradient applied at update t was produced
  tau updates earlier.

Readings where the paper is silent (listed in the design notes as well):
U_0 = V_0 = I; M_0 = V~_0 = L_0 = R_0 = 0; L and R are accumulated at every
update (``accum="every_step"``) unless ``accum="on_refresh"`` asks for the
literal placement inside Algorithm 2; V~ is not re-expressed when the basis
changes; QR is made unique by a positive diagonal of R; no column sorting; the
refresh counter is the update counter t; the first tau calls are warm-up and
apply no update.

Pins: tests/test_oracle_pins.py (orthogonality, reduction to plain Adam,
diagonal quadratic, dense eigendecomposition, Kronecker identities, round
trips, delay-as-index-shift, the memory table of App. H).  Columns produced by
the rank-deficient branch of ``qr_pos`` are *parity unpinned*: only
orthonormality is asserted for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

GEOM_NONE, GEOM_UNI, GEOM_BI = 0, 1, 2
SRC_FIRST, SRC_SECOND = 1, 2
STATUS_OK, STATUS_WARMUP, STATUS_RANK_DEFICIENT = 0, 1, 2

RANK_TOL = 1e-12


# ----------------------------------------------------------------------------
# QR with positive diagonal (Sec. 3.2: "power iteration followed by QR")
# ----------------------------------------------------------------------------
def qr_pos(A: np.ndarray):
    """Householder QR of a square (or tall) matrix, R's diagonal made positive.

    Returns (Q, R, deficient).  For a full-column-rank A this is the unique
    factorisation A = Q R with Q^T Q = I and diag(R) > 0.  ``deficient`` is set
    when some |R_jj| <= RANK_TOL * max_k |R_kk|; those columns of Q are still
    orthonormal (Householder guarantees that) but not unique.
    """
    A = np.array(A, dtype=np.float64, copy=True)
    rows, cols = A.shape
    assert rows >= cols
    vs = []
    for j in range(cols):
        x = A[j:, j]
        alpha = np.linalg.norm(x)
        v = x.copy()
        if alpha > 0.0:
            # reflect x onto -sign(x0) * alpha * e1 (no cancellation)
            s = 1.0 if x[0] >= 0.0 else -1.0
            v[0] += s * alpha
            vn = np.linalg.norm(v)
            v /= vn
            A[j:, j:] -= 2.0 * np.outer(v, v @ A[j:, j:])
        else:
            v[:] = 0.0
        vs.append(v)
    R = np.triu(A[:cols, :])
    # accumulate Q = H_0 H_1 ... H_{cols-1} applied to the first `cols` columns of I
    Q = np.eye(rows, cols)
    for j in reversed(range(cols)):
        v = vs[j]
        Q[j:, :] -= 2.0 * np.outer(v, v @ Q[j:, :])
    d = np.diag(R).copy()
    sgn = np.where(d < 0.0, -1.0, 1.0)
    Q = Q * sgn[None, :]
    R = R * sgn[:, None]
    dmax = np.max(np.abs(d)) if cols else 0.0
    deficient = bool(dmax == 0.0 or np.any(np.abs(d) <= RANK_TOL * dmax))
    return Q, R, deficient


def qr_pos_lapack(A: np.ndarray):
    """The same factorisation with the library's Householder QR (numpy.linalg.qr, i.e. LAPACK) as the
    step, followed by the same sign fix.  For a full-column-rank A the factorisation with
    diag(R) > 0 is unique, so this and `qr_pos` compute one definition (Sec. 3.2 only says "QR
    decomposition"); `qr_pos` is the written-out form that can be checked by eye, this one is what
    makes orders in the thousands affordable (`Hyper.qr = "lapack"`).  Pinned against `qr_pos` and
    against the defining properties (Q^T Q = I, Q R = A, R upper triangular with a positive
    diagonal) in tests/test_oracle_pins.py.  Returns (Q, R, deficient) like `qr_pos`."""
    A = np.asarray(A, dtype=np.float64)
    rows, cols = A.shape
    assert rows >= cols
    Q, R = np.linalg.qr(A, mode="reduced")
    d = np.diag(R).copy()
    sgn = np.where(d < 0.0, -1.0, 1.0)
    Q = Q * sgn[None, :]
    R = R * sgn[:, None]
    dmax = np.max(np.abs(d)) if cols else 0.0
    deficient = bool(dmax == 0.0 or np.any(np.abs(d) <= RANK_TOL * dmax))
    return Q, R, deficient


QR_IMPLS = {"householder": qr_pos, "lapack": qr_pos_lapack}

COMPLETION = 1e-6


def qr_completed(A: np.ndarray, Qprev: np.ndarray, qr=qr_pos):
    """Q factor of A with a positive diagonal of R.  The paper does not say what Power() returns
    when F Q is rank-deficient (S = 1st on the larger side of a bilateral layer: M M^T has rank
    <= min(m, n)).  Reading taken here: whenever the plain factorisation meets a negligible pivot,
    the directions outside the range of A are completed from the current basis, by factorising
    A with COMPLETION * ||A_j|| * Qprev_j added to every column j (a zero column becomes Qprev_j),
    which has full rank when Qprev has.  The rule is invariant to a rescaling of A or of its columns."""
    Q, R, d = qr(A)
    if d:
        cn = np.linalg.norm(A, axis=0)
        w = np.where(cn > 0.0, COMPLETION * cn, 1.0)
        Q, R, _ = qr(A + Qprev * w[None, :])
    return Q, R, d


def power(F: np.ndarray, Q: np.ndarray, iters: int = 1, qr=qr_pos):
    """Power(F, Q): `iters` times Q <- qr(F Q).Q (Sec. 3.2; the paper uses 1)."""
    deficient = False
    for _ in range(iters):
        Q, _, d = qr_completed(F @ Q, Q, qr)
        deficient |= d
    return Q, deficient


def power_sensitivity(F: np.ndarray, Q: np.ndarray, rel: float = 2.0 ** -24, seed: int = 0, qr=qr_pos) -> float:
    """Diagnostic of how well posed one Power(F, Q) is: the largest entry by which the sign-normalised
    result moves when every entry of F is perturbed by a relative `rel` (symmetric Gaussian pattern;
    the default is one fp32 rounding of the stored factor).  The unique Q factor can be numerically
    fragile (trailing columns come out of a cancellation against the leading eigen-directions): a
    basis mismatch of this size against an implementation that keeps F in fp32 says nothing about
    its arithmetic.  Not a step of the method."""
    F = np.asarray(F, dtype=np.float64)
    Z = np.random.default_rng(seed).standard_normal(F.shape)
    Z = (Z + Z.T) / np.sqrt(2.0)
    Q0, _ = power(F, Q, 1, qr)
    Q1, _ = power(F * (1.0 + rel * Z), Q, 1, qr)
    return float(np.max(np.abs(sign_normalise(Q0) - sign_normalise(Q1))))


def sign_normalise(Q: np.ndarray) -> np.ndarray:
    """Flip each column so that its entry of largest magnitude is positive
    (lowest index on ties).  The update is invariant to such flips, so bases
    are compared after this normalisation."""
    Q = np.asarray(Q, dtype=np.float64)
    idx = np.argmax(np.abs(Q), axis=0)
    s = np.sign(Q[idx, np.arange(Q.shape[1])])
    s[s == 0] = 1.0
    return Q * s[None, :]


# ----------------------------------------------------------------------------
# Plain Adam exactly as Eq. (adam) writes it
# ----------------------------------------------------------------------------
def plain_adam_update(w, m, v, g, lr, beta1, beta2, eps, weight_decay=0.0):
    """One update of Eq. (adam): eps inside the sqrt, no bias correction.
    Returns (w, m, v, dw)."""
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    dw = -lr * m / np.sqrt(v + eps)
    if weight_decay:
        w = (1.0 - lr * weight_decay) * w
    return w + dw, m, v, dw


# ----------------------------------------------------------------------------
# State
# ----------------------------------------------------------------------------
def rotated_sides(m: int, n: int, geom: int):
    """(left, right): which sides carry a rotation.  Unilateral rotates the
    smaller dimension (Sec. 3.2); ties go to the left."""
    if geom == GEOM_BI:
        return True, True
    if geom == GEOM_UNI:
        return (m <= n), (m > n)
    return False, False


def overhead_elements(m: int, n: int, geom: int, src: int):
    """(rotation, moment) element counts of App. H's memory table."""
    left, right = rotated_sides(m, n, geom)
    rot = (m * m if left else 0) + (n * n if right else 0)
    mom = rot if src == SRC_SECOND else 0
    return rot, mom


@dataclass
class Hyper:
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.0
    beta_factor: float = -1.0      # < 0 -> beta2 (Algorithm 2 reuses beta2)
    freq: int = 10
    power_iters: int = 1
    accum: str = "every_step"      # or "on_refresh" (literal Algorithm 2)
    clip_norm: float = 0.0         # global-norm gradient clipping (App. D.2 uses 1.0); 0 = off
    qr: str = "householder"        # QR step of Power(): "householder" (written out) or "lapack" (library routine)


class OracleLayer:
    """State of one weight matrix."""

    def __init__(self, W0, geom=GEOM_BI, src=SRC_SECOND, tau_max=0, freq=0):
        self.W = np.array(W0, dtype=np.float64, copy=True)
        self.m, self.n = self.W.shape
        self.geom, self.src = geom, src
        self.left, self.right = rotated_sides(self.m, self.n, geom)
        self.tau_max, self.freq = int(tau_max), int(freq)
        self.M = np.zeros_like(self.W)
        self.V2 = np.zeros_like(self.W)                      # V~ (rotated space)
        self.U = np.eye(self.m) if self.left else None
        self.V = np.eye(self.n) if self.right else None
        second = src == SRC_SECOND
        self.L = np.zeros((self.m, self.m)) if (self.left and second) else None
        self.R = np.zeros((self.n, self.n)) if (self.right and second) else None
        self.ring: List[Optional[np.ndarray]] = [None] * self.tau_max
        # integer state
        self.t = 0
        self.ring_slot = 0          # slot the next call writes
        self.refresh_count = 0
        self.last_dW = None
        self.last_min_pivot = None  # min_j R_jj / ||a_j|| of the last refresh

    # -- pieces of Algorithm 1 / 2 -------------------------------------------------
    def rotate(self, X):
        """U^T X V with the identity on an unrotated side (Alg. 1 (rotation of G and M))."""
        Y = X
        if self.left:
            Y = self.U.T @ Y
        if self.right:
            Y = Y @ self.V
        return Y

    def rotate_back(self, X):
        """U X V^T (Alg. 1 (weight update))."""
        Y = X
        if self.left:
            Y = self.U @ Y
        if self.right:
            Y = Y @ self.V.T
        return Y

    def accumulate_factors(self, G, beta):
        """L <- beta L + (1-beta) G G^T ; R <- beta R + (1-beta) G^T G (Alg. 2)."""
        if self.L is not None:
            self.L = beta * self.L + (1.0 - beta) * (G @ G.T)
        if self.R is not None:
            self.R = beta * self.R + (1.0 - beta) * (G.T @ G)

    def refresh(self, power_iters=1, qr=qr_pos):
        """The Power part of Algorithm 2 on the current L, R (S=2nd) or M (S=1st)."""
        deficient = False
        piv = []
        if self.left:
            F = self.L if self.src == SRC_SECOND else self.M @ self.M.T
            self.U, d, p = _power_with_pivot(F, self.U, power_iters, qr)
            deficient |= d
            piv.append(p)
        if self.right:
            F = self.R if self.src == SRC_SECOND else self.M.T @ self.M
            self.V, d, p = _power_with_pivot(F, self.V, power_iters, qr)
            deficient |= d
            piv.append(p)
        self.refresh_count += 1
        self.last_min_pivot = min(piv) if piv else None
        return deficient


def _power_with_pivot(F, Q, iters, qr=qr_pos):
    deficient, piv = False, np.inf
    for _ in range(iters):
        A = F @ Q
        Q, R, d = qr_completed(A, Q, qr)
        deficient |= d
        cn = np.linalg.norm(A, axis=0)
        cn[cn == 0] = 1.0
        piv = min(piv, float(np.min(np.abs(np.diag(R)) / cn)))
    return Q, deficient, piv


class Oracle:
    """A set of independent layers stepped together (the library's handle)."""

    def __init__(self, layers: Sequence[OracleLayer], hp: Hyper):
        self.layers = list(layers)
        self.hp = hp
        self.calls = 0
        self.clip_of_call = {}     # call index -> clipping factor of that call's gradients

    def _beta_factor(self):
        return self.hp.beta2 if self.hp.beta_factor < 0 else self.hp.beta_factor

    def step(self, grads: Sequence[np.ndarray], tau: int = -1):
        """One call: submit g_c for every layer, apply the update that is due.

        `tau` in [0, tau_max]; -1 means each layer's own tau_max.  Returns
        STATUS_WARMUP when no layer applied an update, STATUS_RANK_DEFICIENT
        when a refresh met a rank-deficient factor, else STATUS_OK.
        """
        hp = self.hp
        self.calls += 1
        if hp.clip_norm > 0.0:
            # App. D.2 ("gradient clipping value of 1.0"): the gradients of one call, all layers
            # together, are scaled to a joint L2 norm of at most clip_norm.  The factor belongs to
            # the call: a layer that applies g_c later applies the clipped g_c.
            nrm = np.sqrt(sum(float(np.sum(np.asarray(g, dtype=np.float64) ** 2)) for g in grads))
            self.clip_of_call[self.calls] = hp.clip_norm / nrm if nrm > hp.clip_norm else 1.0
        applied, deficient = False, False
        for lay, g in zip(self.layers, grads):
            g = np.asarray(g, dtype=np.float64)
            tl = lay.tau_max if tau < 0 else tau
            assert 0 <= tl <= lay.tau_max
            # Eq. (delayed_grad): consume the gradient submitted tau calls ago.
            src_call = self.calls - tl
            G = None
            if src_call >= 1:
                G = g if tl == 0 else lay.ring[(src_call - 1) % lay.tau_max]
            if lay.tau_max > 0:
                lay.ring[(self.calls - 1) % lay.tau_max] = g.copy()
                lay.ring_slot = self.calls % lay.tau_max
            if G is None:
                lay.last_dW = None
                continue
            applied = True
            if hp.clip_norm > 0.0:
                G = self.clip_of_call[src_call] * G
            deficient |= self._update(lay, G)
        if not applied:
            return STATUS_WARMUP
        return STATUS_RANK_DEFICIENT if deficient else STATUS_OK

    def _update(self, lay: OracleLayer, G: np.ndarray) -> bool:
        hp = self.hp
        deficient = False
        lay.t += 1
        if lay.geom == GEOM_NONE:
            lay.W, lay.M, lay.V2, lay.last_dW = plain_adam_update(
                lay.W, lay.M, lay.V2, G, hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay)
            return False
        # Alg. 1 (momentum update)
        lay.M = hp.beta1 * lay.M + (1.0 - hp.beta1) * G
        second = lay.src == SRC_SECOND
        if second and hp.accum == "every_step":
            lay.accumulate_factors(G, self._beta_factor())
        # Alg. 1 (periodic refresh)
        freq = lay.freq if lay.freq > 0 else hp.freq
        if lay.t % freq == 0:
            if second and hp.accum == "on_refresh":
                lay.accumulate_factors(G, self._beta_factor())
            deficient = lay.refresh(hp.power_iters, QR_IMPLS[hp.qr])
        # Alg. 1 (rotation, second moment, weight update)
        Gt = lay.rotate(G)
        Mt = lay.rotate(lay.M)
        lay.V2 = hp.beta2 * lay.V2 + (1.0 - hp.beta2) * Gt * Gt
        X = Mt / np.sqrt(lay.V2 + hp.eps)
        dW = -hp.lr * lay.rotate_back(X)
        if hp.weight_decay:
            lay.W = (1.0 - hp.lr * hp.weight_decay) * lay.W
        lay.W = lay.W + dW
        lay.last_dW = dW
        return deficient

    def refresh_basis(self, layer: int = -1):
        """Forced refresh from the current L, R or M; does not touch t."""
        deficient = False
        targets = self.layers if layer < 0 else [self.layers[layer]]
        for lay in targets:
            if lay.geom == GEOM_NONE:
                continue
            if lay.t == 0:
                raise ValueError("refresh before the first update: the factor is all zero")
            deficient |= lay.refresh(self.hp.power_iters, QR_IMPLS[self.hp.qr])
        return STATUS_RANK_DEFICIENT if deficient else STATUS_OK

    def counters(self, layer: int):
        lay = self.layers[layer]
        freq = lay.freq if lay.freq > 0 else self.hp.freq
        return dict(calls=self.calls, t=lay.t, ring_slot=lay.ring_slot,
                    refresh_count=lay.refresh_count,
                    next_refresh_t=(lay.t // freq + 1) * freq)


def stage_aware_freq(P: int, tau: int, f0: int) -> int:
    """Stage-aware refresh period, App. I ("Stage-aware basis rotation implementation"):
    mid = floor(P/2) - 1; n = mid - tau if tau > mid else mid + 1 - tau; f = floor(f0 / (1 - n/mid)),
    written out in exact rational arithmetic.  The printed rule is undefined where 1 - n/mid <= 0
    (or mid <= 0): ValueError there.  A period below 1 is raised to 1."""
    from fractions import Fraction
    from math import floor
    if P < 1 or tau < 0 or f0 < 1:
        raise ValueError("bad argument")
    mid = P // 2 - 1
    if mid <= 0:
        raise ValueError("the rule needs floor(P/2) - 1 > 0")
    n = mid - tau if tau > mid else mid + 1 - tau
    den = 1 - Fraction(n, mid)
    if den <= 0:
        raise ValueError("the rule divides by zero or goes negative at this delay")
    return max(1, floor(Fraction(f0) / den))


def lr_warmup_cosine(step: int, total_steps: int, warmup_fraction: float, base_lr: float, min_lr: float = 0.0) -> float:
    """Learning-rate schedule of the paper's runs (App. D.2): linear warm-up over the first
    warmup_fraction of the iterations (0.012 in the paper), cosine decay for the rest (towards min_lr,
    which it would reach at step = total_steps).  `step` counts from 0."""
    import math
    W = math.ceil(warmup_fraction * total_steps)
    if step < W:
        return base_lr * (step + 1) / W
    rest = max(1, total_steps - W)
    return min_lr + (base_lr - min_lr) * 0.5 * (1.0 + math.cos(math.pi * (step - W) / rest))


def effective_delay(consts, taus) -> float:
    """Effective delay of stage-dependent delays, Sec. 2.3, Eq. (effective-delay):
    tau' = sqrt(sum_i C_i^2 tau_i^2 / sum_i C_i^2)."""
    c2 = np.asarray(consts, dtype=np.float64) ** 2
    t = np.asarray(taus, dtype=np.float64)
    return float(np.sqrt(np.sum(c2 * t * t) / np.sum(c2)))


def make_oracle(workload, weights: Sequence[np.ndarray], **hp_over) -> Oracle:
    """Build an Oracle for a `workloads.Workload` (shapes and hyper-parameters only)."""
    hp = Hyper(lr=workload.lr, beta1=workload.beta1, beta2=workload.beta2, eps=workload.eps,
               weight_decay=workload.weight_decay, freq=workload.freq)
    for k, v in hp_over.items():
        setattr(hp, k, v)
    layers = [OracleLayer(w0, s.geom, s.src, s.tau_max, s.freq)
              for s, w0 in zip(workload.layers, weights)]
    return Oracle(layers, hp)
